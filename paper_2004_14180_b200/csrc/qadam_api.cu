// Host side of the C interface declared in include/qadam.h: argument checks,
// the tile table, launch configuration and the step bookkeeping.  Every step of
// the method itself runs in the kernels of qadam_kernels.cuh.
#include "qadam.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "qadam_host.h"
#include "qadam_kernels.cuh"
#include "qadam_server_pipe.cuh"
#include "qadam_worker_resident.cuh"

using namespace qadam;

namespace {

thread_local int g_last_cuda_error = 0;

inline bool cuda_ok(cudaError_t e) {
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return false;
  }
  return true;
}

}  // namespace

void qadam::record_cuda_error(int cuda_error) { g_last_cuda_error = cuda_error; }

namespace {

inline int64_t round_up64(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int bits_for(int num_codes) {
  int b = 0;
  while ((1 << b) < num_codes) ++b;
  return b;
}

// Positive levels L of G for (kg, grid), or a negative error.
int grad_levels(int kg, int grid) {
  if (grid == QADAM_GRID_STOCHASTIC) return kg == 0 ? 1 : QADAM_ERR_LEVEL;
  if (grid != QADAM_GRID_POW2 && grid != QADAM_GRID_UNIFORM) return QADAM_ERR_LEVEL;
  if (kg < 0) return QADAM_ERR_LEVEL;
  if (kg <= 1) return kg + 1;                          // both grids: {0,1}, {0,1/2,1}
  if (grid == QADAM_GRID_POW2) return kg <= 14 ? kg + 1 : QADAM_ERR_LEVEL;
  return kg <= 6 ? (1 << kg) : QADAM_ERR_LEVEL;
}

constexpr int kWordCtas = 256;                       // CTAs the per-pair words are sized for
constexpr size_t kWordBudget = (size_t)32 << 20;     // bytes of workspace they may take

struct Geometry {
  std::vector<int64_t> seg_len, seg_off;
  int64_t D = 0;
  std::vector<Tile> tiles;        // runs of at most kTileElems
  std::vector<Tile> ptiles;       // the same vector cut into runs of at most kPipeTile
  int gbits = 0, xbits = 0, L = 0;
  GMode gmode = G_TERNARY;
  size_t gcode_bytes = 0, wcode_bytes = 0, workspace_bytes = 0;
  std::vector<int> seg_tiles;        // tiles per segment
  size_t off_ptiles = 0, off_done = 0;
  // on-chip worker kernel: tiles of the segments that fit on chip (one vector) and the tiles
  // of the remaining segments (two streaming passes)
  std::vector<RTile> rtiles;
  std::vector<Tile> btiles;
  long long resident_elems = 0;      // padded elements of the resident segments (one vector)
  size_t off_rtiles = 0, off_btiles = 0, off_words = 0;
  size_t words_bytes = 0;            // room for the per-(pair, CTA) words of the on-chip worker kernel
};

// Splits the segments into those the on-chip worker kernel can hold (at most `capacity`
// tiles per (worker, segment) pair) and the rest, each with a tile table of its own.
void build_resident(long long capacity, int missing_tiles, Geometry* g) {
  g->rtiles.clear();
  g->btiles.clear();
  g->resident_elems = 0;
  for (const Tile& t : g->tiles) {
    if (g->seg_tiles[t.seg] <= capacity) {
      RTile r;
      r.off = t.off; r.count = t.count; r.seg = t.seg; r.need = g->seg_tiles[t.seg] + missing_tiles;
      // the segment's first tile: the previous entry belongs to another segment
      r.first = (!g->rtiles.empty() && g->rtiles.back().seg == t.seg) ? g->rtiles.back().first
                                                                      : (int)g->rtiles.size();
      g->rtiles.push_back(r);
      g->resident_elems += t.count;
    } else {
      g->btiles.push_back(t);
    }
  }
}

int validate_config(const qadam_config* c) {
  if (!c) return QADAM_ERR_NULL;
  if (c->d < 1 || c->n < 1 || c->n > 4096 || c->num_segments < 1) return QADAM_ERR_SIZE;
  if (c->num_segments > 1 && !c->seg_len) return QADAM_ERR_NULL;
  if (c->placement != QADAM_PLACE_SERVER && c->placement != QADAM_PLACE_WORKER)
    return QADAM_ERR_PLACEMENT;
  if (c->kg < -1 || c->kx < -1 || c->kx > 14) return QADAM_ERR_LEVEL;
  if (c->kg >= 0 && grad_levels(c->kg, c->grid_g) < 0) return QADAM_ERR_LEVEL;
  if (c->kg < 0 && c->grid_g != QADAM_GRID_POW2 && c->grid_g != QADAM_GRID_UNIFORM)
    return QADAM_ERR_LEVEL;      // the stochastic operator has no identity form
  if (!(c->beta1 >= 0.0f && c->beta1 < 1.0f) || !(c->beta2 >= 0.0f && c->beta2 < 1.0f) ||
      !(c->eps > 0.0f) || !std::isfinite(c->eps) || !std::isfinite(c->lr))
    return QADAM_ERR_HYPER;
  return QADAM_OK;
}

int build_geometry(const qadam_config* c, Geometry* g) {
  int rc = validate_config(c);
  if (rc != QADAM_OK) return rc;
  const int S = c->num_segments;
  g->seg_len.resize(S);
  g->seg_off.resize(S);
  int64_t sum = 0, off = 0;
  for (int s = 0; s < S; ++s) {
    const int64_t len = (S == 1 && !c->seg_len) ? c->d : c->seg_len[s];
    if (len < 1) return QADAM_ERR_SIZE;
    g->seg_len[s] = len;
    g->seg_off[s] = off;
    off += round_up64(len, kAlign);
    sum += len;
  }
  if (sum != c->d) return QADAM_ERR_SIZE;
  g->D = off;
  if (g->D / kAlign > (int64_t)1 << 30) return QADAM_ERR_SIZE;
  g->tiles.clear();
  g->ptiles.clear();
  for (int s = 0; s < S; ++s) {
    const int64_t plen = round_up64(g->seg_len[s], kAlign);
    for (int64_t o = 0; o < plen; o += kTileElems) {
      Tile t;
      t.off = g->seg_off[s] + o;
      t.count = (int)std::min<int64_t>(kTileElems, plen - o);
      t.seg = s;
      g->tiles.push_back(t);
    }
    for (int64_t o = 0; o < plen; o += kPipeTile) {
      Tile t;
      t.off = g->seg_off[s] + o;
      t.count = (int)std::min<int64_t>(kPipeTile, plen - o);
      t.seg = s;
      g->ptiles.push_back(t);
    }
  }
  if (c->kg < 0) {
    g->gmode = G_IDENTITY; g->L = 0; g->gbits = 32;
  } else {
    g->L = grad_levels(c->kg, c->grid_g);
    g->gbits = bits_for(2 * g->L + 1);
    g->gmode = c->grid_g == QADAM_GRID_STOCHASTIC ? G_STOCHASTIC
             : c->kg == 0 ? G_TERNARY : c->kg == 1 ? G_FIVE
             : c->grid_g == QADAM_GRID_POW2 ? G_POW2 : G_UNIFORM;
  }
  g->xbits = c->kx < 0 ? 0 : c->kx + 2;
  g->gcode_bytes = (size_t)(g->D * g->gbits / 8);
  g->wcode_bytes = (size_t)(g->D * g->xbits / 8);
  g->seg_tiles.assign(S, 0);
  for (const Tile& t : g->tiles) g->seg_tiles[t.seg] += 1;
  size_t wo = (size_t)round_up64((int64_t)g->tiles.size() * sizeof(Tile), 256);
  g->off_ptiles = wo;
  wo += (size_t)round_up64((int64_t)g->ptiles.size() * sizeof(Tile), 256);
  g->off_done = wo;
  wo += (size_t)round_up64((int64_t)c->n * c->num_segments * sizeof(unsigned), 256);
  // upper bounds (the split into resident and other segments is made at creation, on the device's sizes)
  g->off_rtiles = wo;
  wo += (size_t)round_up64((int64_t)g->tiles.size() * sizeof(RTile), 256);
  g->off_btiles = wo;
  wo += (size_t)round_up64((int64_t)g->tiles.size() * sizeof(Tile), 256);
  // one 64-bit word per (worker, segment) pair and CTA (at most kWordCtas CTAs), as long as
  // that stays modest; beyond it the on-chip kernel falls back to one counter per pair
  g->off_words = wo;
  {
    const size_t want = (size_t)c->n * c->num_segments * kWordCtas * sizeof(unsigned long long);
    g->words_bytes = want <= kWordBudget ? want : 0;
    wo += (size_t)round_up64((int64_t)g->words_bytes, 256);
  }
  g->workspace_bytes = wo + 256;
  return QADAM_OK;
}

}  // namespace

struct qadam_ctx {
  qadam_config cfg;
  qadam_buffers buf;
  Geometry geo;
  Hyper h;
  cudaStream_t stream;
  Tile* d_tiles;
  Tile* d_ptiles;
  int sm_count;
  int64_t last_server_step;     // steps completed by the server
  int64_t workers_done;         // workers compressed for step last_server_step + 1
  int64_t launches;
  int grid_absmax, grid_quant, grid_ident, grid_server, grid_bcast;
  size_t server_smem;
  // persistent pipelined server pass (ternary codes): stages > 0 when in use
  float lambda = 0.0f;       // l2 term (qadam_set_regularization)
  int pipe_stages = 0;
  size_t pipe_smem = 0;
  bool pipe_wide = false;    // the pipelined pass walks the 4096-element tiles (four rows) instead of the 2048-element ones
  qadam_options opt = {};
  unsigned spin_limit = kSpinLimit;
  bool range_open = false;   // a range of the current step has been served (qadam_server_step_range)
  CUtensorMap codes_map;
  unsigned* d_done = nullptr;
  // on-chip worker kernel: grid > 0 when in use
  int grid_resident = 0;
  int res_slots = 0, res_estages = 0;
  size_t res_smem = 0;
  RTile* d_rtiles = nullptr;
  Tile* d_btiles = nullptr;
  unsigned long long* d_words = nullptr;   // nullptr: one counter per pair instead
  // qadam_step_host: the copy of worker i + 1 runs on a stream of its own while worker i is compressed
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t copy_done[2] = {nullptr, nullptr};
  cudaEvent_t stage_free = nullptr;
  // instrumentation: event pairs of the launches since the last read
  bool profiling = false;
  struct Timed { int kind; cudaEvent_t start, stop; };
  std::vector<Timed> timed;
  std::vector<cudaEvent_t> spare_events;
};

namespace {

template <typename K>
int resident_grid(K kernel, size_t smem, int sm_count) {
  int per_sm = 0;
  if (!cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, smem)))
    return -1;
  return std::max(1, per_sm) * sm_count;
}

using WorkerKernel = void (*)(const WorkerParams);
using ServerKernel = void (*)(const ServerParams);

WorkerKernel pick_absmax(const qadam_ctx* c) {
  const bool w = c->cfg.placement == QADAM_PLACE_WORKER;
  if (c->lambda != 0.0f) return w ? worker_absmax_kernel<true, true> : worker_absmax_kernel<false, true>;
  return w ? worker_absmax_kernel<true> : worker_absmax_kernel<false>;
}

WorkerKernel pick_identity(const qadam_ctx* c) {
  const bool w = c->cfg.placement == QADAM_PLACE_WORKER;
  if (c->lambda != 0.0f) return w ? worker_identity_kernel<true, true> : worker_identity_kernel<false, true>;
  return w ? worker_identity_kernel<true> : worker_identity_kernel<false>;
}

WorkerKernel pick_quantize(const qadam_ctx* c) {
  const bool w = c->cfg.placement == QADAM_PLACE_WORKER;
  if (!w && c->lambda != 0.0f) {
    // moments on the server: phase 2 forms u = g + e again, l2 term included
    switch (c->geo.gmode) {
      case G_STOCHASTIC: return worker_quantize_kernel<false, G_STOCHASTIC, true>;
      case G_TERNARY: return worker_quantize_kernel<false, G_TERNARY, true>;
      case G_FIVE:    return worker_quantize_kernel<false, G_FIVE, true>;
      case G_POW2:    return worker_quantize_kernel<false, G_POW2, true>;
      default:        return worker_quantize_kernel<false, G_UNIFORM, true>;
    }
  }
  switch (c->geo.gmode) {
    case G_STOCHASTIC: return w ? worker_quantize_kernel<true, G_STOCHASTIC> : worker_quantize_kernel<false, G_STOCHASTIC>;
    case G_TERNARY: return w ? worker_quantize_kernel<true, G_TERNARY> : worker_quantize_kernel<false, G_TERNARY>;
    case G_FIVE:    return w ? worker_quantize_kernel<true, G_FIVE>    : worker_quantize_kernel<false, G_FIVE>;
    case G_POW2:    return w ? worker_quantize_kernel<true, G_POW2>    : worker_quantize_kernel<false, G_POW2>;
    default:        return w ? worker_quantize_kernel<true, G_UNIFORM> : worker_quantize_kernel<false, G_UNIFORM>;
  }
}

ServerKernel pick_server(const qadam_ctx* c) {
  const bool s = c->cfg.placement == QADAM_PLACE_SERVER;
  switch (c->geo.gmode) {
    case G_STOCHASTIC:
    case G_TERNARY:  return s ? server_step_kernel<true, G_TERNARY>  : server_step_kernel<false, G_TERNARY>;
    case G_FIVE:     return s ? server_step_kernel<true, G_FIVE>     : server_step_kernel<false, G_FIVE>;
    case G_POW2:     return s ? server_step_kernel<true, G_POW2>     : server_step_kernel<false, G_POW2>;
    case G_UNIFORM:  return s ? server_step_kernel<true, G_UNIFORM>  : server_step_kernel<false, G_UNIFORM>;
    default:         return s ? server_step_kernel<true, G_IDENTITY> : server_step_kernel<false, G_IDENTITY>;
  }
}

using PipeKernel = void (*)(const ServerParams, const CUtensorMap, const Tile*, int, int, int);

template <bool SM, int GB, int XB, int ROWS>
PipeKernel pick_pipe_n(int n) {
  switch (n) {
    case 4: return server_pipe_kernel<SM, 4, GB, XB, ROWS>;
    case 8: return server_pipe_kernel<SM, 8, GB, XB, ROWS>;
    case 16: return server_pipe_kernel<SM, 16, GB, XB, ROWS>;
    case 32: return server_pipe_kernel<SM, 32, GB, XB, ROWS>;
    default: return server_pipe_kernel<SM, 0, GB, XB, ROWS>;
  }
}

PipeKernel pick_pipe(const qadam_ctx* c) {
  const bool sm = c->cfg.placement == QADAM_PLACE_SERVER;
  const int n = c->cfg.n;
  if (c->geo.gmode == G_FIVE) return sm ? pick_pipe_n<true, 3, 0, 2>(n) : pick_pipe_n<false, 3, 0, 2>(n);
  if (c->geo.gmode == G_TERNARY || c->geo.gmode == G_STOCHASTIC) {
    // ternary gradient codes; ternary weights (kx = 0) have a path of their own; with the
    // moments on the workers the pass is decode bound and takes tiles of four rows
    if (c->pipe_wide)
      return c->cfg.kx == 0 ? pick_pipe_n<false, 2, 2, 4>(n) : pick_pipe_n<false, 2, 0, 4>(n);
    if (c->cfg.kx == 0) return sm ? pick_pipe_n<true, 2, 2, 2>(n) : pick_pipe_n<false, 2, 2, 2>(n);
    return sm ? pick_pipe_n<true, 2, 0, 2>(n) : pick_pipe_n<false, 2, 0, 2>(n);
  }
  // any other grid of at most 8 bits: table decode, worker count at run time
  return sm ? server_pipe_kernel<true, 0, 0, 0, 2> : server_pipe_kernel<false, 0, 0, 0, 2>;
}

using WorkerResidentKernel = void (*)(const WorkerResidentParams);

// With the l2 term the counter hand-over runs (the words were measured slower there).
template <int MODE>
WorkerResidentKernel pick_worker_resident_mode(bool worker_moments, bool l2, bool words) {
  if (l2) return worker_moments ? worker_resident_kernel<MODE, true, true, false>
                                : worker_resident_kernel<MODE, false, true, false>;
  if (worker_moments) return words ? worker_resident_kernel<MODE, true, false, true>
                                   : worker_resident_kernel<MODE, true, false, false>;
  return words ? worker_resident_kernel<MODE, false, false, true>
               : worker_resident_kernel<MODE, false, false, false>;
}

WorkerResidentKernel pick_worker_resident(const qadam_ctx* c, bool l2, bool words) {
  const bool w = c->cfg.placement == QADAM_PLACE_WORKER;
  switch (c->geo.gmode) {
    case G_TERNARY: return pick_worker_resident_mode<G_TERNARY>(w, l2, words);
    case G_FIVE:    return pick_worker_resident_mode<G_FIVE>(w, l2, words);
    case G_POW2:    return pick_worker_resident_mode<G_POW2>(w, l2, words);
    default:        return pick_worker_resident_mode<G_UNIFORM>(w, l2, words);
  }
}

// grids of the split worker kernels (they depend on whether the l2 term is on)
bool plan_worker_grids(qadam_ctx* c) {
  const int a = resident_grid(pick_absmax(c), 0, c->sm_count);
  const int q = resident_grid(pick_quantize(c), 0, c->sm_count);
  const int i = resident_grid(pick_identity(c), 0, c->sm_count);
  if (a < 0 || q < 0 || i < 0) return false;
  c->grid_absmax = a; c->grid_quant = q; c->grid_ident = i;
  return true;
}

cudaEvent_t take_event(qadam_ctx* c) {
  if (!c->spare_events.empty()) {
    cudaEvent_t e = c->spare_events.back();
    c->spare_events.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cuda_ok(cudaEventCreate(&e));
  return e;
}

// Brackets one kernel launch with events while profiling is on.
struct LaunchTimer {
  qadam_ctx* c;
  qadam_ctx::Timed t;
  LaunchTimer(qadam_ctx* ctx, int kind) : c(ctx) {
    t.kind = kind; t.start = t.stop = nullptr;
    if (c->profiling) {
      t.start = take_event(c);
      t.stop = take_event(c);
      if (t.start) cudaEventRecord(t.start, c->stream);
    }
  }
  ~LaunchTimer() {
    if (c->profiling && t.start && t.stop) {
      cudaEventRecord(t.stop, c->stream);
      c->timed.push_back(t);
    }
  }
};

ServerParams make_server_params(const qadam_ctx* c, float alpha) {
  ServerParams p;
  p.x = c->buf.x; p.m = c->buf.m; p.v = c->buf.v;
  p.scales = c->buf.scales;
  p.gcodes = static_cast<const unsigned char*>(c->buf.gcodes);
  p.wcodes = static_cast<unsigned char*>(c->buf.wcodes);
  p.wresid = c->buf.wresid;
  p.wfeedback = c->buf.wfeedback;
  p.tiles = c->d_tiles;
  p.D = c->geo.D;
  p.gcode_bytes = (long long)c->geo.gcode_bytes;
  p.tiles_per_worker = (int)c->geo.tiles.size();
  p.S = c->cfg.num_segments;
  p.n = c->cfg.n;
  p.k = c->cfg.kg; p.L = c->geo.L; p.gbits = c->geo.gbits;
  p.gmode = c->geo.gmode == G_STOCHASTIC ? G_TERNARY : c->geo.gmode;   // stochastic codes are ternary codes
  p.kx = c->cfg.kx; p.xbits = c->geo.xbits;
  p.alpha = alpha;
  p.nf = (float)c->cfg.n;
  p.inv_nf = 1.0f / (float)c->cfg.n;
  p.status = c->buf.status;
  p.h = c->h;
  p.spin_limit = c->spin_limit;
  return p;
}

}  // namespace

extern "C" {

int qadam_grad_code_bits(int32_t kg, int32_t grid_g) {
  if (kg == -1) return 32;
  const int L = grad_levels(kg, grid_g);
  return L < 0 ? L : bits_for(2 * L + 1);
}

int qadam_weight_code_bits(int32_t kx) {
  if (kx == -1) return 0;
  if (kx < 0 || kx > 14) return QADAM_ERR_LEVEL;
  return kx + 2;
}

int qadam_query_sizes(const qadam_config* cfg, int64_t* D, int64_t* seg_off,
                      size_t* gcode_bytes, size_t* wcode_bytes, size_t* workspace_bytes) {
  Geometry g;
  const int rc = build_geometry(cfg, &g);
  if (rc != QADAM_OK) return rc;
  if (D) *D = g.D;
  if (seg_off) std::memcpy(seg_off, g.seg_off.data(), g.seg_off.size() * sizeof(int64_t));
  if (gcode_bytes) *gcode_bytes = g.gcode_bytes;
  if (wcode_bytes) *wcode_bytes = g.wcode_bytes;
  if (workspace_bytes) *workspace_bytes = g.workspace_bytes;
  return QADAM_OK;
}

int qadam_create(const qadam_config* cfg, const qadam_buffers* b, qadam_ctx** out) {
  return qadam_create_ex(cfg, b, nullptr, out);
}

int qadam_create_ex(const qadam_config* cfg, const qadam_buffers* b, const qadam_options* opt,
                    qadam_ctx** out) {
  if (!cfg || !b || !out) return QADAM_ERR_NULL;
  *out = nullptr;
  qadam_options o = {};
  if (opt) o = *opt;
  if ((o.server_kernel != QADAM_SERVER_AUTO && o.server_kernel != QADAM_SERVER_PLAIN) ||
      (o.worker_kernel != QADAM_WORKER_AUTO && o.worker_kernel != QADAM_WORKER_STREAMING) ||
      (o.hand_over != QADAM_HANDOVER_AUTO && o.hand_over != QADAM_HANDOVER_COUNTERS) ||
      o.test_missing_tiles < 0 || o.reserved[0] || o.reserved[1] || o.reserved[2])
    return QADAM_ERR_SIZE;
  qadam_ctx* c = new (std::nothrow) qadam_ctx();
  if (!c) return QADAM_ERR_CUDA;
  int rc = build_geometry(cfg, &c->geo);
  if (rc != QADAM_OK) { delete c; return rc; }
  const bool quant_x = cfg->kx >= 0;
  if (!b->x || !b->m || !b->v || !b->e || !b->scales || !b->gcodes || !b->workspace ||
      !b->status || (quant_x && !b->wcodes)) {
    delete c; return QADAM_ERR_NULL;
  }
  if (b->wfeedback && !quant_x) { delete c; return QADAM_ERR_LEVEL; }     // a feedback buffer needs a weight quantizer
  const void* ptrs[] = {b->x, b->m, b->v, b->e, b->scales, b->gcodes, b->wcodes, b->wresid, b->wfeedback, b->status};
  for (const void* p : ptrs) {
    if (p && !aligned(p, p == b->status || p == b->scales ? 4 : 16)) { delete c; return QADAM_ERR_ALIGN; }
  }
  if (!aligned(b->workspace, 256)) { delete c; return QADAM_ERR_ALIGN; }
  if (b->workspace_bytes < c->geo.workspace_bytes) { delete c; return QADAM_ERR_WORKSPACE; }

  c->opt = o;
  c->spin_limit = o.wait_polls ? o.wait_polls : kSpinLimit;
  c->cfg = *cfg;
  c->cfg.seg_len = nullptr;            // the caller's array is not kept; geo has a copy
  c->buf = *b;
  c->stream = static_cast<cudaStream_t>(cfg->stream);
  c->h.beta = cfg->beta1; c->h.theta = cfg->beta2; c->h.eps = cfg->eps;
  c->h.one_minus_beta = 1.0f - cfg->beta1;
  c->h.one_minus_theta = 1.0f - cfg->beta2;
  c->last_server_step = 0;
  c->workers_done = 0;
  c->launches = 0;
  c->d_tiles = static_cast<Tile*>(b->workspace);
  {
    unsigned char* ws = static_cast<unsigned char*>(b->workspace);
    c->d_ptiles = reinterpret_cast<Tile*>(ws + c->geo.off_ptiles);
    c->d_done = reinterpret_cast<unsigned*>(ws + c->geo.off_done);
    c->d_rtiles = reinterpret_cast<RTile*>(ws + c->geo.off_rtiles);
    c->d_btiles = reinterpret_cast<Tile*>(ws + c->geo.off_btiles);
    c->d_words = c->geo.words_bytes ? reinterpret_cast<unsigned long long*>(ws + c->geo.off_words) : nullptr;
  }

  int dev = 0;
  if (!cuda_ok(cudaGetDevice(&dev)) ||
      !cuda_ok(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev))) {
    delete c; return QADAM_ERR_CUDA;
  }
  c->server_smem = sizeof(float) * (size_t)cfg->n;
  if (c->geo.gmode != G_TERNARY && c->geo.gmode != G_STOCHASTIC && c->geo.gmode != G_IDENTITY)
    c->server_smem += sizeof(float) * (size_t)cfg->n * ((size_t)1 << c->geo.gbits);
  if (c->server_smem > 200 * 1024) { delete c; return QADAM_ERR_SIZE; }
  ServerKernel sk = pick_server(c);
  if (c->server_smem > 48 * 1024 &&
      !cuda_ok(cudaFuncSetAttribute(sk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->server_smem))) {
    delete c; return QADAM_ERR_CUDA;
  }
  // The pipelined server pass needs ternary or five-level codes, at most kPipeMaxWorkers streams and room
  // for at least two stages in shared memory; otherwise the plain grid-stride kernel runs.
  {
    int max_smem = 0;
    if (!cuda_ok(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev))) {
      delete c; return QADAM_ERR_CUDA;
    }
    const bool sm_mom = cfg->placement == QADAM_PLACE_SERVER;
    const bool table = c->geo.gmode == G_POW2 || c->geo.gmode == G_UNIFORM;
    const bool pipe_codes = c->geo.gmode == G_TERNARY || c->geo.gmode == G_STOCHASTIC || c->geo.gmode == G_FIVE ||
                            (table && c->geo.gbits <= 8);
    const size_t head = pipe_head_bytes(table);
    const bool want_plain = o.server_kernel == QADAM_SERVER_PLAIN;
    auto stages_for = [&](int tile_elems) {
      const size_t sb = pipe_stage_bytes(cfg->n, sm_mom, pipe_codes ? c->geo.gbits : 2, tile_elems);
      return pipe_legal_stages(std::min((int)(((size_t)max_smem - head) / sb), kPipeMaxStages));
    };
    // With the moments on the workers the quantized quantity is Adam's normalised update,
    // whose codes are dense, and the pass is bound by the decode, not by memory: tiles of four
    // rows give a thread twice the independent work per tile, as long as four stages still fit.
    const bool ternary_codes = c->geo.gmode == G_TERNARY || c->geo.gmode == G_STOCHASTIC;
    c->pipe_wide = !sm_mom && ternary_codes && stages_for(kPipeWideTile) >= 4;
    const int tile_elems = c->pipe_wide ? kPipeWideTile : kPipeTile;
    const size_t sb = pipe_stage_bytes(cfg->n, sm_mom, pipe_codes ? c->geo.gbits : 2, tile_elems);
    int stages = stages_for(tile_elems);
    // the tensor copy addresses a tile's codes by a 32-bit coordinate in words of the stream
    // (32-bit words, 64-bit for the table decode): longer streams take the plain kernel
    const bool coord_fits = (long long)c->geo.gcode_bytes / (table ? 8 : 4) < (1ll << 31);
    if (!want_plain && pipe_codes && coord_fits && cfg->n <= kPipeMaxWorkers && stages >= 2 &&
        make_codes_tensor_map(&c->codes_map, b->gcodes, (long long)c->geo.gcode_bytes, cfg->n,
                              c->geo.gbits, table, tile_elems)) {
      c->pipe_stages = stages;
      c->pipe_smem = head + (size_t)stages * sb;
      if (!cuda_ok(cudaFuncSetAttribute(pick_pipe(c), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)c->pipe_smem))) {
        delete c; return QADAM_ERR_CUDA;
      }
    }
  }
  if (!plan_worker_grids(c)) { delete c; return QADAM_ERR_CUDA; }
  c->grid_server = resident_grid(sk, c->server_smem, c->sm_count);
  c->grid_bcast = resident_grid(weight_broadcast_kernel, 0, c->sm_count);
  // Worker side.  Segments small enough to be held by the
  // on-chip kernel (u stays in shared memory between the
  // max-abs reduction and the quantization, so g and e are read once) go through that
  // kernel; larger segments need two passes over memory whatever is done and take the two
  // plain streaming launches, over a tile table of their own.  The on-chip kernel needs
  // every CTA resident at once (its store side waits for other CTAs' load sides): one
  // CTA per SM, launched cooperatively.
  {
    int coop = 0, max_smem = 0;
    const bool want_split = o.worker_kernel == QADAM_WORKER_STREAMING;
    const bool wm = cfg->placement == QADAM_PLACE_WORKER;
    // (the stochastic operator runs in the streaming launches only)
    const bool eligible = !want_split && c->geo.gmode != G_IDENTITY && c->geo.gmode != G_STOCHASTIC &&
        cuda_ok(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev)) && coop &&
        cuda_ok(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (eligible) {
      // the CTA's shared memory: a ring of slots for u and a few stages for e (227 KB: 14 in all)
      const int estages = 2;                  // measured: 12 slots + 2 stages beat 11 + 3 and 10 + 4
      const int slots = std::min(((int)max_smem - kRHeadBytes - estages * resident_stage_bytes(wm)) / kRSlotBytes,
                                 kRMaxSlots);
      // a pair may give a CTA at most slots - 2 tiles: the rest of the ring lets the load side
      // run ahead into the next pair while this one is quantized and stored
      const int spare = 2;
      if (slots - spare >= 1) {
        build_resident((long long)c->sm_count * (slots - spare), o.test_missing_tiles, &c->geo);
        c->res_slots = slots;
        c->res_estages = estages;
        c->res_smem = resident_smem_bytes(slots, estages, wm);
        bool fits = !c->geo.rtiles.empty();
        for (int variant = 0; variant < 3 && fits; ++variant) {          // plain + words, plain, l2
          WorkerResidentKernel k = pick_worker_resident(c, variant == 2, variant == 0);
          int per_sm = 0;
          fits = cuda_ok(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->res_smem)) &&
                 cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kRThreads, c->res_smem)) &&
                 per_sm >= 1;
        }
        if (fits)
          c->grid_resident = c->sm_count;
      }
    }
  }
  if (c->grid_server < 0 || c->grid_bcast < 0) {
    delete c; return QADAM_ERR_CUDA;
  }

  // tables and status: synchronous, so the host vector may go away
  if (!cuda_ok(cudaMemcpyAsync(c->d_tiles, c->geo.tiles.data(), c->geo.tiles.size() * sizeof(Tile),
                               cudaMemcpyHostToDevice, c->stream)) ||
      !cuda_ok(cudaMemcpyAsync(c->d_ptiles, c->geo.ptiles.data(), c->geo.ptiles.size() * sizeof(Tile),
                               cudaMemcpyHostToDevice, c->stream)) ||
      (c->grid_resident > 0 &&
       (!cuda_ok(cudaMemcpyAsync(c->d_rtiles, c->geo.rtiles.data(), c->geo.rtiles.size() * sizeof(RTile),
                                 cudaMemcpyHostToDevice, c->stream)) ||
        (!c->geo.btiles.empty() &&
         !cuda_ok(cudaMemcpyAsync(c->d_btiles, c->geo.btiles.data(), c->geo.btiles.size() * sizeof(Tile),
                                  cudaMemcpyHostToDevice, c->stream))))) ||
      !cuda_ok(cudaMemsetAsync(b->status, 0, sizeof(uint32_t), c->stream)) ||
      !cuda_ok(cudaStreamSynchronize(c->stream))) {
    delete c; return QADAM_ERR_CUDA;
  }
  if (quant_x) {
    const ServerParams p = make_server_params(c, 0.0f);
    const int grid = (int)std::min<int64_t>(c->grid_bcast, (int64_t)c->geo.tiles.size());
    {
      LaunchTimer lt(c, QADAM_K_BROADCAST);
      weight_broadcast_kernel<<<grid, kThreads, 0, c->stream>>>(p);
    }
    if (!cuda_ok(cudaGetLastError())) { delete c; return QADAM_ERR_CUDA; }
    c->launches++;
  }
  *out = c;
  return QADAM_OK;
}

int qadam_worker_compress(qadam_ctx* c, int64_t step, const float* g,
                          int32_t worker_begin, int32_t worker_count, float lr_t) {
  if (!c || !g) return QADAM_ERR_NULL;
  if (!aligned(g, 16)) return QADAM_ERR_ALIGN;
  if (step != c->last_server_step + 1) return QADAM_ERR_STEP;
  if (worker_begin < 0 || worker_count < 1 || (int64_t)worker_begin + worker_count > c->cfg.n)
    return QADAM_ERR_WORKER;
  const float alpha = lr_t < 0.0f ? c->cfg.lr : lr_t;
  if (!std::isfinite(alpha)) return QADAM_ERR_HYPER;

  WorkerParams p;
  p.g = g;
  p.m = c->buf.m; p.v = c->buf.v; p.e = c->buf.e;
  p.scale_bits = reinterpret_cast<unsigned*>(c->buf.scales);
  p.gcodes = static_cast<unsigned char*>(c->buf.gcodes);
  p.tiles = c->d_tiles;
  p.status = c->buf.status;
  p.D = c->geo.D;
  p.gcode_bytes = (long long)c->geo.gcode_bytes;
  p.tiles_per_worker = (int)c->geo.tiles.size();
  p.total_tiles = (long long)worker_count * p.tiles_per_worker;
  p.S = c->cfg.num_segments;
  p.worker_begin = worker_begin;
  p.k = c->cfg.kg; p.L = c->geo.L; p.bits = c->geo.gbits;
  p.alpha = alpha;
  p.h = c->h;
  p.x = c->buf.x;
  p.wcodes = static_cast<const unsigned char*>(c->buf.wcodes);
  p.kx = c->cfg.kx; p.xbits = c->geo.xbits;
  p.lambda = c->lambda;
  p.spin_limit = c->spin_limit;
  p.seed_lo = (unsigned)c->cfg.seed;
  p.seed_hi = (unsigned)(c->cfg.seed >> 32);
  p.step = (unsigned)step;

  // the two streaming launches over a tile table: max-abs, then quantize
  auto streaming = [&](const Tile* tiles, int tiles_per_worker) -> int {
    WorkerParams q = p;
    q.tiles = tiles;
    q.tiles_per_worker = tiles_per_worker;
    q.total_tiles = (long long)worker_count * tiles_per_worker;
    int grid = (int)std::min<int64_t>(c->grid_absmax, q.total_tiles);
    {
      LaunchTimer lt(c, QADAM_K_ABSMAX);
      pick_absmax(c)<<<grid, kThreads, 0, c->stream>>>(q);
    }
    if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
    c->launches += 1;
    grid = (int)std::min<int64_t>(c->grid_quant, q.total_tiles);
    {
      LaunchTimer lt(c, QADAM_K_QUANTIZE);
      pick_quantize(c)<<<grid, kThreads, 0, c->stream>>>(q);
    }
    if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
    c->launches += 1;
    return QADAM_OK;
  };

  if (c->geo.gmode == G_IDENTITY) {
    const int grid = (int)std::min<int64_t>(c->grid_ident, p.total_tiles);
    {
      LaunchTimer lt(c, QADAM_K_IDENTITY);
      pick_identity(c)<<<grid, kThreads, 0, c->stream>>>(p);
    }
    if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
    c->launches += 1;
  } else {
    // the scales of these workers start at zero (the kernels fold maxima into them)
    if (!cuda_ok(cudaMemsetAsync(p.scale_bits + (size_t)worker_begin * p.S, 0,
                                 sizeof(unsigned) * (size_t)worker_count * p.S, c->stream)))
      return QADAM_ERR_CUDA;
    bool on_chip = c->grid_resident > 0;
    if (on_chip) {
      const size_t pairs = (size_t)c->cfg.n * p.S;     // all pairs' records are cleared, the call's are used
      const bool l2 = c->lambda != 0.0f;
      const bool use_words = !l2 && c->d_words != nullptr && c->grid_resident <= kWordCtas &&
                             c->opt.hand_over == QADAM_HANDOVER_AUTO;
      if (!cuda_ok(cudaMemsetAsync(c->d_done, 0, sizeof(unsigned) * pairs, c->stream)) ||
          (use_words && !cuda_ok(cudaMemsetAsync(c->d_words, 0, sizeof(unsigned long long) * pairs * c->grid_resident,
                                                 c->stream))))
        return QADAM_ERR_CUDA;
      WorkerResidentParams rp;
      rp.w = p;
      rp.words = use_words ? c->d_words : nullptr;
      rp.rtiles = c->d_rtiles;
      rp.done = c->d_done;
      rp.TR = (int)c->geo.rtiles.size();
      rp.total = (long long)worker_count * rp.TR;
      rp.slots = c->res_slots;
      rp.estages = c->res_estages;
      void* args[] = {&rp};
      cudaError_t e;
      {
        LaunchTimer lt(c, QADAM_K_WORKER_FUSED);
        e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(pick_worker_resident(c, l2, use_words)),
                                        dim3(c->grid_resident), dim3(kRThreads), args, c->res_smem, c->stream);
      }
      if (cuda_ok(e)) {
        c->launches += 1;
        if (!c->geo.btiles.empty()) {
          // the segments too large for the chip: two streaming passes over their own tile table
          const int rc = streaming(c->d_btiles, (int)c->geo.btiles.size());
          if (rc != QADAM_OK) return rc;
        }
      } else {
        // the cooperative launch was refused (the error is kept for qadam_last_cuda_error):
        // nothing of it runs, and the streaming launches over the whole vector still can
        (void)cudaGetLastError();
        on_chip = false;
      }
    }
    if (!on_chip) {
      const int rc = streaming(c->d_tiles, (int)c->geo.tiles.size());
      if (rc != QADAM_OK) return rc;
    }
  }
  c->workers_done += worker_count;
  return QADAM_OK;
}

int qadam_set_moment_rates(qadam_ctx* c, float beta_t, float theta_t) {
  if (!c) return QADAM_ERR_NULL;
  if (!(beta_t >= 0.0f && beta_t < 1.0f) || !(theta_t >= 0.0f && theta_t < 1.0f)) return QADAM_ERR_HYPER;
  c->h.beta = beta_t;
  c->h.theta = theta_t;
  c->h.one_minus_beta = 1.0f - beta_t;
  c->h.one_minus_theta = 1.0f - theta_t;
  return QADAM_OK;
}

int qadam_set_regularization(qadam_ctx* c, float lambda) {
  if (!c) return QADAM_ERR_NULL;
  if (!(lambda >= 0.0f) || !std::isfinite(lambda)) return QADAM_ERR_HYPER;
  const bool changed = (c->lambda != 0.0f) != (lambda != 0.0f);
  const float before = c->lambda;
  c->lambda = lambda;
  // the streaming kernels with and without the term differ: their grids are planned again
  if (changed && !plan_worker_grids(c)) {
    c->lambda = before;
    return QADAM_ERR_CUDA;
  }
  return QADAM_OK;
}

namespace {

// Index of the tile that starts at element `elem` in a tile table sorted by offset
// (tiles.size() for elem = D), or -1 when no tile starts there.
long long tile_index_at(const std::vector<Tile>& tiles, int64_t D, int64_t elem) {
  if (elem == D) return (long long)tiles.size();
  auto it = std::lower_bound(tiles.begin(), tiles.end(), elem,
                             [](const Tile& t, int64_t e) { return t.off < e; });
  if (it == tiles.end() || it->off != elem) return -1;
  return (long long)(it - tiles.begin());
}

// The server pass over tiles [tb, te) of the 4096-element table, which are ptiles
// [pb, pe) of the 2048-element table.
int launch_server(qadam_ctx* c, float alpha, long long tb, long long te, long long pb, long long pe) {
  if (te <= tb) return QADAM_OK;
  ServerParams p = make_server_params(c, alpha);
  {
    LaunchTimer lt(c, QADAM_K_SERVER);
    if (c->pipe_stages > 0) {
      const int n = c->cfg.n;
      const int inv_exact = (n & (n - 1)) == 0 ? 1 : 0;
      // the walk is over the 2048-element tiles, or over the 4096-element ones (four rows)
      const Tile* table = c->pipe_wide ? c->d_tiles + tb : c->d_ptiles + pb;
      const int np = (int)(c->pipe_wide ? te - tb : pe - pb);
      const int pgrid = std::min(c->sm_count, np);
      pick_pipe(c)<<<pgrid, kPipeThreads, c->pipe_smem, c->stream>>>(p, c->codes_map, table, np,
                                                                      c->pipe_stages, inv_exact);
    } else {
      p.tiles = c->d_tiles + tb;
      p.tiles_per_worker = (int)(te - tb);
      const int grid = (int)std::min<int64_t>(c->grid_server, te - tb);
      pick_server(c)<<<grid, kThreads, c->server_smem, c->stream>>>(p);
    }
  }
  if (!cuda_ok(cudaGetLastError())) return QADAM_ERR_CUDA;
  c->launches += 1;
  return QADAM_OK;
}

}  // namespace

int qadam_server_step(qadam_ctx* c, int64_t step, float lr_t) {
  if (!c) return QADAM_ERR_NULL;
  if (step != c->last_server_step + 1 || c->workers_done < c->cfg.n || c->range_open) return QADAM_ERR_STEP;
  const float alpha = lr_t < 0.0f ? c->cfg.lr : lr_t;
  if (!std::isfinite(alpha)) return QADAM_ERR_HYPER;
  const int rc = launch_server(c, alpha, 0, (long long)c->geo.tiles.size(), 0, (long long)c->geo.ptiles.size());
  if (rc != QADAM_OK) return rc;
  c->last_server_step = step;
  c->workers_done = 0;
  return QADAM_OK;
}

int qadam_server_step_range(qadam_ctx* c, int64_t step, float lr_t, int64_t elem_begin, int64_t elem_end) {
  if (!c) return QADAM_ERR_NULL;
  if (step != c->last_server_step + 1) return QADAM_ERR_STEP;
  const float alpha = lr_t < 0.0f ? c->cfg.lr : lr_t;
  if (!std::isfinite(alpha)) return QADAM_ERR_HYPER;
  if (elem_begin < 0 || elem_end < elem_begin || elem_end > c->geo.D) return QADAM_ERR_SIZE;
  const long long tb = tile_index_at(c->geo.tiles, c->geo.D, elem_begin);
  const long long te = tile_index_at(c->geo.tiles, c->geo.D, elem_end);
  const long long pb = tile_index_at(c->geo.ptiles, c->geo.D, elem_begin);
  const long long pe = tile_index_at(c->geo.ptiles, c->geo.D, elem_end);
  if (tb < 0 || te < 0 || pb < 0 || pe < 0) return QADAM_ERR_SIZE;
  const int rc = launch_server(c, alpha, tb, te, pb, pe);
  if (rc != QADAM_OK) return rc;
  c->range_open = true;
  return QADAM_OK;
}

int qadam_finish_step(qadam_ctx* c, int64_t step) {
  if (!c) return QADAM_ERR_NULL;
  if (step != c->last_server_step + 1) return QADAM_ERR_STEP;
  c->last_server_step = step;
  c->workers_done = 0;
  c->range_open = false;
  return QADAM_OK;
}

int qadam_shard_cuts(const qadam_config* cfg, int32_t shards, int64_t* cuts) {
  if (!cfg || !cuts) return QADAM_ERR_NULL;
  if (shards < 1) return QADAM_ERR_SIZE;
  Geometry geo;
  const int rc = build_geometry(cfg, &geo);
  if (rc != QADAM_OK) return rc;
  // cut g: the first tile whose start is at or beyond g * D / shards
  const std::vector<Tile>& tiles = geo.tiles;
  cuts[0] = 0;
  for (int32_t g = 1; g < shards; ++g) {
    const int64_t want = (int64_t)(((__int128)geo.D * g) / shards);
    auto it = std::lower_bound(tiles.begin(), tiles.end(), want,
                               [](const Tile& t, int64_t e) { return t.off < e; });
    cuts[g] = it == tiles.end() ? geo.D : it->off;
  }
  cuts[shards] = geo.D;
  return QADAM_OK;
}

int qadam_step_host(qadam_ctx* c, int64_t step, const float* g_host, float* g_stage,
                    void* out_host, float lr_t) {
  if (!c || !g_host || !g_stage) return QADAM_ERR_NULL;
  if (!aligned(g_stage, 16)) return QADAM_ERR_ALIGN;
  if (step != c->last_server_step + 1 || c->workers_done != 0 || c->range_open) return QADAM_ERR_STEP;
  const float alpha = lr_t < 0.0f ? c->cfg.lr : lr_t;
  if (!std::isfinite(alpha)) return QADAM_ERR_HYPER;
  // Worker by worker: the gradients of worker i + 1 cross the bus on a copy stream while the
  // kernels of worker i run on the context's stream.
  if (c->copy_stream == nullptr) {
    if (!cuda_ok(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking)) ||
        !cuda_ok(cudaEventCreateWithFlags(&c->copy_done[0], cudaEventDisableTiming)) ||
        !cuda_ok(cudaEventCreateWithFlags(&c->copy_done[1], cudaEventDisableTiming)) ||
        !cuda_ok(cudaEventCreateWithFlags(&c->stage_free, cudaEventDisableTiming)))
      return QADAM_ERR_CUDA;
  }
  // the staging buffer may still be read by work already on the context's stream
  if (!cuda_ok(cudaEventRecord(c->stage_free, c->stream)) ||
      !cuda_ok(cudaStreamWaitEvent(c->copy_stream, c->stage_free, 0)))
    return QADAM_ERR_CUDA;
  const size_t wbytes = sizeof(float) * (size_t)c->geo.D;
  int rc = QADAM_OK;
  for (int i = 0; i < c->cfg.n; ++i) {
    const size_t o = (size_t)i * (size_t)c->geo.D;
    if (!cuda_ok(cudaMemcpyAsync(g_stage + o, g_host + o, wbytes, cudaMemcpyHostToDevice, c->copy_stream)) ||
        !cuda_ok(cudaEventRecord(c->copy_done[i & 1], c->copy_stream)) ||
        !cuda_ok(cudaStreamWaitEvent(c->stream, c->copy_done[i & 1], 0)))
      return QADAM_ERR_CUDA;
    rc = qadam_worker_compress(c, step, g_stage + o, i, 1, lr_t);
    if (rc != QADAM_OK) return rc;
  }
  rc = qadam_server_step(c, step, lr_t);
  if (rc != QADAM_OK) return rc;
  if (out_host) {
    const bool packed = c->cfg.kx >= 0;
    const void* src = packed ? c->buf.wcodes : static_cast<const void*>(c->buf.x);
    const size_t bytes = packed ? c->geo.wcode_bytes : sizeof(float) * (size_t)c->geo.D;
    if (!cuda_ok(cudaMemcpyAsync(out_host, src, bytes, cudaMemcpyDeviceToHost, c->stream)))
      return QADAM_ERR_CUDA;
  }
  if (!cuda_ok(cudaStreamSynchronize(c->stream))) return QADAM_ERR_CUDA;
  return QADAM_OK;
}

int qadam_poll_status(qadam_ctx* c, uint32_t* host_status) {
  if (!c || !host_status) return QADAM_ERR_NULL;
  if (!cuda_ok(cudaMemcpyAsync(host_status, c->buf.status, sizeof(uint32_t),
                               cudaMemcpyDeviceToHost, c->stream)) ||
      !cuda_ok(cudaStreamSynchronize(c->stream)))
    return QADAM_ERR_CUDA;
  return QADAM_OK;
}

int qadam_profile_enable(qadam_ctx* c, int enable) {
  if (!c) return QADAM_ERR_NULL;
  c->profiling = enable != 0;
  return QADAM_OK;
}

int qadam_profile_read(qadam_ctx* c, double* ms, int64_t* launches) {
  if (!c || !ms || !launches) return QADAM_ERR_NULL;
  if (!cuda_ok(cudaStreamSynchronize(c->stream))) return QADAM_ERR_CUDA;
  for (const qadam_ctx::Timed& t : c->timed) {
    float el = 0.0f;
    if (cuda_ok(cudaEventElapsedTime(&el, t.start, t.stop))) {
      ms[t.kind] += el;
      launches[t.kind] += 1;
    }
    c->spare_events.push_back(t.start);
    c->spare_events.push_back(t.stop);
  }
  c->timed.clear();
  return QADAM_OK;
}

int qadam_worker_pass_model(const qadam_ctx* c, int64_t* one_pass, int64_t* two_pass) {
  if (!c || !one_pass || !two_pass) return QADAM_ERR_NULL;
  if (c->grid_resident > 0) {
    *one_pass = (int64_t)c->cfg.n * c->geo.resident_elems;
    *two_pass = (int64_t)c->cfg.n * (c->geo.D - c->geo.resident_elems);
  } else {
    *one_pass = 0;
    *two_pass = (int64_t)c->cfg.n * c->geo.D;
  }
  return QADAM_OK;
}

int64_t qadam_launch_count(const qadam_ctx* c) { return c ? c->launches : 0; }

int qadam_destroy(qadam_ctx* c) {
  if (!c) return QADAM_ERR_NULL;
  for (const qadam_ctx::Timed& t : c->timed) {
    cudaEventDestroy(t.start);
    cudaEventDestroy(t.stop);
  }
  for (cudaEvent_t e : c->spare_events) cudaEventDestroy(e);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  for (cudaEvent_t e : c->copy_done) if (e) cudaEventDestroy(e);
  if (c->stage_free) cudaEventDestroy(c->stage_free);
  delete c;
  return QADAM_OK;
}

const char* qadam_strerror(int err) {
  switch (err) {
    case QADAM_OK: return "ok";
    case QADAM_ERR_NULL: return "a required pointer is NULL";
    case QADAM_ERR_SIZE: return "invalid d, n, num_segments or segment length";
    case QADAM_ERR_LEVEL: return "quantizer level parameter out of the supported range";
    case QADAM_ERR_ALIGN: return "device pointer not sufficiently aligned";
    case QADAM_ERR_WORKSPACE: return "workspace too small";
    case QADAM_ERR_STEP: return "step out of order";
    case QADAM_ERR_WORKER: return "worker range outside 0..n";
    case QADAM_ERR_HYPER: return "invalid beta, theta, epsilon or step size";
    case QADAM_ERR_CUDA: return "a CUDA call failed";
    case QADAM_ERR_PLACEMENT: return "invalid placement";
    case QADAM_ERR_CAPACITY: return "size beyond the fixed capacity of the allocation-free entry point";
    default: return "unknown error";
  }
}

int qadam_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
