// The step kernels: worker phase 1 (form u, reduce max|u|), worker phase 2
// (quantize, pack, residual), the identity worker, the fused server pass and the
// stand-alone weight broadcast.  All are grid-stride loops over a tile table.
//
// Thread/tile mapping (all kernels): a CTA of 256 threads owns a tile of up to
// 4096 consecutive padded elements as 4 CTA-wide rows of 1024; in row r thread t
// owns the 4 consecutive elements starting at r*1024 + 4*t, so every global
// access of fp32 state is one coalesced 128-bit access per thread, and one warp
// in one row owns 128 elements = one aligned run of the packed code stream.
#pragma once

#include "qadam_device.cuh"

namespace qadam {

struct WorkerParams {
  const float* g;        // [worker_count][D] gradients of the workers of this call
  float* m;              // [n][D] worker moments (PLACE_WORKER) or nullptr
  float* v;
  float* e;              // [n][D]
  unsigned* scale_bits;  // [n][S] the scales buffer, seen as bit patterns
  unsigned char* gcodes; // [n][gcode_bytes]
  const Tile* tiles;     // [tiles_per_worker]
  unsigned* status;
  long long D;
  long long gcode_bytes;
  long long total_tiles; // worker_count * tiles_per_worker
  int tiles_per_worker;
  int S;
  int worker_begin;
  int k, L, bits;        // level parameter, positive levels, code width
  float alpha;
  Hyper h;
  // l2 term (kernels instantiated with L2 = true): lambda * (held weights) is added to g
  const float* x;               // [D] master copy (held as is when kx < 0)
  const unsigned char* wcodes;  // packed Q_x(x) (kx >= 0)
  int kx, xbits;
  float lambda;
  unsigned spin_limit;          // persistent kernels: polls of one wait before it gives up
  // stochastic operator: key of the random stream and the step number
  unsigned seed_lo, seed_hi, step;
};

// Packed weight codes of at most 8 bits: the two 32-bit words that hold this lane's 4 codes
// of a 128-element row (row_elem: first element of the row).  Split from the decode so
// that a kernel can issue the loads a tile ahead of their use.
__device__ __forceinline__ void held_fetch8(const WorkerParams& p, long long row_elem, int lane,
                                            unsigned& lo, unsigned& hi) {
  const unsigned* words = reinterpret_cast<const unsigned*>(p.wcodes + row_elem * p.xbits / 8);
  const int F = 4 * p.xbits;                            // bits per lane = words per row
  const int w = (F * lane) >> 5;
  lo = __ldg(words + w);
  // the lane's field runs into the next word only for widths that do not divide 32
  hi = ((F * lane) & 31) + F > 32 ? __ldg(words + w + 1) : 0u;
}
// ... and their values: (code - 2^kx) times the grid step, exact.
__device__ __forceinline__ void held_decode8(const WorkerParams& p, int lane, unsigned lo, unsigned hi,
                                             float out[4]) {
  const int F = 4 * p.xbits;
  const unsigned v = __funnelshift_r(lo, hi, (F * lane) & 31);
  const unsigned f = F == 32 ? v : (v & ((1u << F) - 1u));
  const unsigned mask = (1u << p.xbits) - 1u;
  const float step = exp2i(-(p.kx + 1));
  // code -> float without a conversion: 2^23 + code as a bit pattern, minus 2^23 + 2^kx
  const float bias = -(8388608.0f + (float)(1 << p.kx));
#pragma unroll
  for (int c = 0; c < 4; ++c)
    out[c] = __fmul_rn(__fadd_rn(__uint_as_float(0x4b000000u | ((f >> (c * p.xbits)) & mask)), bias), step);
}

// The weights a worker holds for this lane's 4 elements of a 128-element row: the broadcast
// Q_x(x) decoded from its packed codes (code - 2^kx times the grid step, exact), or x itself
// when the weights are not quantized.  row_elem: first element of the row.
__device__ __forceinline__ void held_weights4(const WorkerParams& p, long long row_elem, int lane,
                                              float out[4]) {
  if (p.kx < 0) {
    const float4 v = *reinterpret_cast<const float4*>(p.x + row_elem + lane * 4);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    return;
  }
  if (p.xbits <= 8) {
    unsigned lo, hi;
    held_fetch8(p, row_elem, lane, lo, hi);
    held_decode8(p, lane, lo, hi, out);
    return;
  }
  const unsigned char* row = p.wcodes + row_elem * p.xbits / 8;
  const unsigned mask = (1u << p.xbits) - 1u;
  const float step = exp2i(-(p.kx + 1));
  const float bias = -(8388608.0f + (float)(1 << p.kx));
  auto value = [&](unsigned code) {
    return __fmul_rn(__fadd_rn(__uint_as_float(0x4b000000u | code), bias), step);
  };
  const unsigned* words = reinterpret_cast<const unsigned*>(row);
  const int row_words = 4 * p.xbits;                    // 128 codes
  const int half = 2 * p.xbits;                         // two codes, at most 32 bits
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int bit = 2 * half * lane + h * half;
    const int w = bit >> 5;
    const unsigned lo = __ldg(words + w);
    const unsigned hi = __ldg(words + (w + 1 < row_words ? w + 1 : w));
    const unsigned f = __funnelshift_r(lo, hi, bit & 31);
    out[2 * h] = value(f & mask);
    out[2 * h + 1] = value((f >> p.xbits) & mask);
  }
}
// The held weights of a thread's 4 elements of a row as they are loaded when the weights are
// packed codes of at most 8 bits: the two words that hold the lane's 4 codes, fetched together
// with the loads of g and e and decoded when the row is processed.  Unquantized weights and
// wider codes are read at the point of use (fetched stays false).
struct HeldRaw {
  unsigned lo, hi;
  bool fetched;
};
__device__ __forceinline__ HeldRaw held_fetch(const WorkerParams& p, long long row_elem, int lane) {
  HeldRaw h;
  h.lo = h.hi = 0u;
  h.fetched = p.kx >= 0 && p.xbits <= 8;
  if (h.fetched) held_fetch8(p, row_elem, lane, h.lo, h.hi);
  return h;
}
// g + lambda * (held weights) from what held_fetch loaded
__device__ __forceinline__ void add_l2_term_held(const WorkerParams& p, long long row_elem, int lane,
                                                 const HeldRaw& h, float gg[4]);

// g + lambda * (held weights), each operation rounded once (Section 5.1's l2 term)
__device__ __forceinline__ void add_l2_term(const WorkerParams& p, long long row_elem, int lane,
                                            float gg[4]) {
  float w[4];
  held_weights4(p, row_elem, lane, w);
#pragma unroll
  for (int c = 0; c < 4; ++c) gg[c] = __fadd_rn(gg[c], __fmul_rn(p.lambda, w[c]));
}

__device__ __forceinline__ void add_l2_term_held(const WorkerParams& p, long long row_elem, int lane,
                                                 const HeldRaw& h, float gg[4]) {
  if (!h.fetched) {
    add_l2_term(p, row_elem, lane, gg);
    return;
  }
  float w[4];
  held_decode8(p, lane, h.lo, h.hi, w);
#pragma unroll
  for (int c = 0; c < 4; ++c) gg[c] = __fadd_rn(gg[c], __fmul_rn(p.lambda, w[c]));
}

// The same from codes fetched earlier with held_fetch8.
__device__ __forceinline__ void add_l2_term_fetched(const WorkerParams& p, int lane, unsigned lo, unsigned hi,
                                                    float gg[4]) {
  float w[4];
  held_decode8(p, lane, lo, hi, w);
#pragma unroll
  for (int c = 0; c < 4; ++c) gg[c] = __fadd_rn(gg[c], __fmul_rn(p.lambda, w[c]));
}

struct ServerParams {
  float* x;              // [D]
  float* m;              // [D] (PLACE_SERVER) or nullptr
  float* v;
  const float* scales;   // [n][S]
  const unsigned char* gcodes;  // [n][gcode_bytes]
  unsigned char* wcodes; // [wcode_bytes] or nullptr
  float* wresid;         // [D] or nullptr
  float* wfeedback;      // [D] or nullptr: error buffer of the broadcast (Q_x is applied to x + wfeedback)
  const Tile* tiles;
  long long D;
  long long gcode_bytes;
  int tiles_per_worker;
  int S;
  int n;
  int k, L, gbits;       // gradient level parameter / levels / code width
  int gmode;             // GMode of the gradient grid
  int kx, xbits;         // weight level parameter (-1: none) / code width
  float alpha;
  float nf;              // (float)n
  float inv_nf;          // 1/n, exact when n is a power of two
  unsigned* status;
  Hyper h;
  unsigned spin_limit;   // pipelined pass: polls of one wait before it gives up
};

__device__ __forceinline__ float4 ld_f4(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
__device__ __forceinline__ float4 ld_f4_stream(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_f4(float* p, const float4& v) {
  *reinterpret_cast<float4*>(p) = v;
}

// CTA-wide max of a 32-bit pattern; result valid in thread 0.
__device__ __forceinline__ unsigned block_max(unsigned v, unsigned* smem8) {
  v = warp_max(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) smem8[warp] = v;
  __syncthreads();
  unsigned r = 0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) r = max(r, smem8[w]);
  }
  __syncthreads();
  return r;
}

// ---------------------------------------------------------------------------
// Worker phase 1.  PLACE_SERVER: u = g + e, nothing written but the running
// max.  PLACE_WORKER: v, m updated in place, u = alpha m/sqrt(v+eps) + e stored
// in e's slot for phase 2.  The max over a (worker, segment) is taken on the bit
// patterns of |u| (monotone for non-negative floats, exact, order-free; a NaN
// or Inf ends up as the maximum and is reported by phase 2).
// ---------------------------------------------------------------------------
template <bool WORKER_MOMENTS, bool L2 = false>
__global__ void __launch_bounds__(kThreads, WORKER_MOMENTS ? 2 : (L2 ? 3 : 4))
worker_absmax_kernel(const WorkerParams p) {
  __shared__ unsigned red[kThreads / 32];
  unsigned mx = 0;
  long long cur_pair = -1;
  for (long long t = blockIdx.x; t < p.total_tiles; t += gridDim.x) {
    const int wl = (int)(t / p.tiles_per_worker);
    const Tile tile = p.tiles[(int)(t - (long long)wl * p.tiles_per_worker)];
    const int w = p.worker_begin + wl;
    const long long pair = (long long)w * p.S + tile.seg;
    if (pair != cur_pair) {
      if (cur_pair >= 0) {
        const unsigned r = block_max(mx, red);
        if (threadIdx.x == 0 && r) atomicMax(p.scale_bits + cur_pair, r);
      }
      mx = 0;
      cur_pair = pair;
    }
    const float* gp = p.g + (long long)wl * p.D + tile.off;
    const long long so = (long long)w * p.D + tile.off;
    float4 gv[kRows], ev[kRows], mv[kRows], vv[kRows];
    HeldRaw hw[L2 ? kRows : 1];
    bool act[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const int idx = r * kRowElems + threadIdx.x * 4;
      act[r] = idx < tile.count;
      if (act[r]) {
        gv[r] = ld_f4_stream(gp + idx);
        ev[r] = ld_f4(p.e + so + idx);
        if constexpr (WORKER_MOMENTS) {
          mv[r] = ld_f4(p.m + so + idx);
          vv[r] = ld_f4(p.v + so + idx);
        }
        if constexpr (L2)
          hw[r] = held_fetch(p, tile.off + r * kRowElems + (threadIdx.x >> 5) * 128, threadIdx.x & 31);
      }
    }
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      if (!act[r]) continue;
      const int idx = r * kRowElems + threadIdx.x * 4;
      float gg[4] = {gv[r].x, gv[r].y, gv[r].z, gv[r].w};
      float ee[4] = {ev[r].x, ev[r].y, ev[r].z, ev[r].w};
      float uu[4];
      if constexpr (L2)
        add_l2_term_held(p, tile.off + r * kRowElems + (threadIdx.x >> 5) * 128, threadIdx.x & 31, hw[r], gg);
      if constexpr (WORKER_MOMENTS) {
        float mm[4] = {mv[r].x, mv[r].y, mv[r].z, mv[r].w};
        float vs[4] = {vv[r].x, vv[r].y, vv[r].z, vv[r].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          moments(p.h, gg[c], mm[c], vs[c]);
          uu[c] = __fadd_rn(adam_step(p.h, mm[c], vs[c], p.alpha), ee[c]);
        }
        st_f4(p.m + so + idx, make_float4(mm[0], mm[1], mm[2], mm[3]));
        st_f4(p.v + so + idx, make_float4(vs[0], vs[1], vs[2], vs[3]));
        st_f4(p.e + so + idx, make_float4(uu[0], uu[1], uu[2], uu[3]));
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) uu[c] = __fadd_rn(gg[c], ee[c]);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) mx = max(mx, __float_as_uint(fabsf(uu[c])));
    }
  }
  if (cur_pair >= 0) {
    const unsigned r = block_max(mx, red);
    if (threadIdx.x == 0 && r) atomicMax(p.scale_bits + cur_pair, r);
  }
}

// ---------------------------------------------------------------------------
// Worker phase 2: codes = Q_g level indices of u against the finished scale,
// packed; e <- u - Q_g(u).  U_IN_E: u was left in e's slot by phase 1.
// Three blocks per SM (at most 80 registers): with one block of 150 registers the
// general grids ran at 0.35 of the copy rate, with three at 0.73 (measured).
// ---------------------------------------------------------------------------
template <bool U_IN_E, int MODE, bool L2 = false>
__global__ void __launch_bounds__(kThreads, MODE == G_STOCHASTIC && !L2 ? 1 : 3)
worker_quantize_kernel(const WorkerParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // Tiles per round of loads, then of arithmetic and stores.  (Two per round when only e is
  // read, to have as many loads in flight as the two-array form, was measured slower.)
  constexpr int kPerRound = 1;
  for (long long t0 = blockIdx.x; t0 < p.total_tiles; t0 += (long long)kPerRound * gridDim.x) {
    Tile tile[kPerRound];
    int wl[kPerRound];
    bool have[kPerRound];
    float4 gv[kPerRound][kRows], ev[kPerRound][kRows];
    HeldRaw hw[kPerRound][L2 ? kRows : 1];
#pragma unroll
    for (int a = 0; a < kPerRound; ++a) {
      const long long t = t0 + (long long)a * gridDim.x;
      have[a] = t < p.total_tiles;
      if (!have[a]) continue;
      wl[a] = (int)(t / p.tiles_per_worker);
      tile[a] = p.tiles[(int)(t - (long long)wl[a] * p.tiles_per_worker)];
      const float* gp = p.g + (long long)wl[a] * p.D + tile[a].off;
      const long long so = (long long)(p.worker_begin + wl[a]) * p.D + tile[a].off;
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const int idx = r * kRowElems + threadIdx.x * 4;
        if (idx < tile[a].count) {
          if constexpr (!U_IN_E) gv[a][r] = ld_f4_stream(gp + idx);
          ev[a][r] = ld_f4(p.e + so + idx);
          if constexpr (L2 && !U_IN_E)
            hw[a][r] = held_fetch(p, tile[a].off + r * kRowElems + warp * 128, lane);
        }
      }
    }
#pragma unroll
    for (int a = 0; a < kPerRound; ++a) {
      if (!have[a]) continue;
      const int w = p.worker_begin + wl[a];
      const unsigned sb = p.scale_bits[(long long)w * p.S + tile[a].seg];
      const float s = __uint_as_float(sb);
      const GradScale gs = grad_scale<MODE == G_STOCHASTIC ? G_TERNARY : MODE>(s, p.k);
      if (sb >= 0x7f800000u && threadIdx.x == 0) atomicOr(p.status, 1u);
      const long long so = (long long)w * p.D + tile[a].off;
      unsigned char* cw = p.gcodes + (long long)w * p.gcode_bytes;
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const int idx = r * kRowElems + threadIdx.x * 4;
        if (idx >= tile[a].count) continue;         // warp-uniform: counts are multiples of 128
        float ee[4] = {ev[a][r].x, ev[a][r].y, ev[a][r].z, ev[a][r].w};
        float uu[4];
        if constexpr (U_IN_E) {
#pragma unroll
          for (int c = 0; c < 4; ++c) uu[c] = ee[c];
        } else {
          float gg[4] = {gv[a][r].x, gv[a][r].y, gv[a][r].z, gv[a][r].w};
          if constexpr (L2) add_l2_term_held(p, tile[a].off + r * kRowElems + warp * 128, lane, hw[a][r], gg);
#pragma unroll
          for (int c = 0; c < 4; ++c) uu[c] = __fadd_rn(gg[c], ee[c]);
        }
        unsigned code[4];
        float en[4];
        if constexpr (MODE == G_STOCHASTIC) {
          // the four coordinates of this thread are one block of the stream: counter
          // (element / 4, worker, step), key = seed
          const unsigned long long block = (unsigned long long)(tile[a].off + idx) >> 2;
          const uint4 rnd = philox4x32_10(make_uint4((unsigned)block, (unsigned)(block >> 32), (unsigned)w, p.step),
                                          make_uint2(p.seed_lo, p.seed_hi));
          code[0] = quantize_grad_stochastic(uu[0], s, rnd.x, en[0]);
          code[1] = quantize_grad_stochastic(uu[1], s, rnd.y, en[1]);
          code[2] = quantize_grad_stochastic(uu[2], s, rnd.z, en[2]);
          code[3] = quantize_grad_stochastic(uu[3], s, rnd.w, en[3]);
        } else if constexpr (MODE == G_TERNARY) {
          code[0] = quantize_ternary4(uu, gs, en);           // the lane's byte of four codes
        } else if constexpr (MODE == G_FIVE) {
          code[0] = quantize_five4(uu, gs, en);              // the lane's 12 bits of four codes
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) code[c] = quantize_grad<MODE>(uu[c], gs, p.k, p.L, en[c]);
        }
        st_f4(p.e + so + idx, make_float4(en[0], en[1], en[2], en[3]));
        const long long row_elem = tile[a].off + r * kRowElems + warp * 128;
        void* dst = cw + row_elem * p.bits / 8;
        if constexpr (MODE == G_TERNARY) {
          store_row_of_code_bytes(code[0], dst, lane);
        } else if constexpr (MODE == G_STOCHASTIC) {
          pack_row_store<2>(code[0], code[1], code[2], code[3], dst, lane);
        } else if constexpr (MODE == G_FIVE) {
          pack_row_store_fields<3>(code[0], dst, lane);
        } else {
          pack_row_store_rt(p.bits, code[0], code[1], code[2], code[3], dst, lane);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Identity Q_g: the stream is u itself, the scale is 1, e <- u - u.
// ---------------------------------------------------------------------------
template <bool WORKER_MOMENTS, bool L2 = false>
__global__ void __launch_bounds__(kThreads)
worker_identity_kernel(const WorkerParams p) {
  for (long long t = blockIdx.x; t < p.total_tiles; t += gridDim.x) {
    const int wl = (int)(t / p.tiles_per_worker);
    const int tl = (int)(t - (long long)wl * p.tiles_per_worker);
    const Tile tile = p.tiles[tl];
    const int w = p.worker_begin + wl;
    if (tl == 0 && threadIdx.x < p.S) {
      for (int s = threadIdx.x; s < p.S; s += kThreads)
        p.scale_bits[(long long)w * p.S + s] = __float_as_uint(1.0f);
    }
    const float* gp = p.g + (long long)wl * p.D + tile.off;
    const long long so = (long long)w * p.D + tile.off;
    float* out = reinterpret_cast<float*>(p.gcodes + (long long)w * p.gcode_bytes) + tile.off;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const int idx = r * kRowElems + threadIdx.x * 4;
      if (idx >= tile.count) continue;
      const float4 g4 = ld_f4_stream(gp + idx);
      const float4 e4 = ld_f4(p.e + so + idx);
      float gg[4] = {g4.x, g4.y, g4.z, g4.w};
      float ee[4] = {e4.x, e4.y, e4.z, e4.w};
      float uu[4], en[4];
      if constexpr (L2)
        add_l2_term(p, tile.off + r * kRowElems + (threadIdx.x >> 5) * 128, threadIdx.x & 31, gg);
      if constexpr (WORKER_MOMENTS) {
        const float4 m4 = ld_f4(p.m + so + idx);
        const float4 v4 = ld_f4(p.v + so + idx);
        float mm[4] = {m4.x, m4.y, m4.z, m4.w};
        float vs[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          moments(p.h, gg[c], mm[c], vs[c]);
          uu[c] = __fadd_rn(adam_step(p.h, mm[c], vs[c], p.alpha), ee[c]);
        }
        st_f4(p.m + so + idx, make_float4(mm[0], mm[1], mm[2], mm[3]));
        st_f4(p.v + so + idx, make_float4(vs[0], vs[1], vs[2], vs[3]));
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) uu[c] = __fadd_rn(gg[c], ee[c]);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) en[c] = __fsub_rn(uu[c], uu[c]);
      st_f4(out + idx, make_float4(uu[0], uu[1], uu[2], uu[3]));
      st_f4(p.e + so + idx, make_float4(en[0], en[1], en[2], en[3]));
    }
  }
}

// ---------------------------------------------------------------------------
// Q_x of 4 consecutive weights of one lane, packed row store, optional residual.
// ---------------------------------------------------------------------------
// With an error buffer for the broadcast (wfeedback, not in the paper) the quantized value is
// y = x + wfeedback and the buffer becomes y - Q_x(y).
__device__ __forceinline__ void broadcast_row(const float xin[4], int kx, int xbits,
                                              unsigned char* wcodes, float* wresid, float* wfeedback,
                                              long long elem, long long row_elem, int lane) {
  unsigned code[4];
  float xx[4] = {xin[0], xin[1], xin[2], xin[3]};
  float xq[4];
  if (wfeedback) {
    const float4 ew = ld_f4(wfeedback + elem);
    xx[0] = __fadd_rn(xx[0], ew.x); xx[1] = __fadd_rn(xx[1], ew.y);
    xx[2] = __fadd_rn(xx[2], ew.z); xx[3] = __fadd_rn(xx[3], ew.w);
  }
#pragma unroll
  for (int c = 0; c < 4; ++c) code[c] = quantize_weight(xx[c], kx, xq[c]);
  if (wresid || wfeedback) {
    const float4 r = make_float4(__fsub_rn(xx[0], xq[0]), __fsub_rn(xx[1], xq[1]),
                                 __fsub_rn(xx[2], xq[2]), __fsub_rn(xx[3], xq[3]));
    if (wresid) st_f4(wresid + elem, r);
    if (wfeedback) st_f4(wfeedback + elem, r);
  }
  void* dst = wcodes + row_elem * xbits / 8;
  switch (xbits) {
    case 2: pack_row_store<2>(code[0], code[1], code[2], code[3], dst, lane); break;
    case 3: pack_row_store<3>(code[0], code[1], code[2], code[3], dst, lane); break;
    case 8: pack_row_store<8>(code[0], code[1], code[2], code[3], dst, lane); break;
    default: pack_row_store_rt(xbits, code[0], code[1], code[2], code[3], dst, lane); break;
  }
}

// Stand-alone Q_x(x) (the broadcast of x_1 before the first step).  Internal linkage:
// this header is included by more than one source file of the library.
static __global__ void __launch_bounds__(kThreads)
weight_broadcast_kernel(const ServerParams p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int t = blockIdx.x; t < p.tiles_per_worker; t += gridDim.x) {
    const Tile tile = p.tiles[t];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const int idx = r * kRowElems + threadIdx.x * 4;
      if (idx >= tile.count) continue;
      const float4 x4 = ld_f4(p.x + tile.off + idx);
      const float xx[4] = {x4.x, x4.y, x4.z, x4.w};
      broadcast_row(xx, p.kx, p.xbits, p.wcodes, p.wresid, p.wfeedback, tile.off + idx,
                    tile.off + r * kRowElems + warp * 128, lane);
    }
  }
}

// ---------------------------------------------------------------------------
// The fused server pass (Algorithm 2's gather/average/update and the next
// broadcast): for every element, decode the n workers' codes and sum them in
// worker order, divide by n, update x (and m, v when they live here), quantize
// the new x for the broadcast.
//
// GDEC selects how a gradient code becomes a value:
//   G_TERNARY  2-bit codes {0,1,2} <-> {-s, 0, +s}.  The code is moved into the
//              mantissa of a float whose exponent gives its bit position the
//              weight 1 (value 2^E + code); subtracting 2^E + 1 leaves the level
//              index q as a float, and fma(q, s, acc) = fl(acc + q*s) is the same
//              rounding as adding the decoded value because q*s is exact.
//   G_IDENTITY the streams are binary32 values.
//   otherwise  a per-CTA table value[worker][code] = +-fl(s * level) in shared
//              memory, rebuilt when the segment changes.
// ---------------------------------------------------------------------------
constexpr int kMaxLutCodes = 256;

template <bool SERVER_MOMENTS, int GDEC>
__global__ void __launch_bounds__(kThreads)
server_step_kernel(const ServerParams p) {
  extern __shared__ float smem[];
  float* s_scale = smem;                 // [n]
  float* s_lut = smem + p.n;             // [n][1 << gbits]   (table decode only)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int cur_seg = -1;
  for (int t = blockIdx.x; t < p.tiles_per_worker; t += gridDim.x) {
    const Tile tile = p.tiles[t];
    if (tile.seg != cur_seg) {
      __syncthreads();
      cur_seg = tile.seg;
      for (int i = threadIdx.x; i < p.n; i += kThreads)
        s_scale[i] = p.scales[(long long)i * p.S + cur_seg];
      if constexpr (GDEC != G_TERNARY && GDEC != G_IDENTITY) {
        const int ncodes = 1 << p.gbits;
        for (int idx = threadIdx.x; idx < p.n * ncodes; idx += kThreads) {
          const int i = idx / ncodes, code = idx - i * ncodes;
          const float s = p.scales[(long long)i * p.S + cur_seg];
          int q = code - p.L;
          const int c = q < 0 ? -q : q;
          float val = 0.0f;
          if (c != 0 && c <= p.L) {
            float lv;
            if (GDEC == G_FIVE) lv = level_value<G_FIVE>(c, p.k);
            else if (GDEC == G_POW2) lv = level_value<G_POW2>(c, p.k);
            else lv = level_value<G_UNIFORM>(c, p.k);
            const float mag = __fmul_rn(s, lv);
            val = q < 0 ? -mag : mag;
          }
          s_lut[idx] = val;
        }
      }
      __syncthreads();
    }

    bool act[kRows];
    float4 xv[kRows], mv[kRows], vv[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const int idx = r * kRowElems + threadIdx.x * 4;
      act[r] = idx < tile.count;
      if (act[r]) {
        xv[r] = ld_f4(p.x + tile.off + idx);
        if constexpr (SERVER_MOMENTS) {
          mv[r] = ld_f4(p.m + tile.off + idx);
          vv[r] = ld_f4(p.v + tile.off + idx);
        }
      }
    }

    float acc[kRows][4];
#pragma unroll
    for (int r = 0; r < kRows; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.0f;

    if constexpr (GDEC == G_TERNARY) {
      // one byte = this thread's 4 codes of a row
      const unsigned char* cb = p.gcodes + (tile.off >> 2) + threadIdx.x;
#pragma unroll 4
      for (int i = 0; i < p.n; ++i) {
        const float s = s_scale[i];
        const unsigned char* ci = cb + (long long)i * p.gcode_bytes;
        unsigned b[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) b[r] = act[r] ? (unsigned)__ldg(ci + r * (kRowElems / 4)) : 0x55u;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const unsigned bits = (b[r] & (3u << (2 * c))) | ((unsigned)(150 - 2 * c) << 23);
            const float q = __fadd_rn(__uint_as_float(bits), -(exp2i(23 - 2 * c) + 1.0f));
            acc[r][c] = __fmaf_rn(q, s, acc[r][c]);
          }
        }
      }
    } else if constexpr (GDEC == G_IDENTITY) {
      for (int i = 0; i < p.n; ++i) {
        const float* ui = reinterpret_cast<const float*>(p.gcodes + (long long)i * p.gcode_bytes) + tile.off;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          if (!act[r]) continue;
          const float4 u4 = ld_f4_stream(ui + r * kRowElems + threadIdx.x * 4);
          acc[r][0] = __fadd_rn(acc[r][0], u4.x);
          acc[r][1] = __fadd_rn(acc[r][1], u4.y);
          acc[r][2] = __fadd_rn(acc[r][2], u4.z);
          acc[r][3] = __fadd_rn(acc[r][3], u4.w);
        }
      }
    } else {
      const int ncodes = 1 << p.gbits;
      const unsigned cmask = (unsigned)ncodes - 1u;
      for (int i = 0; i < p.n; ++i) {
        const unsigned char* ci = p.gcodes + (long long)i * p.gcode_bytes;
        const float* lut = s_lut + i * ncodes;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          if (!act[r]) continue;
          const long long row_elem = tile.off + r * kRowElems + warp * 128;
          const unsigned f = unpack_row_field(ci + row_elem * p.gbits / 8, p.gbits, lane);
#pragma unroll
          for (int c = 0; c < 4; ++c)
            acc[r][c] = __fadd_rn(acc[r][c], lut[(f >> (c * p.gbits)) & cmask]);
        }
      }
    }

#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      if (!act[r]) continue;
      const int idx = r * kRowElems + threadIdx.x * 4;
      float xx[4] = {xv[r].x, xv[r].y, xv[r].z, xv[r].w};
      if constexpr (SERVER_MOMENTS) {
        float mm[4] = {mv[r].x, mv[r].y, mv[r].z, mv[r].w};
        float vs[4] = {vv[r].x, vv[r].y, vv[r].z, vv[r].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float dhat = __fdiv_rn(acc[r][c], p.nf);
          moments(p.h, dhat, mm[c], vs[c]);
          xx[c] = __fsub_rn(xx[c], adam_step(p.h, mm[c], vs[c], p.alpha));
        }
        st_f4(p.m + tile.off + idx, make_float4(mm[0], mm[1], mm[2], mm[3]));
        st_f4(p.v + tile.off + idx, make_float4(vs[0], vs[1], vs[2], vs[3]));
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) xx[c] = __fsub_rn(xx[c], __fdiv_rn(acc[r][c], p.nf));
      }
      st_f4(p.x + tile.off + idx, make_float4(xx[0], xx[1], xx[2], xx[3]));
      if (p.kx >= 0) {
        broadcast_row(xx, p.kx, p.xbits, p.wcodes, p.wresid, p.wfeedback, tile.off + idx,
                      tile.off + r * kRowElems + warp * 128, lane);
      }
    }
  }
}

}  // namespace qadam
