// The worker side for tensors that fit ON CHIP: one persistent kernel that reads g and e
// (and, with the moments on the workers, m and v) once, keeps u in shared memory until
// the tensor's scale is known, and quantizes from there.  u = g + e with the moments on
// the server, u = alpha m / sqrt(v + eps) + e after the moment updates of Algorithm 3
// with the moments on the workers.
//
// The scale of Q_g is the maximum of |u| over a whole (worker, segment) pair, so no
// element of a pair can be quantized before all of the pair has been read.  Going back
// to memory for the second look costs as much through L2 as from HBM on this machine
// (the path from L2 into an SM carries little more than HBM delivers: measured), so the
// only way to touch each element once is to hold u where it was computed.  Each of the
// 148 SMs keeps a ring of 12 slots of 4096 values (8 when m and v are staged too); a pair
// spread over all SMs may therefore be up to a few million elements long.  Per pair and
// element this moves g, e in and e', the packed code out: 12 + b_g / 8 bytes (28 + b_g / 8
// with m, v read and written), the least the method allows.
//
// The resident tiles of the call's workers are numbered worker-major, t = worker * TR + j
// (j: index in the per-vector list of resident tiles), so the tiles of a pair are
// consecutive.  Tile t belongs to CTA t mod gridDim.x; a CTA takes its tiles in
// increasing order and its i-th tile lives in slot i mod slots.  Per CTA, one per SM:
//   load side    a producer warp brings g into the tile's slot and e (m, v) into a small
//                ring with bulk copies that complete on an mbarrier; consumer warps form u
//                in place, fold max |u| (and write m, v back); a publisher warp adds the
//                CTA's maximum and tile count to the pair's global record;
//   store side   a dispatcher warp waits until all tiles of the pair have been counted
//                (every CTA's, hence the final scale); consumer warps take u out of the
//                slot into registers, free the slot at once, quantize, and write the
//                packed codes and e' straight to global memory.
// The two sides run as independent loops over the CTA's tiles, coupled only by the
// pair records in global memory and the slots' "free" barriers: the load side runs
// ahead of the store side by as many tiles as there are slots, which is what hides the
// latency of the grid-wide hand-over (last load of a pair lands somewhere -> every CTA
// learns the scale).  A pair of a single tile (a bias vector, a block of a block-wise
// scale that fits one tile) skips the global record: the dispatcher takes the maximum
// from the tile's header in shared memory.  No deadlock: a load waits for the store of the tile `slots`
// places earlier in the same CTA, which waits for that tile's pair to be complete, which
// waits for loads of that pair only; a pair gives a CTA fewer tiles than it has slots
// (the host sends larger pairs elsewhere), so those loads wait, in turn, only for
// stores of OLDER pairs, and the oldest unfinished pair can always finish, provided
// every CTA is resident (cooperative launch).  All waits are bounded: when one runs out
// the TIMEOUT bit of the status word is set and every role leaves its loop.
#pragma once

#include "qadam_server_pipe.cuh"

namespace qadam {


__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// A tile of a resident segment (padded layout, one vector).
struct __align__(8) RTile {
  long long off;   // first element
  int count;       // elements, multiple of kAlign, at most kTileElems
  int seg;         // segment
  int need;        // tiles of that segment: what the pair's counter must reach
  int first;       // index of the segment's first tile in the list of resident tiles
};

struct WorkerResidentParams {
  WorkerParams w;
  const RTile* rtiles;    // [TR]
  unsigned* done;         // [n][S] tiles counted per pair, zeroed before the launch (as are the scales)
  unsigned long long* words;  // [n][S][gridDim.x] or nullptr: per (pair, CTA) {tiles : 32, max |u| bits : 32},
                              // zeroed before the launch; when given, it replaces `done` and the atomics
  long long total;        // resident tiles of the call: its workers x TR
  int TR;                 // resident tiles per worker
  int slots;              // slots of the CTA's ring (a pair gives a CTA fewer tiles than this)
  int estages;            // stages of the e ring
};

// 24 consumer warps, split between the two sides by where the arithmetic is: with the
// moments on the server the load side only adds (8 warps, 4 rows of 1024 elements per
// thread and tile) and the store side quantizes (16 warps, 2 rows); with the moments on
// the workers the load side also runs the moment updates, a root and a division per
// element (16 warps) and the store side gets 8; the same 16 / 8 split serves the l2 term,
// whose decode of the held weights is load-side work (measured: 3.59 -> 3.28 ms on the
// BERT-shaped set, while without the term 8 / 16 stays the faster split).
constexpr int kRColThreads = 256;       // threads across a 1024-element row, 4 elements each
constexpr int kRConsumerWarps = 24;
constexpr int kRRoleWarp0 = kRConsumerWarps;      // producer, publisher, dispatcher follow
constexpr int kRThreads = 32 * (kRRoleWarp0 + 3);
__host__ __device__ constexpr int resident_load_warps(bool heavy_load_side) { return heavy_load_side ? 16 : 8; }
constexpr int kRSlotBytes = kTileElems * 4;
constexpr int kRCmds = 4;               // quantize commands in flight
constexpr int kRMaxEStages = 8;
constexpr int kRMaxSlots = 16;
constexpr int kRHeaders = 32;           // ring of tile headers; more than slots + e stages, see the publisher
constexpr int kRHeadBytes = 2048;       // barriers, headers, commands

struct RLoadHeader {       // one per tile in flight on the load side (ring of kRHeaders)
  long long pair;          // worker * S + segment
  int slot;                // where g lands and u stays
  int count;               // elements of the tile
  int publish;             // 1: last tile of the CTA's streak of this pair; 2: the pair is this one tile and
                           // is handed over inside the CTA (nothing to publish or to count)
  unsigned max_bits;       // max |u| of the tile, folded in by the consumer warps
  long long elem;          // worker * D + first element: where m, v go back (moments on the workers)
  long long off;           // first element in the vector: where the held weights are (l2 term)
};
struct RCommand {          // one per quantize command
  long long off;           // first element (padded layout)
  int slot;
  int count;
  int worker;
  unsigned scale_bits;     // the pair's final scale
};

struct RSmem {
  unsigned long long e_full[kRMaxEStages];
  unsigned long long e_empty[kRMaxEStages];
  unsigned long long hd_ready[kRHeaders];     // consumers -> publisher: the tile's maximum is in its header
  unsigned long long slot_free[kRMaxSlots];
  unsigned long long cmd_full[kRCmds];
  unsigned long long cmd_empty[kRCmds];
  RLoadHeader load_hd[kRHeaders];
  RCommand cmd[kRCmds];
  int abort_flag;
};
static_assert(sizeof(RSmem) <= kRHeadBytes, "head of the shared-memory layout");

// A stage of the ring holds the tile's e, and with the moments on the workers its m and v.
__host__ __device__ constexpr int resident_stage_bytes(bool worker_moments) {
  return (worker_moments ? 3 : 1) * kRSlotBytes;
}
__host__ __device__ inline size_t resident_smem_bytes(int slots, int estages, bool worker_moments) {
  return kRHeadBytes + (size_t)slots * kRSlotBytes + (size_t)estages * resident_stage_bytes(worker_moments);
}

// MODE: grid of Q_g; WM: moments on the workers; L2: the l2 term lambda * (held weights) is
// added to g first (the held weights are decoded from the packed broadcast, or read from x);
// WORDS: the hand-over goes through one word per (pair, CTA) (rp.words) instead of one
// counter per pair (rp.done) and atomics.
template <int MODE, bool WM, bool L2, bool WORDS>
__global__ void __launch_bounds__(kRThreads, 1)
worker_resident_kernel(const WorkerResidentParams rp) {
  constexpr int kLWarps = resident_load_warps(WM || L2);    // load-side consumer warps
  constexpr int kQWarps = kRConsumerWarps - kLWarps;        // store-side consumer warps
  constexpr int kLRowStep = kLWarps / 8, kQRowStep = kQWarps / 8;
  constexpr int kStageBytes = resident_stage_bytes(WM);
  extern __shared__ __align__(128) unsigned char smem_raw[];
  RSmem* ps = reinterpret_cast<RSmem*>(smem_raw);
  unsigned char* slot_base = smem_raw + kRHeadBytes;
  unsigned char* ering_base = slot_base + (size_t)rp.slots * kRSlotBytes;
  const WorkerParams& p = rp.w;
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int cta = (int)blockIdx.x, ctas = (int)gridDim.x;
  const int estages = rp.estages;
  const unsigned spin = p.spin_limit;                           // polls of one wait before giving up
  const unsigned pair_spin = spin > 1u ? spin >> 1 : 1u;        // polls of a pair's record

  if (tid == 0) {
    for (int s = 0; s < estages; ++s) {
      mbar_init(&ps->e_full[s], 1);
      mbar_init(&ps->e_empty[s], kLWarps);
    }
    for (int s = 0; s < kRHeaders; ++s) mbar_init(&ps->hd_ready[s], kLWarps);
    for (int s = 0; s < rp.slots; ++s) mbar_init(&ps->slot_free[s], kQWarps);
    for (int s = 0; s < kRCmds; ++s) {
      mbar_init(&ps->cmd_full[s], 1);
      mbar_init(&ps->cmd_empty[s], kQWarps);
    }
    ps->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &ps->abort_flag;
  // the CTA's tiles: t = cta, cta + ctas, ... < total
  const long long my_tiles = cta < rp.total ? (rp.total - cta + ctas - 1) / ctas : 0;

  if (warp == kRRoleWarp0) {
    // ------------------------------------------------------------------ load side: producer
    int s = 0;
    unsigned ph = 0;
    int slot = 0;
    unsigned slot_ph = 0;                  // parity of the number of times the ring of slots has been gone round
    unsigned armed_mask = 0, armed_par = 0;
    bool ok = true;
    long long t = cta;
    int worker = my_tiles > 0 ? (int)(t / rp.TR) : 0;
    int j = my_tiles > 0 ? (int)(t - (long long)worker * rp.TR) : 0;
    RTile cur = my_tiles > 0 ? rp.rtiles[j] : RTile{0, 0, 0, 0, 0};
    for (long long i = 0; i < my_tiles; ++i, t += ctas) {
      // the CTA's next tile, for the end of the streak of tiles of one pair
      int worker_n = worker, jn = j + ctas;
      while (jn >= rp.TR) { jn -= rp.TR; ++worker_n; }
      RTile next = cur;
      const bool has_next = i + 1 < my_tiles;
      if (has_next) next = rp.rtiles[jn];
      const int publish = cur.need == 1 ? 2 : !(has_next && worker_n == worker && next.seg == cur.seg);
      if (lane == 0) {
        // the slot must have been read out by the store side (a fresh barrier passes a wait on
        // the parity opposite to its first phase), the ring stage by the consumers
        ok = mbar_wait_bounded(&ps->slot_free[slot], slot_ph ^ 1u, abort_flag, p.status, spin) &&
             mbar_wait_bounded(&ps->e_empty[s], ph ^ 1u, abort_flag, p.status, spin);
        if (ok) {
          RLoadHeader* hd = &ps->load_hd[i & (kRHeaders - 1)];
          // `worker` counts from the first worker of this call: g holds only the call's
          // workers, every other array all n of them
          hd->pair = (long long)(p.worker_begin + worker) * p.S + cur.seg;
          hd->slot = slot;
          hd->count = cur.count;
          hd->publish = publish;
          hd->max_bits = 0u;
          const unsigned bytes = (unsigned)cur.count * 4u;
          const long long eo = (long long)(p.worker_begin + worker) * p.D + cur.off;
          hd->elem = eo;
          hd->off = cur.off;
          unsigned char* st = ering_base + (size_t)s * kStageBytes;
          mbar_arrive_expect_tx(&ps->e_full[s], (WM ? 4u : 2u) * bytes);
          bulk_load(slot_base + (size_t)slot * kRSlotBytes, p.g + (long long)worker * p.D + cur.off, bytes,
                    &ps->e_full[s]);
          bulk_load(st, p.e + eo, bytes, &ps->e_full[s]);
          if constexpr (WM) {
            bulk_load(st + kRSlotBytes, p.m + eo, bytes, &ps->e_full[s]);
            bulk_load(st + 2 * kRSlotBytes, p.v + eo, bytes, &ps->e_full[s]);
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      armed_mask |= 1u << s;
      armed_par = (armed_par & ~(1u << s)) | (ph << s);
      if (++s == estages) { s = 0; ph ^= 1u; }
      if (++slot == rp.slots) { slot = 0; slot_ph ^= 1u; }
      worker = worker_n;
      j = jn;
      cur = next;
    }
    // drain after an abort: nothing may still be landing in shared memory when the CTA exits
    __syncwarp();
    if (lane == 0 && *abort_flag) {
      for (int ds = 0; ds < estages; ++ds) {
        if (!((armed_mask >> ds) & 1u)) continue;
        for (unsigned it = 0; it < kSpinLimit; ++it) {
          if (mbar_try_wait(&ps->e_full[ds], (armed_par >> ds) & 1u)) break;
          __nanosleep(100);
        }
      }
    }
  } else if (warp == kRRoleWarp0 + 1) {
    // ------------------------------------------------------------------ load side: publisher
    // The publisher may fall behind the consumers (its atomics take a round trip to L2), so
    // it has a barrier and a header per tile in a ring of its own rather than sharing the e
    // stages.  It cannot fall behind by a whole ring: the producer reuses a slot only after
    // the tile that held it has been stored, which needs that tile's pair complete, which
    // needs this warp to have published it, and kRHeaders exceeds the slots.
    unsigned acc_max = 0, acc_cnt = 0;
    if (lane == 0) {
      for (long long i = 0; i < my_tiles; ++i) {
        const int hi = (int)(i & (kRHeaders - 1));
        if (!mbar_wait_bounded(&ps->hd_ready[hi], (unsigned)(i / kRHeaders) & 1u, abort_flag, p.status, spin)) break;
        const RLoadHeader hd = ps->load_hd[hi];
        if (hd.publish == 2) continue;                   // a one-tile pair: the dispatcher reads the header itself
        acc_max = max(acc_max, hd.max_bits);
        acc_cnt += 1;
        if (WORDS && hd.publish) {
          // one word per (pair, CTA): count and maximum travel in a single plain store, so there
          // is nothing to order across locations (the fence is for this CTA's own dispatcher,
          // which will read u out of the slots after seeing the word)
          __threadfence_block();
          st_relaxed_u64(rp.words + hd.pair * ctas + cta, ((unsigned long long)acc_cnt << 32) | acc_max);
          acc_max = 0;
          acc_cnt = 0;
        } else if (hd.publish) {
          // the maximum first, then (fence) the count that lets the store side of this pair go
          if (acc_max) atomicMax(p.scale_bits + hd.pair, acc_max);
          __threadfence();
          atomicAdd(rp.done + hd.pair, acc_cnt);
          acc_max = 0;
          acc_cnt = 0;
        }
      }
    }
  } else if (warp == kRRoleWarp0 + 2) {
    // ------------------------------------------------------------------ store side: dispatcher
    int cs = 0;
    unsigned cph = 0;
    long long ready_pair = -1;
    unsigned ready_scale = 0;
    bool ok = true;
    if (my_tiles > 0) {
      long long t = cta;
      int worker = (int)(t / rp.TR);
      int j = (int)(t - (long long)worker * rp.TR);
      int slot = 0;
      for (long long i = 0; i < my_tiles; ++i) {
        const RTile cur = rp.rtiles[j];
        const long long pair = (long long)(p.worker_begin + worker) * p.S + cur.seg;
        if (pair != ready_pair) {                        // warp-uniform
          ok = false;
          if (cur.need == 1) {
            // The pair is this one tile, which this CTA loaded: its maximum is complete in the
            // tile's header once the load-side warps have arrived there, and nothing has to
            // cross to another CTA.  The header is still the tile's own: the load side runs at
            // most `slots` tiles ahead of this warp, fewer than the ring of headers holds, and
            // for the same reason the barrier's phase is the one the tile armed.
            const int hi = (int)(i & (kRHeaders - 1));
            if (lane == 0) {
              ok = mbar_wait_bounded(&ps->hd_ready[hi], (unsigned)(i / kRHeaders) & 1u, abort_flag, p.status, spin);
              if (ok) {
                ready_scale = ps->load_hd[hi].max_bits;
                p.scale_bits[pair] = ready_scale;
                if (ready_scale >= 0x7f800000u) atomicOr(p.status, 1u);
              }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ready_scale = __shfl_sync(0xffffffffu, ready_scale, 0);
          } else if constexpr (WORDS) {
            // the whole warp gathers the words of the CTAs that hold tiles of the pair:
            // CTAs (t0 + k) mod ctas, k < min(need, ctas), t0 the pair's first tile
            const long long t0 = (long long)worker * rp.TR + cur.first;
            const int c0 = (int)(t0 % ctas);
            const int kmax = cur.need < ctas ? cur.need : ctas;
            const unsigned long long* w = rp.words + pair * ctas;
            unsigned mx = 0;
            if constexpr (WM) {
              // With the moments on the workers the load side is the slower one, so a pair is
              // rarely complete when the dispatcher first asks.  It then waits for the CTA that
              // holds the pair's last tile, as a rule the last to publish, before it gathers: one
              // word polled by one lane.  (All lanes polling all words of the pair is 1 KB per
              // round and CTA, which takes a good part of the L2's bandwidth when many CTAs wait
              // at once.)  Whatever this wait sees, the gather below decides.  With the moments on
              // the server pairs are complete as a rule and the extra round trip costs more than
              // it saves (measured both ways).
              int c_last = c0 + (cur.need - 1) % ctas;
              if (c_last >= ctas) c_last -= ctas;
              if (lane == 0) {
                for (unsigned it = 0; it < pair_spin; ++it) {
                  if (ld_relaxed_u64(w + c_last) != 0ull || *abort_flag) break;
                  __nanosleep(it < 64 ? 40 : 400);
                }
              }
              __syncwarp();
            }
            for (unsigned it = 0; it < pair_spin; ++it) {
              unsigned cnt = 0;
              mx = 0;
              for (int k = lane; k < kmax; k += 32) {
                int c = c0 + k;
                if (c >= ctas) c -= ctas;
                const unsigned long long v = ld_relaxed_u64(w + c);
                cnt += (unsigned)(v >> 32);
                mx = max(mx, (unsigned)v);
              }
              cnt = __reduce_add_sync(0xffffffffu, cnt);
              mx = __reduce_max_sync(0xffffffffu, mx);
              if (cnt >= (unsigned)cur.need) { ok = true; break; }
              // the flag is raised by other warps at any moment: the lanes must agree on
              // what they saw, or some would leave while the rest wait in the next reduction
              if (__any_sync(0xffffffffu, *abort_flag != 0)) break;
              __nanosleep(it < 64 ? 40 : 400);
            }
            __threadfence_block();                       // the words, before u is read out of the slots
            ready_scale = mx;
            if (ok && lane == 0 && c0 == cta) {          // the CTA of the pair's first tile reports the scale
              p.scale_bits[pair] = mx;
              if (mx >= 0x7f800000u) atomicOr(p.status, 1u);
            }
          } else {
            if (lane == 0) {
              for (unsigned it = 0; it < pair_spin; ++it) {
                if (ld_acquire_u32(rp.done + pair) >= (unsigned)cur.need) { ok = true; break; }
                if (*abort_flag) break;
                __nanosleep(it < 64 ? 40 : 400);
              }
              if (ok) {
                ready_scale = __ldcg(p.scale_bits + pair);
                if (ready_scale >= 0x7f800000u) atomicOr(p.status, 1u);
              }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ready_scale = __shfl_sync(0xffffffffu, ready_scale, 0);
          }
          if (!ok) {
            if (lane == 0) {
              if (!*abort_flag) atomicOr(p.status, 2u);
              *abort_flag = 1;
            }
            break;
          }
          ready_pair = pair;
        }
        if (lane == 0) {
          ok = mbar_wait_bounded(&ps->cmd_empty[cs], cph ^ 1u, abort_flag, p.status, spin);
          if (ok) {
            RCommand* cd = &ps->cmd[cs];
            cd->off = cur.off;
            cd->slot = slot;
            cd->count = cur.count;
            cd->worker = p.worker_begin + worker;
            cd->scale_bits = ready_scale;
            mbar_arrive(&ps->cmd_full[cs]);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (++cs == kRCmds) { cs = 0; cph ^= 1u; }
        if (++slot == rp.slots) slot = 0;
        j += ctas;
        while (j >= rp.TR) { j -= rp.TR; ++worker; }
      }
    }
  } else if (warp < kLWarps) {
    // ------------------------------------------------------------------ load side: u into the slot, max |u|
    // thread (row group, column): rows row0, row0 + kLRowStep, ... of the tile, 4 elements at column gt
    const int gt = tid & (kRColThreads - 1);
    const int row0 = tid / kRColThreads;
    int s = 0;
    unsigned ph = 0;
    // l2 term with packed weights of at most 8 bits: the code words of a tile are fetched
    // while the tile before it is processed (and the descriptor of the tile after it is
    // read), so that their latency stays off the path.  hw_*: words of the tile about to be
    // processed, one pair per row of this thread.
    constexpr int kMineL = kRows / kLRowStep;
    // (With the moments on the workers the 16 load-side warps hide that latency themselves,
    // and the extra registers cost more than the fetch ahead gains: measured.)
    const bool pref = L2 && !WM && p.kx >= 0 && p.xbits <= 8;
    unsigned hw_lo[kMineL], hw_hi[kMineL];
    int pj = my_tiles > 0 ? (int)((long long)cta % rp.TR) : 0;      // index of the tile whose descriptor is in `ahead`
    RTile ahead = RTile{0, 0, 0, 0, 0};
    auto step_j = [&]() { pj += ctas; while (pj >= rp.TR) pj -= rp.TR; };
    auto fetch_rows = [&](const RTile& t, unsigned (&lo)[kMineL], unsigned (&hi)[kMineL]) {
#pragma unroll
      for (int r = 0; r < kMineL; ++r) {
        const int q = row0 + r * kLRowStep;
        lo[r] = hi[r] = 0u;
        if (q * kRowElems + gt * 4 < t.count)
          held_fetch8(p, t.off + q * kRowElems + (gt >> 5) * 128, lane, lo[r], hi[r]);
      }
    };
    if (pref && my_tiles > 0) {
      fetch_rows(rp.rtiles[pj], hw_lo, hw_hi);                       // tile 0
      step_j();
      if (my_tiles > 1) ahead = rp.rtiles[pj];                       // descriptor of tile 1
    }
    for (long long i = 0; i < my_tiles; ++i) {
      unsigned nx_lo[kMineL], nx_hi[kMineL];
      if (pref && i + 1 < my_tiles) {
        fetch_rows(ahead, nx_lo, nx_hi);                             // words of tile i + 1
        step_j();
        if (i + 2 < my_tiles) ahead = rp.rtiles[pj];                 // descriptor of tile i + 2
      }
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(&ps->e_full[s], ph, abort_flag, p.status, spin))) break;
      RLoadHeader* hdp = &ps->load_hd[i & (kRHeaders - 1)];
      const int slot = hdp->slot, count = hdp->count;
      float* su = reinterpret_cast<float*>(slot_base + (size_t)slot * kRSlotBytes) + gt * 4;
      const float* se = reinterpret_cast<const float*>(ering_base + (size_t)s * kStageBytes) + gt * 4;
      unsigned mx = 0;
      if constexpr (WM) {
        // Algorithm 3: v, m updates, u = alpha m / sqrt(v + eps) + e; m, v go straight back
        const long long elem = hdp->elem;
        const long long off = hdp->off;
        float4 g4[kRows / kLRowStep], e4[kRows / kLRowStep], m4[kRows / kLRowStep], v4[kRows / kLRowStep];
#pragma unroll
        for (int r = 0; r < kRows / kLRowStep; ++r) {
          const int q = row0 + r * kLRowStep;
          if (q * kRowElems + gt * 4 < count) {
            g4[r] = *reinterpret_cast<const float4*>(su + q * kRowElems);
            e4[r] = *reinterpret_cast<const float4*>(se + q * kRowElems);
            m4[r] = *reinterpret_cast<const float4*>(se + kTileElems + q * kRowElems);
            v4[r] = *reinterpret_cast<const float4*>(se + 2 * kTileElems + q * kRowElems);
          }
        }
#pragma unroll
        for (int r = 0; r < kRows / kLRowStep; ++r) {
          const int q = row0 + r * kLRowStep;
          if (q * kRowElems + gt * 4 >= count) continue;               // warp-uniform
          float gg[4] = {g4[r].x, g4[r].y, g4[r].z, g4[r].w};
          float ee[4] = {e4[r].x, e4[r].y, e4[r].z, e4[r].w};
          if constexpr (L2) {
            if (pref) add_l2_term_fetched(p, lane, hw_lo[r], hw_hi[r], gg);
            else add_l2_term(p, off + q * kRowElems + (gt >> 5) * 128, lane, gg);
          }
          float mm[4] = {m4[r].x, m4[r].y, m4[r].z, m4[r].w};
          float vs[4] = {v4[r].x, v4[r].y, v4[r].z, v4[r].w};
          float uu[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            moments(p.h, gg[c], mm[c], vs[c]);
            uu[c] = __fadd_rn(adam_step(p.h, mm[c], vs[c], p.alpha), ee[c]);
            mx = max(mx, __float_as_uint(fabsf(uu[c])));
          }
          *reinterpret_cast<float4*>(su + q * kRowElems) = make_float4(uu[0], uu[1], uu[2], uu[3]);
          const long long o = elem + q * kRowElems + gt * 4;
          *reinterpret_cast<float4*>(p.m + o) = make_float4(mm[0], mm[1], mm[2], mm[3]);
          *reinterpret_cast<float4*>(p.v + o) = make_float4(vs[0], vs[1], vs[2], vs[3]);
        }
      } else {
#pragma unroll
        for (int r = 0; r < kMineL; ++r) {
          const int q = row0 + r * kLRowStep;
          if (q * kRowElems + gt * 4 < count) {
            const float4 g4 = *reinterpret_cast<const float4*>(su + q * kRowElems);
            const float4 e4 = *reinterpret_cast<const float4*>(se + q * kRowElems);
            float gg[4] = {g4.x, g4.y, g4.z, g4.w};
            if constexpr (L2) {
              if (pref) add_l2_term_fetched(p, lane, hw_lo[r], hw_hi[r], gg);
              else add_l2_term(p, hdp->off + q * kRowElems + (gt >> 5) * 128, lane, gg);
            }
            const float4 u4 = make_float4(__fadd_rn(gg[0], e4.x), __fadd_rn(gg[1], e4.y), __fadd_rn(gg[2], e4.z),
                                          __fadd_rn(gg[3], e4.w));
            *reinterpret_cast<float4*>(su + q * kRowElems) = u4;
            mx = max(mx, __float_as_uint(fabsf(u4.x)));
            mx = max(mx, __float_as_uint(fabsf(u4.y)));
            mx = max(mx, __float_as_uint(fabsf(u4.z)));
            mx = max(mx, __float_as_uint(fabsf(u4.w)));
          }
        }
      }
      const unsigned wm = warp_max(mx);
      if (lane == 0 && wm) atomicMax(&hdp->max_bits, wm);
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&ps->e_empty[s]);                            // the stage has been read: it can be refilled
        mbar_arrive(&ps->hd_ready[i & (kRHeaders - 1)]);         // the header's maximum is complete
      }
      if constexpr (L2) {
#pragma unroll
        for (int r = 0; r < kMineL; ++r) { hw_lo[r] = nx_lo[r]; hw_hi[r] = nx_hi[r]; }
      }
      if (++s == estages) { s = 0; ph ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------------ store side: quantize, pack, e'
    // thread (row group, column): rows row0, row0 + kQRowStep, ... of the tile, 4 elements at column gt
    const int gt = (tid - 32 * kLWarps) & (kRColThreads - 1);          // 0..255
    const int row0 = (tid - 32 * kLWarps) / kRColThreads;
    const int gwarp = gt >> 5;
    constexpr int kMine = kRows / kQRowStep;                            // rows per thread
    int cs = 0;
    unsigned cph = 0;
    for (long long i = 0; i < my_tiles; ++i) {
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(&ps->cmd_full[cs], cph, abort_flag, p.status, spin))) break;
      const RCommand cd = ps->cmd[cs];
      const float* su = reinterpret_cast<const float*>(slot_base + (size_t)cd.slot * kRSlotBytes) + gt * 4;
      // u into registers; from here on neither the slot nor the command is needed
      float4 u4[kMine];
#pragma unroll
      for (int r = 0; r < kMine; ++r) {
        const int q = row0 + r * kQRowStep;
        u4[r] = q * kRowElems + gt * 4 < cd.count ? *reinterpret_cast<const float4*>(su + q * kRowElems)
                                                  : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&ps->slot_free[cd.slot]);
        mbar_arrive(&ps->cmd_empty[cs]);
      }
      const GradScale gs = grad_scale<MODE>(__uint_as_float(cd.scale_bits), p.k);
      unsigned char* cw = p.gcodes + (long long)cd.worker * p.gcode_bytes;
      float* ew = p.e + (long long)cd.worker * p.D + cd.off + gt * 4;
#pragma unroll
      for (int r = 0; r < kMine; ++r) {
        const int q = row0 + r * kQRowStep;
        if (q * kRowElems + gt * 4 >= cd.count) continue;              // warp-uniform
        const float uu[4] = {u4[r].x, u4[r].y, u4[r].z, u4[r].w};
        unsigned code[4];
        float en[4];
        if constexpr (MODE == G_TERNARY) {
          code[0] = quantize_ternary4(uu, gs, en);             // the lane's byte of four codes
        } else if constexpr (MODE == G_FIVE) {
          code[0] = quantize_five4(uu, gs, en);                // the lane's 12 bits of four codes
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) code[c] = quantize_grad<MODE>(uu[c], gs, p.k, p.L, en[c]);
        }
        *reinterpret_cast<float4*>(ew + q * kRowElems) = make_float4(en[0], en[1], en[2], en[3]);
        const long long row_elem = cd.off + q * kRowElems + gwarp * 128;
        void* dst = cw + row_elem * p.bits / 8;
        if constexpr (MODE == G_TERNARY) {
          store_row_of_code_bytes(code[0], dst, lane);
        } else if constexpr (MODE == G_FIVE) {
          pack_row_store_fields<3>(code[0], dst, lane);
        } else {
          pack_row_store_rt(p.bits, code[0], code[1], code[2], code[3], dst, lane);
        }
      }
      if (++cs == kRCmds) { cs = 0; cph ^= 1u; }
    }
  }
  __syncthreads();
}

}  // namespace qadam
