// The worker side (moments on the server) as ONE persistent, warp-specialised kernel
// that keeps L2-sized tensors on chip between its two phases.
//
// The scale of Q_g is a maximum over a whole (worker, segment) pair, so a pair must be
// read completely (phase 1) before any of it can be quantized (phase 2).  Run as two
// launches over everything, phase 2 finds nothing of what phase 1 read in L2.  Here
// the pairs are cut into groups of a few megabytes and the phases are interleaved,
//     P1(G0) P1(G1) P2(G0) P1(G2) P2(G1) ... P2(Glast),
// so that phase 2 of a group runs while its g and e are still in L2: tensors that fit
// are read from HBM once (12.25 instead of 20.25 bytes per element).  A pair larger
// than a group is finished at once, its phase 2 walking backwards over the tail that
// phase 1 has just left in L2.
//
// Work items (one 4096-element tile in one phase) are numbered in that order and
// dealt to the CTAs in chunks of kChunk consecutive items, round-robin; a CTA takes
// its items in increasing order.  One CTA per SM:
//   producer warp   walks the CTA's items and brings each tile's g and e into a ring
//                   of shared-memory stages with bulk copies that complete on an
//                   mbarrier (phase 1 asks L2 to keep the lines, phase 2 to drop them);
//   consumer warps  (two groups of eight taking alternate items) phase 1: max |g + e|
//                   into the stage header; phase 2: wait for the pair's scale,
//                   quantize, write the packed codes, leave e' in the stage;
//   storer warp     phase 1: folds the item's maximum into the CTA's running one and,
//                   at the end of the CTA's streak of tiles of that pair, publishes
//                   maximum and tile count; phase 2: bulk-stores e'; frees the stage.
// A phase-2 item waits until every phase-1 tile of its pair has been counted in
// `done[pair]`.  Those tiles have smaller item numbers and a streak is published as
// soon as its last tile is through, whatever comes next, so the smallest unfinished
// item can always run provided all CTAs are resident, which the cooperative launch
// guarantees.  All waits are bounded: when one runs out the TIMEOUT bit of the status
// word is set and every role leaves its loop.
#pragma once

#include "qadam_server_pipe.cuh"

namespace qadam {

// A run: all tiles of one (worker, segment) pair in one phase, as consecutive items.
struct __align__(8) Run {
  long long first_item;   // number of the run's first work item
  long long seg_off;      // first element of the segment (padded layout)
  int plen;               // padded length of the segment
  int ntiles;             // its tiles of kTileElems elements (the last may be shorter)
  int worker;
  int seg;
  int phase;              // 0: phase 1, 1: phase 2
  int dir;                // +1: tiles ascending, -1: descending
  int keep;               // phase 1: ask L2 to hold on to the lines (phase 2 will find them there)
  int pad;
};

struct WorkerPipeParams {
  WorkerParams w;
  const Run* runs;
  unsigned* done;               // [n][S] phase-1 tiles published, zeroed before the launch
  long long total_items;
  int num_runs;
};

constexpr unsigned kWSpinLimit = 1u << 21;

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

constexpr int kWTile = kTileElems;                  // 4096 elements per item
constexpr int kWGroups = 2;
constexpr int kWGroupThreads = 256;                 // 8 warps x 4 rows x 128 elements
constexpr int kWConsumers = kWGroups * kWGroupThreads;
constexpr int kWProducers = 2;                      // producer warps, taking alternate items
constexpr int kWThreads = kWConsumers + 32 * (kWProducers + 1);   // + producer warps + storer warp
constexpr int kWMaxStages = 6;
constexpr int kChunk = 4;                           // consecutive items a CTA takes per turn (default)
constexpr int kWHeaderBytes = 128;
constexpr int kWStageBytes = kWHeaderBytes + 2 * kWTile * 4;      // header, g tile, e tile

struct WStageHeader {
  long long off;        // first element of the tile (padded layout)
  long long pair;       // worker * S + segment
  int count;            // elements in the tile
  int phase;            // 0 / 1
  int worker;
  int publish;          // phase 1: this item ends the CTA's streak of tiles of `pair`
  unsigned max_bits;    // phase 1: max |u| of the tile, folded in by the consumer warps
  unsigned scale_bits;  // phase 2: the pair's finished scale, fetched by the producer
};

struct WPipeSmem {
  unsigned long long full[kWMaxStages];
  unsigned long long computed[kWMaxStages];
  unsigned long long empty[kWMaxStages];
  int abort_flag;
};

constexpr int kWBarrierBytes = 256;
constexpr int kWRunWindow = 128;                    // run records the producer keeps in shared memory

__host__ __device__ inline size_t wpipe_smem_bytes(int stages) {
  return kWBarrierBytes + sizeof(Run) * kWRunWindow * kWProducers + (size_t)stages * kWStageBytes;
}

// L2 eviction-priority policies for the bulk copies.
__device__ __forceinline__ unsigned long long policy_evict_last() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, unsigned bytes,
                                               unsigned long long* bar, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void* gdst, const void* smem_src, unsigned bytes,
                                                unsigned long long policy) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
               "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy)
               : "memory");
}

// The CTA's j-th item: chunks of kChunk consecutive items, dealt round-robin.
__device__ __forceinline__ long long cta_item(long long j, int cta, int ctas, int chunk) {
  return ((j / chunk) * ctas + cta) * chunk + (j % chunk);
}
// How many items the CTA owns.
__device__ __forceinline__ long long cta_item_count(long long total, int cta, int ctas, int kChunk) {
  const long long chunks = (total + kChunk - 1) / kChunk;
  if (cta >= chunks) return 0;
  const long long mine = (chunks - cta + ctas - 1) / ctas;          // chunks cta, cta + ctas, ...
  const long long last_chunk = cta + (mine - 1) * (long long)ctas;
  const long long in_last = total - last_chunk * kChunk;             // 1..kChunk (or more)
  return (mine - 1) * kChunk + (in_last < kChunk ? in_last : kChunk);
}

template <int MODE>
__global__ void __launch_bounds__(kWThreads, 1)
worker_pipe_kernel(const WorkerPipeParams fp, const int stages, const int chunk) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  WPipeSmem* ps = reinterpret_cast<WPipeSmem*>(smem_raw);
  Run* s_run_all = reinterpret_cast<Run*>(smem_raw + kWBarrierBytes);     // one window per producer warp
  unsigned char* stage_base = smem_raw + kWBarrierBytes + sizeof(Run) * kWRunWindow * kWProducers;
  const WorkerParams& p = fp.w;
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&ps->full[s], 1);
      mbar_init(&ps->computed[s], kWGroupThreads / 32);
      mbar_init(&ps->empty[s], 1);
    }
    ps->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &ps->abort_flag;
  const long long my_items = cta_item_count(fp.total_items, (int)blockIdx.x, (int)gridDim.x, chunk);

  if (warp >= kWConsumers / 32 && warp < kWConsumers / 32 + kWProducers) {
    // ------------------------------------------------------------------ producers
    // Both walk the CTA's whole item list (a cheap, mostly cached lookup); each issues
    // the items of its own parity, so that the per-item cost of one thread (barrier wait,
    // header, copy issue, now and then a poll) is paid twice as fast.
    const int pidx = warp - kWConsumers / 32;
    Run* s_run = s_run_all + pidx * kWRunWindow;
    struct Desc { long long off, pair; int count, phase, worker, need, keep; };
    int win_base = -1, r = 0;
    // Item t -> its tile.  The run records come through a shared-memory window that
    // the warp refills 128 at a time; runs are ordered by first item, so the run of
    // t is found by bisection from the current one onwards.
    Run run = Run{0, 0, 0, 0, 0, 0, 0, 1, 0, 0};       // the run of the last item looked up
    long long run_end = 0;                             // first item after it (0: none yet)
    auto lookup = [&](long long t) -> Desc {
      while (t >= run_end) {                           // only when the item leaves the current run
        if (win_base < 0 || r >= win_base + kWRunWindow - 1) {
          __syncwarp();
          win_base = r;
          for (int i = lane; i < kWRunWindow; i += 32) {
            const int idx = win_base + i;
            if (idx < fp.num_runs) {
              s_run[i] = fp.runs[idx];
            } else {
              Run sentinel = Run{fp.total_items, 0, 0, 0, 0, 0, 0, 1, 0, 0};
              s_run[i] = sentinel;
            }
          }
          __syncwarp();
        }
        int lo = r - win_base, hi = kWRunWindow - 1;
        while (lo < hi) {
          const int mid = (lo + hi + 1) >> 1;
          if (s_run[mid].first_item <= t) lo = mid; else hi = mid - 1;
        }
        r = win_base + lo;
        if (lo < kWRunWindow - 1) {                    // the next record starts after t: found
          run = s_run[lo];
          run_end = s_run[lo + 1].first_item;
        }
      }
      const int k = (int)(t - run.first_item);
      const int ti = run.dir > 0 ? k : run.ntiles - 1 - k;
      Desc d;
      d.off = run.seg_off + (long long)ti * kWTile;
      const int left = run.plen - ti * kWTile;
      d.count = left < kWTile ? left : kWTile;
      d.phase = run.phase;
      d.worker = run.worker;
      d.pair = (long long)run.worker * p.S + run.seg;
      d.need = run.ntiles;
      d.keep = run.keep;
      return d;
    };
    const unsigned long long keep = policy_evict_last(), drop = policy_evict_first();
    int s = 0;
    unsigned ph = 0;
    unsigned armed_mask = 0, armed_par = 0;            // stages this warp has armed, and with which parity
    long long ready_pair = -1;                         // pair whose scale is known to be final
    unsigned ready_scale = 0;
    Desc cur = Desc{0, 0, 0, 0, 0, 0, 0}, next = cur;
    // item numbers of this CTA, advanced without divisions: `within` counts inside a chunk
    long long t_next = (long long)blockIdx.x * chunk;
    int within = 0;
    auto advance = [&]() {
      if (++within == chunk) { within = 0; t_next += (long long)(gridDim.x - 1) * chunk + 1; }
      else t_next += 1;
    };
    if (my_items > 0) { next = lookup(t_next); advance(); }
    for (long long j = 0; j < my_items; ++j) {
      cur = next;
      const bool more = j + 1 < my_items;
      if (more) { next = lookup(t_next); advance(); }
      const int publish = cur.phase == 0 && !(more && next.phase == 0 && next.pair == cur.pair);
      if ((int)(j % kWProducers) != pidx) {            // the other producer's item
        if (++s == stages) { s = 0; ph ^= 1u; }
        continue;
      }
      bool ok = true;
      if (lane == 0) ok = mbar_wait_bounded(&ps->empty[s], ph ^ 1u, abort_flag, p.status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        unsigned char* st = stage_base + (size_t)s * kWStageBytes;
        WStageHeader* hd = reinterpret_cast<WStageHeader*>(st);
        const unsigned bytes = (unsigned)cur.count * 4u;
        // The copies go out first (g and e are inputs nobody has touched yet); the stage is
        // handed to the consumers by the arrive below, once the header is complete.
        mbar_expect_tx(&ps->full[s], 2u * bytes);
        const long long eo = (long long)cur.worker * p.D + cur.off;
        if (cur.phase == 0 && !cur.keep) {
          // phase 1 of a pair too large for L2: plain streaming loads
          bulk_load(st + kWHeaderBytes, p.g + eo, bytes, &ps->full[s]);
          bulk_load(st + kWHeaderBytes + kWTile * 4, p.e + eo, bytes, &ps->full[s]);
        } else {
          const unsigned long long pol = cur.phase == 0 ? keep : drop;
          bulk_load_hint(st + kWHeaderBytes, p.g + eo, bytes, &ps->full[s], pol);
          bulk_load_hint(st + kWHeaderBytes + kWTile * 4, p.e + eo, bytes, &ps->full[s], pol);
        }
        if (cur.phase != 0 && cur.pair != ready_pair) {
          // phase 2 needs the pair's scale: wait until all its phase-1 tiles are published
          ok = false;
          for (unsigned it = 0; it < kWSpinLimit; ++it) {
            if (ld_acquire_u32(fp.done + cur.pair) >= (unsigned)cur.need) { ok = true; break; }
            if (*abort_flag) break;
            __nanosleep(it < 64 ? 40 : 400);
          }
          if (ok) {
            ready_pair = cur.pair;
            ready_scale = __ldcg(p.scale_bits + cur.pair);
            if (ready_scale >= 0x7f800000u) atomicOr(p.status, 1u);
          } else {
            *abort_flag = 1;
            atomicOr(p.status, 2u);
          }
        }
        hd->off = cur.off; hd->pair = cur.pair; hd->count = cur.count; hd->phase = cur.phase;
        hd->worker = cur.worker; hd->publish = publish; hd->max_bits = 0u; hd->scale_bits = ready_scale;
        mbar_arrive(&ps->full[s]);
      }
      armed_mask |= 1u << s;
      armed_par = (armed_par & ~(1u << s)) | (ph << s);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (++s == stages) { s = 0; ph ^= 1u; }
    }
    // drain after an abort: nothing may still be landing in shared memory when the CTA exits
    __syncwarp();
    if (lane == 0 && *abort_flag) {
      for (int ds = 0; ds < stages; ++ds) {
        if (!((armed_mask >> ds) & 1u)) continue;
        for (unsigned it = 0; it < kSpinLimit; ++it) {
          if (mbar_try_wait(&ps->full[ds], (armed_par >> ds) & 1u)) break;
          __nanosleep(100);
        }
      }
    }
  } else if (warp == kWConsumers / 32 + kWProducers) {
    // ------------------------------------------------------------------ storer
    int s = 0;
    unsigned ph = 0;
    unsigned acc_max = 0, acc_cnt = 0;
    int owed_stage = -1;                               // stage of the last e' store, not yet freed
    const unsigned long long drop = policy_evict_first();
    for (long long j = 0; j < my_items; ++j) {
      bool ok = true;
      if (lane == 0) ok = mbar_wait_bounded(&ps->computed[s], ph, abort_flag, p.status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        unsigned char* st = stage_base + (size_t)s * kWStageBytes;
        const WStageHeader hd = *reinterpret_cast<const WStageHeader*>(st);
        if (hd.phase == 0) {
          if (owed_stage >= 0) {                       // an earlier e' store: surely read out by now
            bulk_wait_read_all();
            mbar_arrive(&ps->empty[owed_stage]);
            owed_stage = -1;
          }
          mbar_arrive(&ps->empty[s]);                  // nothing of the stage is needed any more
          acc_max = max(acc_max, hd.max_bits);
          acc_cnt += 1;
          if (hd.publish) {
            // the maximum first, then the count that lets phase 2 of this pair go
            if (acc_max) atomicMax(p.scale_bits + hd.pair, acc_max);
            __threadfence();
            atomicAdd(fp.done + hd.pair, acc_cnt);
            acc_max = 0;
            acc_cnt = 0;
          }
        } else {
          // e' goes back with a bulk store; the stage is freed one item later, when the
          // copy engine has certainly read it, so that this warp never sits in the wait
          bulk_store_hint(p.e + (long long)hd.worker * p.D + hd.off, st + kWHeaderBytes + kWTile * 4,
                          (unsigned)hd.count * 4u, drop);
          bulk_commit();
          if (owed_stage >= 0) {
            bulk_wait_read_1();                        // all but the store just issued
            mbar_arrive(&ps->empty[owed_stage]);
          }
          owed_stage = s;
        }
      }
      if (++s == stages) { s = 0; ph ^= 1u; }
    }
    if (lane == 0) {
      if (owed_stage >= 0) {
        bulk_wait_read_all();
        mbar_arrive(&ps->empty[owed_stage]);
      }
      bulk_wait_all();
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const int group = tid / kWGroupThreads;
    const int gt = tid - group * kWGroupThreads;
    const int gwarp = gt >> 5;
    int s = 0;
    unsigned ph = 0;
    for (long long j = 0; j < my_items; ++j) {
      if ((int)(j % kWGroups) == group) {
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(&ps->full[s], ph, abort_flag, p.status))) break;
        unsigned char* st = stage_base + (size_t)s * kWStageBytes;
        WStageHeader* hdp = reinterpret_cast<WStageHeader*>(st);
        const WStageHeader hd = *hdp;
        const float* sg = reinterpret_cast<const float*>(st + kWHeaderBytes) + gt * 4;
        float* se = reinterpret_cast<float*>(st + kWHeaderBytes + kWTile * 4) + gt * 4;
        if (hd.phase == 0) {
          unsigned mx = 0;
#pragma unroll
          for (int q = 0; q < kRows; ++q) {
            if (q * kRowElems + gt * 4 < hd.count) {
              const float4 g4 = *reinterpret_cast<const float4*>(sg + q * kRowElems);
              const float4 e4 = *reinterpret_cast<const float4*>(se + q * kRowElems);
              mx = max(mx, __float_as_uint(fabsf(__fadd_rn(g4.x, e4.x))));
              mx = max(mx, __float_as_uint(fabsf(__fadd_rn(g4.y, e4.y))));
              mx = max(mx, __float_as_uint(fabsf(__fadd_rn(g4.z, e4.z))));
              mx = max(mx, __float_as_uint(fabsf(__fadd_rn(g4.w, e4.w))));
            }
          }
          const unsigned wm = warp_max(mx);
          if (lane == 0 && wm) atomicMax(&hdp->max_bits, wm);
        } else {
          const float sc = __uint_as_float(hd.scale_bits);
          unsigned char* cw = p.gcodes + (long long)hd.worker * p.gcode_bytes;
#pragma unroll
          for (int q = 0; q < kRows; ++q) {
            if (q * kRowElems + gt * 4 >= hd.count) continue;          // warp-uniform
            const float4 g4 = *reinterpret_cast<const float4*>(sg + q * kRowElems);
            const float4 e4 = *reinterpret_cast<const float4*>(se + q * kRowElems);
            const float uu[4] = {__fadd_rn(g4.x, e4.x), __fadd_rn(g4.y, e4.y), __fadd_rn(g4.z, e4.z),
                                 __fadd_rn(g4.w, e4.w)};
            unsigned code[4];
            float en[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) code[c] = quantize_grad<MODE>(uu[c], sc, p.k, p.L, en[c]);
            *reinterpret_cast<float4*>(se + q * kRowElems) = make_float4(en[0], en[1], en[2], en[3]);
            const long long row_elem = hd.off + q * kRowElems + gwarp * 128;
            void* dst = cw + row_elem * p.bits / 8;
            if constexpr (MODE == G_TERNARY) {
              pack_row_store<2>(code[0], code[1], code[2], code[3], dst, lane);
            } else if constexpr (MODE == G_FIVE) {
              pack_row_store<3>(code[0], code[1], code[2], code[3], dst, lane);
            } else {
              pack_row_store_rt(p.bits, code[0], code[1], code[2], code[3], dst, lane);
            }
          }
          fence_async_shared();                          // e' before the storer's bulk read
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ps->computed[s]);
      }
      if (++s == stages) { s = 0; ph ^= 1u; }
    }
  }
  __syncthreads();
}

}  // namespace qadam
