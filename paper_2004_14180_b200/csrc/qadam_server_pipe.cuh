// The server pass for ternary codes as a persistent, warp-specialised pipeline.
//
// One CTA per SM loops over 2048-element tiles.  A producer warp brings each
// tile's inputs (x, m, v and the n workers' 512-byte code runs) into a ring of
// shared-memory stages with bulk asynchronous copies that complete on an
// mbarrier; sixteen consumer warps decode, average and update in place in shared
// memory and write the packed broadcast; a storer warp sends the updated x, m, v
// back with bulk stores and frees the stage.  Global-memory latency is covered by
// the copies in flight (stages x tile bytes per SM), not by occupancy, so the
// consumers keep their registers for arithmetic.
//
// Every wait on an mbarrier is bounded: when a wait runs out the thread raises a
// CTA-wide abort flag and the TIMEOUT bit of the status word, every role leaves
// its loop, outstanding copies are drained and the kernel returns.
#pragma once

#include "qadam_kernels.cuh"

namespace qadam {

constexpr int kPipeTile = 2048;                 // elements per pipeline tile
constexpr int kPipeConsumers = 512;             // 16 warps, 4 elements per thread
constexpr int kPipeThreads = kPipeConsumers + 64;   // + producer warp + storer warp
constexpr int kPipeMaxWorkers = 64;
constexpr int kPipeMaxStages = 8;
constexpr unsigned kSpinLimit = 1u << 22;

__device__ __forceinline__ unsigned smem_u32(const void* p) {
  return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// global -> shared, completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes,
                                          unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
// shared -> global, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Waits for the phase with the given parity; gives up after kSpinLimit polls or
// as soon as another thread has raised the abort flag.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity,
                                                  volatile int* abort_flag, unsigned* status) {
  for (unsigned it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it >= 32) {
      if (*abort_flag) return false;
      __nanosleep(100);
    }
  }
  *abort_flag = 1;
  atomicOr(status, 2u);
  return false;
}

struct PipeSmem {
  unsigned long long full[kPipeMaxStages];      // producer -> consumers (bytes landed, scales written)
  unsigned long long computed[kPipeMaxStages];  // consumers -> storer
  unsigned long long empty[kPipeMaxStages];     // storer -> producer
  int abort_flag;
};

// Bytes of one stage: x, m, v tiles, the code runs of n workers, n scales.
__host__ __device__ inline size_t pipe_stage_bytes(int n, bool server_moments) {
  const size_t state = (server_moments ? 3 : 1) * (size_t)kPipeTile * sizeof(float);
  const size_t codes = (size_t)n * (kPipeTile / 4);
  const size_t scales = ((size_t)n * sizeof(float) + 127) / 128 * 128;
  return state + codes + scales;
}

template <bool SERVER_MOMENTS>
__global__ void __launch_bounds__(kPipeThreads, 1)
server_pipe_kernel(const ServerParams p, const int stages, const int inv_n_exact) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  PipeSmem* ps = reinterpret_cast<PipeSmem*>(smem_raw);
  unsigned char* stage_base = smem_raw + 256;
  const size_t stage_bytes = pipe_stage_bytes(p.n, SERVER_MOMENTS);
  constexpr int kState = SERVER_MOMENTS ? 3 : 1;
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&ps->full[s], 1);
      mbar_init(&ps->computed[s], kPipeConsumers / 32);
      mbar_init(&ps->empty[s], 1);
    }
    ps->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // Tiles of this CTA: halves h = blockIdx.x, blockIdx.x + gridDim.x, ... of the 4096-element table.
  const long long num_halves = 2LL * p.tiles_per_worker;
  volatile int* abort_flag = &ps->abort_flag;

  auto stage_ptr = [&](int s) { return stage_base + (size_t)s * stage_bytes; };
  auto half_tile = [&](long long h, long long& off, int& count, int& seg) {
    const Tile t = p.tiles[(int)(h >> 1)];
    const int skip = (int)(h & 1) * kPipeTile;
    off = t.off + skip;
    count = t.count - skip;
    count = count > kPipeTile ? kPipeTile : count;
    seg = t.seg;
  };

  if (warp == kPipeConsumers / 32) {
    // ------------------------------------------------------------------ producer
    int cur_seg = -1;
    float sc0 = 0.0f, sc1 = 0.0f;                       // scales of workers lane, lane + 32
    long long j = 0;
    for (long long h = blockIdx.x; h < num_halves; h += gridDim.x) {
      long long off; int count, seg;
      half_tile(h, off, count, seg);
      if (count <= 0) continue;
      const int s = (int)(j % stages);
      const unsigned k = (unsigned)(j / stages);
      if (seg != cur_seg) {
        cur_seg = seg;
        if (lane < p.n) sc0 = p.scales[(long long)lane * p.S + seg];
        if (lane + 32 < p.n) sc1 = p.scales[(long long)(lane + 32) * p.S + seg];
      }
      if (k > 0) {
        bool ok = true;
        if (lane == 0) ok = mbar_wait_bounded(&ps->empty[s], (k - 1) & 1, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
      } else if (*abort_flag) {
        break;
      }
      unsigned char* st = stage_ptr(s);
      float* s_scale = reinterpret_cast<float*>(st + (size_t)kState * kPipeTile * 4 + (size_t)p.n * (kPipeTile / 4));
      if (lane < p.n) s_scale[lane] = sc0;
      if (lane + 32 < p.n) s_scale[lane + 32] = sc1;
      __syncwarp();
      const unsigned fbytes = (unsigned)count * 4u;
      const unsigned cbytes = (unsigned)count / 4u;
      if (lane == 0) mbar_arrive_expect_tx(&ps->full[s], kState * fbytes + (unsigned)p.n * cbytes);
      __syncwarp();
      if (lane == 0) bulk_load(st, p.x + off, fbytes, &ps->full[s]);
      if (SERVER_MOMENTS) {
        if (lane == 1) bulk_load(st + kPipeTile * 4, p.m + off, fbytes, &ps->full[s]);
        if (lane == 2) bulk_load(st + 2 * kPipeTile * 4, p.v + off, fbytes, &ps->full[s]);
      }
      unsigned char* s_codes = st + (size_t)kState * kPipeTile * 4;
      for (int i = lane; i < p.n; i += 32) {
        bulk_load(s_codes + (size_t)i * (kPipeTile / 4), p.gcodes + (long long)i * p.gcode_bytes + (off >> 2),
                  cbytes, &ps->full[s]);
      }
      ++j;
    }
    // drain: nothing may still be landing in shared memory when the CTA exits
    __syncwarp();
    if (lane == 0 && *abort_flag) {
      for (long long jj = (j > stages ? j - stages : 0); jj < j; ++jj) {
        const int s = (int)(jj % stages);
        const unsigned k = (unsigned)(jj / stages);
        for (unsigned it = 0; it < kSpinLimit; ++it) {
          if (mbar_try_wait(&ps->full[s], k & 1)) break;
          __nanosleep(100);
        }
      }
    }
  } else if (warp == kPipeConsumers / 32 + 1) {
    // ------------------------------------------------------------------ storer
    long long j = 0;
    for (long long h = blockIdx.x; h < num_halves; h += gridDim.x) {
      long long off; int count, seg;
      half_tile(h, off, count, seg);
      if (count <= 0) continue;
      const int s = (int)(j % stages);
      const unsigned k = (unsigned)(j / stages);
      bool ok = true;
      if (lane == 0) ok = mbar_wait_bounded(&ps->computed[s], k & 1, abort_flag, p.status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        unsigned char* st = stage_ptr(s);
        const unsigned fbytes = (unsigned)count * 4u;
        bulk_store(p.x + off, st, fbytes);
        if (SERVER_MOMENTS) {
          bulk_store(p.m + off, st + kPipeTile * 4, fbytes);
          bulk_store(p.v + off, st + 2 * kPipeTile * 4, fbytes);
        }
        bulk_commit();
        bulk_wait_read_all();                    // the stage has been read out
        mbar_arrive(&ps->empty[s]);
      }
      ++j;
    }
    if (lane == 0) bulk_wait_all();               // writes are complete before the kernel ends
  } else {
    // ------------------------------------------------------------------ consumers
    long long j = 0;
    for (long long h = blockIdx.x; h < num_halves; h += gridDim.x) {
      long long off; int count, seg;
      half_tile(h, off, count, seg);
      if (count <= 0) continue;
      const int s = (int)(j % stages);
      const unsigned k = (unsigned)(j / stages);
      // every lane waits for itself; the warp then agrees on the outcome so that it never splits
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(&ps->full[s], k & 1, abort_flag, p.status))) break;
      unsigned char* st = stage_ptr(s);
      const bool act = tid * 4 < count;                 // warp-uniform
      if (act) {
        float* sx = reinterpret_cast<float*>(st) + tid * 4;
        const unsigned char* s_codes = st + (size_t)kState * kPipeTile * 4 + tid;
        const float* s_scale = reinterpret_cast<const float*>(st + (size_t)kState * kPipeTile * 4 +
                                                               (size_t)p.n * (kPipeTile / 4));
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 4
        for (int i = 0; i < p.n; ++i) {
          const float sc = s_scale[i];
          const unsigned b = s_codes[(size_t)i * (kPipeTile / 4)];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const unsigned bits = (b & (3u << (2 * c))) | ((unsigned)(150 - 2 * c) << 23);
            const float q = __fadd_rn(__uint_as_float(bits), -(exp2i(23 - 2 * c) + 1.0f));
            acc[c] = __fmaf_rn(q, sc, acc[c]);
          }
        }
        const float4 x4 = *reinterpret_cast<const float4*>(sx);
        float xx[4] = {x4.x, x4.y, x4.z, x4.w};
        float dh[4];
#pragma unroll
        for (int c = 0; c < 4; ++c)
          dh[c] = inv_n_exact ? __fmul_rn(acc[c], p.inv_nf) : __fdiv_rn(acc[c], p.nf);
        if constexpr (SERVER_MOMENTS) {
          float* sm = sx + kPipeTile;
          float* sv = sx + 2 * kPipeTile;
          const float4 m4 = *reinterpret_cast<const float4*>(sm);
          const float4 v4 = *reinterpret_cast<const float4*>(sv);
          float mm[4] = {m4.x, m4.y, m4.z, m4.w};
          float vs[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            moments(p.h, dh[c], mm[c], vs[c]);
            xx[c] = __fsub_rn(xx[c], adam_step(p.h, mm[c], vs[c], p.alpha));
          }
          *reinterpret_cast<float4*>(sm) = make_float4(mm[0], mm[1], mm[2], mm[3]);
          *reinterpret_cast<float4*>(sv) = make_float4(vs[0], vs[1], vs[2], vs[3]);
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) xx[c] = __fsub_rn(xx[c], dh[c]);
        }
        *reinterpret_cast<float4*>(sx) = make_float4(xx[0], xx[1], xx[2], xx[3]);
        if (p.kx >= 0) {
          broadcast_row(xx, p.kx, p.xbits, p.wcodes, p.wresid, off + tid * 4, off + warp * 128, lane);
        }
      }
      fence_async_shared();                              // my writes, before the storer's bulk reads
      __syncwarp();
      if (lane == 0) mbar_arrive(&ps->computed[s]);
      ++j;
    }
  }
  __syncthreads();
}

}  // namespace qadam
