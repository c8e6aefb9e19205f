// The server pass for ternary and five-level codes as a persistent, warp-specialised
// pipeline.
//
// One CTA per SM loops over 2048-element tiles.  A producer warp brings each
// tile's inputs (x, m, v and the n workers' code runs of 512 or 768 bytes) into a ring of
// shared-memory stages with bulk asynchronous copies that complete on an
// mbarrier; two groups of eight consumer warps take alternate tiles.  A consumer
// warp first finds out which workers have anything but level 0 in its 256 codes
// (one 16-byte load per lane covers a quarter of a worker's codes, a ballot gives
// the answer for eight workers at once), decodes those in worker order, takes the
// tile's x, m, v into registers and hands the stage back to the producer at once;
// the update, the weight quantizer and the stores to global memory follow from
// registers, while the stage is already being refilled.  Global-memory latency is
// covered by the copies in flight (stages x tile bytes per SM), not by occupancy,
// so the consumers keep their registers for arithmetic.
//
// Every wait on an mbarrier is bounded: when a wait runs out the thread raises a
// CTA-wide abort flag and the TIMEOUT bit of the status word, every role leaves
// its loop, outstanding copies are drained and the kernel returns.
#pragma once

#include <cuda.h>

#include "qadam_kernels.cuh"

namespace qadam {

constexpr int kPipeRowElems = 1024;             // a tile is 2 or 4 rows of 1024 elements (4 per consumer thread)
constexpr int kPipeTile = 2 * kPipeRowElems;    // elements per pipeline tile (the default, two rows)
constexpr int kPipeWideTile = 4 * kPipeRowElems;// four rows: decode-bound passes get more work per thread and tile
constexpr int kPipeGroups = 2;                  // consumer groups; group g takes tiles g, g + groups, ...
constexpr int kPipeGroupThreads = 256;          // 8 warps per group, 8 elements per thread and tile
constexpr int kPipeConsumers = kPipeGroups * kPipeGroupThreads;
constexpr int kPipeThreads = kPipeConsumers + 32;   // + producer warp
constexpr int kPipeMaxWorkers = 64;
constexpr int kPipeMaxStages = 16;
constexpr unsigned kSpinLimit = 1u << 22;       // default bound on the polls of one wait

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
// adds to the bytes the current phase waits for, without arriving
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
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
// The same, but the hardware may keep the thread suspended for up to `ns` nanoseconds while
// the phase is incomplete (it resumes at once when the phase completes): a waiting warp then
// takes no issue slots from the warps that have work.
__device__ __forceinline__ bool mbar_try_wait_suspend(unsigned long long* bar, unsigned parity, unsigned ns) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
constexpr unsigned kWaitSuspendNs = 1000;       // per poll; a wait gives up after `limit` polls
// global -> shared, completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes,
                                          unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
// One tiled 2-D tensor copy global -> shared: the box of `map` whose corner is at
// (c0, c1) in elements; completion counted in bytes (always the whole box) on `bar`.
__device__ __forceinline__ void tensor_load_2d(void* smem_dst, const CUtensorMap* map, int c0, int c1,
                                               unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
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
__device__ __forceinline__ void bulk_wait_read_1() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_shared() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Waits for the phase with the given parity; gives up after `limit` polls or
// as soon as another thread has raised the abort flag.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity,
                                                  volatile int* abort_flag, unsigned* status,
                                                  unsigned limit) {
  if (mbar_try_wait(bar, parity)) return true;
  for (unsigned it = 0; it < limit; ++it) {
    if (mbar_try_wait_suspend(bar, parity, kWaitSuspendNs)) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1;
  atomicOr(status, 2u);
  return false;
}

// Tensor map over the n packed code streams of gbits (2 or 3) bits per code, seen as a 2-D
// array of 32-bit words [n rows][gcode_bytes / 4], with a box of one tile's words
// (kPipeTile * gbits / 32) by all n rows: one request brings every worker's codes of a tile, row after row,
// into shared memory.  Encoded through the driver entry point the runtime hands out,
// so the library links against the runtime only.  Returns false if unavailable.
// wide: 64-bit words instead (a box side holds at most 256 elements, which 32-bit words
// exceed from 5 bits per code on); coordinates and extents are then in 8-byte units.
inline bool make_codes_tensor_map(CUtensorMap* map, const void* gcodes, long long gcode_bytes, int n,
                                  int gbits, bool wide = false, int tile_elems = kPipeTile) {
  typedef CUresult (*EncodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr)
    return false;
  const int word = wide ? 8 : 4;
  const cuuint64_t dims[2] = {(cuuint64_t)(gcode_bytes / word), (cuuint64_t)n};
  const cuuint64_t strides[1] = {(cuuint64_t)gcode_bytes};          // bytes between rows
  const cuuint32_t box[2] = {(cuuint32_t)(tile_elems * gbits / (8 * word)), (cuuint32_t)n};
  if (box[0] > 256 || box[1] > 256) return false;
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiled>(fn)(
      map, wide ? CU_TENSOR_MAP_DATA_TYPE_UINT64 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(gcodes), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The ring must hold a multiple of kPipeGroups stages.  A stage is then always served by
// the same consumer group, so a thread that waits on a stage's barrier for use k + 1 has
// itself seen use k complete.  With any other count the groups would alternate on a stage,
// and a group running ahead could ask for the parity of use k + 1 while use k is still in
// flight, which the barrier answers with "complete" (it reports the phase before the
// current one): the group would then work on a stage that has not been loaded.
__host__ __device__ inline int pipe_legal_stages(int stages) {
  return stages / kPipeGroups * kPipeGroups;
}

struct PipeSmem {
  unsigned long long full[kPipeMaxStages];      // producer -> consumers (bytes landed, header and scales written)
  unsigned long long empty[kPipeMaxStages];     // consumers -> producer (the stage has been read out)
  int abort_flag;
};

// A stage: [header 128 B][x tile][m tile][v tile][n code runs of 256 * gbits B][n scales, each stored twice]
struct StageHeader {
  long long off;   // first element of the tile
  int count;       // its length (multiple of 128, at most kPipeTile)
  int tiny;        // five-level codes: some scale is so small that half of it may not be a float
};
constexpr int kStageHeaderBytes = 128;

__host__ __device__ inline size_t pipe_stage_bytes(int n, bool server_moments, int gbits,
                                                   int tile_elems = kPipeTile) {
  const size_t state = (server_moments ? 3 : 1) * (size_t)tile_elems * sizeof(float);
  const size_t codes = (size_t)n * (tile_elems * gbits / 8);
  const size_t scales = ((size_t)n * 2 * sizeof(float) + 127) / 128 * 128;
  return kStageHeaderBytes + state + codes + scales;
}

// v, m updates of Algorithm 1 / 3 on two coordinates at once.  Only the products
// are packed: the assembler fuses a packed multiply that feeds a packed add into one
// fused multiply-add even when both carry an explicit rounding mode (measured), which
// would drop a rounding; the scalar add with explicit rounding is never fused.
__device__ __forceinline__ void moments2(const Hyper& h, float2 g, float2& m, float2& v) {
  const float2 gg = mul2_rn(g, g);
  const float2 tv = mul2_rn(make_float2(h.theta, h.theta), v);
  const float2 og = mul2_rn(make_float2(h.one_minus_theta, h.one_minus_theta), gg);
  const float2 bm = mul2_rn(make_float2(h.beta, h.beta), m);
  const float2 ob = mul2_rn(make_float2(h.one_minus_beta, h.one_minus_beta), g);
  v = make_float2(__fadd_rn(tv.x, og.x), __fadd_rn(tv.y, og.y));
  m = make_float2(__fadd_rn(bm.x, ob.x), __fadd_rn(bm.y, ob.y));
}

// One worker's contribution to the 8 running sums of a consumer thread.
//   sc    (scale, scale) of the worker
//   b0,b1 the thread's code bytes of the tile's two rows (4 two-bit codes each)
// A code c sits in mantissa bits [2c', 2c'+2) of a float whose exponent gives that
// position the weight 1 (value 2^E + code); subtracting 2^E + 1 leaves the level
// index (-1, 0, 1) as a float, and fma(index, scale, sum) = fl(sum + index*scale)
// rounds exactly like adding the decoded value because the product is exact.
// mg[c']: the bit pattern of 2^(23 - 2c'), held in registers that the compiler
// cannot see through, so that (byte & mask) | pattern is one three-input logic
// operation with a single immediate instead of two operations.
template <unsigned MASK_LO, unsigned MASK_HI>
__device__ __forceinline__ float2 code_pair_minus_bias(unsigned b, unsigned mg_lo, unsigned mg_hi,
                                                       float2 k) {
  // {lo, hi} = {(b & MASK_LO) | mg_lo, (b & MASK_HI) | mg_hi}, each one three-input
  // logic operation (truth table 0xEA = (a & b) | c), built straight into the two
  // halves of the packed operand; then the packed subtraction of 2^E + 1.
  unsigned long long r;
  asm("{\n\t.reg .b32 lo, hi;\n\t.reg .b64 t;\n\t"
      "lop3.b32 lo, %1, %2, %3, 0xEA;\n\t"
      "lop3.b32 hi, %1, %4, %5, 0xEA;\n\t"
      "mov.b64 t, {lo, hi};\n\t"
      "add.rn.f32x2 %0, t, %6;\n\t}"
      : "=l"(r)
      : "r"(b), "n"(MASK_LO), "r"(mg_lo), "n"(MASK_HI), "r"(mg_hi), "l"(pack_f2(k)));
  return unpack_f2(r);
}

__device__ __forceinline__ void decode_accumulate(float2 sc, unsigned b0, unsigned b1, float2 k01,
                                                  float2 k23, const unsigned (&mg)[4], float2 (&a)[4]) {
  a[0] = fma2_rn(code_pair_minus_bias<0x03u, 0x0cu>(b0, mg[0], mg[1], k01), sc, a[0]);
  a[1] = fma2_rn(code_pair_minus_bias<0x30u, 0xc0u>(b0, mg[2], mg[3], k23), sc, a[1]);
  a[2] = fma2_rn(code_pair_minus_bias<0x03u, 0x0cu>(b1, mg[0], mg[1], k01), sc, a[2]);
  a[3] = fma2_rn(code_pair_minus_bias<0x30u, 0xc0u>(b1, mg[2], mg[3], k23), sc, a[3]);
}

// The same for 3-bit codes of the five-level grid {0, 1/2, 1} (code = level index + 2).
// A lane's four codes of a row are 12 bits that start at bit 0 (even lanes) or bit 4 (odd
// lanes) of a 16-bit window, so masks and exponents differ between lanes and sit in
// registers.  The exponent gives a code's lowest bit the weight 1/2: the float reads
// 2^E + code / 2, and subtracting 2^E + 1 leaves the level value (-1, -1/2, 0, 1/2, 1).
struct FiveLevelLane {
  unsigned mask[4];   // 7 << position of code c
  unsigned mg[4];     // bit pattern of 2^E, E = 22 - position
  float2 k01, k23;    // -(2^E + 1) for codes 0, 1 and 2, 3
  unsigned zero;      // the 12 bits of four level-0 codes, at the lane's position
  unsigned field;     // the lane's 12 bits
};
__device__ __forceinline__ FiveLevelLane five_level_lane(int lane) {
  FiveLevelLane f;
  const int sh = 4 * (lane & 1);
  float kk[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int pos = sh + 3 * c;
    f.mask[c] = 7u << pos;
    f.mg[c] = (unsigned)(149 - pos) << 23;
    kk[c] = -(exp2i(22 - pos) + 1.0f);
  }
  f.k01 = make_float2(kk[0], kk[1]);
  f.k23 = make_float2(kk[2], kk[3]);
  f.zero = 0x492u << sh;
  f.field = 0xfffu << sh;
  return f;
}
__device__ __forceinline__ float2 level_pair(unsigned w, unsigned m_lo, unsigned mg_lo, unsigned m_hi,
                                             unsigned mg_hi, float2 k) {
  unsigned long long r;
  asm("{\n\t.reg .b32 lo, hi;\n\t.reg .b64 t;\n\t"
      "lop3.b32 lo, %1, %2, %3, 0xEA;\n\t"
      "lop3.b32 hi, %1, %4, %5, 0xEA;\n\t"
      "mov.b64 t, {lo, hi};\n\t"
      "add.rn.f32x2 %0, t, %6;\n\t}"
      : "=l"(r)
      : "r"(w), "r"(m_lo), "r"(mg_lo), "r"(m_hi), "r"(mg_hi), "l"(pack_f2(k)));
  return unpack_f2(r);
}
// One worker's contribution from its 16-bit windows w0, w1 of the tile's two rows.
// EXACT = false: fma(level, scale, sum); the product is exact unless scale / 2 is not a
// float, which the producer rules out per tile.  EXACT = true: the product is rounded
// first, then added (scalar adds: a packed product feeding a packed add would be fused).
template <bool EXACT>
__device__ __forceinline__ void decode_accumulate5(float2 sc, unsigned w0, unsigned w1,
                                                   const FiveLevelLane& f, float2 (&a)[4]) {
  const float2 l0 = level_pair(w0, f.mask[0], f.mg[0], f.mask[1], f.mg[1], f.k01);
  const float2 l1 = level_pair(w0, f.mask[2], f.mg[2], f.mask[3], f.mg[3], f.k23);
  const float2 l2 = level_pair(w1, f.mask[0], f.mg[0], f.mask[1], f.mg[1], f.k01);
  const float2 l3 = level_pair(w1, f.mask[2], f.mg[2], f.mask[3], f.mg[3], f.k23);
  if constexpr (EXACT) {
    const float2 q0 = mul2_rn(l0, sc), q1 = mul2_rn(l1, sc), q2 = mul2_rn(l2, sc), q3 = mul2_rn(l3, sc);
    a[0] = make_float2(__fadd_rn(a[0].x, q0.x), __fadd_rn(a[0].y, q0.y));
    a[1] = make_float2(__fadd_rn(a[1].x, q1.x), __fadd_rn(a[1].y, q1.y));
    a[2] = make_float2(__fadd_rn(a[2].x, q2.x), __fadd_rn(a[2].y, q2.y));
    a[3] = make_float2(__fadd_rn(a[3].x, q3.x), __fadd_rn(a[3].y, q3.y));
  } else {
    a[0] = fma2_rn(l0, sc, a[0]);
    a[1] = fma2_rn(l1, sc, a[1]);
    a[2] = fma2_rn(l2, sc, a[2]);
    a[3] = fma2_rn(l3, sc, a[3]);
  }
}

__device__ __forceinline__ unsigned opaque_u32(unsigned v) {
  unsigned r;
  asm volatile("mov.u32 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}

// Bytes ahead of the stage ring: the barriers and, for the table decode, 256 level values.
constexpr int kPipeBarrierBytes = 512;
static_assert(sizeof(PipeSmem) <= kPipeBarrierBytes, "head of the shared-memory layout");
__host__ __device__ inline size_t pipe_head_bytes(bool table_decode) {
  return kPipeBarrierBytes + (table_decode ? 256 * sizeof(float) : 0);
}

// Slots of the liveness vote.  A warp's codes of one worker are one window per row of the tile
// (16 * gb bytes, i.e. gb pieces of 16 bytes each); a worker gets ROWS * P slots, P the next
// power of two >= gb, so that a ballot holds a whole number of workers.  Slot (row, piece) of
// worker i is lane-slot i * ROWS * P + row * P + piece.
__host__ __device__ constexpr int vote_pieces_pow2(int gb) { return gb <= 2 ? 2 : gb <= 4 ? 4 : 8; }

// Q_x for the grid {-1/2, 0, 1/2} (kx = 0) of 4 consecutive weights of one lane and the
// packed store of the warp's row of 128 two-bit codes (32 bytes): the four codes of a lane
// are one byte; two shuffle steps gather four lanes' bytes into a word, which lanes
// 0, 4, ..., 28 store.  row_dst: address of the row's first code.
// wfeedback_elem (optional): the thread's 4 values of the broadcast's error buffer, see broadcast_row;
// ew_fetched (optional): their old contents, read by the caller ahead of time.
__device__ __forceinline__ void broadcast_row_ternary(const float xin[4], unsigned char* row_dst,
                                                      float* wresid_elem, float* wfeedback_elem,
                                                      const float4* ew_fetched, int lane) {
  float xx[4] = {xin[0], xin[1], xin[2], xin[3]};
  float xq[4];
  if (wfeedback_elem) {
    const float4 ew = ew_fetched ? *ew_fetched : ld_f4(wfeedback_elem);
    xx[0] = __fadd_rn(xx[0], ew.x); xx[1] = __fadd_rn(xx[1], ew.y);
    xx[2] = __fadd_rn(xx[2], ew.z); xx[3] = __fadd_rn(xx[3], ew.w);
  }
  // Level index q = [x > 1/4] - [x < -1/4] (midpoint 1/4, ties toward zero), code = q + 1,
  // taken on the fp32 pipe, which has slots to spare when the integer pipe is busy decoding:
  // sat(x 2^30 - 2^28) is 1 for every float above 1/4 (the smallest such difference times
  // 2^30 is 32) and 0 for 1/4 and below, exactly; likewise for -1/4.  The four codes are
  // gathered by exact multiply-adds (c0 + 4 c1 + 16 c2 + 64 c3 <= 170) and read out of the
  // mantissa of 2^23 + that.
  float cf[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float up, down;
    asm("fma.rn.sat.f32 %0, %1, 0f4E800000, 0fCD800000;" : "=f"(up) : "f"(xx[c]));     // x * 2^30 - 2^28
    asm("fma.rn.sat.f32 %0, %1, 0fCE800000, 0fCD800000;" : "=f"(down) : "f"(xx[c]));   // -x * 2^30 - 2^28
    const float q = __fsub_rn(up, down);
    xq[c] = __fmul_rn(0.5f, q);
    cf[c] = __fadd_rn(q, 1.0f);
  }
  const float packed = __fmaf_rn(__fmaf_rn(__fmaf_rn(cf[3], 4.0f, cf[2]), 4.0f, cf[1]), 4.0f, cf[0]);
  const unsigned field = __float_as_uint(__fadd_rn(packed, 8388608.0f)) & 0xffu;
  if (wresid_elem || wfeedback_elem) {
    const float4 r = make_float4(__fsub_rn(xx[0], xq[0]), __fsub_rn(xx[1], xq[1]),
                                 __fsub_rn(xx[2], xq[2]), __fsub_rn(xx[3], xq[3]));
    if (wresid_elem) st_f4(wresid_elem, r);
    if (wfeedback_elem) st_f4(wfeedback_elem, r);
  }
  unsigned w = field | (__shfl_down_sync(0xffffffffu, field, 1) << 8);
  w |= __shfl_down_sync(0xffffffffu, w, 2) << 16;
  if ((lane & 3) == 0) reinterpret_cast<unsigned*>(row_dst)[lane >> 2] = w;
}

// NW > 0: the worker count, known at compile time (the decode loop is unrolled and
// every shared-memory offset is an immediate).  NW = 0: p.n workers, run-time loop.
// GB: bits per gradient code, 2 (ternary) or 3 (five levels); 0: any grid with p.gbits
// (3..8) bits per code, decoded through a table of the signed level values.
// XB: 2 when the weights are quantized to {-1/2, 0, 1/2} (kx = 0), which gets a path of its
// own; 0: any p.kx, decided at run time.
// ROWS: rows of 1024 elements per tile, 2 or 4 (a thread owns 4 elements of each row).
template <bool SERVER_MOMENTS, int NW, int GB, int XB, int ROWS>
__global__ void __launch_bounds__(kPipeThreads, 1)
server_pipe_kernel(const ServerParams p, const __grid_constant__ CUtensorMap codes_map,
                   const Tile* __restrict__ ptiles, const int num_ptiles, const int stages,
                   const int inv_n_exact) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  PipeSmem* ps = reinterpret_cast<PipeSmem*>(smem_raw);
  static_assert(GB == 0 || GB == 2 || GB == 3, "code widths of the pipelined decode");
  static_assert(XB == 0 || XB == 2, "weight code widths with a path of their own");
  static_assert(ROWS == 2 || ROWS == 4, "rows per tile");
  constexpr int kTile = ROWS * kPipeRowElems;
  unsigned char* stage_base = smem_raw + pipe_head_bytes(GB == 0);
  float* s_lut = reinterpret_cast<float*>(smem_raw + kPipeBarrierBytes);      // table decode only
  const int n = NW > 0 ? NW : p.n;
  const int gb = GB > 0 ? GB : p.gbits;
  const unsigned stage_bytes = (unsigned)pipe_stage_bytes(n, SERVER_MOMENTS, gb, kTile);
  constexpr int kState = SERVER_MOMENTS ? 3 : 1;
  constexpr unsigned kCodesOff = kStageHeaderBytes + kState * kTile * 4;
  const int kRunBytes = kTile * gb / 8;                  // one worker's codes of a tile
  const int kRowBytes = kRunBytes / ROWS;                // of one of its 1024-element rows
  const unsigned scales_off = kCodesOff + (unsigned)n * kRunBytes;
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const unsigned spin = p.spin_limit;

  if constexpr (GB == 0) {
    // signed level value of every code (code = level index + L); codes past 2L never occur
    for (int c = tid; c < 256; c += kPipeThreads) {
      const int q = c - p.L;
      const int a = q < 0 ? -q : q;
      float lv = 0.0f;
      if (a != 0 && a <= p.L)
        lv = p.gmode == G_POW2 ? level_value<G_POW2>(a, p.k)
                               : (p.gmode == G_FIVE ? level_value<G_FIVE>(a, p.k) : level_value<G_UNIFORM>(a, p.k));
      s_lut[c] = q < 0 ? -lv : lv;
    }
  }
  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&ps->full[s], 1);
      mbar_init(&ps->empty[s], kPipeGroupThreads / 32);
    }
    ps->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  volatile int* abort_flag = &ps->abort_flag;
  // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const int my_tiles = (int)blockIdx.x < num_ptiles
                           ? (num_ptiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  if (warp == kPipeConsumers / 32) {
    // ------------------------------------------------------------------ producer
    int cur_seg = -1;
    float sc0 = 0.0f, sc1 = 0.0f;                       // scales of workers lane, lane + 32
    int tiny = 0;
    int s = 0;
    unsigned ph = 0;
    int issued = 0;
    Tile t = my_tiles > 0 ? ptiles[blockIdx.x] : Tile{0, 0, 0};
    for (int j = 0; j < my_tiles; ++j) {
      // next tile's descriptor is fetched while this one is issued
      Tile tn = t;
      if (j + 1 < my_tiles) tn = ptiles[blockIdx.x + (long long)(j + 1) * gridDim.x];
      if (t.seg != cur_seg) {
        cur_seg = t.seg;
        if (lane < n) sc0 = p.scales[(long long)lane * p.S + t.seg];
        if (lane + 32 < n) sc1 = p.scales[(long long)(lane + 32) * p.S + t.seg];
        if (GB == 3) {
          // half of a scale below 2^-120 may fall between floats; such a segment is summed
          // with a rounded product instead of a fused one
          const float lim = exp2i(-120);
          tiny = __any_sync(0xffffffffu, (lane < n && sc0 != 0.0f && sc0 < lim) ||
                                             (lane + 32 < n && sc1 != 0.0f && sc1 < lim));
        }
      }
      // a fresh barrier passes a wait on the parity opposite to its first phase
      bool ok = true;
      if (lane == 0) ok = mbar_wait_bounded(&ps->empty[s], ph ^ 1u, abort_flag, p.status, spin);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      unsigned char* st = stage_base + (size_t)s * stage_bytes;
      float2* s_scale = reinterpret_cast<float2*>(st + scales_off);
      if (lane < n) s_scale[lane] = make_float2(sc0, sc0);
      if (lane + 32 < n) s_scale[lane + 32] = make_float2(sc1, sc1);
      if (lane == 0) {
        StageHeader* hd = reinterpret_cast<StageHeader*>(st);
        hd->off = t.off;
        hd->count = t.count;
        hd->tiny = tiny;
      }
      __syncwarp();
      // one elected lane issues the tile's requests: x, m, v runs and the code box.
      // The box always carries n full rows of kRunBytes (beyond a short tile's length it holds
      // the neighbouring codes or zero fill, which nobody reads).
      if (lane == 0) {
        const unsigned fbytes = (unsigned)t.count * 4u;
        mbar_arrive_expect_tx(&ps->full[s], kState * fbytes + (unsigned)n * kRunBytes);
        float* sx = reinterpret_cast<float*>(st + kStageHeaderBytes);
        bulk_load(sx, p.x + t.off, fbytes, &ps->full[s]);
        if (SERVER_MOMENTS) {
          bulk_load(sx + kTile, p.m + t.off, fbytes, &ps->full[s]);
          bulk_load(sx + 2 * kTile, p.v + t.off, fbytes, &ps->full[s]);
        }
        // coordinate in words of the map: 32-bit (GB > 0) or 64-bit (table decode); the host
        // only selects this kernel when the last tile's coordinate fits an int
        const int c0 = GB > 0 ? (int)(t.off >> 5) * GB : (int)(t.off >> 6) * gb;
        tensor_load_2d(st + kCodesOff, &codes_map, c0, 0, &ps->full[s]);
      }
      ++issued;
      if (++s == stages) { s = 0; ph ^= 1u; }
      t = tn;
    }
    // drain after an abort: nothing may still be landing in shared memory when the CTA exits
    __syncwarp();
    if (lane == 0 && *abort_flag) {
      const int back = issued < stages ? issued : stages;
      int ds = s;
      unsigned dph = ph;
      for (int b = 0; b < back; ++b) {
        if (--ds < 0) { ds = stages - 1; dph ^= 1u; }
        for (unsigned it = 0; it < kSpinLimit; ++it) {
          if (mbar_try_wait(&ps->full[ds], dph)) break;
          __nanosleep(100);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    // Two groups of 8 warps take alternate tiles, so that one group computes while
    // the other waits for its data.  In a tile a thread owns elements 4t..4t+3 of every
    // 1024-element row.  The ring holds a multiple of the group count, so a group steps
    // through its own stages only.
    const int group = tid / kPipeGroupThreads;
    const int gt = tid - group * kPipeGroupThreads;           // 0..255
    const int gwarp = gt >> 5;
    // -(2^E + 1) for the four code positions of a byte (E = 23, 21, 19, 17)
    const float2 k01 = make_float2(-(exp2i(23) + 1.0f), -(exp2i(21) + 1.0f));
    const float2 k23 = make_float2(-(exp2i(19) + 1.0f), -(exp2i(17) + 1.0f));
    const unsigned mg[4] = {opaque_u32(150u << 23), opaque_u32(148u << 23), opaque_u32(146u << 23),
                            opaque_u32(144u << 23)};
    const FiveLevelLane fl = five_level_lane(lane);          // used by the 3-bit decode only
    // the 3-bit decode holds more per worker in registers: unroll it by 8 at most
    constexpr int kUnroll = NW > 0 ? (GB == 0 && NW > 4 ? 4 : (GB == 3 && NW > 8 ? 8 : NW)) : 1;
    // table decode: the lane's 4 codes are the 4 * gb bits from bit 4 * gb * lane of the
    // warp's packed row (16 * gb bytes = 4 * gb words)
    const int tb_word = (4 * gb * lane) >> 5;
    const int tb_next = tb_word + 1 < 4 * gb ? tb_word + 1 : tb_word;
    const int tb_shift = (4 * gb * lane) & 31;
    const unsigned tb_cmask = (1u << gb) - 1u;

    // Liveness vote.  With a max-abs scale most codes are level 0, and a worker whose 256
    // codes in this warp's two rows are all level 0 adds +0 to every sum, which changes
    // nothing (a sum is never -0).  Each lane compares one 16-byte piece of one worker's
    // window with the pattern of level-0 codes; a ballot then tells, for 32 / v_slots workers
    // at once, which have anything to add, and only those are decoded, in increasing worker
    // order (the order of the sum is unchanged).
    const int v_p2 = vote_pieces_pow2(gb);
    const int v_slots = ROWS * v_p2;                          // per worker: 4, 8, 16 or 32
    const int sl_log = v_slots == 4 ? 2 : v_slots == 8 ? 3 : v_slots == 16 ? 4 : 5;
    const int v_slot = lane & (v_slots - 1);
    const int v_row = v_slot / v_p2;
    const int v_piece = v_slot & (v_p2 - 1);
    const bool v_piece_ok = v_piece < gb;
    const int v_worker0 = lane >> sl_log;                     // worker of this lane in ballot 0
    const int v_per_ballot = 32 >> sl_log;                    // workers per ballot
    const int v_off = v_row * kRowBytes + v_piece * 16 + gwarp * 16 * gb;
    const unsigned v_gmask = v_slots == 4 ? 0xfu : v_slots == 8 ? 0xffu : v_slots == 16 ? 0xffffu : 0xffffffffu;
    // level-0 codes (code L) as they sit in the four words of the lane's piece: the window
    // starts on a code boundary, so word j of it is the endless repetition of L in fields of
    // gb bits, read from bit 32 j on
    unsigned kz[4];
    {
      unsigned long long rep = (unsigned long long)p.L;
      for (int width = gb; width < 64; width *= 2) rep |= rep << width;
#pragma unroll
      for (int t = 0; t < 4; ++t) kz[t] = (unsigned)(rep >> ((32 * (4 * v_piece + t)) % gb));
    }
    // per-thread pieces of the output addresses
    float* const gx = p.x + gt * 4;
    float* const gm = SERVER_MOMENTS ? p.m + gt * 4 : nullptr;
    float* const gv = SERVER_MOMENTS ? p.v + gt * 4 : nullptr;
    int dense_tiles_left = 0;         // warp-uniform: tiles for which the search for sparse structure is skipped
    int dense_span = 8;
    int all_live_left = 0;            // warp-uniform: tiles for which even the vote is skipped (every worker decoded)
    int all_live_span = 4;

    int s = group;
    unsigned ph = 0;
    for (int j = group; j < my_tiles; j += kPipeGroups) {
      // every lane waits for itself; the warp then agrees on the outcome so that it never splits
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(&ps->full[s], ph, abort_flag, p.status, spin))) break;
      unsigned char* st = stage_base + (size_t)s * stage_bytes;
      const StageHeader hd = *reinterpret_cast<const StageHeader*>(st);
      const bool act0 = gt * 4 < hd.count;                   // warp-uniform
      auto active = [&](int r) { return r * kPipeRowElems + gt * 4 < hd.count; };   // monotone in r
      float2 a[2 * ROWS];
      float4 x4[ROWS], m4[ROWS], v4[ROWS];
      // the broadcast's own error buffer (optional) is not staged: its values are asked for
      // now and used after the decode, which hides the latency of the plain loads (where the
      // registers allow: two-row tiles with the ternary broadcast; elsewhere they are read in place)
      constexpr bool kFetchEwAhead = XB == 2 && ROWS == 2;
      float4 ew4[ROWS];
      if (kFetchEwAhead && p.wfeedback != nullptr && act0) {
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
          if (active(r)) ew4[r] = ld_f4(p.wfeedback + hd.off + r * kPipeRowElems + gt * 4);
      }
      if (act0) {
        // ternary: the thread's byte of a row; five levels: the first of its two bytes
        // (table decode: the first byte of the warp's packed row)
        const unsigned char* s_codes =
            st + kCodesOff + (GB == 2 ? gt : GB == 3 ? gwarp * 48 + ((lane * 3) >> 1) : gwarp * 16 * gb);
        const bool tiny = GB == 3 && hd.tiny != 0;
        const float2* s_scale = reinterpret_cast<const float2*>(st + scales_off);
#pragma unroll
        for (int c = 0; c < 2 * ROWS; ++c) a[c] = make_float2(0.0f, 0.0f);
        auto window = [&](int i, int r) -> unsigned {       // 3-bit codes: the lane's 16-bit window
          const unsigned char* q = s_codes + i * kRunBytes + r * kRowBytes;
          return (unsigned)q[0] | ((unsigned)q[1] << 8);
        };
        auto field = [&](int i, int r) -> unsigned {         // table decode: the lane's 4 codes
          const unsigned* w = reinterpret_cast<const unsigned*>(s_codes + i * kRunBytes + r * kRowBytes);
          return __funnelshift_r(w[tb_word], w[tb_next], tb_shift);
        };
        // value = fl(scale * signed level), then the rounded add: the decode as defined
        // (rows 2q and 2q + 1 go to accumulators a[4q] .. a[4q + 3]: two per row)
        auto table_accumulate = [&](float sc, unsigned f0, unsigned f1, int q) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float v0 = __fmul_rn(sc, s_lut[(f0 >> (c * gb)) & tb_cmask]);
            const float v1 = __fmul_rn(sc, s_lut[(f1 >> (c * gb)) & tb_cmask]);
            float2& r0 = a[4 * q + (c >> 1)];
            float2& r1 = a[4 * q + 2 + (c >> 1)];
            if (c & 1) { r0.y = __fadd_rn(r0.y, v0); r1.y = __fadd_rn(r1.y, v1); }
            else       { r0.x = __fadd_rn(r0.x, v0); r1.x = __fadd_rn(r1.x, v1); }
          }
        };
        auto row_pair = [&](int q) -> float2(&)[4] { return *reinterpret_cast<float2(*)[4]>(&a[4 * q]); };
        auto contribute = [&](int i) {
          const float2 sc = s_scale[i];
#pragma unroll
          for (int q = 0; q < ROWS / 2; ++q) {
            if constexpr (GB == 2) {
              decode_accumulate(sc, s_codes[i * kRunBytes + 2 * q * kRowBytes],
                                s_codes[i * kRunBytes + (2 * q + 1) * kRowBytes], k01, k23, mg, row_pair(q));
            } else if constexpr (GB == 3) {
              decode_accumulate5<false>(sc, window(i, 2 * q), window(i, 2 * q + 1), fl, row_pair(q));
            } else {
              table_accumulate(sc.x, field(i, 2 * q), field(i, 2 * q + 1), q);
            }
          }
        };
        // ballot b: one bit per slot of workers b * v_per_ballot ... ; a slot beyond the
        // window's pieces or the last worker votes "nothing"
        const unsigned char* v_base = st + kCodesOff + v_off;
        auto vote = [&](int b) -> unsigned {
          const int i = b * v_per_ballot + v_worker0;
          bool nz = false;
          if (v_piece_ok && i < n) {
            const uint4 w = *reinterpret_cast<const uint4*>(v_base + i * kRunBytes);
            nz = (((w.x ^ kz[0]) | (w.y ^ kz[1])) | ((w.z ^ kz[2]) | (w.w ^ kz[3]))) != 0u;
          }
          return __ballot_sync(0xffffffffu, nz);
        };
        auto for_each_live = [&](int b, unsigned bal, auto&& fn) {   // live workers of one ballot, in order
          while (bal) {
            const int g = (__ffs((int)bal) - 1) >> sl_log;
            bal &= ~(v_gmask << (g << sl_log));
            fn(b * v_per_ballot + g);
          }
        };
        if (tiny) {
          // rare: every worker, products rounded before they are added
#pragma unroll 1
          for (int i = 0; i < n; ++i)
#pragma unroll
            for (int q = 0; q < ROWS / 2; ++q)
              decode_accumulate5<true>(s_scale[i], window(i, 2 * q), window(i, 2 * q + 1), fl, row_pair(q));
        } else if constexpr (NW > 0 && GB > 0) {
          constexpr int kSlots = ROWS * vote_pieces_pow2(GB);      // v_slots, at compile time
          constexpr int kBallots = (NW * kSlots + 31) / 32;
          unsigned bal[kBallots];
          int live = 0;
          bool done = false;
          if (all_live_left > 0) {
            // Every worker was live in the last tile looked at (dense codes, as always with the
            // moments on the workers): decoding a worker that has nothing to add is harmless
            // (+0), so for 8, 16, ... 256 tiles the vote itself is left out.
            --all_live_left;
#pragma unroll kUnroll
            for (int i = 0; i < NW; ++i) contribute(i);
            done = true;
          } else {
#pragma unroll
            for (int b = 0; b < kBallots; ++b) {
              bal[b] = vote(b);
              unsigned t = bal[b];                             // folded to one bit per live worker
              t |= t >> 1;
              t |= t >> 2;
              if (kSlots >= 8) t |= t >> 4;
              if (kSlots >= 16) t |= t >> 8;
              live += __popc(t & (kSlots == 4 ? 0x11111111u : kSlots == 8 ? 0x01010101u : 0x00010001u));
            }
            if (live == NW) {
              all_live_span = all_live_span < 256 ? 2 * all_live_span : 256;
              all_live_left = all_live_span;
            } else {
              all_live_span = 4;
            }
          }
          if constexpr (GB == 2 && NW <= 32) if (!done) {
            // Between "a few live workers" and "codes everywhere": a live worker still has
            // level 0 in nearly all of its bytes.  Each lane notes, per row, which live workers
            // have anything in ITS byte; the warp then works in rounds, lane by lane taking its
            // next such worker (increasing worker order per lane, which is all the sum's order
            // asks for: different lanes hold different elements).  A lane with nothing left
            // decodes a byte of level-0 codes, which adds +0.  The rounds are the largest
            // number of such workers any lane has, usually a fraction of the live workers.
            if (live >= 3 && dense_tiles_left <= 0) {
              unsigned mk[ROWS];
#pragma unroll
              for (int r = 0; r < ROWS; ++r) mk[r] = 0u;
#pragma unroll
              for (int b = 0; b < kBallots; ++b)
                for_each_live(b, bal[b], [&](int i) {
#pragma unroll
                  for (int r = 0; r < ROWS; ++r)
                    mk[r] |= (s_codes[i * kRunBytes + r * kRowBytes] != 0x55u ? 1u : 0u) << i;
                });
              int rounds[ROWS], total_rounds = 0;
#pragma unroll
              for (int r = 0; r < ROWS; ++r) {
                rounds[r] = (int)__reduce_max_sync(0xffffffffu, (unsigned)__popc(mk[r]));
                total_rounds += rounds[r];
              }
              if (3 * total_rounds <= ROWS * live) {
                auto round = [&](unsigned& m, int row_off, float2& lo, float2& hi) {
                  const bool has = m != 0u;
                  const int i = has ? __ffs((int)m) - 1 : 0;
                  m &= m - 1u;
                  const unsigned byte = has ? (unsigned)s_codes[i * kRunBytes + row_off] : 0x55u;
                  const float2 sc = s_scale[i];
                  lo = fma2_rn(code_pair_minus_bias<0x03u, 0x0cu>(byte, mg[0], mg[1], k01), sc, lo);
                  hi = fma2_rn(code_pair_minus_bias<0x30u, 0xc0u>(byte, mg[2], mg[3], k23), sc, hi);
                };
#pragma unroll
                for (int r = 0; r < ROWS; ++r)
                  for (int k = 0; k < rounds[r]; ++k) round(mk[r], r * kRowBytes, a[2 * r], a[2 * r + 1]);
                done = true;
                dense_span = 8;
              } else {
                // codes too dense for rounds to pay: stop looking for a while (16, 32, ... 1024 tiles)
                dense_span = dense_span < 1024 ? 2 * dense_span : 1024;
                dense_tiles_left = dense_span;
              }
            }
            --dense_tiles_left;
          }
          if (!done) {
            if (4 * live >= 3 * NW) {
              // nearly every worker has something to add: the unrolled loop over all of them
#pragma unroll kUnroll
              for (int i = 0; i < NW; ++i) contribute(i);
            } else {
#pragma unroll
              for (int b = 0; b < kBallots; ++b) for_each_live(b, bal[b], contribute);
            }
          }
        } else {
          // run-time worker count or code width: ballots taken and served one at a time
          const int nb = (n * v_slots + 31) >> 5;
          for (int b = 0; b < nb; ++b) for_each_live(b, vote(b), contribute);
        }
        // the tile's state into registers; pads beyond the tile's length are not used
        const float* sx = reinterpret_cast<const float*>(st + kStageHeaderBytes) + gt * 4;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
          if (r > 0 && !active(r)) break;
          x4[r] = *reinterpret_cast<const float4*>(sx + r * kPipeRowElems);
          if constexpr (SERVER_MOMENTS) {
            m4[r] = *reinterpret_cast<const float4*>(sx + kTile + r * kPipeRowElems);
            v4[r] = *reinterpret_cast<const float4*>(sx + 2 * kTile + r * kPipeRowElems);
          }
        }
      }
      // everything this warp needs of the stage is in registers: hand it back
      __syncwarp();
      if (lane == 0) mbar_arrive(&ps->empty[s]);
      if (act0) {
        float2 d[2 * ROWS];
        if (inv_n_exact) {
          const float2 inv = make_float2(p.inv_nf, p.inv_nf);
#pragma unroll
          for (int c = 0; c < 2 * ROWS; ++c) d[c] = mul2_rn(a[c], inv);
        } else {
#pragma unroll
          for (int c = 0; c < 2 * ROWS; ++c) d[c] = make_float2(__fdiv_rn(a[c].x, p.nf), __fdiv_rn(a[c].y, p.nf));
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
          if (r > 0 && !active(r)) break;
          const long long e0 = hd.off + r * kPipeRowElems;
          float xx[4];
          if constexpr (SERVER_MOMENTS) {
            float2 m01 = make_float2(m4[r].x, m4[r].y), m23 = make_float2(m4[r].z, m4[r].w);
            float2 v01 = make_float2(v4[r].x, v4[r].y), v23 = make_float2(v4[r].z, v4[r].w);
            moments2(p.h, d[2 * r], m01, v01);
            moments2(p.h, d[2 * r + 1], m23, v23);
            xx[0] = __fsub_rn(x4[r].x, adam_step(p.h, m01.x, v01.x, p.alpha));
            xx[1] = __fsub_rn(x4[r].y, adam_step(p.h, m01.y, v01.y, p.alpha));
            xx[2] = __fsub_rn(x4[r].z, adam_step(p.h, m23.x, v23.x, p.alpha));
            xx[3] = __fsub_rn(x4[r].w, adam_step(p.h, m23.y, v23.y, p.alpha));
            st_f4(gm + e0, make_float4(m01.x, m01.y, m23.x, m23.y));
            st_f4(gv + e0, make_float4(v01.x, v01.y, v23.x, v23.y));
          } else {
            xx[0] = __fsub_rn(x4[r].x, d[2 * r].x);
            xx[1] = __fsub_rn(x4[r].y, d[2 * r].y);
            xx[2] = __fsub_rn(x4[r].z, d[2 * r + 1].x);
            xx[3] = __fsub_rn(x4[r].w, d[2 * r + 1].y);
          }
          st_f4(gx + e0, make_float4(xx[0], xx[1], xx[2], xx[3]));
          if constexpr (XB == 2) {
            broadcast_row_ternary(xx, p.wcodes + ((e0 + gwarp * 128) >> 2),
                                  p.wresid ? p.wresid + e0 + gt * 4 : nullptr,
                                  p.wfeedback ? p.wfeedback + e0 + gt * 4 : nullptr,
                                  kFetchEwAhead ? &ew4[r] : nullptr, lane);
          } else {
            if (p.kx >= 0)
              broadcast_row(xx, p.kx, p.xbits, p.wcodes, p.wresid, p.wfeedback, e0 + gt * 4, e0 + gwarp * 128, lane);
          }
        }
      }
      s += kPipeGroups;
      if (s >= stages) { s -= stages; ph ^= 1u; }
    }
  }
  __syncthreads();
}

}  // namespace qadam
