/*
 * qadam.h - C interface of the quantized-Adam-with-error-feedback step library
 * for NVIDIA B200 (sm_100a).
 *
 * One context is one parameter-server problem of the paper "Quantized Adam with
 * Error Feedback": a parameter vector x in R^d (Eq. 1), N workers, a gradient
 * quantizer Q_g and a weight quantizer Q_x (Section 5.1), Adam parameters
 * beta, theta, epsilon and a step size alpha_t (Algorithms 1-3).  The N workers
 * are a batch dimension on one GPU; what a worker would send to the server, and
 * what the server would broadcast, are packed device buffers.
 *
 * Conventions
 *  - Every pointer in qadam_buffers, and `g`, is a DEVICE pointer owned by the
 *    caller, 16-byte aligned, valid until qadam_destroy.  The library allocates
 *    and frees no device memory; its scratch space is `workspace`.
 *  - Host pointers are marked "host".
 *  - Calls enqueue work on the context's stream and return without waiting,
 *    unless stated otherwise.
 *  - Return value: QADAM_OK, or a negative qadam_error.  Arguments are checked
 *    before anything is enqueued, so every error but QADAM_ERR_CUDA means that
 *    the call has done nothing.  QADAM_ERR_CUDA (a CUDA call failed) may come
 *    after clears of the scales and of the library's counters, or after the
 *    host-to-device copy of qadam_step_host, have been enqueued; the state
 *    buffers x, m, v, e are untouched unless a kernel was launched, and the
 *    step counter is not advanced.  Conditions found on the device (a
 *    non-finite input, a wait that gave up) set bits of the status word.
 *  - A context is not thread-safe; distinct contexts are independent.
 *
 * Layout ("padded layout")
 *  The parameter vector is a list of segments (tensors).  Segment s starts at
 *  element seg_off[s], the running sum of the previous segments' lengths each
 *  rounded up to a multiple of 128 elements; D is the padded total.  Pad
 *  elements must be 0 in g, x, m, v, e when the context is created and stay 0.
 *  Q_g uses one max-abs scale per (worker, segment); num_segments = 1 is the
 *  paper's literal whole-vector infinity norm.
 *
 * Packed streams
 *  A code is an unsigned integer of b bits; element j of a stream occupies bits
 *  [j*b, (j+1)*b) of the stream read as a little-endian bit string (bit p is bit
 *  p mod 8 of byte p / 8).  Gradient code = level index + L, where the level
 *  index runs over -L..L and L is the number of positive levels of G; weight
 *  code = level index + 2^kx.  Pads carry level index 0.
 *  b_g = ceil(log2(2L+1)) (3 levels: 2 bits, 5 levels: 3 bits), b_x = kx + 2:
 *  the fixed widths behind the "Comm" and "Size" columns of Tables 1-2.
 *  With kg = -1 (Q_g = identity) the "codes" of a worker are the D binary32
 *  values it would send and its scales are 1.
 */
#ifndef QADAM_H_
#define QADAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qadam_ctx qadam_ctx;

/* Where Adam's moments m, v live and what Q_g is applied to.
 *  QADAM_PLACE_WORKER: Algorithms 2-3 as printed.  Each worker keeps its own
 *    m, v, forms alpha_t m/sqrt(v+eps) + e, quantizes THAT, and the server only
 *    averages and subtracts.
 *  QADAM_PLACE_SERVER: the plain distributed Adam the end of Section 3 compares
 *    with.  Each worker quantizes g + e; the server averages the decoded
 *    gradients and runs the moment and parameter updates of Algorithm 1. */
enum { QADAM_PLACE_SERVER = 0, QADAM_PLACE_WORKER = 1 };

/* Reading of the level set G of Section 5.1 for kg >= 2 (identical for kg = 0, 1):
 *  POW2:    {0, 2^-kg, 2^-kg+1, ..., 1}  (as printed: geometric; L = kg + 1)
 *  UNIFORM: {0, 1/2^kg, 2/2^kg, ..., 1}  (the spacing printed for X; L = 2^kg) */
/*  STOCHASTIC (kg = 0 only): not a grid of Section 5.1 but the stochastic ternary operator of
 *    the method that section compares with (TernGrad): coordinate j becomes scale * sign(u_j)
 *    with probability |u_j| / scale and 0 otherwise (unbiased), the scale again max|u| per
 *    (worker, segment).  The coin of padded element j of worker i at step t is word j mod 4
 *    of the Philox4x32-10 block with counter (j/4 low, j/4 high, i, t) and key (seed low, seed
 *    high); level 1 iff (word >> 8) * 2^-24 < fl(|u_j| / scale).  Codes, packing, the error
 *    update and the server side are those of kg = 0. */
enum { QADAM_GRID_POW2 = 0, QADAM_GRID_UNIFORM = 1, QADAM_GRID_STOCHASTIC = 2 };

enum qadam_error {
  QADAM_OK = 0,
  QADAM_ERR_NULL = -1,        /* a required pointer is NULL                         */
  QADAM_ERR_SIZE = -2,        /* d, n, num_segments or a segment length is invalid  */
  QADAM_ERR_LEVEL = -3,       /* kg, kx or grid_g outside the supported range       */
  QADAM_ERR_ALIGN = -4,       /* a device pointer is not 16-byte aligned            */
  QADAM_ERR_WORKSPACE = -5,   /* workspace_bytes is smaller than qadam_query_sizes says */
  QADAM_ERR_STEP = -6,        /* step out of order (see the step functions)         */
  QADAM_ERR_WORKER = -7,      /* worker range outside 0..n                          */
  QADAM_ERR_HYPER = -8,       /* beta/theta outside [0,1), eps <= 0 or a bad step size */
  QADAM_ERR_CUDA = -9,        /* a CUDA call failed; see qadam_last_cuda_error      */
  QADAM_ERR_PLACEMENT = -10,  /* placement is not one of the two values             */
  QADAM_ERR_CAPACITY = -11    /* beyond the fixed capacity of qadam_worker_scales_static */
};

/* Bits of the device status word. */
enum {
  QADAM_ST_NONFINITE = 1u,    /* a max-abs scale was Inf or NaN: outputs of that step are unspecified */
  QADAM_ST_TIMEOUT = 2u       /* a bounded wait inside a kernel ran out and the kernel returned early:
                                 x, m, v, e and the outputs of that step are partly written and the
                                 context cannot continue; restore the state from a copy and create a
                                 new context */
};

typedef struct {
  int64_t d;                  /* logical number of parameters (Eq. 1: x in R^d)                 */
  int32_t n;                  /* N, the number of workers (Algorithms 2-3); 1 gives Algorithm 1 */
  int32_t num_segments;       /* S >= 1                                                          */
  const int64_t* seg_len;     /* host, [S], each >= 1, sum = d; may be NULL when S = 1           */
  int32_t kg;                 /* level parameter of G (Section 5.1), 0 = {-1,0,1}; -1: identity.
                                 Supported: POW2 0..14, UNIFORM 0..6                            */
  int32_t kx;                 /* level parameter of X (Section 5.1), 0..14; -1: no weight
                                 quantization (nothing is broadcast in packed form)             */
  int32_t grid_g;             /* QADAM_GRID_*                                                    */
  int32_t placement;          /* QADAM_PLACE_*                                                   */
  float beta1;                /* beta  of the m update, in [0, 1)                                */
  float beta2;                /* theta of the v update, in [0, 1)                                */
  float eps;                  /* epsilon, > 0, added to v INSIDE the square root                 */
  float lr;                   /* default alpha, used when a step is given a negative lr_t        */
  void* stream;               /* cudaStream_t all work is enqueued on (NULL: the default stream) */
  uint64_t seed;              /* key of the random stream; read only with QADAM_GRID_STOCHASTIC
                                 (the quantizers of Section 5.1 are deterministic)                */
} qadam_config;

/* Which kernels a context uses where it has a choice, and two hooks for tests.  All
 * zero (or a NULL pointer to qadam_create_ex) gives the defaults, which is what
 * qadam_create uses.  Nothing here changes a result: every route computes the same bits.
 *  server_kernel  AUTO: the pipelined server pass (bulk and tensor copies into shared
 *                 memory, one CTA per SM) whenever the codes are at most 8 bits wide and
 *                 n <= 64, else the plain grid-stride kernel.  PLAIN: always the latter.
 *  worker_kernel  AUTO: (worker, segment) pairs that fit in the SMs' shared memory go
 *                 through one persistent kernel that reads g and e once; larger pairs take
 *                 two streaming launches (max-abs, then quantize), and so does everything
 *                 under the stochastic operator.  STREAMING: always the two launches.
 *  hand_over      how the persistent worker kernel passes a pair's scale between CTAs.
 *                 AUTO: one 64-bit word per (pair, CTA) while those fit in 32 MB of
 *                 workspace, else one counter per pair and atomics.  COUNTERS: always the
 *                 latter.
 *  wait_polls     bound on the polls of every wait inside the persistent kernels before
 *                 the kernel gives up with QADAM_ST_TIMEOUT; 0: the default (2^22, seconds).
 *  test_missing_tiles  TESTING ONLY.  The persistent worker kernel is told that every pair
 *                 has this many more tiles than it has, so its waits run out: the way to
 *                 see QADAM_ST_TIMEOUT without a fault.  Leave 0. */
enum { QADAM_SERVER_AUTO = 0, QADAM_SERVER_PLAIN = 1 };
enum { QADAM_WORKER_AUTO = 0, QADAM_WORKER_STREAMING = 1 };
enum { QADAM_HANDOVER_AUTO = 0, QADAM_HANDOVER_COUNTERS = 1 };
typedef struct {
  int32_t server_kernel;      /* QADAM_SERVER_*   */
  int32_t worker_kernel;      /* QADAM_WORKER_*   */
  int32_t hand_over;          /* QADAM_HANDOVER_* */
  uint32_t wait_polls;
  int32_t test_missing_tiles;
  int32_t reserved[3];        /* must be 0 */
} qadam_options;

typedef struct {
  float* x;                   /* [D] master copy x_t, updated in place                            */
  float* m;                   /* first moment:  [D] (PLACE_SERVER) or [n][D] (PLACE_WORKER)       */
  float* v;                   /* second moment: same shape as m                                   */
  float* e;                   /* [n][D] error-feedback buffers e^(i), updated in place            */
  float* scales;              /* [n][S] out: max-abs scale of each (worker, segment)              */
  void* gcodes;               /* [n][gcode_bytes] out: what each worker sends                     */
  void* wcodes;               /* [wcode_bytes] out: packed Q_x(x); may be NULL when kx = -1       */
  float* wresid;              /* [D] out, optional (NULL to skip): x - Q_x(x)                     */
  void* workspace;            /* scratch, workspace_bytes of qadam_query_sizes, 256-byte aligned;
                                 the library keeps tables here between calls: do not touch it   */
  size_t workspace_bytes;
  uint32_t* status;           /* one word; qadam_create clears it                                 */
  float* wfeedback;           /* [D] optional (NULL: off; needs kx >= 0), zeros at creation.  An
                                 error buffer for the broadcast, which the paper does not have
                                 (its server keeps the master copy and forgets what Q_x drops):
                                 what is broadcast becomes Q_x(y), y = x + wfeedback, and
                                 wfeedback <- y - Q_x(y), so that successive broadcasts add up
                                 to the master weights.  x itself is unaffected.  With it,
                                 wresid (if given) receives the new wfeedback                    */
} qadam_buffers;

/* Sizes for a configuration.  Any output pointer may be NULL.
 *  D: padded length; seg_off: host [S] padded segment offsets;
 *  gcode_bytes: bytes ONE worker sends per step (D*b_g/8, or 4*D when kg = -1);
 *  wcode_bytes: bytes of the packed broadcast (D*b_x/8, 0 when kx = -1).
 * Per step the workers send n*(gcode_bytes + 4*S) bytes against 4*d*n unquantized. */
int qadam_query_sizes(const qadam_config* cfg, int64_t* D, int64_t* seg_off,
                      size_t* gcode_bytes, size_t* wcode_bytes, size_t* workspace_bytes);

/* Code widths: b_g for (kg, grid_g) (32 when kg = -1), b_x for kx (0 when kx = -1);
 * negative qadam_error when unsupported. */
int qadam_grad_code_bits(int32_t kg, int32_t grid_g);
int qadam_weight_code_bits(int32_t kx);

/* Creates a context.  The caller has put x_1 into x and zeros into m, v, e
 * (Algorithm 1 / 3: m_0 = v_0 = 0, e_1 = 0).  Writes the library's tables into
 * the workspace (synchronously) and, when kx >= 0, enqueues the first broadcast
 * Q_x(x_1) into wcodes (and wresid), the first line of Algorithm 2's loop. */
int qadam_create(const qadam_config* cfg, const qadam_buffers* bufs, qadam_ctx** out);

/* The same with explicit options (host, may be NULL).  QADAM_ERR_SIZE for an unknown
 * enumerator or a non-zero reserved field. */
int qadam_create_ex(const qadam_config* cfg, const qadam_buffers* bufs, const qadam_options* opt,
                    qadam_ctx** out);

/* Worker side of step `step` (1-based) for workers [worker_begin, worker_begin +
 * worker_count): Algorithm 3, lines from "v = ..." to the error update.
 *   g: [worker_count][D] stochastic gradients of those workers (padded layout).
 *   PLACE_WORKER: v, m updates; u = lr_t*m/sqrt(v+eps) + e.   PLACE_SERVER: u = g + e.
 *   scale = max|u| per segment; codes = nearest level of u/scale in G (ties toward
 *   zero; all-zero segment: level 0), packed; e <- u - scale*level (Algorithm 1's
 *   last line).
 * Steps must be taken in order: `step` must be one more than the last completed
 * server step, and each worker compresses once per step (not checked: compressing
 * a worker twice applies the error feedback twice).
 * lr_t < 0 selects cfg.lr. */
int qadam_worker_compress(qadam_ctx* ctx, int64_t step, const float* g,
                          int32_t worker_begin, int32_t worker_count, float lr_t);

/* Server side of step `step`: Algorithm 2's gather-average-update, then the next
 * broadcast.  Decodes the n streams, delta^ = (sum in worker order 0..n-1)/n,
 *   PLACE_WORKER: x <- x - delta^              (the printed '+' is read as '-')
 *   PLACE_SERVER: v, m updates with delta^ as the gradient; x <- x - lr_t*m/sqrt(v+eps)
 * then, when kx >= 0, wcodes <- packed Q_x(x) (nearest point of the grid of step
 * 2^-(kx+1) on [-1/2, 1/2], clipped, ties toward zero) and wresid <- x - Q_x(x).
 * Requires that all n workers were compressed for `step`. */
int qadam_server_step(qadam_ctx* ctx, int64_t step, float lr_t);

/* The server side of step `step` for a part of the vector: Algorithm 2 when the server
 * is sharded, each shard owning a contiguous range of x (and of m, v under
 * PLACE_SERVER) and receiving, from every worker, the codes of that range ("Gathering
 * all updates").  Elements [elem_begin, elem_end) of the padded layout are served
 * exactly as qadam_server_step serves them: the same sums in the same order, the same
 * bits in x, m, v, wcodes and wresid on that range; nothing outside it is read or
 * written (gcodes: bytes [elem_begin*b_g/8, elem_end*b_g/8) of each worker's stream, and
 * every worker's scales).  Both ends must be tile boundaries, such as the cuts that
 * qadam_shard_cuts returns (any start of a 4096-element tile of a segment, or D), else
 * QADAM_ERR_SIZE.  The caller vouches that all n workers' codes of the range and all
 * scales are in gcodes / scales (compressed here or received from elsewhere): the check of
 * qadam_server_step on the workers compressed by THIS context does not apply.
 * A step served by ranges stays open until qadam_finish_step; ranges of one step must not
 * overlap (not checked: a range served twice is updated twice). */
int qadam_server_step_range(qadam_ctx* ctx, int64_t step, float lr_t, int64_t elem_begin,
                            int64_t elem_end);

/* Closes a step that was served through qadam_server_step_range (here for some ranges,
 * by other processes for the rest): the next worker and server calls expect step + 1.
 * Host call, nothing is enqueued.  QADAM_ERR_STEP unless `step` is the open step. */
int qadam_finish_step(qadam_ctx* ctx, int64_t step);

/* Cuts of the padded vector into `shards` contiguous ranges of nearly equal length for a
 * sharded server: cuts[0] = 0 <= cuts[1] <= ... <= cuts[shards] = D (host array of
 * shards + 1 entries).  Every cut falls on a boundary of the 4096-element tiles the
 * kernels walk (tiles never straddle a segment), so a range is a whole number of tiles
 * and its code bytes are 16-byte aligned in every stream.  With more shards than tiles
 * some ranges are empty.  A function of the configuration only (host call, no device
 * needed): every process of a sharded run computes the same cuts.  QADAM_ERR_SIZE for
 * shards < 1. */
int qadam_shard_cuts(const qadam_config* cfg, int32_t shards, int64_t* cuts);

/* One whole step from HOST memory, for callers whose gradients live on the host:
 * copies g_host ([n][D], host, ideally pinned) into g_stage (device, [n][D],
 * caller-owned) one worker at a time on a copy stream of the context's own (created by
 * the first call), compressing worker i (qadam_worker_compress) while worker i + 1
 * crosses the bus, then runs qadam_server_step and copies the result back to out_host
 * (host): the packed broadcast (wcode_bytes) when kx >= 0, else x (4*D bytes).  Waits
 * for the stream before returning.  out_host may be NULL to skip the read-back.  If a
 * worker's call fails, the workers before it have been compressed: the context cannot
 * continue with this step. */
int qadam_step_host(qadam_ctx* ctx, int64_t step, const float* g_host, float* g_stage,
                    void* out_host, float lr_t);

/* Algorithm 1's step-dependent rates: beta_t and theta_t used by every later call (the
 * moments are updated by the workers under PLACE_WORKER and by the server under
 * PLACE_SERVER, so call it between steps, not between a step's worker and server
 * halves).  The caller computes the schedule, e.g. Assumption 2's theta_t = 1 - theta/t
 * with beta_t in [0, beta]; the base learning rate alpha_t = alpha/sqrt(t) is each call's
 * lr_t.  Host call, nothing is enqueued.  0 <= beta_t < 1 and 0 <= theta_t < 1, else
 * QADAM_ERR_HYPER and nothing changes. */
int qadam_set_moment_rates(qadam_ctx* ctx, float beta_t, float theta_t);

/* The l2 term of Section 5.1 ("l2 regularization with a scalar 5e-4 as the weight decay
 * term"): every later qadam_worker_compress uses g + lambda * w in place of g, where w is
 * the weight vector the workers hold during the step: the broadcast Q_x(x_t) decoded from
 * wcodes (kx >= 0), or x itself (kx = -1).  Rounded as fl(g + fl(lambda * w)).  lambda = 0
 * (the state after qadam_create) switches the term off.  Host call, nothing is enqueued.
 * lambda must be finite and >= 0, else QADAM_ERR_HYPER. */
int qadam_set_regularization(qadam_ctx* ctx, float lambda);

/* Worker scales without any allocation (no counterpart in the paper: a service
 * entry point for callers that cannot allocate device memory at all, such as a
 * process that sizes its device memory once at start-up and forbids cudaMalloc
 * afterwards, and therefore cannot provide the workspace the context-based calls
 * need).
 *   scales[i] = max_j |g[i][j] + e[i][j]|,  i = 0..n-1,
 * i.e. exactly what qadam_worker_compress writes into `scales` for a problem with
 * num_segments = 1 and the moments on the server (bit-identical).  g, e: device,
 * [n][D] binary32, 16-byte aligned, D a multiple of 128 (pads zero); scales: device,
 * [n] out; stream: cudaStream_t.  Enqueues on `stream` and returns.
 * The kernel's scratch (tile table, running maxima) is a fixed 260 KiB array inside
 * the library image, held by every GPU that loads the library until the process
 * ends.  Limits: D <= QADAM_STATIC_MAX_ELEMENTS and n <= QADAM_STATIC_MAX_WORKERS,
 * else QADAM_ERR_CAPACITY and nothing is enqueued.  There is no status word here: a
 * non-finite input shows only as an Inf or NaN scale.  The call allocates and frees
 * nothing.  The first call on each device looks the array's address up; make that
 * first call outside any stream capture.  All calls on a device share the one
 * array (each call rewrites and clears what it uses), so two calls that may overlap
 * on the GPU (different streams, no dependency between them) race: serialise them. */
#define QADAM_STATIC_MAX_ELEMENTS (1ll << 26)
#define QADAM_STATIC_MAX_WORKERS 1024
int qadam_worker_scales_static(const float* g, const float* e, int64_t D, int32_t n,
                               float* scales, void* stream);

/* Waits for the context's stream, then copies the status word to *host_status. */
int qadam_poll_status(qadam_ctx* ctx, uint32_t* host_status);

/* Instrumentation (no counterpart in the paper).  While enabled, every kernel the
 * context launches is bracketed by CUDA events on the context's stream.
 * qadam_profile_read waits for the stream, adds the elapsed device time of the
 * launches since the last read to ms[kind] and their number to launches[kind]
 * (host arrays of QADAM_NUM_KERNELS entries, which the caller zeroes), and
 * forgets them. */
enum {
  QADAM_K_ABSMAX = 0,      /* worker phase 1: form u, max|u| per (worker, segment)  */
  QADAM_K_QUANTIZE = 1,    /* worker phase 2: level indices, packing, e <- u - Q_g(u) */
  QADAM_K_IDENTITY = 2,    /* worker with Q_g = identity                              */
  QADAM_K_SERVER = 3,      /* fused server pass                                       */
  QADAM_K_BROADCAST = 4,   /* stand-alone Q_x(x_1)                                    */
  QADAM_K_WORKER_FUSED = 5,/* both worker phases in one persistent kernel, for the
                              (worker, segment) pairs that fit on chip                */
  QADAM_NUM_KERNELS = 6
};
int qadam_profile_enable(qadam_ctx* ctx, int enable);
int qadam_profile_read(qadam_ctx* ctx, double* ms, int64_t* launches);

/* Instrumentation: how the worker side of this context moves its data when all
 * workers are compressed.  one_pass: padded (worker, element) pairs that
 * belong to (worker, segment) pairs small enough to be held on chip between the
 * max-abs reduction and the quantization (read from HBM once); two_pass: pairs in
 * segments too large for that (read twice).  The sum is n * D. */
int qadam_worker_pass_model(const qadam_ctx* ctx, int64_t* one_pass, int64_t* two_pass);

/* Number of kernels this context has launched since it was created. */
int64_t qadam_launch_count(const qadam_ctx* ctx);

/* Releases the host-side context.  Device buffers stay the caller's. */
int qadam_destroy(qadam_ctx* ctx);

const char* qadam_strerror(int err);

/* The cudaError_t of the last failed CUDA call made through this library (0 if none). */
int qadam_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif  /* QADAM_H_ */
