// Quantized Adam with error feedback: the slow CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, single-threaded statement
// of what one parameter-server step computes.  It exists so that the CUDA
// library can be checked against it and so that a CPU baseline can be timed.
// It shares no code, header, table or helper with the CUDA path, and nothing
// in the product imports, links or calls it.
//
// Arithmetic: every floating-point step is ONE IEEE-754 binary32 operation
// (round to nearest even), in the order written here; no fused multiply-add
// (build with -ffp-contract=off, no -ffast-math), division and square root
// correctly rounded, subnormals kept.  The paper does not fix a precision;
// binary32 is the precision the decisions (which level a value rounds to) are
// taken in.
//
// What follows the paper:
//   * Q_g, Q_x and their level sets G, X ........ Section 5.1 (implementation
//     details); contraction / bounded-error properties: Assumptions 2 and 3
//   * moments, step, error feedback ............. Algorithm 1 and Algorithm 3
//   * server average and update ................. Algorithm 2
// Readings taken where the paper is silent or garbled are marked "READING".
//
// Parity status: every function here is pinned by the CPU test-suite (brute
// force over the level set with exact rationals, hand-worked vectors, closed
// forms, invariants, reduction to an independently written generic Adam).
// Unpinned: nothing in this file.  (Which k_g, k_x the paper's tables used is
// not something code can pin; only the byte ratios are.)

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr int64_t kAlign = 128;  // elements; every segment starts on a multiple of this

int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------------------
// Level set G of the gradient quantizer (Section 5.1):
//   G = {-1, ..., -2^-k, 0, 2^-k, 2^-k+1, ..., 1}
// READING (grid): the printed progression 2^-k, 2^-k+1, ..., 1 is geometric
// (grid 0, "POW2": 0 and 2^(c-1-k) for c = 1..k+1).  The weight set X is
// printed as 1/2^k, 2/2^k, ..., 1, a uniform grid; grid 1 ("UNIFORM") offers
// the same spacing for G: c * 2^-k for c = 0..2^k.  Both give {0, 1} for k = 0
// and {0, 1/2, 1} for k = 1.
// ---------------------------------------------------------------------------
struct GradLevels {
  int L = 0;                  // number of positive levels; codes run 0..2L
  int bits = 0;               // fixed width of one code
  std::vector<float> level;   // level[c], c = 0..L   (level[0] = 0, level[L] = 1)
  std::vector<float> mid;     // mid[c] = (level[c-1] + level[c]) / 2, c = 1..L; mid[0] unused
};

int bits_for(int num_codes) {
  int b = 0;
  while ((1 << b) < num_codes) ++b;
  return b;
}

bool make_grad_levels(int kg, int grid, GradLevels* out) {
  if (grid == 2) {                        // stochastic ternary: the level set {0, 1}, kg = 0 only
    if (kg != 0) return false;
    grid = 0;
  }
  if (kg < 0 || kg > 14 || (grid != 0 && grid != 1)) return false;
  GradLevels g;
  if (grid == 1) {
    g.L = 1 << kg;
    g.level.resize(g.L + 1);
    for (int c = 0; c <= g.L; ++c) g.level[c] = std::ldexp((float)c, -kg);
  } else {
    g.L = kg + 1;
    g.level.resize(g.L + 1);
    g.level[0] = 0.0f;
    for (int c = 1; c <= g.L; ++c) g.level[c] = std::ldexp(1.0f, c - 1 - kg);
  }
  g.mid.assign(g.L + 1, 0.0f);
  for (int c = 1; c <= g.L; ++c) {
    // exactly representable: a sum of two dyadic numbers a few binades apart
    g.mid[c] = (float)(((double)g.level[c - 1] + (double)g.level[c]) * 0.5);
  }
  g.bits = bits_for(2 * g.L + 1);   // fixed width: the tables' 3 levels -> 2 bits, 5 -> 3 bits
  *out = g;
  return true;
}

// ---------------------------------------------------------------------------
// Q_g on one segment (Section 5.1):  Q_g(u) = |u|_inf * argmin_{g^ in G^d} |u/|u|_inf - g^|
// The argmin separates per coordinate: each coordinate goes to its nearest level.
// READING (ties): a value exactly half-way between two levels goes to the one
// nearer zero (strict '>' against every midpoint), as in the ternary example
// where only values strictly above |u|_inf / 2 map to |u|_inf.
// READING (zero vector): |u|_inf = 0 gives level 0 everywhere.
//   q[j]     signed level index in -L..L
//   resid[j] = u[j] - Q_g(u)[j], the next error-feedback buffer (Algorithm 1,
//              last line; Algorithm 3, last line)
// ---------------------------------------------------------------------------
void quantize_grad_segment(const float* u, int64_t len, const GradLevels& G,
                           float* scale_out, int32_t* q, float* resid) {
  float s = 0.0f;
  for (int64_t j = 0; j < len; ++j) {
    float a = std::fabs(u[j]);
    if (a > s) s = a;
  }
  *scale_out = s;
  for (int64_t j = 0; j < len; ++j) {
    int c = 0;
    if (s > 0.0f) {
      float y = std::fabs(u[j]) / s;                 // normalised magnitude in [0, 1]
      for (int cc = 1; cc <= G.L; ++cc) c += (y > G.mid[cc]) ? 1 : 0;
    }
    float deq = s * G.level[c];                      // magnitude of the quantized value
    if (u[j] < 0.0f) { deq = -deq; c = -c; }
    if (c == 0) deq = 0.0f;                          // level 0 carries no sign
    q[j] = c;
    resid[j] = u[j] - deq;
  }
}

// Value a received code stands for: scale * level, signed.
float dequantize_grad(int32_t qv, float s, const GradLevels& G) {
  int c = qv < 0 ? -qv : qv;
  float deq = s * G.level[c];
  if (qv < 0) deq = -deq;
  if (qv == 0) deq = 0.0f;
  return deq;
}

// ---------------------------------------------------------------------------
// Philox4x32-10, the counter-based generator of Salmon, Moraes, Dror and Shaw
// ("Parallel random numbers: as easy as 1, 2, 3", SC 2011), written from its
// published definition: a 128-bit counter (four 32-bit words) and a 64-bit key
// (two words) go through ten rounds; a round multiplies words 0 and 2 by two fixed
// odd constants, keeps both halves of the 64-bit products and mixes in the other
// two words and the key; between rounds the key words grow by two Weyl constants
// (the golden ratio and sqrt(3) - 1 in 32-bit fixed point).
// It is the only source of randomness anywhere in this file and is used only by the
// stochastic ternary operator below.
// ---------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = M0 * (uint64_t)c0;
    const uint64_t p1 = M1 * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0;
    k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---------------------------------------------------------------------------
// The stochastic ternary operator of the method Section 5.1 compares with
// (TernGrad): with s = |u|_inf, coordinate j becomes s * sign(u_j) with probability
// |u_j| / s and 0 otherwise, which makes the operator unbiased, E Q(u) = u.
// READING (how the coin is tossed): y = |u_j| / s in binary32; the coin is the top
// 24 bits of one Philox word read as r = bits * 2^-24 in [0, 1); the level is 1 iff
// r < y.  So the arg-max (y = 1) is always kept and a zero is never raised.
// READING (which word): element j of the padded layout takes word j mod 4 of the
// block with counter (low and high half of j / 4, worker, step) and key (low and
// high half of the seed): any element of any worker at any step can be drawn alone.
// ---------------------------------------------------------------------------
void quantize_grad_segment_stochastic(const float* u, int64_t len, int64_t first_elem,
                                      uint64_t seed, uint32_t step, uint32_t worker,
                                      float* scale_out, int32_t* q, float* resid) {
  float s = 0.0f;
  for (int64_t j = 0; j < len; ++j) {
    float a = std::fabs(u[j]);
    if (a > s) s = a;
  }
  *scale_out = s;
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  for (int64_t j = 0; j < len; ++j) {
    int c = 0;
    if (s > 0.0f) {
      const int64_t elem = first_elem + j;
      const uint64_t block = (uint64_t)elem >> 2;
      const uint32_t ctr[4] = {(uint32_t)block, (uint32_t)(block >> 32), worker, step};
      uint32_t words[4];
      philox4x32_10(ctr, key, words);
      const float r = (float)(words[elem & 3] >> 8) * 5.9604644775390625e-08f;   // 2^-24, exact
      const float y = std::fabs(u[j]) / s;
      c = (r < y) ? 1 : 0;
    }
    float deq = (c != 0) ? s : 0.0f;
    if (u[j] < 0.0f) { deq = -deq; c = -c; }
    if (c == 0) deq = 0.0f;
    q[j] = c;
    resid[j] = u[j] - deq;
  }
}

// ---------------------------------------------------------------------------
// Q_x (Section 5.1):  Q_x(x) = 0.5 * argmin_{x^ in X^d} |2x - x^|,
//   X = {-1, ..., -1/2^k, 0, 1/2^k, 2/2^k, ..., 1}
// i.e. the nearest point of a fixed uniform grid of step 2^-(k+1) on [-1/2, 1/2]
// (no scale), values outside clipped to the ends.  Level index c = number of
// half-integers c' - 1/2 (c' = 1..2^k) strictly below y = |x| * 2^(k+1); with
// y = f + frac (f = floor) that count is f + [frac > 1/2], capped at 2^k.
// Ties toward zero, as for Q_g.
// ---------------------------------------------------------------------------
void quantize_weights(const float* x, int64_t len, int kx,
                      int32_t* q, float* xhat, float* resid) {
  const int L = 1 << kx;
  const float up = std::ldexp(1.0f, kx + 1);
  for (int64_t j = 0; j < len; ++j) {
    float y = std::fabs(x[j]) * up;       // exact (power-of-two factor)
    int c;
    if (y >= (float)L) {
      c = L;
    } else {
      float f = std::floor(y);
      float frac = y - f;                 // exact
      c = (int)f + (frac > 0.5f ? 1 : 0);
    }
    if (x[j] < 0.0f) c = -c;
    float xq = std::ldexp((float)c, -(kx + 1));   // exact
    if (q) q[j] = c;
    if (xhat) xhat[j] = xq;
    if (resid) resid[j] = x[j] - xq;
  }
}

// ---------------------------------------------------------------------------
// Fixed-width packing.  Element j holds code[j] in bits [j*b, (j+1)*b) of the
// stream read as one little-endian bit string: bit p of the stream is bit
// (p mod 8) of byte p / 8.  The "Comm" and "Size" columns of Tables 1-2 count
// exactly such fixed-width codes (32 -> 3 -> 2 bits; 32 -> 16 -> 8 bits).
// ---------------------------------------------------------------------------
void pack_bits(const uint32_t* code, int64_t count, int bits, uint8_t* out) {
  std::memset(out, 0, (size_t)((count * bits + 7) / 8));
  for (int64_t j = 0; j < count; ++j) {
    for (int b = 0; b < bits; ++b) {
      int64_t p = j * bits + b;
      if ((code[j] >> b) & 1u) out[p >> 3] |= (uint8_t)(1u << (p & 7));
    }
  }
}

void unpack_bits(const uint8_t* in, int64_t count, int bits, uint32_t* code) {
  for (int64_t j = 0; j < count; ++j) {
    uint32_t c = 0;
    for (int b = 0; b < bits; ++b) {
      int64_t p = j * bits + b;
      if ((in[p >> 3] >> (p & 7)) & 1u) c |= (1u << b);
    }
    code[j] = c;
  }
}

// ---------------------------------------------------------------------------
// Adam pieces ("generic Adam": no bias correction, epsilon inside the root;
// Algorithm 1 / Algorithm 3, the v, m and step lines).
// ---------------------------------------------------------------------------
struct Hyper {
  float beta, theta, eps, one_minus_beta, one_minus_theta;
};

Hyper make_hyper(float beta, float theta, float eps) {
  Hyper h;
  h.beta = beta; h.theta = theta; h.eps = eps;
  h.one_minus_beta = 1.0f - beta;
  h.one_minus_theta = 1.0f - theta;
  return h;
}

inline void moments(const Hyper& h, float g, float* m, float* v) {
  float gg = g * g;
  float a = h.theta * (*v);
  float b = h.one_minus_theta * gg;
  *v = a + b;                                   // v_t = theta v_{t-1} + (1 - theta) g^2
  float c = h.beta * (*m);
  float d = h.one_minus_beta * g;
  *m = c + d;                                   // m_t = beta m_{t-1} + (1 - beta) g
}

inline float adam_step(const Hyper& h, float m, float v, float alpha) {
  float num = alpha * m;
  float den = std::sqrt(v + h.eps);
  return num / den;                             // alpha_t m_t / sqrt(v_t + eps)
}

}  // namespace

// ===========================================================================
// C interface (loaded with ctypes by the tests and the CPU-baseline timer)
// ===========================================================================
extern "C" {

enum { QO_PLACE_SERVER = 0, QO_PLACE_WORKER = 1 };

typedef struct {
  int64_t d;                 // logical elements
  int64_t D;                 // padded elements (qo_layout)
  int32_t n;                 // workers N
  int32_t S;                 // segments (1: one max-abs scale for the whole vector)
  const int64_t* seg_len;    // [S] logical lengths
  const int64_t* seg_off;    // [S] padded start offsets
  int32_t kg;                // -1: Q_g = identity
  int32_t kx;                // -1: Q_x = identity (nothing broadcast in packed form)
  int32_t grid_g;            // 0 POW2, 1 UNIFORM, 2 STOCHASTIC (kg = 0 only: the stochastic ternary operator)
  int32_t placement;         // where m, v live
  float beta, theta, eps;    // beta_t, theta_t of the step at hand (the caller may change them
                             // between steps: Assumption 2's theta_t = 1 - theta/t)
  float weight_decay;        // lambda of the l2 term (Section 5.1); 0: none
  uint64_t seed;             // key of the random stream (stochastic operator only)
} qo_problem;

// Padded layout: segment s starts at the next multiple of 128 elements.
// Returns D.  Pad elements hold 0 in every state buffer and encode level 0.
int64_t qo_layout(int32_t S, const int64_t* seg_len, int64_t* seg_off) {
  int64_t off = 0;
  for (int32_t s = 0; s < S; ++s) {
    if (seg_off) seg_off[s] = off;
    off += round_up(seg_len[s], kAlign);
  }
  return off;
}

int32_t qo_grad_levels(int32_t kg, int32_t grid, float* level_out, int32_t cap) {
  GradLevels G;
  if (!make_grad_levels(kg, grid, &G)) return -1;
  for (int c = 0; c <= G.L && c < cap; ++c) level_out[c] = G.level[c];
  return G.L;
}

int32_t qo_grad_code_bits(int32_t kg, int32_t grid) {
  if (kg < 0) return 32;
  GradLevels G;
  if (!make_grad_levels(kg, grid, &G)) return -1;
  return G.bits;
}

int32_t qo_weight_code_bits(int32_t kx) {
  if (kx < 0) return 32;
  return bits_for((2 << kx) + 1);               // 2^(k+1) + 1 levels -> k + 2 bits
}

int64_t qo_gcode_bytes(const qo_problem* p) {
  return p->D * qo_grad_code_bits(p->kg, p->grid_g) / 8;
}

int64_t qo_wcode_bytes(const qo_problem* p) {
  return p->kx < 0 ? 0 : p->D * qo_weight_code_bits(p->kx) / 8;
}

int32_t qo_quantize_grad_segment(const float* u, int64_t len, int32_t kg, int32_t grid,
                                 float* scale_out, int32_t* q, float* resid) {
  GradLevels G;
  if (!make_grad_levels(kg, grid, &G)) return -1;
  quantize_grad_segment(u, len, G, scale_out, q, resid);
  return 0;
}

void qo_quantize_weights(const float* x, int64_t len, int32_t kx,
                         int32_t* q, float* xhat, float* resid) {
  quantize_weights(x, len, kx, q, xhat, resid);
}

void qo_pack_bits(const uint32_t* code, int64_t count, int32_t bits, uint8_t* out) {
  pack_bits(code, count, bits, out);
}

void qo_unpack_bits(const uint8_t* in, int64_t count, int32_t bits, uint32_t* code) {
  unpack_bits(in, count, bits, code);
}

// ---------------------------------------------------------------------------
// One worker, one step (Algorithm 3; with N = 1 also Algorithm 1).
//   g      [D] this worker's stochastic gradient (pads 0)
//   m, v   [D] this worker's moments        (PLACE_WORKER only, else NULL)
//   e      [D] this worker's error buffer, updated in place
//   scales [S] out: |u|_inf per segment (1 when Q_g is the identity)
//   codes      out: packed stream, qo_gcode_bytes(p) bytes
// PLACE_WORKER (the paper's placement): u = alpha m/sqrt(v+eps) + e
// PLACE_SERVER (plain distributed Adam, which the closing remark of Section 3
//   contrasts with): u = g + e, moments are the server's.
// READING (identity Q_g): the stream is the raw binary32 of u, scale 1, e = 0.
// ---------------------------------------------------------------------------
void qo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

int32_t qo_quantize_grad_segment_stochastic(const float* u, int64_t len, int64_t first_elem,
                                            uint64_t seed, uint32_t step, uint32_t worker,
                                            float* scale_out, int32_t* q, float* resid) {
  quantize_grad_segment_stochastic(u, len, first_elem, seed, step, worker, scale_out, q, resid);
  return 0;
}

// worker, step: this worker's index and the step number (1-based); they only select the
// random stream of the stochastic operator.
int32_t qo_worker_step(const qo_problem* p, const float* g, const float* xhat, float* m, float* v,
                       float* e, float alpha, float* scales, uint8_t* codes,
                       int32_t worker, int64_t step) {
  const Hyper h = make_hyper(p->beta, p->theta, p->eps);
  GradLevels G;
  if (p->kg >= 0 && !make_grad_levels(p->kg, p->grid_g, &G)) return -1;
  if (p->placement == QO_PLACE_WORKER && (!m || !v)) return -2;
  const float lambda = p->weight_decay;
  if (lambda != 0.0f && !xhat) return -3;

  std::vector<float> u;
  std::vector<int32_t> q;
  std::vector<uint32_t> code;
  for (int32_t s = 0; s < p->S; ++s) {
    const int64_t off = p->seg_off[s], len = p->seg_len[s];
    const int64_t plen = round_up(len, kAlign);
    u.assign((size_t)len, 0.0f);
    for (int64_t j = 0; j < len; ++j) {
      const int64_t k = off + j;
      // READING (l2 term): "l2 regularization with a scalar 5e-4 as the weight decay term"
      // (Section 5.1) adds lambda/2 |x|^2 to each worker's loss, i.e. lambda times the weight
      // the worker holds, which is the broadcast Q_x(x_t), to its stochastic gradient.
      float gk = g[k];
      if (lambda != 0.0f) {
        const float term = lambda * xhat[k];
        gk = gk + term;
      }
      if (p->placement == QO_PLACE_WORKER) {
        moments(h, gk, &m[k], &v[k]);
        u[j] = adam_step(h, m[k], v[k], alpha) + e[k];
      } else {
        u[j] = gk + e[k];
      }
    }
    if (p->kg < 0) {
      scales[s] = 1.0f;
      u.resize((size_t)plen, 0.0f);                       // pads are sent as zeros
      std::memcpy(codes + 4 * off, u.data(), sizeof(float) * u.size());
      for (int64_t j = 0; j < len; ++j) e[off + j] = u[j] - u[j];
      continue;
    }
    q.assign((size_t)len, 0);
    if (p->grid_g == 2)
      quantize_grad_segment_stochastic(u.data(), len, off, p->seed, (uint32_t)step, (uint32_t)worker,
                                       &scales[s], q.data(), e + off);
    else
      quantize_grad_segment(u.data(), len, G, &scales[s], q.data(), e + off);
    code.assign((size_t)plen, (uint32_t)G.L);            // pads: level 0
    for (int64_t j = 0; j < len; ++j) code[j] = (uint32_t)(q[j] + G.L);
    pack_bits(code.data(), plen, G.bits, codes + off * G.bits / 8);
  }
  return 0;
}

// ---------------------------------------------------------------------------
// Q_x(x) as the server broadcasts it (Algorithm 2, first line of the loop and
// the output line).  wcodes: qo_wcode_bytes(p) bytes; wresid (optional) [D]:
// x - Q_x(x).
// READING (weight error feedback): the server keeps the full-precision x_t and
// only the broadcast is quantized, so the part Q_x drops is never lost; the
// residual is a derived quantity, written out only when asked for.
// BEYOND THE PAPER (wfeedback, optional): a separate error buffer for the broadcast in
// the manner of Algorithm 1's e for the gradients ("sigma-delta" form): what is sent is
// Q_x(y) with y = x + e^w, and e^w <- y - Q_x(y), so that the quantization error of one
// broadcast is carried into the next instead of being forgotten: the broadcasts then add
// up to the master weights, sum_t Q_x(y_t) + e^w_{T+1} = sum_t x_t + e^w_1.  The master
// copy x is not touched by it.  With a buffer, wresid (if asked for) is the new e^w.
// ---------------------------------------------------------------------------
int32_t qo_broadcast_weights(const qo_problem* p, const float* x, uint8_t* wcodes, float* wresid,
                             float* wfeedback) {
  if (p->kx < 0) return 0;
  const int bits = qo_weight_code_bits(p->kx);
  const int L = 1 << p->kx;
  std::vector<int32_t> q;
  std::vector<uint32_t> code;
  std::vector<float> y, r;
  for (int32_t s = 0; s < p->S; ++s) {
    const int64_t off = p->seg_off[s], len = p->seg_len[s];
    const int64_t plen = round_up(len, kAlign);
    q.assign((size_t)len, 0);
    if (wfeedback) {
      y.resize((size_t)len);
      r.resize((size_t)len);
      for (int64_t j = 0; j < len; ++j) y[j] = x[off + j] + wfeedback[off + j];
      quantize_weights(y.data(), len, p->kx, q.data(), nullptr, r.data());
      for (int64_t j = 0; j < len; ++j) {
        wfeedback[off + j] = r[j];
        if (wresid) wresid[off + j] = r[j];
      }
    } else {
      quantize_weights(x + off, len, p->kx, q.data(), nullptr, wresid ? wresid + off : nullptr);
    }
    code.assign((size_t)plen, (uint32_t)L);
    for (int64_t j = 0; j < len; ++j) code[j] = (uint32_t)(q[j] + L);
    if (wcodes) pack_bits(code.data(), plen, bits, wcodes + off * bits / 8);
  }
  return 0;
}

// ---------------------------------------------------------------------------
// The server, one step (Algorithm 2): average the N decoded streams in worker
// order, update x, then emit Q_x(x_{t+1}) for the next round's broadcast.
//   scales [n][S], codes [n][qo_gcode_bytes]
//   x [D]; m, v [D] (PLACE_SERVER only)
// READING (sign): the printed update is x + delta^ while Algorithm 1 and the
// virtual-iterate identity of the proofs use x - Q_g(.); the step is subtracted.
// PLACE_SERVER: delta^ is an averaged gradient; moments and step as Algorithm 1.
// ---------------------------------------------------------------------------
int32_t qo_server_step(const qo_problem* p, const float* scales, const uint8_t* codes,
                       float* x, float* m, float* v, float alpha,
                       uint8_t* wcodes, float* wresid, float* wfeedback) {
  const Hyper h = make_hyper(p->beta, p->theta, p->eps);
  GradLevels G;
  if (p->kg >= 0 && !make_grad_levels(p->kg, p->grid_g, &G)) return -1;
  if (p->placement == QO_PLACE_SERVER && (!m || !v)) return -2;
  const int64_t gbytes = qo_gcode_bytes(p);
  const float nf = (float)p->n;

  std::vector<uint32_t> code;
  std::vector<float> acc;
  for (int32_t s = 0; s < p->S; ++s) {
    const int64_t off = p->seg_off[s], len = p->seg_len[s];
    acc.assign((size_t)len, 0.0f);
    for (int32_t i = 0; i < p->n; ++i) {               // fixed order i = 0..N-1
      const uint8_t* stream = codes + (int64_t)i * gbytes;
      if (p->kg < 0) {
        for (int64_t j = 0; j < len; ++j) {
          float uj;
          std::memcpy(&uj, stream + 4 * (off + j), 4);
          acc[j] = acc[j] + uj;
        }
      } else {
        code.resize((size_t)len);
        unpack_bits(stream + off * G.bits / 8, len, G.bits, code.data());
        const float sc = scales[(int64_t)i * p->S + s];
        for (int64_t j = 0; j < len; ++j) {
          acc[j] = acc[j] + dequantize_grad((int32_t)code[j] - G.L, sc, G);
        }
      }
    }
    for (int64_t j = 0; j < len; ++j) {
      const int64_t k = off + j;
      const float dhat = acc[j] / nf;                   // (1/N) sum_i delta^(i)
      if (p->placement == QO_PLACE_SERVER) {
        moments(h, dhat, &m[k], &v[k]);
        x[k] = x[k] - adam_step(h, m[k], v[k], alpha);
      } else {
        x[k] = x[k] - dhat;
      }
    }
  }
  return qo_broadcast_weights(p, x, wcodes, wresid, wfeedback);
}

// Decode a packed weight broadcast back to values (what a worker receives).
int32_t qo_decode_weights(const qo_problem* p, const uint8_t* wcodes, float* xhat) {
  if (p->kx < 0) return -1;
  const int bits = qo_weight_code_bits(p->kx);
  const int L = 1 << p->kx;
  std::vector<uint32_t> code((size_t)p->D);
  unpack_bits(wcodes, p->D, bits, code.data());
  for (int64_t j = 0; j < p->D; ++j) {
    xhat[j] = std::ldexp((float)((int32_t)code[j] - L), -(p->kx + 1));
  }
  return 0;
}

}  // extern "C"
