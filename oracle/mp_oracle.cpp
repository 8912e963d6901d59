// CPU oracle for the mixed-precision training step of a stack of linear layers.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// method computes (paper Section 3.1: FP16 operands, FP32 accumulation, loss
// scaling, FP32 master weights; Section 3.2: FP16 gradients -> FP32 -> optimizer
// on the FP32 master -> FP16 working copy; Section 3.3: weight decay applied to
// the FP32 copy).  It shares no code with the CUDA path and is never called by
// it: only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
//
// No hardware half type is used: FP16 values are uint16_t bit patterns handled by
// h2f/f2h below.  Compile with -ffp-contract=off so that every FP32 operation is
// rounded on its own, in the order written.
//
// Parity pins (tests/test_oracle_*.py): h2f and f2h exhaustively against the
// closed form of IEEE binary16 and against an independent library conversion;
// the matmuls by brute force in double, by an integer-exact family and by
// permutation matrices; Adam and momentum against closed forms and a library
// optimizer run in float64; the scaler against the closed-form trajectory.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <algorithm>

namespace {

inline uint32_t f32_bits(float x) { uint32_t u; std::memcpy(&u, &x, 4); return u; }
inline float bits_f32(uint32_t u) { float x; std::memcpy(&x, &u, 4); return x; }

// IEEE binary16 -> binary32, exact for every one of the 65536 patterns.
inline float h2f(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const uint32_t e = (h >> 10) & 0x1Fu;
  const uint32_t f = h & 0x3FFu;
  if (e == 0x1Fu) {                         // inf or NaN (payload kept, quiet bit kept)
    return bits_f32(sign | 0x7F800000u | (f << 13));
  }
  if (e == 0) {
    if (f == 0) return bits_f32(sign);      // signed zero
    // subnormal: value = f * 2^-24; normalise into a binary32 normal
    int shift = 0;
    uint32_t m = f;
    while ((m & 0x400u) == 0) { m <<= 1; ++shift; }
    m &= 0x3FFu;
    const uint32_t e32 = (uint32_t)(127 - 15 - shift + 1);
    return bits_f32(sign | (e32 << 23) | (m << 13));
  }
  return bits_f32(sign | ((e + 127 - 15) << 23) | (f << 13));
}

// binary32 -> binary16, round to nearest, ties to even; |x| >= 65520 becomes inf
// (never saturates: the loss scaler must see the overflow); results below the
// smallest normal are produced as subnormals (no flush to zero); NaN -> quiet NaN.
inline uint16_t f2h(float x) {
  const uint32_t u = f32_bits(x);
  const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
  const uint32_t a = u & 0x7FFFFFFFu;
  if (a > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);           // NaN
  if (a == 0x7F800000u) return (uint16_t)(sign | 0x7C00u);          // inf
  const int e = (int)(a >> 23) - 127;                                 // unbiased
  uint32_t m = (a & 0x7FFFFFu) | 0x800000u;                           // 24-bit significand
  if (e > 15) return (uint16_t)(sign | 0x7C00u);                      // >= 2^16
  if (e >= -14) {
    // normal half candidate: drop 13 bits with RNE; a carry may bump the exponent,
    // and a carry out of exponent 15 yields 0x7C00 = inf, which is the right answer.
    uint32_t half = (uint32_t)((e + 15) << 10) | ((m >> 13) & 0x3FFu);
    const uint32_t rem = m & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (half & 1u))) half += 1;
    return (uint16_t)(sign | half);
  }
  if (e < -25) return sign;                                           // < 2^-25: rounds to zero
  // subnormal result: value = m * 2^(e-23); target unit is 2^-24 -> shift right by (-e-1)
  const int shift = -e - 1;                                           // 14..24
  uint32_t q = m >> shift;
  const uint32_t rem = m & ((1u << shift) - 1u);
  const uint32_t halfway = 1u << (shift - 1);
  if (rem > halfway || (rem == halfway && (q & 1u))) q += 1;          // may reach 0x400 = min normal
  return (uint16_t)(sign | q);
}

inline bool h_nonfinite(uint16_t h) { return (h & 0x7C00u) == 0x7C00u; }

template <class F>
void parallel_rows(int64_t rows, int nthreads, F fn) {
  if (nthreads <= 1 || rows < 2) { fn((int64_t)0, rows); return; }
  nthreads = (int)std::min<int64_t>(nthreads, rows);
  std::vector<std::thread> th;
  const int64_t per = (rows + nthreads - 1) / nthreads;
  for (int t = 0; t < nthreads; ++t) {
    const int64_t lo = t * per, hi = std::min<int64_t>(rows, lo + per);
    if (lo >= hi) break;
    th.emplace_back([=] { fn(lo, hi); });
  }
  for (auto& t : th) t.join();
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------- FP16 (O1)
float orc_h2f(uint16_t h) { return h2f(h); }
uint16_t orc_f2h(float x) { return f2h(x); }
void orc_h2f_array(const uint16_t* h, float* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = h2f(h[i]);
}
void orc_f2h_array(const float* x, uint16_t* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = f2h(x[i]);
}

// ------------------------------------------------------------- matmuls (O2)
// Section 3.1: operands FP16, every product exact in FP32 (11+11 significand bits),
// running sum kept in FP32, reduction index ascending, one rounding to FP16 at the end.
// Row-major throughout; ld* are leading dimensions in elements.

// forward:  Y[m,n] = rn16( sum_k X[m,k] * W[k,n] )
void orc_linear_fwd(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                    uint16_t* Y, int64_t ldy, int64_t M, int64_t K, int64_t N, int nthreads) {
  parallel_rows(M, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t m = lo; m < hi; ++m)
      for (int64_t n = 0; n < N; ++n) {
        float acc = 0.0f;
        for (int64_t k = 0; k < K; ++k) acc = acc + h2f(X[m * ldx + k]) * h2f(W[k * ldw + n]);
        Y[m * ldy + n] = f2h(acc);
      }
  });
}

// data gradient:  dX[m,k] = rn16( sum_n dY[m,n] * W[k,n] )
void orc_linear_bwd_dgrad(const uint16_t* dY, int64_t lddy, const uint16_t* W, int64_t ldw,
                          uint16_t* dX, int64_t lddx, int64_t M, int64_t K, int64_t N,
                          int nthreads) {
  parallel_rows(M, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t m = lo; m < hi; ++m)
      for (int64_t k = 0; k < K; ++k) {
        float acc = 0.0f;
        for (int64_t n = 0; n < N; ++n) acc = acc + h2f(dY[m * lddy + n]) * h2f(W[k * ldw + n]);
        dX[m * lddx + k] = f2h(acc);
      }
  });
}

// weight gradient:  dW[k,n] = rn16( sum_m X[m,k] * dY[m,n] )   (still multiplied by S)
void orc_linear_bwd_wgrad(const uint16_t* X, int64_t ldx, const uint16_t* dY, int64_t lddy,
                          uint16_t* dW, int64_t lddw, int64_t M, int64_t K, int64_t N,
                          int nthreads) {
  parallel_rows(K, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t k = lo; k < hi; ++k)
      for (int64_t n = 0; n < N; ++n) {
        float acc = 0.0f;
        for (int64_t m = 0; m < M; ++m) acc = acc + h2f(X[m * ldx + k]) * h2f(dY[m * lddy + n]);
        dW[k * lddw + n] = f2h(acc);
      }
  });
}

// Sampled outputs of the three products, for sizes the full loops cannot finish.
// op: 0 fwd (row=m, col=n), 1 dgrad (row=m, col=k), 2 wgrad (row=k, col=n).
// A and B are the two operands in the order of the functions above.  Writes the
// FP16 result, the same sum carried in double (un-rounded) and sum |a||b|.
void orc_linear_sampled(int op, const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                        int64_t M, int64_t K, int64_t N, const int64_t* rows, const int64_t* cols,
                        int64_t count, uint16_t* out16, double* out_exact, double* out_abs) {
  for (int64_t i = 0; i < count; ++i) {
    const int64_t r = rows[i], c = cols[i];
    const int64_t red = (op == 0) ? K : (op == 1) ? N : M;
    float acc = 0.0f;
    double ex = 0.0, ab = 0.0;
    for (int64_t j = 0; j < red; ++j) {
      float a, b;
      if (op == 0)      { a = h2f(A[r * lda + j]); b = h2f(B[j * ldb + c]); }
      else if (op == 1) { a = h2f(A[r * lda + j]); b = h2f(B[c * ldb + j]); }
      else              { a = h2f(A[j * lda + r]); b = h2f(B[j * ldb + c]); }
      acc = acc + a * b;
      ex += (double)a * (double)b;
      ab += std::fabs((double)a * (double)b);
    }
    out16[i] = f2h(acc);
    if (out_exact) out_exact[i] = ex;
    if (out_abs) out_abs[i] = ab;
  }
}

// Full-matrix double accumulation (error bounds and overflow margins only).
// op as above; out_exact/out_abs are dense [rows_out, cols_out].
void orc_linear_exact(int op, const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                      int64_t M, int64_t K, int64_t N, double* out_exact, double* out_abs,
                      int nthreads) {
  const int64_t R = (op == 2) ? K : M, C = (op == 1) ? K : N;
  const int64_t red = (op == 0) ? K : (op == 1) ? N : M;
  parallel_rows(R, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t r = lo; r < hi; ++r)
      for (int64_t c = 0; c < C; ++c) {
        double ex = 0.0, ab = 0.0;
        for (int64_t j = 0; j < red; ++j) {
          float a, b;
          if (op == 0)      { a = h2f(A[r * lda + j]); b = h2f(B[j * ldb + c]); }
          else if (op == 1) { a = h2f(A[r * lda + j]); b = h2f(B[c * ldb + j]); }
          else              { a = h2f(A[j * lda + r]); b = h2f(B[j * ldb + c]); }
          ex += (double)a * (double)b;
          ab += std::fabs((double)a * (double)b);
        }
        out_exact[r * C + c] = ex;
        if (out_abs) out_abs[r * C + c] = ab;
      }
  });
}

// ------------------------------------------- layers with bias and activation
// The paper's models put a bias and a nonlinearity after their dense products (ReLU in the
// Transformer feed-forward block, clipped ReLU in DeepSpeech2; Section 5).  Readings, since the
// paper states none: the bias is added to the FP32 sum before the one rounding to FP16; the
// activation acts on that FP32 value; the backward pass masks the FP16 data gradient with the
// derivative taken from the stored FP16 output (1 where the output is strictly inside the
// activation's linear range, else 0).
// act: 0 identity, 1 max(x,0), 2 min(max(x,0),clip).
static inline float apply_act(float x, int act, float clip) {
  if (act == 1) return x > 0.0f ? x : 0.0f;
  if (act == 2) { x = x > 0.0f ? x : 0.0f; return x < clip ? x : clip; }
  return x;
}
static inline bool act_passes(float y, int act, float clip) {
  if (act == 1) return y > 0.0f;
  if (act == 2) return y > 0.0f && y < clip;
  return true;
}

// Y[m,n] = rn16( act( sum_k X[m,k] W[k,n] + b[n] ) ); b may be null.
void orc_linear_fwd_act(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                        const uint16_t* b, uint16_t* Y, int64_t ldy, int64_t M, int64_t K,
                        int64_t N, int act, float clip, int nthreads) {
  parallel_rows(M, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t m = lo; m < hi; ++m)
      for (int64_t n = 0; n < N; ++n) {
        float acc = 0.0f;
        for (int64_t k = 0; k < K; ++k) acc = acc + h2f(X[m * ldx + k]) * h2f(W[k * ldw + n]);
        if (b) acc = acc + h2f(b[n]);
        Y[m * ldy + n] = f2h(apply_act(acc, act, clip));
      }
  });
}

// dX[m,k] = rn16( sum_n dY[m,n] W[k,n] ) where the layer's input A[m,k] (the previous layer's
// activated output) lies strictly inside the linear range of that layer's activation, else +0.
void orc_linear_bwd_dgrad_act(const uint16_t* dY, int64_t lddy, const uint16_t* W, int64_t ldw,
                              const uint16_t* A, int64_t lda, uint16_t* dX, int64_t lddx,
                              int64_t M, int64_t K, int64_t N, int act, float clip, int nthreads) {
  parallel_rows(M, nthreads, [=](int64_t lo, int64_t hi) {
    for (int64_t m = lo; m < hi; ++m)
      for (int64_t k = 0; k < K; ++k) {
        float acc = 0.0f;
        for (int64_t n = 0; n < N; ++n) acc = acc + h2f(dY[m * lddy + n]) * h2f(W[k * ldw + n]);
        dX[m * lddx + k] = act_passes(h2f(A[m * lda + k]), act, clip) ? f2h(acc) : (uint16_t)0;
      }
  });
}

// db[n] = rn16( sum_m dY[m,n] ), FP32 running sum, m ascending (still multiplied by S).
void orc_bias_grad(const uint16_t* dY, int64_t lddy, uint16_t* db, int64_t M, int64_t N) {
  for (int64_t n = 0; n < N; ++n) {
    float acc = 0.0f;
    for (int64_t m = 0; m < M; ++m) acc = acc + h2f(dY[m * lddy + n]);
    db[n] = f2h(acc);
  }
}

// ------------------------------------------------------------------ LSTM cell
// The GNMT-like models of Section 5 feed their gate product [x;h] W (four gates of H columns
// each, order i, f, g, o) to an LSTM cell.  Reading (the paper states no arithmetic): gates and
// states are stored FP16, the cell is evaluated in FP32 from those FP16 values with
// sigma(x) = 1 / (1 + exp(-x)) and tanh, and each output is rounded to FP16 once.
static inline float sigm(float x) { return 1.0f / (1.0f + std::exp(-x)); }

// c_new = sigma(f) c_prev + sigma(i) tanh(g);  h = sigma(o) tanh(c_new)
void orc_lstm_cell_fwd(const uint16_t* G, int64_t ldg, const uint16_t* c_prev, uint16_t* c_new,
                       uint16_t* h, int64_t M, int64_t H) {
  for (int64_t m = 0; m < M; ++m)
    for (int64_t j = 0; j < H; ++j) {
      const float i = sigm(h2f(G[m * ldg + j])), f = sigm(h2f(G[m * ldg + H + j]));
      const float g = std::tanh(h2f(G[m * ldg + 2 * H + j])), o = sigm(h2f(G[m * ldg + 3 * H + j]));
      const float c = f * h2f(c_prev[m * H + j]) + i * g;
      c_new[m * H + j] = f2h(c);
      h[m * H + j] = f2h(o * std::tanh(c));
    }
}

// Backward of the cell from the stored FP16 gates and states.  dh: gradient at h; dc_in:
// gradient arriving at c_new from the next time step (may be null = 0).  tanh(c_new) is taken
// from the stored FP16 c_new.  Writes dG [M,4H] (gradient at the gate pre-activations) and
// dc_prev, all FP16, still multiplied by the loss scale.
void orc_lstm_cell_bwd(const uint16_t* G, int64_t ldg, const uint16_t* c_prev,
                       const uint16_t* c_new, const uint16_t* dh, const uint16_t* dc_in,
                       uint16_t* dG, int64_t lddg, uint16_t* dc_prev, int64_t M, int64_t H) {
  for (int64_t m = 0; m < M; ++m)
    for (int64_t j = 0; j < H; ++j) {
      const float i = sigm(h2f(G[m * ldg + j])), f = sigm(h2f(G[m * ldg + H + j]));
      const float g = std::tanh(h2f(G[m * ldg + 2 * H + j])), o = sigm(h2f(G[m * ldg + 3 * H + j]));
      const float tc = std::tanh(h2f(c_new[m * H + j]));
      const float dhv = h2f(dh[m * H + j]);
      float dc = dhv * o * (1.0f - tc * tc);
      if (dc_in) dc = dc + h2f(dc_in[m * H + j]);
      dG[m * lddg + j] = f2h(dc * g * (i * (1.0f - i)));
      dG[m * lddg + H + j] = f2h(dc * h2f(c_prev[m * H + j]) * (f * (1.0f - f)));
      dG[m * lddg + 2 * H + j] = f2h(dc * i * (1.0f - g * g));
      dG[m * lddg + 3 * H + j] = f2h(dhv * tc * (o * (1.0f - o)));
      dc_prev[m * H + j] = f2h(dc * f);
    }
}

// ----------------------------------------------------- upstream scaling (O3)
// Section 3.1 item 1: the loss (here: the gradient entering the top layer) is
// multiplied by the current scale S, in FP32, then stored as FP16.
void orc_scale_upstream(const float* g32, float S, uint16_t* dY16, int64_t n) {
  for (int64_t i = 0; i < n; ++i) dY16[i] = f2h(S * g32[i]);
}

// ------------------------------------------------------------------ flag (O4)
// Section 3.1 item 1, "inspects gradients": 1 iff any element is inf or NaN.
int orc_found_inf(const uint16_t* g16, int64_t n) {
  int flag = 0;
  for (int64_t i = 0; i < n; ++i) flag |= h_nonfinite(g16[i]) ? 1 : 0;
  return flag;
}

// ---------------------------------------------------------------- update (O5)
// Section 3.2: FP16 gradient -> FP32, unscale by 1/S, optimizer on the FP32
// master, FP16 working copy rewritten from the master.  Section 3.3: the decay
// term is formed from the FP32 master and added to the FP32 gradient.
// The caller decides whether the step is applied (flag clear) and passes t, the
// count of applied steps including this one.
void orc_adam_update(const uint16_t* g16, float* w32, float* m, float* v, uint16_t* w16,
                     int64_t n, float S, float lr, float b1, float b2, float eps,
                     float weight_decay, int64_t t) {
  const float inv = 1.0f / S;
  const float c1 = (float)(1.0 - std::pow((double)b1, (double)t));
  const float c2 = (float)(1.0 - std::pow((double)b2, (double)t));
  const float omb1 = 1.0f - b1, omb2 = 1.0f - b2;
  for (int64_t i = 0; i < n; ++i) {
    float g = h2f(g16[i]) * inv;
    if (weight_decay != 0.0f) g = g + weight_decay * w32[i];
    const float mi = b1 * m[i] + omb1 * g;
    const float vi = b2 * v[i] + omb2 * (g * g);
    const float mh = mi / c1;
    const float vh = vi / c2;
    const float w = w32[i] - lr * (mh / (std::sqrt(vh) + eps));
    m[i] = mi; v[i] = vi; w32[i] = w;
    w16[i] = f2h(w);
  }
}

void orc_momentum_update(const uint16_t* g16, float* w32, float* u, uint16_t* w16, int64_t n,
                         float S, float lr, float mu, float weight_decay) {
  const float inv = 1.0f / S;
  for (int64_t i = 0; i < n; ++i) {
    float g = h2f(g16[i]) * inv;
    if (weight_decay != 0.0f) g = g + weight_decay * w32[i];
    const float ui = mu * u[i] + g;
    const float w = w32[i] - lr * ui;
    u[i] = ui; w32[i] = w;
    w16[i] = f2h(w);
  }
}

// ---------------------------------------------------------------- scaler (O6)
// Section 3.1 item 1: the scale for the NEXT iteration is chosen from this
// iteration's inspection.  Halve on overflow, double after `interval` clean steps
// in a row, clamp to [s_min, s_max].  dynamic == 0: S never changes (static loss
// scaling), but the counters still advance.
// Second policy, not in the paper (which only names "Backoff"): with tolerance H > 1 the
// scale is halved at the H-th overflow since it last changed, so that an isolated overflow
// costs one skipped step but no precision; every overflow step is still skipped and still
// restarts the count of clean steps.  H = 1 is the plain policy.
struct orc_scaler {
  float S;
  float s_min, s_max;
  int32_t interval;
  int32_t dynamic;
  int32_t good;       // clean steps since the last change of S
  int64_t t;          // applied optimizer steps
  int64_t step;       // all steps
  int64_t skipped;    // overflow steps
  int32_t tolerance;  // overflows that it takes to halve S (1: every overflow halves)
  int32_t strikes;    // overflows since S last changed
};

void orc_scaler_update(orc_scaler* s, int found_inf) {
  if (found_inf) {
    s->skipped += 1;
    s->good = 0;
    s->strikes += 1;
    if (s->dynamic && s->strikes >= s->tolerance) {
      s->S = std::max(s->S * 0.5f, s->s_min);
      s->strikes = 0;
    }
  } else {
    s->t += 1;
    s->good += 1;
    if (s->dynamic && s->good >= s->interval) {
      s->S = std::min(s->S * 2.0f, s->s_max);
      s->good = 0;
      s->strikes = 0;
    }
  }
  s->step += 1;
}

int orc_hardware_threads(void) { return (int)std::thread::hardware_concurrency(); }

}  // extern "C"
