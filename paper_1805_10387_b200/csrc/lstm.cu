// LSTM cell (forward and backward) for the gate product of the GNMT-like layers: elementwise,
// HBM-streaming kernels.  Gates and states are FP16 in memory; the cell is evaluated in FP32
// (sigma(x) = 1 / (1 + exp(-x)), tanh) and every output is rounded to FP16 once.  Gate order
// in the 4H columns of the gate matrix: i, f, g, o.  Each thread handles 8 hidden units of one
// row with 128-bit loads and stores.
//
// What bounds these kernels next to HBM is the special-function unit (16 results per clock
// and SM): a hidden unit may spend about 9 of its operations before that unit, not memory,
// sets the time.  sigma and tanh therefore use the hardware's exponential and reciprocal
// approximations (a few FP32 units in the last place, far inside half an FP16 unit), and
// several quotients share ONE reciprocal: 1/a, 1/b, 1/c, 1/d are formed from r = 1/(abcd) with
// nine multiplications.  Forward: five exponentials and two reciprocals per hidden unit
// (sigma(i), sigma(f), sigma(o), tanh(g) share one; tanh(c_new) needs c_new first); backward:
// five and two (the three sigmas; tanh(g) and tanh(c_new), both from stored values).
//
// The shared product must not overflow, so arguments are limited where the limit cannot be
// seen in an FP16 result: sigma's argument to >= -L with L = 21 (forward) or 28 (backward),
// where sigma(-L) <= 7.6e-10 stands in for a still smaller number; tanh's to |x| <= 10, where the
// quotient form gives exactly 1.0f as tanh itself does from 9.02 on.  A gate
// below -87.4, where exp(-x) overflows and the plain form gives exactly 0, is set to exactly 0,
// and a NaN gate gives NaN for that gate alone (the clamps would otherwise swallow it, and the
// shared reciprocal must not spread it to the other gates).

#include <cuda_fp16.h>

#include "common.h"

namespace {

constexpr int kThreads = 256;

// FP16 values as loaded (packed words, two per word); elements are converted where they are
// used, so a thread holds a vector in half as many registers as it has elements.  A thread takes
// kUnits = 8 hidden units (128-bit loads and stores).  Four units per thread (64-bit accesses,
// 32 - 45 registers, up to 64 warps per SM instead of 32 - 40) were measured and are no faster:
// 25.6 against 24.2 us forward, 33.8 against 32.6 us backward on 6400 x 1024; the kernels are
// bound by instruction issue (75 % of the issue slots), not by latency.
constexpr int kUnits = 8;
struct VU {
  uint32_t w[kUnits / 2];
};

__device__ __forceinline__ VU loadu(const uint16_t* p) {
  const uint4 q = __ldcs(reinterpret_cast<const uint4*>(p));
  return VU{{q.x, q.y, q.z, q.w}};
}
__device__ __forceinline__ float2 pair_at(const VU& x, int j) {      // elements 2j and 2j + 1
  return __half22float2(*reinterpret_cast<const __half2*>(&x.w[j]));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void storeu(uint16_t* p, const VU& x) {
  __stcs(reinterpret_cast<uint4*>(p), make_uint4(x.w[0], x.w[1], x.w[2], x.w[3]));
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kSigmaZeroBelow = -87.4f;   // exp(-x) overflows FP32 below this: sigma is exactly 0

// 1 + exp(-x), the denominator of sigma(x), with the exponent limited to L (i.e. x to >= -L; a
// large positive x needs no limit: exp(-x) just vanishes).  A NaN x gives a finite value here
// (the minimum drops it); sigma_fix puts the NaN back.
__device__ __forceinline__ float sigma_den(float x, float L) {
  return 1.0f + ex2_approx(fminf(-kLog2e * x, kLog2e * L));
}
// sigma(x) from the reciprocal of its denominator: exact 0 where the plain form gives it, NaN kept.
__device__ __forceinline__ float sigma_fix(float x, float inv_den) {
  const float s = x < kSigmaZeroBelow ? 0.0f : inv_den;
  return x != x ? x : s;
}
// exp(2 |x|) + 1 with |x| limited to 10: the denominator of tanh(|x|) = 1 - 2 / (exp(2|x|) + 1).
// At the limit the quotient form gives exactly 1.0f, which is what tanh rounds to from 9.02 on.
__device__ __forceinline__ float tanh_den(float x) {
  return ex2_approx(fminf((2.0f * kLog2e) * fabsf(x), 20.0f * kLog2e)) + 1.0f;
}
// tanh(x) from the reciprocal of its denominator; x (1 - x^2 / 3) below 0.02 (the next term,
// 2 x^5 / 15, is under 3e-8 of x there, and the quotient form would cancel); NaN kept.
__device__ __forceinline__ float tanh_fix(float x, float inv_den) {
  float t = copysignf(fmaf(-2.0f, inv_den, 1.0f), x);
  t = fabsf(x) < 0.02f ? x * fmaf(x * x, -1.0f / 3.0f, 1.0f) : t;
  return x != x ? x : t;
}

// Reciprocals of a, b, c, d from one hardware reciprocal (all four finite, >= 1, product finite).
__device__ __forceinline__ void rcp4(float a, float b, float c, float d, float& ia, float& ib,
                                     float& ic, float& id) {
  const float ab = a * b, cd = c * d;
  const float r = rcp_approx(ab * cd);
  const float rab = r * cd, rcd = r * ab;     // 1 / (a b), 1 / (c d)
  ia = rab * b; ib = rab * a; ic = rcd * d; id = rcd * c;
}
__device__ __forceinline__ void rcp3(float a, float b, float c, float& ia, float& ib, float& ic) {
  const float ab = a * b;
  const float r = rcp_approx(ab * c);
  const float rab = r * c;                    // 1 / (a b)
  ia = rab * b; ib = rab * a; ic = r * ab;
}
__device__ __forceinline__ void rcp2(float a, float b, float& ia, float& ib) {
  const float r = rcp_approx(a * b);
  ia = r * b; ib = r * a;
}

struct FwdOut { float c, h; };
__device__ __forceinline__ FwdOut cell_fwd(float xi, float xf, float xg, float xo, float cp) {
  float ri, rf, ro, rg;
  // (1 + e^21)^3 (e^20 + 1) < 1.2e36: the product is finite and its reciprocal a normal number
  rcp4(sigma_den(xi, 21.0f), sigma_den(xf, 21.0f), sigma_den(xo, 21.0f), tanh_den(xg), ri, rf, ro, rg);
  const float i = sigma_fix(xi, ri), f = sigma_fix(xf, rf), o = sigma_fix(xo, ro);
  const float gt = tanh_fix(xg, rg);
  FwdOut r;
  r.c = fmaf(f, cp, i * gt);
  r.h = o * tanh_fix(r.c, rcp_approx(tanh_den(r.c)));
  return r;
}

__global__ void __launch_bounds__(kThreads)
mp_lstm_cell_fwd_kernel(const uint16_t* __restrict__ G, int64_t ldg, const uint16_t* __restrict__ c_prev,
                        uint16_t* __restrict__ c_new, uint16_t* __restrict__ h, int64_t M, int64_t H) {
  const int64_t per_row = H / kUnits, total = M * per_row;
  for (int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kThreads) {
    const int64_t m = t / per_row, j = (t % per_row) * kUnits;
    const uint16_t* g = G + m * ldg + j;
    const VU gi = loadu(g), gf = loadu(g + H), gg = loadu(g + 2 * H), go = loadu(g + 3 * H);
    const VU cp = loadu(c_prev + m * H + j);
    VU cn, hh;
#pragma unroll
    for (int k = 0; k < kUnits / 2; ++k) {
      const float2 xi = pair_at(gi, k), xf = pair_at(gf, k), xg = pair_at(gg, k), xo = pair_at(go, k);
      const float2 c0 = pair_at(cp, k);
      const FwdOut a = cell_fwd(xi.x, xf.x, xg.x, xo.x, c0.x), b = cell_fwd(xi.y, xf.y, xg.y, xo.y, c0.y);
      cn.w[k] = pack2(a.c, b.c);
      hh.w[k] = pack2(a.h, b.h);
    }
    storeu(c_new + m * H + j, cn);
    storeu(h + m * H + j, hh);
  }
}

struct BwdOut { float di, df, dg, dout, dcp; };
template <bool HAS_DC>
__device__ __forceinline__ BwdOut cell_bwd(float xi, float xf, float xg, float xo, float cp, float cn,
                                           float dh, float dci) {
  float ri, rf, ro, rg, rc;
  // (1 + e^28)^3 < 3.1e36 and (e^20 + 1)^2 < 2.4e17: finite products, normal reciprocals
  rcp3(sigma_den(xi, 28.0f), sigma_den(xf, 28.0f), sigma_den(xo, 28.0f), ri, rf, ro);
  rcp2(tanh_den(xg), tanh_den(cn), rg, rc);
  const float i = sigma_fix(xi, ri), f = sigma_fix(xf, rf), o = sigma_fix(xo, ro);
  const float gt = tanh_fix(xg, rg), tc = tanh_fix(cn, rc);
  // s (1 - s) as s - s^2 and 1 - t^2 in one fused operation each: these kernels are bound by
  // instruction issue, and the quotients above already differ from an exactly rounded
  // evaluation by a few FP32 units in the last place
  const float dho = dh * o;
  float dc = dho * fmaf(-tc, tc, 1.0f);
  if (HAS_DC) dc = fmaf(dho, fmaf(-tc, tc, 1.0f), dci);
  BwdOut r;
  r.di = (dc * gt) * fmaf(-i, i, i);
  r.df = (dc * cp) * fmaf(-f, f, f);
  r.dg = (dc * i) * fmaf(-gt, gt, 1.0f);
  r.dout = (dh * tc) * fmaf(-o, o, o);
  r.dcp = dc * f;
  return r;
}

template <bool HAS_DC>
__global__ void __launch_bounds__(kThreads)
mp_lstm_cell_bwd_kernel(const uint16_t* __restrict__ G, int64_t ldg, const uint16_t* __restrict__ c_prev,
                        const uint16_t* __restrict__ c_new, const uint16_t* __restrict__ dh,
                        const uint16_t* __restrict__ dc_in, uint16_t* __restrict__ dG, int64_t lddg,
                        uint16_t* __restrict__ dc_prev, int64_t M, int64_t H) {
  const int64_t per_row = H / kUnits, total = M * per_row;
  for (int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kThreads) {
    const int64_t m = t / per_row, j = (t % per_row) * kUnits;
    const uint16_t* g = G + m * ldg + j;
    const VU gi = loadu(g), gf = loadu(g + H), gg = loadu(g + 2 * H), go = loadu(g + 3 * H);
    const VU cp = loadu(c_prev + m * H + j), cn = loadu(c_new + m * H + j), dhv = loadu(dh + m * H + j);
    VU dci = {{0u, 0u, 0u, 0u}};
    if (HAS_DC) dci = loadu(dc_in + m * H + j);
    VU di, df, dg, dout, dcp;
#pragma unroll
    for (int k = 0; k < kUnits / 2; ++k) {
      const float2 xi = pair_at(gi, k), xf = pair_at(gf, k), xg = pair_at(gg, k), xo = pair_at(go, k);
      const float2 c0 = pair_at(cp, k), c1 = pair_at(cn, k), d0 = pair_at(dhv, k), e0 = pair_at(dci, k);
      const BwdOut a = cell_bwd<HAS_DC>(xi.x, xf.x, xg.x, xo.x, c0.x, c1.x, d0.x, e0.x);
      const BwdOut b = cell_bwd<HAS_DC>(xi.y, xf.y, xg.y, xo.y, c0.y, c1.y, d0.y, e0.y);
      di.w[k] = pack2(a.di, b.di);
      df.w[k] = pack2(a.df, b.df);
      dg.w[k] = pack2(a.dg, b.dg);
      dout.w[k] = pack2(a.dout, b.dout);
      dcp.w[k] = pack2(a.dcp, b.dcp);
    }
    uint16_t* d = dG + m * lddg + j;
    storeu(d, di);
    storeu(d + H, df);
    storeu(d + 2 * H, dg);
    storeu(d + 3 * H, dout);
    storeu(dc_prev + m * H + j, dcp);
  }
}

// One resident round of blocks (what fits on the device at the kernel's register use): a grid
// a little larger than that runs a nearly empty second round.
template <class K>
int grid_for(K kernel, int64_t threads_needed) {
  int dev = 0, sms = 148, per_sm = 1;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0);
  if (per_sm < 1) per_sm = 1;
  const int64_t blocks = (threads_needed + kThreads - 1) / kThreads;
  const int64_t cap = (int64_t)sms * per_sm;
  return (int)(blocks < cap ? (blocks > 0 ? blocks : 1) : cap);
}

int check_common(const char* name, const void* G16, int64_t ldg, int64_t M, int64_t H) {
  if (!G16 || M <= 0 || H <= 0 || ldg < 4 * H)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: bad argument", name);
  if ((H & 7) || (ldg & 7))
    return mp::set_error(MP_ERR_ALIGNMENT, "%s: H and the leading dimension must be multiples of 8", name);
  return mp::check_device();
}

}  // namespace

extern "C" {

int mp_lstm_cell_fwd(const void* G16, int64_t ldg, const void* c_prev16, void* c_new16, void* h16,
                     int64_t M, int64_t H, void* stream) {
  if (int rc = check_common("mp_lstm_cell_fwd", G16, ldg, M, H)) return rc;
  if (!c_prev16 || !c_new16 || !h16)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_lstm_cell_fwd: null pointer");
  if (!mp::aligned16(G16) || !mp::aligned16(c_prev16) || !mp::aligned16(c_new16) || !mp::aligned16(h16))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_lstm_cell_fwd: pointers must be 16-byte aligned");
  mp_lstm_cell_fwd_kernel<<<grid_for(mp_lstm_cell_fwd_kernel, M * (H / kUnits)), kThreads, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)G16, ldg, (const uint16_t*)c_prev16, (uint16_t*)c_new16, (uint16_t*)h16, M, H);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

int mp_lstm_cell_bwd(const void* G16, int64_t ldg, const void* c_prev16, const void* c_new16,
                     const void* dh16, const void* dc_in16, void* dG16, int64_t lddg, void* dc_prev16,
                     int64_t M, int64_t H, void* stream) {
  if (int rc = check_common("mp_lstm_cell_bwd", G16, ldg, M, H)) return rc;
  if (!c_prev16 || !c_new16 || !dh16 || !dG16 || !dc_prev16 || lddg < 4 * H)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_lstm_cell_bwd: bad argument");
  if ((lddg & 7) || !mp::aligned16(G16) || !mp::aligned16(c_prev16) || !mp::aligned16(c_new16) ||
      !mp::aligned16(dh16) || !mp::aligned16(dG16) || !mp::aligned16(dc_prev16) ||
      (dc_in16 && !mp::aligned16(dc_in16)))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_lstm_cell_bwd: 16-byte alignment and lddg %% 8 == 0 required");
  if (dc_in16 != nullptr)
    mp_lstm_cell_bwd_kernel<true><<<grid_for(mp_lstm_cell_bwd_kernel<true>, M * (H / kUnits)), kThreads, 0, (cudaStream_t)stream>>>(
        (const uint16_t*)G16, ldg, (const uint16_t*)c_prev16, (const uint16_t*)c_new16, (const uint16_t*)dh16,
        (const uint16_t*)dc_in16, (uint16_t*)dG16, lddg, (uint16_t*)dc_prev16, M, H);
  else
    mp_lstm_cell_bwd_kernel<false><<<grid_for(mp_lstm_cell_bwd_kernel<false>, M * (H / kUnits)), kThreads, 0, (cudaStream_t)stream>>>(
        (const uint16_t*)G16, ldg, (const uint16_t*)c_prev16, (const uint16_t*)c_new16, (const uint16_t*)dh16,
        (const uint16_t*)dc_in16, (uint16_t*)dG16, lddg, (uint16_t*)dc_prev16, M, H);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

}  // extern "C"
