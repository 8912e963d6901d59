// LSTM cell (forward and backward) for the gate product of the GNMT-like layers: elementwise,
// HBM-streaming kernels.  Gates and states are FP16 in memory; the cell is evaluated in FP32
// (sigma(x) = 1 / (1 + exp(-x)), tanh) and every output is rounded to FP16 once.  Eight
// sigma / tanh evaluations per hidden unit (forward three and two, backward the same again):
// with the library's exactly rounded division and its expf / tanhf the kernels were bound by
// instruction issue at a third of the HBM rate, so sigma and tanh use the hardware's
// exponential and reciprocal approximations (a few FP32 units in the last place, far inside
// half an FP16 unit), with tanh's small-argument and saturated ranges handled apart.  Gate order
// in the 4H columns of the gate matrix: i, f, g, o.  Each thread handles 8 hidden units of one
// row with 128-bit loads and stores.

#include <cuda_fp16.h>

#include "common.h"

namespace {

constexpr int kThreads = 256;

struct H8 {
  float v[8];
};

__device__ __forceinline__ H8 load8(const uint16_t* p) {
  const uint4 q = __ldcs(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  H8 r;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    r.v[2 * j] = __half2float(__ushort_as_half((uint16_t)(w[j] & 0xFFFFu)));
    r.v[2 * j + 1] = __half2float(__ushort_as_half((uint16_t)(w[j] >> 16)));
  }
  return r;
}

__device__ __forceinline__ void store8(uint16_t* p, const H8& x) {
  uint32_t w[4];
#pragma unroll
  for (int j = 0; j < 4; ++j)
    w[j] = (uint32_t)__half_as_ushort(__float2half_rn(x.v[2 * j])) |
           ((uint32_t)__half_as_ushort(__float2half_rn(x.v[2 * j + 1])) << 16);
  __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
}

__device__ __forceinline__ float sigm(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }

// tanh(x): x (1 - x^2 / 3) below 0.02 (the next term, 2 x^5 / 15, is under 3e-8 of x there, and
// the exponential form would cancel); +-1 beyond 9 (tanh(9) rounds to 1 in FP32); else
// (e^{2|x|} - 1) / (e^{2|x|} + 1) with the sign of x.  NaN falls through to the last form.
__device__ __forceinline__ float tanh_fast(float x) {
  const float ax = fabsf(x);
  if (ax < 0.02f) return x * (1.0f - x * x * (1.0f / 3.0f));
  if (ax > 9.0f) return copysignf(1.0f, x);
  const float t = __expf(2.0f * ax);
  return copysignf(__fdividef(t - 1.0f, t + 1.0f), x);
}

__global__ void __launch_bounds__(kThreads)
mp_lstm_cell_fwd_kernel(const uint16_t* __restrict__ G, int64_t ldg, const uint16_t* __restrict__ c_prev,
                        uint16_t* __restrict__ c_new, uint16_t* __restrict__ h, int64_t M, int64_t H) {
  const int64_t per_row = H / 8, total = M * per_row;
  for (int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kThreads) {
    const int64_t m = t / per_row, j = (t % per_row) * 8;
    const uint16_t* g = G + m * ldg + j;
    const H8 gi = load8(g), gf = load8(g + H), gg = load8(g + 2 * H), go = load8(g + 3 * H);
    const H8 cp = load8(c_prev + m * H + j);
    H8 cn, hh;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float i = sigm(gi.v[k]), f = sigm(gf.v[k]), gt = tanh_fast(gg.v[k]), o = sigm(go.v[k]);
      const float c = __fadd_rn(__fmul_rn(f, cp.v[k]), __fmul_rn(i, gt));
      cn.v[k] = c;
      hh.v[k] = __fmul_rn(o, tanh_fast(c));
    }
    store8(c_new + m * H + j, cn);
    store8(h + m * H + j, hh);
  }
}

__global__ void __launch_bounds__(kThreads)
mp_lstm_cell_bwd_kernel(const uint16_t* __restrict__ G, int64_t ldg, const uint16_t* __restrict__ c_prev,
                        const uint16_t* __restrict__ c_new, const uint16_t* __restrict__ dh,
                        const uint16_t* __restrict__ dc_in, uint16_t* __restrict__ dG, int64_t lddg,
                        uint16_t* __restrict__ dc_prev, int64_t M, int64_t H) {
  const int64_t per_row = H / 8, total = M * per_row;
  for (int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kThreads) {
    const int64_t m = t / per_row, j = (t % per_row) * 8;
    const uint16_t* g = G + m * ldg + j;
    const H8 gi = load8(g), gf = load8(g + H), gg = load8(g + 2 * H), go = load8(g + 3 * H);
    const H8 cp = load8(c_prev + m * H + j), cn = load8(c_new + m * H + j), dhv = load8(dh + m * H + j);
    H8 dci;
    if (dc_in != nullptr) dci = load8(dc_in + m * H + j);
    H8 di, df, dg, dout, dcp;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float i = sigm(gi.v[k]), f = sigm(gf.v[k]), gt = tanh_fast(gg.v[k]), o = sigm(go.v[k]);
      const float tc = tanh_fast(cn.v[k]);
      float dc = __fmul_rn(__fmul_rn(dhv.v[k], o), __fsub_rn(1.0f, __fmul_rn(tc, tc)));
      if (dc_in != nullptr) dc = __fadd_rn(dc, dci.v[k]);
      di.v[k] = __fmul_rn(__fmul_rn(dc, gt), __fmul_rn(i, __fsub_rn(1.0f, i)));
      df.v[k] = __fmul_rn(__fmul_rn(dc, cp.v[k]), __fmul_rn(f, __fsub_rn(1.0f, f)));
      dg.v[k] = __fmul_rn(__fmul_rn(dc, i), __fsub_rn(1.0f, __fmul_rn(gt, gt)));
      dout.v[k] = __fmul_rn(__fmul_rn(dhv.v[k], tc), __fmul_rn(o, __fsub_rn(1.0f, o)));
      dcp.v[k] = __fmul_rn(dc, f);
    }
    uint16_t* d = dG + m * lddg + j;
    store8(d, di);
    store8(d + H, df);
    store8(d + 2 * H, dg);
    store8(d + 3 * H, dout);
    store8(dc_prev + m * H + j, dcp);
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
  mp_lstm_cell_fwd_kernel<<<grid_for(mp_lstm_cell_fwd_kernel, M * (H / 8)), kThreads, 0, (cudaStream_t)stream>>>(
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
  mp_lstm_cell_bwd_kernel<<<grid_for(mp_lstm_cell_bwd_kernel, M * (H / 8)), kThreads, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)G16, ldg, (const uint16_t*)c_prev16, (const uint16_t*)c_new16, (const uint16_t*)dh16,
      (const uint16_t*)dc_in16, (uint16_t*)dG16, lddg, (uint16_t*)dc_prev16, M, H);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

}  // extern "C"
