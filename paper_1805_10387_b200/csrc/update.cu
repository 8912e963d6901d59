// HBM-streaming kernels of the step: upstream scaling, gradient inspection, the fused
// unscale + optimizer + FP16 recast over all tensors of a plan, and the loss-scale state
// machine.  Host entry points for them and for the state / plan objects.
//
// Every FP32 operation of the update is written with a round-to-nearest intrinsic so that
// the compiler cannot contract a multiply and an add into one fused operation: the update
// is then the sequence of individually rounded operations that Section 3.2 of the paper
// implies for an FP32 optimizer.  The kernels are bandwidth bound, so this costs nothing.

#include <cuda_fp16.h>
#include <math.h>
#include <stdarg.h>
#include <string.h>

#include <atomic>
#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.h"

// ------------------------------------------------------------------ host helpers
namespace mp {

static thread_local char g_err[512] = "";
static std::atomic<int64_t> g_launches{0};

int set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int check_device() {
  int dev = 0;
  MP_CUDA_TRY(cudaGetDevice(&dev));
  static thread_local int cached_dev = -1, cached_major = 0;
  if (cached_dev != dev) {
    int major = 0;
    MP_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    cached_dev = dev;
    cached_major = major;
  }
  if (cached_major != 10)
    return set_error(MP_ERR_UNSUPPORTED_ARCH,
                     "device %d has compute capability %d.x; this library is built for 10.x only",
                     dev, cached_major);
  return MP_OK;
}

}  // namespace mp

// ------------------------------------------------------------------ plan layout
namespace {

constexpr int kThreads = 256;
constexpr int kVec = 8;                           // elements per 128-bit FP16 vector
constexpr int kGroups = 4;                        // 8-element groups per thread and chunk
constexpr int kChunk = kThreads * kVec * kGroups; // 8192 elements per chunk (measured best of 4096..32768)

struct TensorRec {
  const uint16_t* g16;
  float* w32;
  float* m;
  float* v;
  uint16_t* w16;
  int64_t count;
};

struct ChunkRec {
  int32_t tensor;
  int32_t chunk;  // element offset = chunk * kChunk
};

struct OptArgs {
  float lr, b1, b2, eps, mu, wd;
};

}  // namespace

struct mp_update_plan {
  TensorRec* d_tensors;
  ChunkRec* d_chunks;
  int64_t n_chunks;
  int64_t total;
  int n_tensors;
  int has_v;
  int device;
  int sm_count;
};

namespace {

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
  return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ float4 ld_stream_f4(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream_f4(float* p, float4 x) {
  __stcs(reinterpret_cast<float4*>(p), x);
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 x) {
  __stcs(reinterpret_cast<uint4*>(p), x);
}

__device__ __forceinline__ float half_bits_to_float(uint16_t h) {
  return __half2float(__ushort_as_half(h));
}
__device__ __forceinline__ uint16_t float_to_half_bits(float x) {
  return __half_as_ushort(__float2half_rn(x));  // RNE, overflow -> inf, subnormals kept
}

// both halves of a packed pair: exponent field all ones <=> inf or NaN
__device__ __forceinline__ uint32_t pair_nonfinite(uint32_t w) {
  return __vcmpeq2(w & 0x7C007C00u, 0x7C007C00u);
}

struct Coef {
  float inv_s, c1, c2, omb1, omb2;
};

template <int KIND>
__device__ __forceinline__ void update_one(float g16f, float& w, float& m, float& v,
                                           const Coef& c, const OptArgs& o) {
  float g = __fmul_rn(g16f, c.inv_s);
  if (o.wd != 0.0f) g = __fadd_rn(g, __fmul_rn(o.wd, w));
  if (KIND == MP_OPT_ADAM) {
    m = __fadd_rn(__fmul_rn(o.b1, m), __fmul_rn(c.omb1, g));
    v = __fadd_rn(__fmul_rn(o.b2, v), __fmul_rn(c.omb2, __fmul_rn(g, g)));
    const float mh = __fdiv_rn(m, c.c1);
    const float vh = __fdiv_rn(v, c.c2);
    w = __fsub_rn(w, __fmul_rn(o.lr, __fdiv_rn(mh, __fadd_rn(__fsqrt_rn(vh), o.eps))));
  } else {
    m = __fadd_rn(__fmul_rn(o.mu, m), g);
    w = __fsub_rn(w, __fmul_rn(o.lr, m));
  }
}

template <int KIND>
__device__ __forceinline__ void update_vec8(const TensorRec& T, int64_t i, const Coef& c,
                                            const OptArgs& o) {
  const uint4 gq = ld_stream_u4(T.g16 + i);
  float4 w0 = ld_stream_f4(T.w32 + i), w1 = ld_stream_f4(T.w32 + i + 4);
  float4 m0 = ld_stream_f4(T.m + i), m1 = ld_stream_f4(T.m + i + 4);
  float4 v0 = make_float4(0, 0, 0, 0), v1 = v0;
  if (KIND == MP_OPT_ADAM) {
    v0 = ld_stream_f4(T.v + i);
    v1 = ld_stream_f4(T.v + i + 4);
  }
  const uint32_t gw[4] = {gq.x, gq.y, gq.z, gq.w};
  float* wp[8] = {&w0.x, &w0.y, &w0.z, &w0.w, &w1.x, &w1.y, &w1.z, &w1.w};
  float* mp_[8] = {&m0.x, &m0.y, &m0.z, &m0.w, &m1.x, &m1.y, &m1.z, &m1.w};
  float* vp[8] = {&v0.x, &v0.y, &v0.z, &v0.w, &v1.x, &v1.y, &v1.z, &v1.w};
  uint32_t out[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float g_lo = half_bits_to_float((uint16_t)(gw[j] & 0xFFFFu));
    const float g_hi = half_bits_to_float((uint16_t)(gw[j] >> 16));
    update_one<KIND>(g_lo, *wp[2 * j], *mp_[2 * j], *vp[2 * j], c, o);
    update_one<KIND>(g_hi, *wp[2 * j + 1], *mp_[2 * j + 1], *vp[2 * j + 1], c, o);
    out[j] = (uint32_t)float_to_half_bits(*wp[2 * j]) |
             ((uint32_t)float_to_half_bits(*wp[2 * j + 1]) << 16);
  }
  st_stream_f4(T.w32 + i, w0);
  st_stream_f4(T.w32 + i + 4, w1);
  st_stream_f4(T.m + i, m0);
  st_stream_f4(T.m + i + 4, m1);
  if (KIND == MP_OPT_ADAM) {
    st_stream_f4(T.v + i, v0);
    st_stream_f4(T.v + i + 4, v1);
  }
  st_stream_u4(T.w16 + i, make_uint4(out[0], out[1], out[2], out[3]));
}

// ------------------------------------------------------------------ kernels

// Fused master update (Section 3.2).  One resident wave of blocks; each block draws the next
// chunk from a device-side ticket counter (ascending, so neighbouring blocks stream
// neighbouring memory, and short chunks of ragged plans cannot unbalance the grid).  Per
// element 14 B read + 14 B written for Adam, 10 B + 10 B for momentum.  Returns at once,
// having written nothing, when the step's flag is set.
template <int KIND>
__global__ void __launch_bounds__(kThreads)
mp_master_update_kernel(const TensorRec* __restrict__ tensors, const ChunkRec* __restrict__ chunks,
                        int64_t n_chunks, mp_dev_state* __restrict__ st, OptArgs o,
                        const int* __restrict__ gemm_status) {
  if (*reinterpret_cast<const volatile int32_t*>(&st->h.found_inf) != 0) return;
  // a product kernel of this step gave up on a wait: its output is incomplete, apply nothing
  if (*reinterpret_cast<const volatile int32_t*>(&st->h.status) != 0 ||
      *reinterpret_cast<const volatile int*>(gemm_status) != 0) return;
  __shared__ Coef s_coef;
  __shared__ unsigned int s_ticket;
  if (threadIdx.x == 0) {
    const double t = (double)(st->h.t + 1);  // applied steps including this one
    Coef c;
    c.inv_s = __fdiv_rn(1.0f, st->h.scale);
    c.c1 = (float)(1.0 - pow((double)o.b1, t));
    c.c2 = (float)(1.0 - pow((double)o.b2, t));
    c.omb1 = __fsub_rn(1.0f, o.b1);
    c.omb2 = __fsub_rn(1.0f, o.b2);
    s_coef = c;
  }
  __syncthreads();
  const Coef c = s_coef;
  for (;;) {
    if (threadIdx.x == 0) s_ticket = atomicAdd(&st->update_ticket, 1u);
    __syncthreads();
    const int64_t ch = s_ticket;
    __syncthreads();                       // everyone has read the ticket before it is redrawn
    if (ch >= n_chunks) break;
    const ChunkRec rec = chunks[ch];
    const TensorRec T = tensors[rec.tensor];
    const int64_t start = (int64_t)rec.chunk * kChunk;
    const int64_t rem = T.count - start;
    const int n = rem < kChunk ? (int)rem : kChunk;
    if (n == kChunk) {
#pragma unroll
      for (int u = 0; u < kGroups; ++u)
        update_vec8<KIND>(T, start + (u * kThreads + threadIdx.x) * kVec, c, o);
    } else {
      const int nvec = n / kVec;
      for (int q = threadIdx.x; q < nvec; q += kThreads)
        update_vec8<KIND>(T, start + (int64_t)q * kVec, c, o);
      const int tail = n - nvec * kVec;  // < 8 elements, past the last full vector
      if ((int)threadIdx.x < tail) {
        const int64_t i = start + nvec * kVec + threadIdx.x;
        float w = T.w32[i], m = T.m[i], v = (KIND == MP_OPT_ADAM) ? T.v[i] : 0.0f;
        update_one<KIND>(half_bits_to_float(T.g16[i]), w, m, v, c, o);
        T.w32[i] = w;
        T.m[i] = m;
        if (KIND == MP_OPT_ADAM) T.v[i] = v;
        T.w16[i] = float_to_half_bits(w);
      }
    }
  }
  // the last block to leave puts both counters back to zero for the next launch
  if (threadIdx.x == 0 && atomicAdd(&st->update_done, 1u) == gridDim.x - 1) {
    st->update_ticket = 0;
    st->update_done = 0;
  }
}

// Gradient inspection over a plan (Section 3.1, item 1): 2 B read per element, OR-reduced
// by warp vote, at most one atomic per block and only when something was found.
__global__ void __launch_bounds__(kThreads)
mp_check_plan_kernel(const TensorRec* __restrict__ tensors, const ChunkRec* __restrict__ chunks,
                     int64_t n_chunks, mp_dev_state* __restrict__ st) {
  uint32_t bad = 0;
  for (int64_t ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
    const ChunkRec rec = chunks[ch];
    const uint16_t* g = tensors[rec.tensor].g16;
    const int64_t start = (int64_t)rec.chunk * kChunk;
    const int64_t rem = tensors[rec.tensor].count - start;
    const int n = rem < kChunk ? (int)rem : kChunk;
    const int nvec = n / kVec;
    for (int q = threadIdx.x; q < nvec; q += kThreads) {
      const uint4 x = ld_stream_u4(g + start + (int64_t)q * kVec);
      bad |= pair_nonfinite(x.x) | pair_nonfinite(x.y) | pair_nonfinite(x.z) | pair_nonfinite(x.w);
    }
    const int tail = n - nvec * kVec;
    if ((int)threadIdx.x < tail) {
      const uint16_t h = g[start + nvec * kVec + threadIdx.x];
      bad |= ((h & 0x7C00u) == 0x7C00u) ? 1u : 0u;
    }
  }
  const int warp_bad = __any_sync(0xFFFFFFFFu, bad != 0);
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  if (warp_bad && (threadIdx.x & 31) == 0) s_bad = 1;
  __syncthreads();
  if (threadIdx.x == 0 && s_bad) atomicOr(&st->h.found_inf, 1);
}

// Inspection of one flat FP16 buffer.
__global__ void __launch_bounds__(kThreads)
mp_check_flat_kernel(const uint16_t* __restrict__ g, int64_t n, mp_dev_state* __restrict__ st) {
  uint32_t bad = 0;
  const int64_t nvec = n / kVec;
  for (int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x; q < nvec;
       q += (int64_t)gridDim.x * kThreads) {
    const uint4 x = ld_stream_u4(g + q * kVec);
    bad |= pair_nonfinite(x.x) | pair_nonfinite(x.y) | pair_nonfinite(x.z) | pair_nonfinite(x.w);
  }
  if (blockIdx.x == 0 && (int64_t)threadIdx.x < n - nvec * kVec) {
    const uint16_t h = g[nvec * kVec + threadIdx.x];
    bad |= ((h & 0x7C00u) == 0x7C00u) ? 1u : 0u;
  }
  const int warp_bad = __any_sync(0xFFFFFFFFu, bad != 0);
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  if (warp_bad && (threadIdx.x & 31) == 0) s_bad = 1;
  __syncthreads();
  if (threadIdx.x == 0 && s_bad) atomicOr(&st->h.found_inf, 1);
}

// dY16 = rn16(S * g32), S read on the device (Section 3.1, item 1).
__global__ void __launch_bounds__(kThreads)
mp_scale_upstream_kernel(const float* __restrict__ g32, uint16_t* __restrict__ out, int64_t n,
                         const mp_dev_state* __restrict__ st) {
  const float S = st->h.scale;
  const int64_t nvec = n / kVec;
  for (int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x; q < nvec;
       q += (int64_t)gridDim.x * kThreads) {
    const float4 a = ld_stream_f4(g32 + q * kVec), b = ld_stream_f4(g32 + q * kVec + 4);
    uint4 r;
    r.x = (uint32_t)float_to_half_bits(__fmul_rn(S, a.x)) | ((uint32_t)float_to_half_bits(__fmul_rn(S, a.y)) << 16);
    r.y = (uint32_t)float_to_half_bits(__fmul_rn(S, a.z)) | ((uint32_t)float_to_half_bits(__fmul_rn(S, a.w)) << 16);
    r.z = (uint32_t)float_to_half_bits(__fmul_rn(S, b.x)) | ((uint32_t)float_to_half_bits(__fmul_rn(S, b.y)) << 16);
    r.w = (uint32_t)float_to_half_bits(__fmul_rn(S, b.z)) | ((uint32_t)float_to_half_bits(__fmul_rn(S, b.w)) << 16);
    *reinterpret_cast<uint4*>(out + q * kVec) = r;
  }
  if (blockIdx.x == 0 && (int64_t)threadIdx.x < n - nvec * kVec) {
    const int64_t i = nvec * kVec + threadIdx.x;
    out[i] = float_to_half_bits(__fmul_rn(S, g32[i]));
  }
}

// Bias gradient, stage 1: FP32 column sums of dY over a slab of rows.  A block owns up to 256
// columns and one slab.  A lane reads one 16-byte vector (8 columns) of a row; when a row has
// fewer than 32 vectors the spare lanes of the warp take further rows (lane = row group *
// vecs + vector), so narrow matrices still fill the warp.  The 8 warps stride over the slab's
// rows, four rows in flight per thread; the per-thread sums are then added through shared
// memory in (warp, row group) order.  partial[slab][n] is written once, no atomics, so the
// result does not depend on timing.  Row pitches are multiples of 8, so a vector that starts
// below N lies inside its row; columns at or beyond N are read and dropped.
constexpr int kBiasSlabs = 512;
constexpr int kBiasCols = 256;
constexpr int kBiasGroup = 4;      // gradients of one shape that may share a launch (blockIdx.z picks one)
struct BiasGroup {
  const uint16_t* dY[kBiasGroup];
  uint16_t* db[kBiasGroup];
};
__global__ void __launch_bounds__(kThreads, 8)
mp_bias_grad_partial_kernel(const BiasGroup group, int64_t lddy, int64_t M, int64_t N,
                            float* __restrict__ partial_all, int slabs, int vecs) {
  const uint16_t* __restrict__ dY = group.dY[blockIdx.z];
  float* __restrict__ partial = partial_all + (int64_t)blockIdx.z * slabs * N;
  // vecs: vectors per row handled by one warp, a power of two <= 32
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int groups = 32 / vecs;                     // rows a warp reads at once
  const int vc = lane & (vecs - 1), rg = lane / vecs;
  const int64_t col = (int64_t)blockIdx.x * kBiasCols + vc * 8;
  const int slab = blockIdx.y;
  const int64_t rows_per = (M + slabs - 1) / slabs;
  const int64_t r0 = slab * rows_per, r1 = r0 + rows_per < M ? r0 + rows_per : M;
  const int64_t stride = 8 * groups;                // rows between two reads of one thread
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // stage 2 may take its place early
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
  if (col < N) {
    const uint16_t* base = dY + col;
    for (int64_t r = r0 + warp * groups + rg; r < r1; r += 4 * stride) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int64_t rr = r + stride * u;
        v[u] = rr < r1 ? __ldcs(reinterpret_cast<const uint4*>(base + rr * lddy)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {          // ascending rows; a row past the slab adds +0
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] = __fadd_rn(acc[2 * j], half_bits_to_float((uint16_t)(w[j] & 0xFFFFu)));
          acc[2 * j + 1] = __fadd_rn(acc[2 * j + 1], half_bits_to_float((uint16_t)(w[j] >> 16)));
        }
      }
    }
  }
  __shared__ float sm[8][8][32];             // [warp][element][lane]
#pragma unroll
  for (int j = 0; j < 8; ++j) sm[warp][j][lane] = acc[j];
  __syncthreads();
  // thread (warp = element j, lane = vector) adds the sums of column col + j over the warps
  // and their row groups in a fixed order
  const int j = warp;
  if (lane < vecs) {
    float t = 0.0f;
    for (int w = 0; w < 8; ++w)
      for (int g = 0; g < groups; ++g) t = __fadd_rn(t, sm[w][j][g * vecs + lane]);
    const int64_t c = (int64_t)blockIdx.x * kBiasCols + lane * 8 + j;
    if (c < N) partial[(int64_t)slab * N + c] = t;
  }
}

// Bias gradient, stage 2: add the slabs in a fixed order, round to FP16, store, inspect.  A block
// of 1024 threads owns 32 columns; thread (group, column) adds its share of the slabs in
// ascending order, eight loads in flight at a time, then the 32 groups are added in ascending
// order through shared memory.
constexpr int kBiasFinalThreads = 1024;
__global__ void __launch_bounds__(kBiasFinalThreads)
mp_bias_grad_final_kernel(const float* __restrict__ partial_all, int slabs, int64_t N,
                          const BiasGroup group, mp_dev_state* st) {
  const float* __restrict__ partial = partial_all + (int64_t)blockIdx.y * slabs * N;
  uint16_t* __restrict__ db = group.db[blockIdx.y];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  const int64_t n = (int64_t)blockIdx.x * 32 + lane;
  const int per = (slabs + 31) / 32;
  asm volatile("griddepcontrol.wait;" ::: "memory");   // stage 1 complete, its sums visible
  const int s_begin = grp * per;
  const int s_end = s_begin + per < slabs ? s_begin + per : slabs;
  float a = 0.0f;
  if (n < N) {
    for (int s0 = s_begin; s0 < s_end; s0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = s0 + u < s_end ? partial[(int64_t)(s0 + u) * N + n] : 0.0f;
#pragma unroll
      for (int u = 0; u < 8; ++u) a = __fadd_rn(a, v[u]);
    }
  }
  __shared__ float sm[32][32];
  sm[grp][lane] = a;
  __syncthreads();
  uint32_t bad = 0;
  if (grp == 0 && n < N) {
    float t = sm[0][lane];
#pragma unroll
    for (int g = 1; g < 32; ++g) t = __fadd_rn(t, sm[g][lane]);
    const uint16_t h = float_to_half_bits(t);
    db[n] = h;
    bad = ((h & 0x7C00u) == 0x7C00u) ? 1u : 0u;
  }
  if (st != nullptr && __any_sync(0xFFFFFFFFu, bad != 0) && (threadIdx.x & 31) == 0)
    atomicOr(&st->h.found_inf, 1);
}

// Loss-scale state machine, one thread (Section 3.1, item 1).
__global__ void mp_loss_scale_update_kernel(mp_dev_state* st, const int* gemm_status) {
  mp_state_host& h = st->h;
  // A device-side error freezes the training state: the update above wrote nothing, and the
  // scale, the counters, the flag and the log stay as they are until the host has read the
  // status and cleared it.
  if (h.status == 0 && *gemm_status != 0) h.status = *gemm_status;
  if (h.status != 0) return;
  mp_log_record rec;
  rec.step = h.step;
  rec.scale_before = h.scale;
  rec.found_inf = h.found_inf != 0;
  if (h.found_inf != 0) {
    h.skipped += 1;
    h.good_steps = 0;
    h.strikes += 1;
    if (h.dynamic && h.strikes >= h.overflow_tolerance) {
      h.scale = fmaxf(__fmul_rn(h.scale, 0.5f), h.min_scale);
      h.strikes = 0;
    }
  } else {
    h.t += 1;
    h.good_steps += 1;
    if (h.dynamic && h.good_steps >= h.growth_interval) {
      h.scale = fminf(__fmul_rn(h.scale, 2.0f), h.max_scale);
      h.good_steps = 0;
      h.strikes = 0;
    }
  }
  h.found_inf = 0;
  h.step += 1;
  rec.t = h.t;
  rec.scale_after = h.scale;
  rec.good_steps = h.good_steps;
  st->log[st->log_count % MP_LOG_CAPACITY] = rec;
  st->log_count += 1;
}

// One-word moves between the device state's overflow flag and a caller-owned device word.
__global__ void mp_flag_export_kernel(const mp_dev_state* st, int32_t* word) {
  *word = st->h.found_inf != 0 ? 1 : 0;
}
__global__ void mp_flag_import_kernel(mp_dev_state* st, const int32_t* word) {
  if (*word != 0) st->h.found_inf = 1;
}

// Blocks of `kernel` that fit on one SM at once, remembered per (device, kernel).  Persistent
// grids are sized to exactly one resident wave: a grid of more blocks than fit runs in rounds
// of unequal length.
template <class K>
int resident_blocks_per_sm(K kernel) {
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, int> cache;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
  const std::pair<int, const void*> key(dev, reinterpret_cast<const void*>(kernel));
  std::lock_guard<std::mutex> lock(mu);
  auto it = cache.find(key);
  if (it != cache.end()) return it->second;
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreads, 0) != cudaSuccess || n < 1) n = 1;
  cache[key] = n;
  return n;
}

int grid_for(int64_t work_blocks, int sm_count, int per_sm) {
  const int64_t cap = (int64_t)sm_count * per_sm;
  return (int)(work_blocks < cap ? (work_blocks > 0 ? work_blocks : 1) : cap);
}

int sm_count_of_current_device(int* out) {
  int dev = 0;
  MP_CUDA_TRY(cudaGetDevice(&dev));
  MP_CUDA_TRY(cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, dev));
  return MP_OK;
}

}  // namespace

// ------------------------------------------------------------------ C ABI
extern "C" {

const char* mp_last_error(void) { return mp::g_err; }
int64_t mp_kernel_launch_count(void) { return mp::g_launches.load(); }

int mp_state_create(const mp_scaler_config* cfg, mp_state** out) {
  if (!cfg || !out) return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_create: null argument");
  if (!(cfg->init_scale > 0) || !(cfg->min_scale > 0) || !(cfg->max_scale >= cfg->min_scale) ||
      cfg->growth_interval < 1 || cfg->overflow_tolerance < 1)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_create: bad scaler configuration");
  if (int rc = mp::check_device()) return rc;
  mp_state* s = new (std::nothrow) mp_state{nullptr, 0};
  if (!s) return mp::set_error(MP_ERR_NOMEM, "mp_state_create: host allocation failed");
  cudaGetDevice(&s->device);
  if (cudaMalloc(&s->dev, sizeof(mp_dev_state)) != cudaSuccess) {
    delete s;
    return mp::set_error(MP_ERR_NOMEM, "mp_state_create: device allocation failed");
  }
  cudaMemset(s->dev, 0, sizeof(mp_dev_state));
  mp_state_host h;
  memset(&h, 0, sizeof(h));
  h.scale = cfg->init_scale;
  h.min_scale = cfg->min_scale;
  h.max_scale = cfg->max_scale;
  h.growth_interval = cfg->growth_interval;
  h.dynamic = cfg->dynamic ? 1 : 0;
  h.overflow_tolerance = cfg->overflow_tolerance;
  cudaError_t e = cudaMemcpy(s->dev, &h, sizeof(h), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    cudaFree(s->dev);
    delete s;
    return mp::set_error(MP_ERR_CUDA, "mp_state_create: %s", cudaGetErrorString(e));
  }
  *out = s;
  return MP_OK;
}

int mp_state_destroy(mp_state* s) {
  if (!s) return MP_OK;
  cudaFree(s->dev);
  delete s;
  return MP_OK;
}

int mp_state_read(mp_state* s, mp_state_host* out, void* stream) {
  if (!s || !out) return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_read: null argument");
  cudaStream_t st = (cudaStream_t)stream;
  MP_CUDA_TRY(cudaMemcpyAsync(out, s->dev, sizeof(*out), cudaMemcpyDeviceToHost, st));
  MP_CUDA_TRY(cudaStreamSynchronize(st));
  return MP_OK;
}

int mp_state_write(mp_state* s, const mp_state_host* in, void* stream) {
  if (!s || !in) return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_write: null argument");
  cudaStream_t st = (cudaStream_t)stream;
  MP_CUDA_TRY(cudaMemcpyAsync(s->dev, in, sizeof(*in), cudaMemcpyHostToDevice, st));
  MP_CUDA_TRY(cudaStreamSynchronize(st));
  return MP_OK;
}

int mp_state_read_log(mp_state* s, mp_log_record* out, int max_records, int* n_out, void* stream) {
  if (!s || !out || !n_out || max_records < 0)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_read_log: bad argument");
  cudaStream_t st = (cudaStream_t)stream;
  int64_t total = 0;
  MP_CUDA_TRY(cudaMemcpyAsync(&total, &s->dev->log_count, sizeof(total), cudaMemcpyDeviceToHost, st));
  MP_CUDA_TRY(cudaStreamSynchronize(st));
  int64_t have = total < MP_LOG_CAPACITY ? total : MP_LOG_CAPACITY;
  if (have > max_records) have = max_records;
  for (int64_t i = 0; i < have; ++i) {
    const int64_t idx = (total - have + i) % MP_LOG_CAPACITY;
    MP_CUDA_TRY(cudaMemcpyAsync(out + i, &s->dev->log[idx], sizeof(mp_log_record),
                                cudaMemcpyDeviceToHost, st));
  }
  MP_CUDA_TRY(cudaStreamSynchronize(st));
  *n_out = (int)have;
  return MP_OK;
}

int mp_state_export_flag(const mp_state* s, int32_t* word, void* stream) {
  if (!s || !word) return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_export_flag: null argument");
  if (reinterpret_cast<uintptr_t>(word) & 3u)
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_state_export_flag: word must be 4-byte aligned");
  if (int rc = mp::check_device()) return rc;
  mp_flag_export_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(s->dev, word);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

int mp_state_import_flag(mp_state* s, const int32_t* word, void* stream) {
  if (!s || !word) return mp::set_error(MP_ERR_INVALID_ARG, "mp_state_import_flag: null argument");
  if (reinterpret_cast<uintptr_t>(word) & 3u)
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_state_import_flag: word must be 4-byte aligned");
  if (int rc = mp::check_device()) return rc;
  mp_flag_import_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(s->dev, word);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

int mp_update_plan_create(int n, void* const* g16, void* const* w32, void* const* m,
                          void* const* v, void* const* w16, const int64_t* count,
                          mp_update_plan** out) {
  if (n <= 0 || !g16 || !w32 || !m || !w16 || !count || !out)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_update_plan_create: null argument or n <= 0");
  if (int rc = mp::check_device()) return rc;
  std::vector<TensorRec> recs(n);
  std::vector<ChunkRec> chunks;
  int64_t total = 0;
  for (int i = 0; i < n; ++i) {
    if (count[i] < 0)
      return mp::set_error(MP_ERR_INVALID_ARG, "mp_update_plan_create: count[%d] < 0", i);
    if (count[i] > 0) {
      if (!g16[i] || !w32[i] || !m[i] || !w16[i] || (v && !v[i]))
        return mp::set_error(MP_ERR_INVALID_ARG, "mp_update_plan_create: tensor %d has a null buffer", i);
      if (!mp::aligned16(g16[i]) || !mp::aligned16(w32[i]) || !mp::aligned16(m[i]) ||
          !mp::aligned16(w16[i]) || (v && !mp::aligned16(v[i])))
        return mp::set_error(MP_ERR_ALIGNMENT, "mp_update_plan_create: tensor %d is not 16-byte aligned", i);
    }
    recs[i] = TensorRec{(const uint16_t*)g16[i], (float*)w32[i], (float*)m[i],
                        v ? (float*)v[i] : nullptr, (uint16_t*)w16[i], count[i]};
    const int64_t nch = (count[i] + kChunk - 1) / kChunk;
    if (nch > INT32_MAX)
      return mp::set_error(MP_ERR_TOO_LARGE, "mp_update_plan_create: tensor %d is too large", i);
    for (int64_t c = 0; c < nch; ++c) chunks.push_back(ChunkRec{i, (int32_t)c});
    total += count[i];
  }
  mp_update_plan* p = new (std::nothrow) mp_update_plan();
  if (!p) return mp::set_error(MP_ERR_NOMEM, "mp_update_plan_create: host allocation failed");
  memset(p, 0, sizeof(*p));
  p->n_tensors = n;
  p->n_chunks = (int64_t)chunks.size();
  p->total = total;
  p->has_v = v != nullptr;
  cudaGetDevice(&p->device);
  if (int rc = sm_count_of_current_device(&p->sm_count)) { delete p; return rc; }
  const size_t chunk_bytes = (chunks.size() ? chunks.size() : 1) * sizeof(ChunkRec);
  if (cudaMalloc(&p->d_tensors, n * sizeof(TensorRec)) != cudaSuccess ||
      cudaMalloc(&p->d_chunks, chunk_bytes) != cudaSuccess) {
    cudaFree(p->d_tensors);
    delete p;
    return mp::set_error(MP_ERR_NOMEM, "mp_update_plan_create: device allocation failed");
  }
  cudaError_t e = cudaMemcpy(p->d_tensors, recs.data(), n * sizeof(TensorRec), cudaMemcpyHostToDevice);
  if (e == cudaSuccess && !chunks.empty())
    e = cudaMemcpy(p->d_chunks, chunks.data(), chunks.size() * sizeof(ChunkRec), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    mp_update_plan_destroy(p);
    return mp::set_error(MP_ERR_CUDA, "mp_update_plan_create: %s", cudaGetErrorString(e));
  }
  *out = p;
  return MP_OK;
}

int mp_update_plan_destroy(mp_update_plan* p) {
  if (!p) return MP_OK;
  cudaFree(p->d_tensors);
  cudaFree(p->d_chunks);
  delete p;
  return MP_OK;
}

int mp_master_update(mp_update_plan* plan, mp_state* state, const mp_optim_config* opt,
                     int check_mode, void* stream) {
  if (!plan || !state || !opt)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_master_update: null argument");
  if (opt->kind != MP_OPT_ADAM && opt->kind != MP_OPT_MOMENTUM)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_master_update: unknown optimizer kind %d", opt->kind);
  if (opt->kind == MP_OPT_ADAM && !plan->has_v)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_master_update: Adam needs a plan created with v");
  if (check_mode != 0 && check_mode != 1)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_master_update: check_mode must be 0 or 1");
  if (int rc = mp::check_device()) return rc;
  if (plan->n_chunks == 0) return MP_OK;
  cudaStream_t st = (cudaStream_t)stream;
  int* gemm_status = nullptr;
  if (int rc = mp::gemm_status_device_ptr(&gemm_status)) return rc;
  const OptArgs o{opt->lr, opt->beta1, opt->beta2, opt->eps, opt->momentum, opt->weight_decay};
  if (check_mode == 1) {
    // (the 2 B/element inspection, unlike the update, is faster as one resident wave)
    mp_check_plan_kernel<<<grid_for(plan->n_chunks, plan->sm_count,
                                    resident_blocks_per_sm(mp_check_plan_kernel)), kThreads, 0, st>>>(
        plan->d_tensors, plan->d_chunks, plan->n_chunks, state->dev);
    mp::count_launch();
  }
  const int per_sm = opt->kind == MP_OPT_ADAM ? resident_blocks_per_sm(mp_master_update_kernel<MP_OPT_ADAM>)
                                              : resident_blocks_per_sm(mp_master_update_kernel<MP_OPT_MOMENTUM>);
  const int grid = grid_for(plan->n_chunks, plan->sm_count, per_sm);
  if (opt->kind == MP_OPT_ADAM)
    mp_master_update_kernel<MP_OPT_ADAM><<<grid, kThreads, 0, st>>>(
        plan->d_tensors, plan->d_chunks, plan->n_chunks, state->dev, o, gemm_status);
  else
    mp_master_update_kernel<MP_OPT_MOMENTUM><<<grid, kThreads, 0, st>>>(
        plan->d_tensors, plan->d_chunks, plan->n_chunks, state->dev, o, gemm_status);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

int mp_loss_scale_update(mp_state* state, void* stream) {
  if (!state) return mp::set_error(MP_ERR_INVALID_ARG, "mp_loss_scale_update: null state");
  if (int rc = mp::check_device()) return rc;
  int* gemm_status = nullptr;
  if (int rc = mp::gemm_status_device_ptr(&gemm_status)) return rc;
  mp_loss_scale_update_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(state->dev, gemm_status);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

int mp_scale_upstream(const float* g32, void* dY16, int64_t n, const mp_state* state, void* stream) {
  if (!g32 || !dY16 || !state || n < 0)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_scale_upstream: bad argument");
  if (!mp::aligned16(g32) || !mp::aligned16(dY16))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_scale_upstream: buffers must be 16-byte aligned");
  if (int rc = mp::check_device()) return rc;
  if (n == 0) return MP_OK;
  int sms = 0;
  if (int rc = sm_count_of_current_device(&sms)) return rc;
  const int64_t blocks = (n / kVec + kThreads - 1) / kThreads;
  mp_scale_upstream_kernel<<<grid_for(blocks, sms, resident_blocks_per_sm(mp_scale_upstream_kernel)),
                             kThreads, 0, (cudaStream_t)stream>>>(
      g32, (uint16_t*)dY16, n, state->dev);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

// Slabs of rows that the first stage sums separately: at most eight blocks per SM (the kernel is
// compiled to fit eight), all resident at
// once (a grid a little larger than what fits runs a second, nearly empty round), each with at
// least 32 rows (8 warps x 4 rows in flight), at most kBiasSlabs.
static int bias_vecs(int64_t N) {        // 16-byte vectors per row and warp, as a power of two
  int vecs = 1;
  while (vecs < 32 && (int64_t)vecs * 8 < N) vecs *= 2;
  return vecs;
}

static int bias_slabs(int64_t M, int64_t N) {
  const int64_t col_blocks = (N + kBiasCols - 1) / kBiasCols;
  int sms = 0;
  if (sm_count_of_current_device(&sms) != MP_OK || sms < 1) sms = 148;   // no device to ask: a B200's count
  int64_t want = 8 * (int64_t)sms / col_blocks;
  const int64_t rows_per_pass = 32 * (32 / bias_vecs(N));     // rows one block reads at once
  const int64_t by_rows = (M + rows_per_pass - 1) / rows_per_pass;
  if (want > by_rows) want = by_rows;
  return (int)(want < 1 ? 1 : (want > kBiasSlabs ? kBiasSlabs : want));
}

size_t mp_bias_grad_workspace_bytes(int64_t M, int64_t N) {
  if (M <= 0 || N <= 0) return 0;
  return (size_t)bias_slabs(M, N) * (size_t)N * sizeof(float);
}

int mp_bias_grad_grouped(int count, const void* const* dY16, int64_t lddy, void* const* db16, int64_t M,
                         int64_t N, mp_state* state, void* workspace, size_t workspace_bytes, void* stream) {
  if (count < 1 || count > kBiasGroup || !dY16 || !db16 || M <= 0 || N <= 0 || lddy < N)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_bias_grad: bad argument (1..%d gradients per call)", kBiasGroup);
  for (int i = 0; i < count; ++i) {
    if (!dY16[i] || !db16[i]) return mp::set_error(MP_ERR_INVALID_ARG, "mp_bias_grad: null pointer");
    if (!mp::aligned16(dY16[i]) || !mp::aligned16(db16[i]))
      return mp::set_error(MP_ERR_ALIGNMENT, "mp_bias_grad: buffers must be 16-byte aligned");
  }
  if ((lddy & 7) || (workspace && !mp::aligned16(workspace)))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_bias_grad: buffers must be 16-byte aligned, lddy a multiple of 8");
  const size_t need = (size_t)count * mp_bias_grad_workspace_bytes(M, N);
  if (!workspace || workspace_bytes < need)
    return mp::set_error(MP_ERR_NOMEM, "mp_bias_grad: workspace of %zu bytes needed", need);
  if (int rc = mp::check_device()) return rc;
  const int slabs = bias_slabs(M, N);
  cudaStream_t st = (cudaStream_t)stream;
  BiasGroup grp;
  for (int i = 0; i < kBiasGroup; ++i) {
    grp.dY[i] = (const uint16_t*)dY16[i < count ? i : 0];
    grp.db[i] = (uint16_t*)db16[i < count ? i : 0];
  }
  const dim3 grid((unsigned)((N + kBiasCols - 1) / kBiasCols), (unsigned)slabs, (unsigned)count);
  const int vecs = bias_vecs(N);
  mp_bias_grad_partial_kernel<<<grid, kThreads, 0, st>>>(grp, lddy, M, N, (float*)workspace, slabs, vecs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((N + 31) / 32), (unsigned)count, 1);
  cfg.blockDim = dim3(kBiasFinalThreads, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute attr;            // resident early, waits on the device for stage 1
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  MP_CUDA_TRY(cudaLaunchKernelEx(&cfg, mp_bias_grad_final_kernel,
      (const float*)workspace, slabs, N, grp, state ? state->dev : (mp_dev_state*)nullptr));
  mp::count_launch(2);
  return MP_OK;
}

int mp_bias_grad(const void* dY16, int64_t lddy, void* db16, int64_t M, int64_t N, mp_state* state,
                 void* workspace, size_t workspace_bytes, void* stream) {
  const void* dys[1] = {dY16};
  void* dbs[1] = {db16};
  return mp_bias_grad_grouped(1, dys, lddy, dbs, M, N, state, workspace, workspace_bytes, stream);
}

int mp_check_finite(const void* g16, int64_t n, mp_state* state, void* stream) {
  if (!g16 || !state || n < 0)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_check_finite: bad argument");
  if (!mp::aligned16(g16))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_check_finite: buffer must be 16-byte aligned");
  if (int rc = mp::check_device()) return rc;
  if (n == 0) return MP_OK;
  int sms = 0;
  if (int rc = sm_count_of_current_device(&sms)) return rc;
  const int64_t blocks = (n / kVec + kThreads - 1) / kThreads;
  mp_check_flat_kernel<<<grid_for(blocks, sms, resident_blocks_per_sm(mp_check_flat_kernel)), kThreads, 0,
                         (cudaStream_t)stream>>>(
      (const uint16_t*)g16, n, state->dev);
  mp::count_launch();
  MP_CUDA_TRY(cudaGetLastError());
  return MP_OK;
}

}  // extern "C"
