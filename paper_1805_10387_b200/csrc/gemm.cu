// FP16-in / FP32-accumulate matrix products of the step (Section 3.1 of the paper) as persistent,
// warp-specialised tcgen05 kernels for sm_100a.  Both kernels share one pipeline:
//
//   warp 0      TMA producer: tensor-map loads into a shared-memory ring (128-byte swizzle)
//   warp 1      MMA issuer: tcgen05.mma (FP16 x FP16 -> FP32) into tensor memory; owns the TMEM
//               allocation (two 256-column accumulators, so the epilogue of one tile overlaps
//               the main loop of the next)
//   warps 2-5   epilogue (warps 2-9 in the fused flavours, two per TMEM lane quarter): tcgen05.ld,
//               optional bias / activation / mask, round to FP16 (nearest even, overflow to
//               inf), stage in shared memory, TMA store; for the weight gradient also the
//               inf/NaN inspection of what is stored
//
//   mp_gemm_pair_kernel  clusters of two CTAs, tcgen05.mma.cta_group::2, one 256 x 256 tile per
//                        pair, 6 stages x 32 KiB per CTA; used for outputs of more than 128 rows
//   mp_gemm_kernel       one CTA per 128 x 256 tile, cta_group::1, 4 stages x 48 KiB
//
// The three products differ only in which operand dimension is contiguous in memory:
//   forward   Y  = X  * W      A = X  (reduction contiguous)   B = W  (output dim contiguous)
//   dgrad     dX = dY * W^T    A = dY (reduction contiguous)   B = W  (reduction contiguous)
//   wgrad     dW = X^T * dY    A = X  (output dim contiguous)  B = dY (output dim contiguous)
// and that is expressed by the TMA box shape and the "major" bits of the MMA descriptors:
// no operand is ever transposed in memory.
//
// A long reduction with few output tiles (the weight gradient) can be split across CTAs:
// each split stores FP32 partial sums to a workspace and a second kernel adds them in a
// fixed order, rounds to FP16 and inspects.  Up to four independent products of one shape can
// share a launch (the *_grouped entry points): one persistent work list over all their tiles.

#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.h"
#include "ptx.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;           // 16 KiB
constexpr int B_BYTES = BN * BK * 2;           // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int CHUNK_BYTES = 64 * BK * 2;       // one 64 x 64 box of an MN-major operand
// warp 0 producer, warp 1 MMA issuer, then 4 or 8 epilogue warps.  Four (one per TMEM lane quarter)
// for the plain flavours, whose epilogue only rounds and stores (eight were measured and are no
// faster).  The bias / activation / mask epilogues are bound by the issue rate of one warp per
// scheduler, so they are launched with eight (two per lane quarter, each taking half of the
// tile's columns): 137 against 154 us on the masked 25600x1600x1600 data gradient.
constexpr int THREADS_PLAIN = 64 + 32 * 4;
constexpr int THREADS_FUSED = 64 + 32 * 8;
constexpr int TMEM_COLS = 512;
constexpr int STAGING_BYTES = 8 * 32 * 64 * 2;  // epilogue staging: 8 slots of 32 rows x 64 FP16 columns
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kFallbackSMs = 148;              // split heuristic when no device can be asked

__device__ int g_gemm_status = 0;              // first device-side error (bounded wait expired)

enum OutMode { OUT_F16 = 0, OUT_F16_FLAG = 1, OUT_PARTIAL = 2 };

// Up to MAX_GROUP independent products of the same shape and layouts run as one launch: the
// work list is problem-major, and every role picks its tensor maps by problem index.
constexpr int MAX_GROUP = 4;
struct GroupMaps {
  CUtensorMap a[MAX_GROUP], b[MAX_GROUP], b32[MAX_GROUP], out[MAX_GROUP], ws[MAX_GROUP];
};

struct GemmParams {
  int group;            // number of problems in this launch
  int work_per_problem; // tiles x splits of one problem; within a problem the tile index runs fastest, so that the
                        // CTAs running at one time work on the same slice of the reduction and share its panels in L2
  int Mo, No, R;        // output rows, output columns, reduction length
  int No8;              // No rounded down to a multiple of 8: the columns the output tensor map covers
  int m_tiles, n_tiles, splits, num_kb;
  int m_fast;           // tile order: 1 = the row-tile index runs fastest, 0 = the column-tile index
  int out_mode;
  uint16_t* out[MAX_GROUP];   // FP16 outputs [Mo, No], leading dimension ldo
  int64_t ldo;
  float* ws;            // FP32 partials [problem][splits][Mo][ws_ld]
  int64_t ws_ld;
  int* flag;            // found_inf word, or null
  int* status;          // status word of the caller's state object, or null
  uint64_t wait_ns;     // limit of every wait on a pipeline barrier
  int no_loads;         // error-path self-test only: the producer issues no load at all
  // Optional fused epilogue (FP16 output only).  Forward flavour: add bias[col] to the FP32 sum,
  // then the activation.  Data-gradient flavour: zero the output where the layer input
  // mask[row, col] (the previous layer's activated FP16 output) is outside the activation's
  // linear range.  act: 0 none, 1 max(x,0), 2 min(max(x,0),clip).
  const uint16_t* bias[MAX_GROUP];   // per problem (all set or all null)
  const uint16_t* mask;
  int64_t ldmask;
  int act;
  float clip;
};

struct Barriers {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__device__ __forceinline__ uint32_t pair_nonfinite(uint32_t w) {
  return __vcmpeq2(w & 0x7C007C00u, 0x7C007C00u);
}

// A bounded wait ran out: the CTA stops taking work.  The error is recorded in the device-wide
// status word (which the update and loss-scale kernels consult before they touch the training
// state) and, when the call was given a state object, in that state's status field.
template <class B>
__device__ __forceinline__ void report_timeout(B* bars, const GemmParams& p) {
  bars->abort = 1;
  atomicCAS(&g_gemm_status, 0, (int)MP_ERR_TIMEOUT);
  if (p.status != nullptr) atomicCAS(p.status, 0, (int)MP_ERR_TIMEOUT);
}

// Row-tile and column-tile index of tile number `tile`.  Consecutive tiles run at the same time
// on the GPU, so the fast index is that of the smaller operand: its panels stay in L2 while the
// larger operand streams through once (with the column index fast, a weight gradient of 8 x 16
// tiles read its 16 dY panels once per wave: 678 MB of DRAM traffic against 381 algorithmic).
__device__ __forceinline__ int tile_m(const GemmParams& p, int tile) {
  return p.m_fast ? tile % p.m_tiles : tile / p.n_tiles;
}
__device__ __forceinline__ int tile_n(const GemmParams& p, int tile) {
  return p.m_fast ? tile / p.m_tiles : tile % p.n_tiles;
}

// Width of the MMAs of the tile whose first column is n_base: the columns that exist, rounded up
// to 32, at most BN.  A ragged last column tile (1600 = 6 x 256 + 64) then issues a quarter of
// the MMA work of a full one instead of multiplying zero-filled columns, and the producer
// fetches only the B boxes those MMAs read (a full tile's loads, 64 B per clock and SM, take
// as long as its MMAs, so a narrow tile gets faster only if its loads shrink too).  Multiples
// of 32 keep every form legal: N % 16 == 0 for both instruction shapes, and each CTA of a pair
// holds N / 2 (a multiple of 16) columns of B.
__device__ __forceinline__ int tile_width(int No, int n_base) {
  const int left = No - n_base;
  return left >= BN ? BN : ((left + 31) & ~31);
}

// Activation mask of one thread's row of a tile, one bit per column (word c = columns
// 32c .. 32c+31): 1 where the layer input (the activated FP16 output of the layer below)
// lies strictly inside the activation's linear range.  Called BEFORE the thread waits for the
// accumulator, so the global loads (a DRAM round trip each when the input has left L2) run
// under the tile's main loop instead of stretching the epilogue.
__device__ __forceinline__ void load_pass_bits(const GemmParams& p, int row, int n0, int c_begin,
                                               int c_count, uint32_t (&bits)[BN / 32]) {
  const bool row_ok = row < p.Mo;
#pragma unroll 4
  for (int cc = 0; cc < c_count; ++cc) {
    const int c = c_begin + cc;
    const int col0 = n0 + c * 32;
    uint32_t b = 0;
    if (row_ok && col0 < p.No) {
      const uint16_t* mrow = p.mask + (int64_t)row * p.ldmask + col0;
      uint32_t mw[16];
      if (col0 + 32 <= p.No) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(mrow) + j);
          mw[4 * j] = q4.x; mw[4 * j + 1] = q4.y; mw[4 * j + 2] = q4.z; mw[4 * j + 3] = q4.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t lo = (col0 + 2 * j < p.No) ? __ldg(mrow + 2 * j) : 0u;
          const uint32_t hi = (col0 + 2 * j + 1 < p.No) ? __ldg(mrow + 2 * j + 1) : 0u;
          mw[j] = lo | (hi << 16);
        }
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const uint16_t hm = (uint16_t)((j & 1) ? (mw[j >> 1] >> 16) : (mw[j >> 1] & 0xFFFFu));
        const float y = __half2float(__ushort_as_half(hm));
        const bool pass = p.act == 2 ? (y > 0.0f && y < p.clip) : (y > 0.0f);
        b |= (pass ? 1u : 0u) << j;
      }
    }
    bits[c] = b;
  }
}

//
// FP16 output leaves through shared memory: the warp's 32 rows x 64 columns (two chunks) are
// written into a 4 KiB staging slot in the 128-byte-swizzled order of the output tensor map and
// one TMA store moves the slot to global memory, whole 128-byte row segments at a time and
// clipped at the matrix edges.  `stage` is this warp's slot area (nslots slots of 4 KiB,
// 1024-byte aligned), `stores` its running count of committed stores, which picks the slot;
// before a slot is rewritten the store that last read it must have finished reading.  A TMA
// store clips the contiguous dimension in units of 16 bytes, not of elements, so the tensor map
// covers only the first No8 = No rounded down to 8 columns; the up to 7 columns after them are
// stored from registers.
//
// One warp per scheduler runs this, so its speed is set by the length of its dependent
// instruction chains: the two chunks of a group are converted side by side, and the inf/NaN
// test (weight gradient only) is two integer operations per packed pair.
constexpr int SLOT_BYTES = 32 * 64 * 2;

// One chunk (32 columns from col0) of this thread's row, FP16 modes: optional bias and
// activation on the FP32 sums, rounding, optional activation mask, columns and rows that do not
// exist, the inf/NaN test, the register-stored tail columns, and the 64 bytes of the row into
// the staging slot (half = 0 / 1: first or second chunk of the 64-column group).
template <bool FUSED>
__device__ __forceinline__ void finish_chunk(const GemmParams& p, uint32_t (&r)[32], int col0, int row,
                                             bool row_ok, int lane, uint8_t* slot, int half,
                                             const uint32_t* pass_bits, int c, uint32_t& flag_acc,
                                             int prob) {
  const uint16_t* bias = FUSED ? p.bias[prob] : nullptr;
  if (FUSED && (bias != nullptr || (p.act != 0 && p.mask == nullptr))) {
    // forward flavour, on the FP32 values: + bias, then the activation
    uint32_t bw[16];                          // 32 bias values as packed halves (0 if absent)
    if (bias != nullptr && col0 + 32 <= p.No) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {           // same address in every thread: one broadcast load
        const uint4 q4 = __ldg(reinterpret_cast<const uint4*>(bias + col0) + j);
        bw[4 * j] = q4.x; bw[4 * j + 1] = q4.y; bw[4 * j + 2] = q4.z; bw[4 * j + 3] = q4.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t lo = (bias != nullptr && col0 + 2 * j < p.No) ? __ldg(bias + col0 + 2 * j) : 0u;
        const uint32_t hi = (bias != nullptr && col0 + 2 * j + 1 < p.No) ? __ldg(bias + col0 + 2 * j + 1) : 0u;
        bw[j] = lo | (hi << 16);
      }
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      float x = __uint_as_float(r[j]);
      if (bias != nullptr) {
        const uint16_t hb = (uint16_t)((j & 1) ? (bw[j >> 1] >> 16) : (bw[j >> 1] & 0xFFFFu));
        x = __fadd_rn(x, __half2float(__ushort_as_half(hb)));
      }
      if (p.act != 0) {
        x = x > 0.0f ? x : 0.0f;
        if (p.act == 2) x = x < p.clip ? x : p.clip;
      }
      r[j] = __float_as_uint(x);
    }
  }
  uint32_t h[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const __half2 v = __floats2half2_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
    h[j] = *reinterpret_cast<const uint32_t*>(&v);
  }
  if (FUSED && pass_bits != nullptr) {
    // data-gradient flavour: keep the value only where the layer input passes the activation
    const uint32_t bits = pass_bits[c];
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (!((bits >> j) & 1u)) h[j >> 1] &= (j & 1) ? 0x0000FFFFu : 0xFFFF0000u;
  }
  if (col0 + 32 > p.No) {
    // columns beyond No (dropped by the store) must not raise the flag: 0 x inf is NaN
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (col0 + j >= p.No) h[j >> 1] &= (j & 1) ? 0x0000FFFFu : 0xFFFF0000u;
  }
  if (row_ok) {                               // rows beyond Mo are dropped by the store
    if (p.out_mode == OUT_F16_FLAG) {
      // a half is inf or NaN iff its exponent field is 0x7C00; adding 0x0400 to the isolated
      // field then carries into bit 15 (and no further), for both halves of the word at once
#pragma unroll
      for (int j = 0; j < 16; ++j) flag_acc |= (h[j] & 0x7C007C00u) + 0x04000400u;
    }
    if (col0 + 32 > p.No8) {                  // the columns past the tensor map's last 16-byte unit
      uint16_t* dst = p.out[prob] + (int64_t)row * p.ldo + col0;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col0 + j >= p.No8 && col0 + j < p.No)
          dst[j] = (uint16_t)((j & 1) ? (h[j >> 1] >> 16) : (h[j >> 1] & 0xFFFFu));
    }
  }
  uint8_t* rowp = slot + lane * 128;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int piece = half * 4 + j;           // 16-byte piece of the 128-byte row segment
    *reinterpret_cast<uint4*>(rowp + ((piece ^ (lane & 7)) << 4)) =
        make_uint4(h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
  }
}

// Epilogue of one accumulator for one warp: this thread owns output row `row` (TMEM lane) and
// the warp walks chunks c_begin .. c_begin + c_count (32 columns each, both even) of the tile
// whose first column is n0.  tmem_acc is the TMEM address of the accumulator's first column in
// this warp's lane quarter.  Returns nonzero if an inf or NaN was stored by the weight gradient.
// The store half of a group: wait for the slot, round and stage both chunks, hand the slot over.
template <bool FUSED>
__device__ __forceinline__ void finish_group(const GemmParams& p, const CUtensorMap* map_out, uint8_t* stage,
                                             int nslots, int& stores, uint32_t (&ra)[32], uint32_t (&rb)[32],
                                             bool second, int colg, int g, int row, bool row_ok, int lane,
                                             const uint32_t* pass_bits, uint32_t& flag_acc, int prob) {
  uint8_t* slot = stage + (stores % nslots) * SLOT_BYTES;
  // the slot must no longer be read by an earlier store
  if (lane == 0) {
    if (nslots == 2) ptx::bulk_wait_group_read<1>(); else ptx::bulk_wait_group_read<0>();
  }
  __syncwarp();
  finish_chunk<FUSED>(p, ra, colg, row, row_ok, lane, slot, 0, pass_bits, 2 * g, flag_acc, prob);
  if (second)
    finish_chunk<FUSED>(p, rb, colg + 32, row, row_ok, lane, slot, 1, pass_bits, 2 * g + 1, flag_acc, prob);
  ptx::fence_proxy_async_smem();                // the slot is complete: hand it to the TMA unit
  __syncwarp();
  if (colg < p.No8) {                           // else: only register-stored columns in this group
    if (lane == 0) {
      ptx::tma_store_2d(map_out, slot, colg, row - lane);
      ptx::bulk_commit_group();
    }
    ++stores;
  }
}

// Epilogue of one accumulator for one warp: this thread owns output row `row` (TMEM lane) and
// the warp walks chunks c_begin .. c_begin + c_count (32 columns each, both even) of the tile
// whose first column is n0.  tmem_acc is the TMEM address of the accumulator's first column in
// this warp's lane quarter.  Returns nonzero if an inf or NaN was stored by the weight gradient.
// FUSED is the kernel's flavour (bias / activation / mask code present, eight epilogue warps);
// the plain flavour carries none of that code: one warp per scheduler runs this, and a short
// instruction stream matters more to it than anything else.
template <bool FUSED>
__device__ __forceinline__ uint32_t epilogue_tile(const GemmParams& p, const CUtensorMap* map_out,
                                                  const CUtensorMap* map_ws, uint8_t* stage, int nslots,
                                                  int& stores,
                                                  uint32_t tmem_acc, int row, int n0, int split,
                                                  int c_begin, int c_count, int prob,
                                                  const uint32_t* pass_bits = nullptr) {
  const bool row_ok = row < p.Mo;
  const int lane = threadIdx.x & 31;
  if (row - lane >= p.Mo) return 0;             // nothing of this warp's rows exists
  if (p.out_mode == OUT_PARTIAL) {
    // FP32 partial sums of a split reduction: a chunk (32 rows x 32 floats = 4 KiB) fills one
    // staging slot; the workspace map is [split][row][column], so rows beyond Mo are clipped
    // instead of landing in the next split's plane (its padded row length is a multiple of 4
    // floats, so the 16-byte clipping of the columns is exact)
#pragma unroll 1
    for (int c = c_begin; c < c_begin + c_count; ++c) {
      const int col0 = n0 + c * 32;
      if (col0 >= p.No) break;                  // warp-uniform
      uint8_t* slot = stage + (stores % nslots) * SLOT_BYTES;
      if (lane == 0) {
        if (nslots == 2) ptx::bulk_wait_group_read<1>(); else ptx::bulk_wait_group_read<0>();
      }
      __syncwarp();
      uint32_t r[32];
      ptx::tmem_ld_32x32(tmem_acc + c * 32, r);
      ptx::tmem_ld_wait();
      uint8_t* rowp = slot + lane * 128;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<uint4*>(rowp + ((j ^ (lane & 7)) << 4)) =
            make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        ptx::tma_store_3d(map_ws, slot, col0, row - lane, split);
        ptx::bulk_commit_group();
      }
      ++stores;
    }
    return 0;
  }
  uint32_t flag_acc = 0;
  // groups of 64 columns g_begin .. g_end that have columns (warp-uniform)
  const int g_begin = c_begin >> 1;
  int g_end = (c_begin + c_count) >> 1;
  if (n0 + g_end * 64 > p.No) g_end = (p.No - n0 + 63) >> 6;
  if (g_end <= g_begin) return 0;
#pragma unroll 1
  for (int g = g_begin; g < g_end; ++g) {
    const int colg = n0 + g * 64;               // first column of the 64-column group
    const bool second = colg + 32 < p.No;       // the group's second chunk has columns
    uint32_t ra[32], rb[32];
    ptx::tmem_ld_32x32(tmem_acc + g * 64, ra);
    if (second) ptx::tmem_ld_32x32(tmem_acc + g * 64 + 32, rb);
    ptx::tmem_ld_wait();
    finish_group<FUSED>(p, map_out, stage, nslots, stores, ra, rb, second, colg, g, row, row_ok, lane,
                        pass_bits, flag_acc, prob);
  }
  return flag_acc & 0x80008000u;
}

template <bool A_MN, bool B_MN, bool WIDE>
__global__ void __launch_bounds__(WIDE ? THREADS_FUSED : THREADS_PLAIN, 1)
mp_gemm_kernel(const __grid_constant__ GroupMaps maps, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* staging = smem + STAGES * STAGE_BYTES;
  Barriers* bars = reinterpret_cast<Barriers*>(staging + STAGING_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  ptx::launch_dependents();    // the next kernel's CTAs may take SMs as soon as ours leave them

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&bars->full[s], 1);
      ptx::mbar_init(&bars->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&bars->tmem_full[a], 1);
      ptx::mbar_init(&bars->tmem_empty[a], blockDim.x - 64);
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&maps.a[0]);
    ptx::prefetch_tensormap(&maps.b[0]);
    ptx::prefetch_tensormap(&maps.out[0]);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  // Everything above (barriers, tensor memory, descriptor prefetch) may overlap the tail of the
  // previous kernel in the stream; nothing below may.
  ptx::grid_dependency_wait();

  const int total_work = p.group * p.work_per_problem;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    // (no_loads: the error-path self-test; nothing is issued, so nothing is in flight at exit)
    for (int w = blockIdx.x; w < total_work && ok && !p.no_loads; w += gridDim.x) {
      const int prob = w / p.work_per_problem, wl = w - prob * p.work_per_problem;
      const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
      const CUtensorMap* map_a = &maps.a[prob];
      const CUtensorMap* map_b = &maps.b[prob];
      const int m0 = tile_m(p, tile) * BM, n0 = tile_n(p, tile) * BN;
      const int b_boxes = B_MN ? (tile_width(p.No, n0) + 63) / 64 : BN / 64;   // 64-column boxes of B
      const int kb0 = (int)((int64_t)split * p.num_kb / p.splits);
      const int kb1 = (int)((int64_t)(split + 1) * p.num_kb / p.splits);
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(&bars->empty[stage], phase ^ 1, p.wait_ns)) { ok = false; break; }
        if (lane == 0) {
          uint8_t* sA = smem + stage * STAGE_BYTES;
          uint8_t* sB = sA + A_BYTES;
          ptx::mbar_arrive_expect_tx(&bars->full[stage], A_BYTES + b_boxes * CHUNK_BYTES);
          const int k = kb * BK;
          if (A_MN) {
#pragma unroll
            for (int c = 0; c < BM / 64; ++c)
              ptx::tma_load_2d(sA + c * CHUNK_BYTES, map_a, &bars->full[stage], m0 + 64 * c, k);
          } else {
            ptx::tma_load_2d(sA, map_a, &bars->full[stage], k, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int c = 0; c < BN / 64; ++c)
              if (c < b_boxes)
                ptx::tma_load_2d(sB + c * CHUNK_BYTES, map_b, &bars->full[stage], n0 + 64 * c, k);
          } else {
            ptx::tma_load_2d(sB, map_b, &bars->full[stage], k, n0);
          }
        }
        __syncwarp();
        ++issued;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
    if (!ok) report_timeout(bars, p);
    if (!ok || bars->abort) {
      // Leaving early: wait (bounded) until the loads already issued have landed, so that no
      // copy is in flight into this CTA's shared memory when it exits.
      const int pending = issued < STAGES ? issued : STAGES;
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = STAGES - 1; phase ^= 1; }
        ptx::mbar_wait(&bars->full[stage], phase, p.wait_ns);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    int stage = 0;
    uint32_t phase = 0;
    int iter = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < total_work && ok; w += gridDim.x, ++iter) {
      const int wl = w % p.work_per_problem;
      const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
      const uint32_t idesc =
          ptx::idesc_f16_f32(BM, tile_width(p.No, tile_n(p, tile) * BN), A_MN, B_MN);
      const int kb0 = (int)((int64_t)split * p.num_kb / p.splits);
      const int kb1 = (int)((int64_t)(split + 1) * p.num_kb / p.splits);
      const int acc = iter & 1;
      const uint32_t acc_phase = (iter >> 1) & 1;
      if (!ptx::mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, p.wait_ns)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(&bars->full[stage], phase, p.wait_ns)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        if (lane == 0) {
          const uint32_t sA = ptx::smem_u32(smem + stage * STAGE_BYTES);
          const uint32_t sB = sA + A_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            // K-major operand: rows of 128 B, 8-row groups 1024 B apart, a K step of 16
            // elements is 32 B inside the swizzled row.  MN-major operand: 64-element column
            // blocks 8 KiB apart (leading offset), 8 reduction rows per 1024 B (stride
            // offset), a K step of 16 rows is 2 KiB.
            const uint64_t da = A_MN ? ptx::smem_desc_sw128(sA + kk * 2048, CHUNK_BYTES, 1024)
                                     : ptx::smem_desc_sw128(sA + kk * 32, 16, 1024);
            const uint64_t db = B_MN ? ptx::smem_desc_sw128(sB + kk * 2048, CHUNK_BYTES, 1024)
                                     : ptx::smem_desc_sw128(sB + kk * 32, 16, 1024);
            ptx::mma_f16_ss(d_tmem, da, db, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
          }
          ptx::mma_commit(&bars->empty[stage]);   // frees the stage when these MMAs are done
        }
        __syncwarp();
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      if (ok && lane == 0) ptx::mma_commit(&bars->tmem_full[acc]);
      __syncwarp();
    }
    if (!ok) report_timeout(bars, p);
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                         // TMEM lane quarter this warp may read
    const int c_count = (BN / 32) / ((int)(blockDim.x / 32 - 2) / 4);   // column chunks per warp: 8 or 4
    const int c_begin = ((warp - 2) >> 2) * c_count;                    // its share of the tile's columns
    const int nslots = 8 / ((int)blockDim.x / 32 - 2);                  // staging slots per warp: 2 or 1
    uint8_t* stage = staging + (warp - 2) * nslots * SLOT_BYTES;
    int stores = 0;
    int iter = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < total_work && ok; w += gridDim.x, ++iter) {
      const int prob = w / p.work_per_problem, wl = w - prob * p.work_per_problem;
      const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
      const int m0 = tile_m(p, tile) * BM, n0 = tile_n(p, tile) * BN;
      const int acc = iter & 1;
      const uint32_t acc_phase = (iter >> 1) & 1;
      const int row = m0 + q * 32 + lane;
      uint32_t pass_bits[BN / 32];
      const bool masked = p.mask != nullptr && p.act != 0 && p.out_mode != OUT_PARTIAL;
      if (masked) load_pass_bits(p, row, n0, c_begin, c_count, pass_bits);   // runs under the tile's main loop
      if (!ptx::mbar_wait(&bars->tmem_full[acc], acc_phase, p.wait_ns)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const uint32_t bad = epilogue_tile<WIDE>(p, &maps.out[prob], &maps.ws[prob], stage, nslots, stores,
                                         tmem_base + acc * BN + ((uint32_t)(q * 32) << 16), row, n0, split,
                                         c_begin, c_count, prob, masked ? pass_bits : nullptr);
      if (p.out_mode == OUT_F16_FLAG && p.flag != nullptr) {
        if (__any_sync(0xFFFFFFFFu, bad != 0) && lane == 0) atomicOr(p.flag, 1);
      }
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(&bars->tmem_empty[acc]);
    }
    if (!ok) report_timeout(bars, p);
    if (lane == 0) ptx::bulk_wait_group_all();   // this warp's output stores have left shared memory
  }

  // ---------------------------------------------------------------- teardown
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------ CTA-pair kernel
// Same pipeline on a cluster of two CTAs (two SMs) that share one 256 x 256 output tile through
// tcgen05.mma.cta_group::2: CTA r of the pair loads rows [128 r, 128 r + 128) of the A tile and
// columns [128 r, 128 r + 128) of the B tile into its own shared memory (plain TMA loads, no
// multicast), the leader CTA issues every MMA, and each CTA's tensor memory receives the 128
// output rows it loaded A for.  Per SM that halves the B bytes read from shared memory per
// flop and shrinks a stage to 32 KiB, so six stages fit.
constexpr int STAGES2 = 6;
constexpr int HALF_BYTES = 128 * BK * 2;            // 16 KiB: half a tile of A or of B
constexpr int STAGE2_BYTES = 2 * HALF_BYTES;
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + STAGING_BYTES + 1024 + 256;

struct Barriers2 {
  uint64_t full[STAGES2];     // used in the leader: both CTAs' loads of a stage have landed
  uint64_t empty[STAGES2];    // in each CTA: the MMAs that read the stage are done
  uint64_t tmem_full[2];      // in each CTA: accumulator ready for the epilogue
  uint64_t tmem_empty[2];     // used in the leader: both CTAs' epilogues have drained it
  uint32_t tmem_base;
  volatile uint32_t abort;
};

template <bool A_MN, bool B_MN, bool WIDE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(WIDE ? THREADS_FUSED : THREADS_PLAIN, 1)
mp_gemm_pair_kernel(const __grid_constant__ GroupMaps maps, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* staging = smem + STAGES2 * STAGE2_BYTES;
  Barriers2* bars = reinterpret_cast<Barriers2*>(staging + STAGING_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const bool leader = rank == 0;
  ptx::launch_dependents();    // the next kernel's CTAs may take SMs as soon as ours leave them

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) {
      ptx::mbar_init(&bars->full[s], 1);            // the leader's arrive; bytes of both CTAs
      ptx::mbar_init(&bars->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&bars->tmem_full[a], 1);
      ptx::mbar_init(&bars->tmem_empty[a], 2 * (blockDim.x / 32 - 2));   // one arrive per epilogue warp of each CTA
    }
    bars->abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&maps.a[0]);
    ptx::prefetch_tensormap(&maps.b[0]);
    if (!B_MN) ptx::prefetch_tensormap(&maps.b32[0]);
    ptx::prefetch_tensormap(&maps.out[0]);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(&bars->tmem_base, TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();                              // both CTAs' barriers exist before any remote arrive
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  // Everything above may overlap the tail of the previous kernel in the stream; nothing below may.
  ptx::grid_dependency_wait();

  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total_work = p.group * p.work_per_problem;   // m_tiles counts 256-row tiles here

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    for (int w = pair; w < total_work && ok; w += npairs) {
      const int prob = w / p.work_per_problem, wl = w - prob * p.work_per_problem;
      const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
      const CUtensorMap* map_a = &maps.a[prob];
      const CUtensorMap* map_b = &maps.b[prob];
      const CUtensorMap* map_b32 = &maps.b32[prob];
      const int m0 = tile_m(p, tile) * 256 + 128 * (int)rank;
      // this CTA's half of the tile's columns: 128 of a full tile, fewer of a narrow last one.
      // B arrives in boxes of 64 columns (output dimension contiguous) or, for a narrow tile
      // of a reduction-contiguous B, in boxes of 32 rows from the second tensor map; only the
      // boxes that the MMAs read are fetched.
      const int n_base = tile_n(p, tile) * BN;
      const int half = tile_width(p.No, n_base) >> 1;
      const int n0 = n_base + half * (int)rank;
      const int b_boxes = B_MN ? (half + 63) / 64 : (half + 31) / 32;
      const uint32_t b_bytes = B_MN ? b_boxes * CHUNK_BYTES : b_boxes * (32 * BK * 2);
      const int kb0 = (int)((int64_t)split * p.num_kb / p.splits);
      const int kb1 = (int)((int64_t)(split + 1) * p.num_kb / p.splits);
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(&bars->empty[stage], phase ^ 1, p.wait_ns)) { ok = false; break; }
        if (lane == 0) {
          uint8_t* sA = smem + stage * STAGE2_BYTES;
          uint8_t* sB = sA + HALF_BYTES;
          const uint32_t full = ptx::map_to_cta(ptx::smem_u32(&bars->full[stage]), 0);
          // Only the leader arrives, expecting both CTAs' bytes.  The peer's bytes can reach the
          // barrier before this arrive (the count of bytes still to come just goes negative
          // for a moment); they cannot reach it before the previous phase has completed,
          // because the peer refills a stage only after the MMAs that read it are done.
          if (leader) ptx::mbar_arrive_expect_tx(&bars->full[stage], 2 * (HALF_BYTES + b_bytes));
          const int k = kb * BK;
          if (A_MN) {
            ptx::tma_load_2d_pair(sA, map_a, full, m0, k);
            ptx::tma_load_2d_pair(sA + CHUNK_BYTES, map_a, full, m0 + 64, k);
          } else {
            ptx::tma_load_2d_pair(sA, map_a, full, k, m0);
          }
          if (B_MN) {
            ptx::tma_load_2d_pair(sB, map_b, full, n0, k);
            if (b_boxes > 1) ptx::tma_load_2d_pair(sB + CHUNK_BYTES, map_b, full, n0 + 64, k);
          } else if (b_boxes == 4) {
            ptx::tma_load_2d_pair(sB, map_b, full, k, n0);
          } else {
            for (int c = 0; c < b_boxes; ++c)   // 32 rows of 128 B each: 4 KiB apart, whole swizzle groups
              ptx::tma_load_2d_pair(sB + c * (32 * BK * 2), map_b32, full, k, n0 + 32 * c);
          }
        }
        __syncwarp();
        ++issued;
        if (++stage == STAGES2) { stage = 0; phase ^= 1; }
      }
    }
    if (!ok) report_timeout(bars, p);
    if (leader && (!ok || bars->abort)) {
      // Leaving early: the leader's "full" barriers count both CTAs' bytes, so waiting on
      // them (bounded) covers every load still in flight into either CTA; the peer cannot
      // exit before the cluster barrier below.
      const int pending = issued < STAGES2 ? issued : STAGES2;
      for (int i = 0; i < pending; ++i) {
        if (--stage < 0) { stage = STAGES2 - 1; phase ^= 1; }
        ptx::mbar_wait(&bars->full[stage], phase, p.wait_ns);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader) {
      int stage = 0;
      uint32_t phase = 0;
      int iter = 0;
      bool ok = true;
      for (int w = pair; w < total_work && ok; w += npairs, ++iter) {
        const int wl = w % p.work_per_problem;
        const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
        const uint32_t idesc =
            ptx::idesc_f16_f32(256, tile_width(p.No, tile_n(p, tile) * BN), A_MN, B_MN);
        const int kb0 = (int)((int64_t)split * p.num_kb / p.splits);
        const int kb1 = (int)((int64_t)(split + 1) * p.num_kb / p.splits);
        const int acc = iter & 1;
        const uint32_t acc_phase = (iter >> 1) & 1;
        if (!ptx::mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, p.wait_ns)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(&bars->full[stage], phase, p.wait_ns)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          if (lane == 0) {
            const uint32_t sA = ptx::smem_u32(smem + stage * STAGE2_BYTES);
            const uint32_t sB = sA + HALF_BYTES;
#pragma unroll
            for (int kk = 0; kk < BK / UMMA_K; ++kk) {
              const uint64_t da = A_MN ? ptx::smem_desc_sw128(sA + kk * 2048, CHUNK_BYTES, 1024)
                                       : ptx::smem_desc_sw128(sA + kk * 32, 16, 1024);
              const uint64_t db = B_MN ? ptx::smem_desc_sw128(sB + kk * 2048, CHUNK_BYTES, 1024)
                                       : ptx::smem_desc_sw128(sB + kk * 32, 16, 1024);
              ptx::mma_f16_ss_pair(d_tmem, da, db, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
            }
            ptx::mma_commit_pair(&bars->empty[stage], 3);   // frees the stage in both CTAs
          }
          __syncwarp();
          if (++stage == STAGES2) { stage = 0; phase ^= 1; }
        }
        if (ok && lane == 0) ptx::mma_commit_pair(&bars->tmem_full[acc], 3);
        __syncwarp();
      }
      if (!ok) report_timeout(bars, p);
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs)
    const int q = warp & 3;
    const int c_count = (BN / 32) / ((int)(blockDim.x / 32 - 2) / 4);
    const int c_begin = ((warp - 2) >> 2) * c_count;
    const int nslots = 8 / ((int)blockDim.x / 32 - 2);
    uint8_t* stage = staging + (warp - 2) * nslots * SLOT_BYTES;
    int stores = 0;
    int iter = 0;
    bool ok = true;
    for (int w = pair; w < total_work && ok; w += npairs, ++iter) {
      const int prob = w / p.work_per_problem, wl = w - prob * p.work_per_problem;
      const int tiles = p.m_tiles * p.n_tiles, split = wl / tiles, tile = wl - split * tiles;
      const int m0 = tile_m(p, tile) * 256 + 128 * (int)rank, n0 = tile_n(p, tile) * BN;
      const int acc = iter & 1;
      const uint32_t acc_phase = (iter >> 1) & 1;
      const int row = m0 + q * 32 + lane;
      uint32_t pass_bits[BN / 32];
      const bool masked = p.mask != nullptr && p.act != 0 && p.out_mode != OUT_PARTIAL;
      if (masked) load_pass_bits(p, row, n0, c_begin, c_count, pass_bits);   // runs under the tile's main loop
      if (!ptx::mbar_wait(&bars->tmem_full[acc], acc_phase, p.wait_ns)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const uint32_t bad =
          epilogue_tile<WIDE>(p, &maps.out[prob], &maps.ws[prob], stage, nslots, stores,
                        tmem_base + acc * BN + ((uint32_t)(q * 32) << 16), row, n0, split, c_begin,
                        c_count, prob, masked ? pass_bits : nullptr);
      if (p.out_mode == OUT_F16_FLAG && p.flag != nullptr) {
        if (__any_sync(0xFFFFFFFFu, bad != 0) && lane == 0) atomicOr(p.flag, 1);
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0)
        ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&bars->tmem_empty[acc]), 0));
    }
    if (!ok) report_timeout(bars, p);
    if (lane == 0) ptx::bulk_wait_group_all();   // this warp's output stores have left shared memory
  }

  // ---------------------------------------------------------------- teardown
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();        // neither CTA's shared or tensor memory goes away under the other
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// Adds the split partial sums in ascending split order, rounds to FP16, stores, inspects.
__global__ void __launch_bounds__(256)
mp_splitk_reduce_kernel(const float* __restrict__ ws, int splits, int Mo, int No, int64_t ws_ld,
                        uint16_t* __restrict__ out, int64_t ldo, int* flag) {
  const int vec_per_row = (No + 3) / 4;
  const int64_t total = (int64_t)Mo * vec_per_row;
  const int64_t split_stride = (int64_t)Mo * ws_ld;
  uint32_t bad = 0;
  // Launched with programmatic stream serialization: the blocks may be resident before the
  // product kernel has finished, and wait here until its partial sums are complete and visible.
  ptx::launch_dependents();
  ptx::grid_dependency_wait();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / vec_per_row);
    const int col = (int)(i % vec_per_row) * 4;
    const float* src = ws + (int64_t)row * ws_ld + col;
    if (col + 4 <= No) {
      float4 acc = *reinterpret_cast<const float4*>(src);
      int s = 1;
      for (; s + 3 < splits; s += 4) {            // four loads in flight, added in ascending order
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = *reinterpret_cast<const float4*>(src + (s + u) * split_stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc.x = __fadd_rn(acc.x, x[u].x); acc.y = __fadd_rn(acc.y, x[u].y);
          acc.z = __fadd_rn(acc.z, x[u].z); acc.w = __fadd_rn(acc.w, x[u].w);
        }
      }
      for (; s < splits; ++s) {
        const float4 x = *reinterpret_cast<const float4*>(src + s * split_stride);
        acc.x = __fadd_rn(acc.x, x.x); acc.y = __fadd_rn(acc.y, x.y);
        acc.z = __fadd_rn(acc.z, x.z); acc.w = __fadd_rn(acc.w, x.w);
      }
      const __half2 lo = __floats2half2_rn(acc.x, acc.y), hi = __floats2half2_rn(acc.z, acc.w);
      const uint2 pk = make_uint2(*reinterpret_cast<const uint32_t*>(&lo),
                                  *reinterpret_cast<const uint32_t*>(&hi));
      *reinterpret_cast<uint2*>(out + (int64_t)row * ldo + col) = pk;
      bad |= pair_nonfinite(pk.x) | pair_nonfinite(pk.y);
    } else {
      for (int j = 0; col + j < No; ++j) {
        float a = src[j];
        for (int s = 1; s < splits; ++s) a = __fadd_rn(a, src[j + s * split_stride]);
        const uint16_t hv = __half_as_ushort(__float2half_rn(a));
        out[(int64_t)row * ldo + col + j] = hv;
        bad |= ((hv & 0x7C00u) == 0x7C00u) ? 1u : 0u;
      }
    }
  }
  if (flag != nullptr && __any_sync(0xFFFFFFFFu, bad != 0) && (threadIdx.x & 31) == 0)
    atomicOr(flag, 1);
}

// ------------------------------------------------------------------ host side
// One-time set-up per device and per kernel flavour (attribute calls, occupancy and symbol
// queries) is serialised by this mutex, so that first calls from several host threads are safe.
std::mutex g_setup_mutex;

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

int load_encoder() {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_encode) return MP_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  MP_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (qres != cudaDriverEntryPointSuccess || !fn)
    return mp::set_error(MP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  return MP_OK;
}

// 2-D FP16 tensor map: `inner` contiguous elements per row, `outer` rows, row pitch ld elements.
int make_map(CUtensorMap* map, const void* ptr, int64_t inner, int64_t outer, int64_t ld,
             int box_inner, int box_outer) {
  const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), dims,
                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return mp::set_error(MP_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return MP_OK;
}

// 3-D FP32 tensor map over the split-reduction workspace: `ld` floats per row (a multiple of 4),
// `rows` rows per split, `splits` planes; one box is 32 floats x 32 rows of one plane.
int make_map_ws(CUtensorMap* map, const void* ptr, int64_t ld, int64_t rows, int64_t splits) {
  const cuuint64_t dims[3] = {(cuuint64_t)ld, (cuuint64_t)rows, (cuuint64_t)splits};
  const cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)rows * (cuuint64_t)ld * 4};
  const cuuint32_t box[3] = {32, 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(ptr), dims,
                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return mp::set_error(MP_ERR_CUDA, "cuTensorMapEncodeTiled (workspace) failed with code %d", (int)r);
  return MP_OK;
}

// SM count of the current device (the heuristics below size waves with it); kFallbackSMs when no
// device can be asked, so that a workspace query still answers.
constexpr int kMaxDevicesCached = 64;
int model_sms() {
  static int sms_of[kMaxDevicesCached] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevicesCached) { cudaGetLastError(); return kFallbackSMs; }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (sms_of[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      cudaGetLastError();
      return kFallbackSMs;
    }
    sms_of[dev] = n;
  }
  return sms_of[dev];
}

// Number of reduction splits: minimise a simple time model (waves of tiles on the SMs plus
// the workspace round trip).  Depends only on the sizes, so that the workspace query and the
// launch always agree.
// Output tiles of more than 128 rows go to the CTA-pair kernel (256 x 256 tiles, one per SM pair).
bool use_pair_kernel(int64_t Mo) { return Mo > 128; }

int choose_splits(int64_t Mo, int64_t No, int64_t R, int64_t count = 1) {
  const bool pair = use_pair_kernel(Mo);
  const int64_t bm = pair ? 256 : BM;
  const int sms = model_sms();
  const int64_t slots = pair ? sms / 2 : sms;
  const int64_t tiles = count * ((Mo + bm - 1) / bm) * ((No + BN - 1) / BN);
  const int64_t num_kb = (R + BK - 1) / BK;
  const double t_kb = 0.42e-6;                   // one 128x256x64 block per SM at ~1.0e13 flop/s
  const double bw = 4.0e12;                      // workspace traffic, bytes/s
  int best = 1;
  double best_t = 1e30;
  for (int s = 1; s <= 16 && s * 4 <= num_kb; ++s) {
    const int64_t work = tiles * s;
    const int64_t waves = (work + slots - 1) / slots;
    double t = (double)waves * (double)((num_kb + s - 1) / s) * t_kb;
    if (s > 1) t += (double)count * ((double)Mo * (double)No * (8.0 * s + 2.0) / bw + 3e-6);
    if (t < best_t * 0.97) { best_t = t; best = s; }
  }
  return best;
}

int64_t ws_ld_for(int64_t No) { return (No + 3) / 4 * 4; }

struct Fuse {
  const void* bias = nullptr;          // single problem
  const void* const* biases = nullptr; // grouped call: one per problem (overrides `bias`)
  const void* mask = nullptr;
  int64_t ldmask = 0;
  int act = 0;
  float clip = 0.0f;
  uint64_t wait_ns = ptx::kWaitNs;     // limit of the kernel's barrier waits
  bool no_loads = false;               // error-path self-test: the producer issues nothing
};

struct Operand {
  const void* ptr;
  int64_t ld;
  bool mn_major;      // true: the output dimension is the contiguous one
  int64_t mn, red;    // extents along the output dimension and the reduction
};

// The per-kernel set-up below (shared-memory opt-in, cluster occupancy) is a property of the
// device the call runs on, so it is remembered per device index.
int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
  return dev % kMaxDevicesCached;
}

template <bool A_MN, bool B_MN, bool WIDE>
int launch(const GroupMaps& maps, const GemmParams& p, int grid, cudaStream_t st) {
  static bool attr_set[kMaxDevicesCached] = {};
  const int slot = current_device_slot();
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!attr_set[slot]) {
      MP_CUDA_TRY(cudaFuncSetAttribute(mp_gemm_kernel<A_MN, B_MN, WIDE>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
      attr_set[slot] = true;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(WIDE ? THREADS_FUSED : THREADS_PLAIN, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  MP_CUDA_TRY(cudaLaunchKernelEx(&cfg, mp_gemm_kernel<A_MN, B_MN, WIDE>, maps, p));
  mp::count_launch();
  return MP_OK;
}

template <bool A_MN, bool B_MN, bool WIDE>
int launch_pair(const GroupMaps& maps, const GemmParams& p, int64_t work, cudaStream_t st) {
  static int max_pairs_of[kMaxDevicesCached] = {};
  std::unique_lock<std::mutex> lock(g_setup_mutex);
  int max_pairs = max_pairs_of[current_device_slot()];
  if (max_pairs == 0) {
    MP_CUDA_TRY(cudaFuncSetAttribute(mp_gemm_pair_kernel<A_MN, B_MN, WIDE>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    int sms = 0, dev = 0;
    MP_CUDA_TRY(cudaGetDevice(&dev));
    MP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * sms, 1, 1);
    cfg.blockDim = dim3(WIDE ? THREADS_FUSED : THREADS_PLAIN, 1, 1);
    cfg.dynamicSmemBytes = SMEM2_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    MP_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, mp_gemm_pair_kernel<A_MN, B_MN, WIDE>, &cfg));
    if (n < 1) return mp::set_error(MP_ERR_CUDA, "no CTA pair of the GEMM kernel fits on this device");
    max_pairs = max_pairs_of[current_device_slot()] = n;
  }
  lock.unlock();
  const int pairs = (int)(work < max_pairs ? work : max_pairs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(WIDE ? THREADS_FUSED : THREADS_PLAIN, 1, 1);
  cfg.dynamicSmemBytes = SMEM2_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  MP_CUDA_TRY(cudaLaunchKernelEx(&cfg, mp_gemm_pair_kernel<A_MN, B_MN, WIDE>, maps, p));
  mp::count_launch();
  return MP_OK;
}

// `count` products of one shape and one set of layouts (operands As[i], Bs[i], outputs outs[i]).
// dstate: the caller's device state or null; its status word receives device-side errors and, when
// want_flag is set, its found_inf word the inspection of what is stored.
int run_gemm(const char* name, int count, const Operand* As, const Operand* Bs, void* const* outs,
             int64_t ldo, mp_dev_state* dstate, bool want_flag, void* workspace, size_t ws_bytes, cudaStream_t st,
             const Fuse& fuse = Fuse()) {
  int* flag = dstate ? &dstate->h.found_inf : nullptr;
  want_flag = want_flag && flag != nullptr;
  if (count < 1 || count > MAX_GROUP)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: between 1 and %d problems per call", name, MAX_GROUP);
  const Operand& A = As[0];
  const Operand& B = Bs[0];
  const int64_t Mo = A.mn, No = B.mn, R = A.red;
  for (int i = 0; i < count; ++i)
    if (!As[i].ptr || !Bs[i].ptr || !outs[i]) return mp::set_error(MP_ERR_INVALID_ARG, "%s: null pointer", name);
  if (Mo <= 0 || No <= 0 || R <= 0)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: sizes must be positive", name);
  if (Mo > INT32_MAX / 2 || No > INT32_MAX / 2 || R > INT32_MAX / 2)
    return mp::set_error(MP_ERR_TOO_LARGE, "%s: a dimension exceeds 2^30", name);
  const int64_t a_inner = A.mn_major ? A.mn : A.red, b_inner = B.mn_major ? B.mn : B.red;
  if (A.ld < a_inner || B.ld < b_inner || ldo < No)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: leading dimension smaller than the row length", name);
  if ((A.ld | B.ld | ldo) & 7)
    return mp::set_error(MP_ERR_ALIGNMENT, "%s: leading dimensions must be multiples of 8", name);
  for (int i = 0; i < count; ++i)
    if (!mp::aligned16(As[i].ptr) || !mp::aligned16(Bs[i].ptr) || !mp::aligned16(outs[i]))
      return mp::set_error(MP_ERR_ALIGNMENT, "%s: pointers must be 16-byte aligned", name);
  if (workspace && !mp::aligned16(workspace))
    return mp::set_error(MP_ERR_ALIGNMENT, "%s: pointers must be 16-byte aligned", name);
  if (int rc = mp::check_device()) return rc;
  if (int rc = load_encoder()) return rc;

  const int64_t No8 = No & ~(int64_t)7;
  GemmParams p;
  p.group = count;
  p.Mo = (int)Mo; p.No = (int)No; p.R = (int)R; p.No8 = (int)No8;
  const bool pair = use_pair_kernel(Mo);
  p.m_tiles = (int)(pair ? (Mo + 255) / 256 : (Mo + BM - 1) / BM);
  p.n_tiles = (int)((No + BN - 1) / BN);
  p.num_kb = (int)((R + BK - 1) / BK);
  p.m_fast = Mo < No ? 1 : 0;
  const bool has_bias = fuse.bias != nullptr || fuse.biases != nullptr;
  const bool fused = has_bias || fuse.act != 0;
  if (fuse.mask != nullptr && count != 1)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: the masked data gradient takes one problem per call", name);
  p.splits = (fused || fuse.no_loads) ? 1 : choose_splits(Mo, No, R, count);   // the fused epilogue needs the whole sum
  p.work_per_problem = p.m_tiles * p.n_tiles * p.splits;
  for (int i = 0; i < MAX_GROUP; ++i)
    p.bias[i] = (const uint16_t*)(fuse.biases ? fuse.biases[i < count ? i : 0] : fuse.bias);
  p.mask = (const uint16_t*)fuse.mask;
  p.ldmask = fuse.ldmask; p.act = fuse.act; p.clip = fuse.clip;
  for (int i = 0; i < MAX_GROUP; ++i) p.out[i] = (uint16_t*)outs[i < count ? i : 0];
  p.ldo = ldo;
  p.ws = (float*)workspace; p.ws_ld = ws_ld_for(No);
  p.flag = flag;
  p.status = dstate ? &dstate->h.status : nullptr;
  p.wait_ns = fuse.wait_ns;
  p.no_loads = fuse.no_loads ? 1 : 0;
  if (fuse.no_loads && (pair || p.splits != 1 || count != 1 || p.m_tiles * p.n_tiles != 1))
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: the error-path self-test takes one tile of at most 128 x 256", name);
  p.out_mode = p.splits > 1 ? OUT_PARTIAL : (want_flag ? OUT_F16_FLAG : OUT_F16);
  const size_t ws_floats_per_problem = (size_t)p.splits * (size_t)Mo * (size_t)p.ws_ld;
  if (p.splits > 1) {
    const size_t need = (size_t)count * ws_floats_per_problem * sizeof(float);
    if (!workspace || ws_bytes < need)
      return mp::set_error(MP_ERR_NOMEM, "%s: workspace of %zu bytes needed, %zu given", name, need,
                           workspace ? ws_bytes : (size_t)0);
  }

  GroupMaps maps;
  for (int i = 0; i < count; ++i) {
    // FP16 output: 32-row x 64-column boxes, the unit one epilogue warp stores at a time
    // (first No8 columns; a map over 8 columns that is never used when No < 8)
    if (int rc = make_map(&maps.out[i], outs[i], No8 > 0 ? No8 : 8, Mo, ldo, 64, 32)) return rc;
    if (int rc = A.mn_major ? make_map(&maps.a[i], As[i].ptr, A.mn, A.red, A.ld, 64, BK)
                            : make_map(&maps.a[i], As[i].ptr, A.red, A.mn, A.ld, BK, BM)) return rc;
    if (int rc = B.mn_major ? make_map(&maps.b[i], Bs[i].ptr, B.mn, B.red, B.ld, 64, BK)
                            : make_map(&maps.b[i], Bs[i].ptr, B.red, B.mn, B.ld, BK, pair ? 128 : BN)) return rc;
    // reduction-contiguous B of the pair kernel: 32-row boxes for a narrow last column tile
    if (pair && !B.mn_major) {
      if (int rc = make_map(&maps.b32[i], Bs[i].ptr, B.red, B.mn, B.ld, BK, 32)) return rc;
    } else {
      maps.b32[i] = maps.b[i];
    }
    // FP32 partial sums of a split reduction: [split][row][padded column], boxes of 32 x 32 floats
    if (p.splits > 1) {
      if (int rc = make_map_ws(&maps.ws[i], p.ws + (size_t)i * ws_floats_per_problem, p.ws_ld, Mo, p.splits))
        return rc;
    } else {
      maps.ws[i] = maps.out[i];
    }
  }
  for (int i = count; i < MAX_GROUP; ++i) {       // unused entries: valid copies of problem 0
    maps.a[i] = maps.a[0]; maps.b[i] = maps.b[0]; maps.b32[i] = maps.b32[0];
    maps.out[i] = maps.out[0]; maps.ws[i] = maps.ws[0];
  }

  int dev = 0, sms = 0;
  MP_CUDA_TRY(cudaGetDevice(&dev));
  MP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int64_t work = (int64_t)count * p.work_per_problem;
  const int grid = (int)(work < sms ? work : sms);

  // eight epilogue warps (two per scheduler) for the bias / activation / mask flavours, four for
  // the plain ones
  int rc;
#define MP_DISPATCH(FN, ...)                                                                   \
  do {                                                                                         \
    if (A.mn_major && B.mn_major) rc = fused ? FN<true, true, true>(__VA_ARGS__) : FN<true, true, false>(__VA_ARGS__); \
    else if (!A.mn_major && B.mn_major) rc = fused ? FN<false, true, true>(__VA_ARGS__) : FN<false, true, false>(__VA_ARGS__); \
    else if (!A.mn_major && !B.mn_major) rc = fused ? FN<false, false, true>(__VA_ARGS__) : FN<false, false, false>(__VA_ARGS__); \
    else rc = fused ? FN<true, false, true>(__VA_ARGS__) : FN<true, false, false>(__VA_ARGS__); \
  } while (0)
  if (pair) MP_DISPATCH(launch_pair, maps, p, work, st);
  else MP_DISPATCH(launch, maps, p, grid, st);
#undef MP_DISPATCH
  if (rc) return rc;

  if (p.splits > 1) {
    const int64_t vecs = Mo * ((No + 3) / 4);
    int64_t blocks = (vecs + 255) / 256;
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    for (int i = 0; i < count; ++i) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)blocks, 1, 1);
      cfg.blockDim = dim3(256, 1, 1);
      cfg.stream = st;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr.val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      MP_CUDA_TRY(cudaLaunchKernelEx(&cfg, mp_splitk_reduce_kernel,
                                     (const float*)(p.ws + (size_t)i * ws_floats_per_problem), p.splits, p.Mo,
                                     p.No, p.ws_ld, p.out[i], p.ldo, want_flag ? flag : (int*)nullptr));
      mp::count_launch();
    }
  }
  return MP_OK;
}

// One product: the common case.
int run_gemm(const char* name, const Operand& A, const Operand& B, void* out, int64_t ldo, mp_dev_state* dstate,
             bool want_flag, void* workspace, size_t ws_bytes, cudaStream_t st, const Fuse& fuse = Fuse()) {
  void* outs[1] = {out};
  return run_gemm(name, 1, &A, &B, outs, ldo, dstate, want_flag, workspace, ws_bytes, st, fuse);
}

// Output rows, output columns and reduction length of a layer's product `op`.
bool product_dims(int64_t M, int64_t K, int64_t N, int op, int64_t* Mo, int64_t* No, int64_t* R) {
  if (op == MP_OP_FWD) { *Mo = M; *No = N; *R = K; }
  else if (op == MP_OP_DGRAD) { *Mo = M; *No = K; *R = N; }
  else if (op == MP_OP_WGRAD) { *Mo = K; *No = N; *R = M; }
  else return false;
  return true;
}

}  // namespace

// Device address, on the current device, of the device-wide status word that the GEMM kernels
// write when a bounded wait runs out.  The update and loss-scale kernels read it.
int mp::gemm_status_device_ptr(int** out) {
  static int* addr_of[kMaxDevicesCached] = {};
  int dev = 0;
  MP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevicesCached)
    return mp::set_error(MP_ERR_INVALID_ARG, "device index %d is outside 0..%d", dev, kMaxDevicesCached - 1);
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (addr_of[dev] == nullptr) {
    int* ptr = nullptr;
    MP_CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_gemm_status));
    addr_of[dev] = ptr;
  }
  *out = addr_of[dev];
  return MP_OK;
}

extern "C" {

size_t mp_gemm_workspace_bytes_grouped(int count, int64_t M, int64_t K, int64_t N, int op) {
  if (M <= 0 || K <= 0 || N <= 0 || count < 1 || count > MAX_GROUP) return 0;
  int64_t Mo, No, R;
  if (!product_dims(M, K, N, op, &Mo, &No, &R)) return 0;
  const int s = choose_splits(Mo, No, R, count);
  return s > 1 ? (size_t)count * (size_t)s * (size_t)Mo * (size_t)ws_ld_for(No) * sizeof(float) : 0;
}

size_t mp_gemm_workspace_bytes(int64_t M, int64_t K, int64_t N, int op) {
  return mp_gemm_workspace_bytes_grouped(1, M, K, N, op);
}

int mp_max_group(void) { return MAX_GROUP; }

// ---- several independent layers of one shape in one launch ---------------------------------
int mp_linear_fwd_grouped(int count, const void* const* X16, int64_t ldx, const void* const* W16,
                          int64_t ldw, void* const* Y16, int64_t ldy, int64_t M, int64_t K, int64_t N,
                          void* workspace, size_t workspace_bytes, void* stream) {
  if (count < 1 || count > MAX_GROUP || !X16 || !W16 || !Y16)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_fwd_grouped: 1..%d problems, non-null arrays", MAX_GROUP);
  Operand A[MAX_GROUP], B[MAX_GROUP];
  for (int i = 0; i < count; ++i) { A[i] = Operand{X16[i], ldx, false, M, K}; B[i] = Operand{W16[i], ldw, true, N, K}; }
  return run_gemm("mp_linear_fwd_grouped", count, A, B, Y16, ldy, nullptr, false, workspace, workspace_bytes,
                  (cudaStream_t)stream);
}

int mp_linear_bwd_dgrad_grouped(int count, const void* const* dY16, int64_t lddy, const void* const* W16,
                                int64_t ldw, void* const* dX16, int64_t lddx, int64_t M, int64_t K,
                                int64_t N, void* workspace, size_t workspace_bytes, void* stream) {
  if (count < 1 || count > MAX_GROUP || !dY16 || !W16 || !dX16)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_bwd_dgrad_grouped: 1..%d problems, non-null arrays", MAX_GROUP);
  Operand A[MAX_GROUP], B[MAX_GROUP];
  for (int i = 0; i < count; ++i) { A[i] = Operand{dY16[i], lddy, false, M, N}; B[i] = Operand{W16[i], ldw, false, K, N}; }
  return run_gemm("mp_linear_bwd_dgrad_grouped", count, A, B, dX16, lddx, nullptr, false, workspace,
                  workspace_bytes, (cudaStream_t)stream);
}

int mp_linear_bwd_wgrad_grouped(int count, const void* const* X16, int64_t ldx, const void* const* dY16,
                                int64_t lddy, void* const* dW16, int64_t lddw, int64_t M, int64_t K,
                                int64_t N, mp_state* state, void* workspace, size_t workspace_bytes,
                                void* stream) {
  if (count < 1 || count > MAX_GROUP || !X16 || !dY16 || !dW16)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_bwd_wgrad_grouped: 1..%d problems, non-null arrays", MAX_GROUP);
  Operand A[MAX_GROUP], B[MAX_GROUP];
  for (int i = 0; i < count; ++i) { A[i] = Operand{X16[i], ldx, true, K, M}; B[i] = Operand{dY16[i], lddy, true, N, M}; }
  return run_gemm("mp_linear_bwd_wgrad_grouped", count, A, B, dW16, lddw, state ? state->dev : nullptr, true, workspace,
                  workspace_bytes, (cudaStream_t)stream);
}

int mp_linear_fwd(const void* X16, int64_t ldx, const void* W16, int64_t ldw, void* Y16,
                  int64_t ldy, int64_t M, int64_t K, int64_t N, void* workspace,
                  size_t workspace_bytes, void* stream) {
  const Operand A{X16, ldx, false, M, K};
  const Operand B{W16, ldw, true, N, K};
  return run_gemm("mp_linear_fwd", A, B, Y16, ldy, nullptr, false, workspace, workspace_bytes,
                  (cudaStream_t)stream);
}

int mp_linear_bwd_dgrad(const void* dY16, int64_t lddy, const void* W16, int64_t ldw,
                        void* dX16, int64_t lddx, int64_t M, int64_t K, int64_t N,
                        void* workspace, size_t workspace_bytes, void* stream) {
  const Operand A{dY16, lddy, false, M, N};
  const Operand B{W16, ldw, false, K, N};
  return run_gemm("mp_linear_bwd_dgrad", A, B, dX16, lddx, nullptr, false, workspace,
                  workspace_bytes, (cudaStream_t)stream);
}

int mp_linear_bwd_wgrad(const void* X16, int64_t ldx, const void* dY16, int64_t lddy,
                        void* dW16, int64_t lddw, int64_t M, int64_t K, int64_t N,
                        mp_state* state, void* workspace, size_t workspace_bytes, void* stream) {
  const Operand A{X16, ldx, true, K, M};
  const Operand B{dY16, lddy, true, N, M};
  return run_gemm("mp_linear_bwd_wgrad", A, B, dW16, lddw, state ? state->dev : nullptr, true, workspace,
                  workspace_bytes, (cudaStream_t)stream);
}

// ---- weight gradient with built-in scratch -------------------------------------------------
// Split-reduction scratch that belongs to the library image instead of the caller.  It is a
// fixed-size device array: every GPU that loads this library reserves it until the process
// exits, and every call on that GPU shares it.
#define MP_STATIC_SCRATCH_FLOATS (8u << 20)   /* 8 Mi floats = 32 MiB */
static_assert((size_t)MP_STATIC_SCRATCH_FLOATS * sizeof(float) == (size_t)MP_STATIC_SCRATCH_BYTES,
              "the array and the size the header states must agree");
static __device__ __align__(256) float g_static_scratch[MP_STATIC_SCRATCH_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device.  In host code the array's name
// is only a handle for the runtime, not an address a kernel could use, so the address is
// asked for once per device (with that device current) and remembered.
int static_scratch_for_current_device(float** out) {
  int dev = 0;
  MP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices)
    return mp::set_error(MP_ERR_INVALID_ARG, "device index %d is outside 0..%d", dev, kMaxDevices - 1);
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    float* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess || ptr == nullptr)
      return mp::set_error(MP_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return MP_OK;
}
}  // namespace

int mp_linear_bwd_wgrad_static(const void* X16, int64_t ldx, const void* dY16, int64_t lddy,
                               void* dW16, int64_t lddw, int64_t M, int64_t K, int64_t N,
                               mp_state* state, void* stream) {
  const size_t need = mp_gemm_workspace_bytes(M, K, N, MP_OP_WGRAD);
  const size_t have = (size_t)MP_STATIC_SCRATCH_FLOATS * sizeof(float);
  if (need > have)
    return mp::set_error(MP_ERR_TOO_LARGE,
                         "mp_linear_bwd_wgrad_static: these sizes need %zu bytes of scratch, the "
                         "built-in array holds %zu; use mp_linear_bwd_wgrad with a caller workspace",
                         need, have);
  if (int rc = mp::check_device()) return rc;
  float* scratch = nullptr;
  if (int rc = static_scratch_for_current_device(&scratch)) return rc;
  const Operand A{X16, ldx, true, K, M};
  const Operand B{dY16, lddy, true, N, M};
  return run_gemm("mp_linear_bwd_wgrad_static", A, B, dW16, lddw, state ? state->dev : nullptr, true, scratch,
                  have, (cudaStream_t)stream);
}

size_t mp_static_scratch_bytes(void) { return (size_t)MP_STATIC_SCRATCH_FLOATS * sizeof(float); }

// ---- layers with bias and activation ----------------------------------------------------------
static int check_act(const char* name, int act, float clip) {
  if (act != MP_ACT_NONE && act != MP_ACT_RELU && act != MP_ACT_CLIPPED_RELU)
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: unknown activation %d", name, act);
  if (act == MP_ACT_CLIPPED_RELU && !(clip > 0.0f))
    return mp::set_error(MP_ERR_INVALID_ARG, "%s: clip must be positive", name);
  return MP_OK;
}

int mp_linear_fwd_act(const void* X16, int64_t ldx, const void* W16, int64_t ldw, const void* bias16,
                      void* Y16, int64_t ldy, int64_t M, int64_t K, int64_t N, int act, float clip,
                      void* workspace, size_t workspace_bytes, void* stream) {
  if (int rc = check_act("mp_linear_fwd_act", act, clip)) return rc;
  if (bias16 && !mp::aligned16(bias16))
    return mp::set_error(MP_ERR_ALIGNMENT, "mp_linear_fwd_act: bias must be 16-byte aligned");
  const Operand A{X16, ldx, false, M, K};
  const Operand B{W16, ldw, true, N, K};
  Fuse f;
  f.bias = bias16; f.act = act; f.clip = clip;
  return run_gemm("mp_linear_fwd_act", A, B, Y16, ldy, nullptr, false, workspace, workspace_bytes,
                  (cudaStream_t)stream, f);
}

int mp_linear_fwd_act_grouped(int count, const void* const* X16, int64_t ldx, const void* const* W16,
                              int64_t ldw, const void* const* bias16, void* const* Y16, int64_t ldy,
                              int64_t M, int64_t K, int64_t N, int act, float clip, void* workspace,
                              size_t workspace_bytes, void* stream) {
  if (int rc = check_act("mp_linear_fwd_act_grouped", act, clip)) return rc;
  if (count < 1 || count > MAX_GROUP || !X16 || !W16 || !Y16)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_fwd_act_grouped: 1..%d problems, non-null arrays", MAX_GROUP);
  if (bias16) {
    for (int i = 0; i < count; ++i)
      if (!bias16[i] || !mp::aligned16(bias16[i]))
        return mp::set_error(MP_ERR_ALIGNMENT, "mp_linear_fwd_act_grouped: every bias must be non-null and 16-byte aligned");
  }
  Operand A[MAX_GROUP], B[MAX_GROUP];
  for (int i = 0; i < count; ++i) { A[i] = Operand{X16[i], ldx, false, M, K}; B[i] = Operand{W16[i], ldw, true, N, K}; }
  Fuse f;
  f.biases = bias16; f.act = act; f.clip = clip;
  return run_gemm("mp_linear_fwd_act_grouped", count, A, B, Y16, ldy, nullptr, false, workspace, workspace_bytes,
                  (cudaStream_t)stream, f);
}

int mp_linear_bwd_dgrad_act(const void* dY16, int64_t lddy, const void* W16, int64_t ldw,
                            const void* A16, int64_t lda, void* dX16, int64_t lddx, int64_t M,
                            int64_t K, int64_t N, int act, float clip, void* workspace,
                            size_t workspace_bytes, void* stream) {
  if (int rc = check_act("mp_linear_bwd_dgrad_act", act, clip)) return rc;
  if (act != MP_ACT_NONE) {
    if (!A16) return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_bwd_dgrad_act: null layer input");
    if (lda < K) return mp::set_error(MP_ERR_INVALID_ARG, "mp_linear_bwd_dgrad_act: lda < K");
    // the epilogue reads the layer input with 128-bit loads
    if (!mp::aligned16(A16) || (lda & 7))
      return mp::set_error(MP_ERR_ALIGNMENT, "mp_linear_bwd_dgrad_act: the layer input must be 16-byte "
                                             "aligned and lda a multiple of 8");
  }
  const Operand A{dY16, lddy, false, M, N};
  const Operand B{W16, ldw, false, K, N};
  Fuse f;
  f.mask = act != MP_ACT_NONE ? A16 : nullptr; f.ldmask = lda; f.act = act; f.clip = clip;
  return run_gemm("mp_linear_bwd_dgrad_act", A, B, dX16, lddx, nullptr, false, workspace,
                  workspace_bytes, (cudaStream_t)stream, f);
}

// Error-path self-test: the forward product's one-CTA kernel on a single tile, with its producer
// warp told to issue no load.  Nothing is ever in flight; the MMA issuer's wait for operands and
// the epilogue's wait for the accumulator run out after wait_us, the CTA records MP_ERR_TIMEOUT,
// releases its tensor memory and returns.  Y16 is not written.
int mp_selftest_wait_timeout(const void* X16, int64_t ldx, const void* W16, int64_t ldw, void* Y16,
                             int64_t ldy, int64_t M, int64_t K, int64_t N, int64_t wait_us,
                             mp_state* state, void* stream) {
  if (wait_us < 1 || wait_us > 2000000)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_selftest_wait_timeout: wait_us must be in 1 .. 2000000");
  if (M > BM || N > BN)
    return mp::set_error(MP_ERR_INVALID_ARG, "mp_selftest_wait_timeout: one tile only (M <= %d, N <= %d)", BM, BN);
  const Operand A{X16, ldx, false, M, K};
  const Operand B{W16, ldw, true, N, K};
  Fuse f;
  f.wait_ns = (uint64_t)wait_us * 1000ull;
  f.no_loads = true;
  return run_gemm("mp_selftest_wait_timeout", A, B, Y16, ldy, state ? state->dev : nullptr, false, nullptr, 0,
                  (cudaStream_t)stream, f);
}

// Synchronises the device and returns the first device-side error recorded by a GEMM kernel
// (MP_OK if none), clearing it.
int mp_gemm_device_status(int* out) {
  if (!out) return mp::set_error(MP_ERR_INVALID_ARG, "mp_gemm_device_status: null argument");
  MP_CUDA_TRY(cudaDeviceSynchronize());
  int v = 0, zero = 0;
  MP_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)));
  MP_CUDA_TRY(cudaMemcpyToSymbol(g_gemm_status, &zero, sizeof(int)));
  *out = v;
  return MP_OK;
}

}  // extern "C"
