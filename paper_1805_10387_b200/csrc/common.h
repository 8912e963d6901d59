// Host-side helpers shared by the translation units of the library: error text,
// launch accounting, device check, and the layout of the device-resident state.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "mp.h"

// Device-resident state.  Its head has the exact layout of mp_state_host so that a read is
// one copy; the log ring follows.
struct mp_dev_state {
  mp_state_host h;
  int64_t log_count;  // records ever written; slot = log_count % MP_LOG_CAPACITY
  // Work distribution of the fused update: next chunk to hand out, and blocks that have finished.
  // Both are zero between launches (the last block to finish clears them).
  unsigned int update_ticket, update_done;
  mp_log_record log[MP_LOG_CAPACITY];
};

struct mp_state {
  mp_dev_state* dev;
  int device;
};

namespace mp {

int set_error(int code, const char* fmt, ...);  // stores the message, returns code
void count_launch(int n = 1);
int check_device();  // MP_OK if the current device is compute capability 10.x
// Device address (on the current device) of the status word that the GEMM kernels set when a
// bounded wait expires; defined beside those kernels.
int gemm_status_device_ptr(int** out);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define MP_CUDA_TRY(expr)                                                            \
  do {                                                                               \
    cudaError_t e__ = (expr);                                                        \
    if (e__ != cudaSuccess)                                                          \
      return mp::set_error(MP_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__));   \
  } while (0)

}  // namespace mp
