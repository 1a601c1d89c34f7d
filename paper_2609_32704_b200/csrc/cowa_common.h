// Shared host-side declarations of the CoWA library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cowa.h"
#include "cowa_sched.h"

#define COWA_MAX_HKV 64  // per-call KV heads whose tuples travel as a kernel argument

// Per-head tuples passed by value to the training kernels.
struct CowaHeadWindows {
  CowaWin w[COWA_MAX_HKV];
};

// Element strides (batch, head, token) of a [B, H, T, D] tensor whose D axis is contiguous.
struct CowaStrides {
  long long b, h, t;
};

// Bits of the device status word (set by kernels whose bounded waits ran out).
enum { COWA_DEV_TIMEOUT = 1u, COWA_DEV_BAD_SEQLENS = 2u, COWA_DEV_DQ_RANGE = 4u };

namespace cowa {

// Records a failing CUDA call for cowa_last_cuda_error(); returns COWA_ERR_CUDA.
int record_cuda_error(cudaError_t e);

// Device address of the status word of the current device (nullptr on failure).
unsigned int* device_status_word();

// Resolves the per-head tuples of a training call (explicit, default rule or FullAttn).
// Returns COWA_OK or an error status.
int resolve_windows(int Nk, int Hkv, const cowa_params_t* p, CowaHeadWindows* out);

// Strides of one tensor of a call: all zeros in `s` mean contiguous head-major [B, H, T, D]; otherwise every
// stride must be a non-negative multiple of 8 elements (TMA and the 128-bit loads need 16-byte steps) and
// the token stride at least D.  Returns COWA_OK, COWA_ERR_INVALID_ARG or COWA_ERR_MISALIGNED.
int resolve_strides(const int64_t s[3], int H, long long T, int D, CowaStrides* out);

// True when any stride of q, k, v or o is set (for the calls that take contiguous tensors only).
bool any_stride_set(const cowa_params_t* p);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace cowa

#define COWA_CUDA_TRY(expr)                                      \
  do {                                                           \
    cudaError_t cowa_e_ = (expr);                                \
    if (cowa_e_ != cudaSuccess) return cowa::record_cuda_error(cowa_e_); \
  } while (0)
