// Shared host/device helpers of liblosa: status word, problem geometry, error macros.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "losa.h"

namespace losa {

// Upper bound on the number of persistent CTAs any kernel here launches; workspace is
// sized for it so that losa_workspace_bytes() needs no GPU.
constexpr int kMaxPersistentCtas = 160;

// Per-device state of the library, created on a device's first call (thread-safe) and kept until
// the process exits: the SM count and the device-visible status word (one int of pinned, mapped
// host memory per device).  Kernels record the first error with a system-scope compare-and-swap;
// the host reads the word after a stream sync.
constexpr int kMaxDevices = 64;
struct DeviceState {
  int sm_count;
  int* status_host;
  int* status_dev;  // the same word as the kernels of this device address it
};
// State of the CURRENT device, or nullptr with *rc = LOSA_ERR_UNSUPPORTED (not an sm_100 GPU, or
// a device ordinal beyond kMaxDevices) or LOSA_ERR_CUDA (a runtime call failed).
const DeviceState* device_state(int* rc);
// LOSA_OK if the current device can run the library's kernels (compute capability 10.x); makes no
// allocation.
int check_device();
const char* set_cuda_error(cudaError_t e, const char* what);

__device__ __forceinline__ void report_error(int* status, int code) {
  atomicCAS_system(status, 0, code);
}

struct Geometry {
  int B, H, N, D, R, C;
  int nQb, nKb;
  int nQt;     // 128-row query tiles per head
  int nPairs;  // pairs of query tiles per head (one CTA work item)
  int64_t sb, sh, sn;
  float scale;
};

int make_geometry(const losa_problem_t* p, Geometry* g);  // LOSA_OK or an error code

#define LOSA_CUDA_TRY(expr)                                        \
  do {                                                             \
    cudaError_t e__ = (expr);                                      \
    if (e__ != cudaSuccess) {                                      \
      ::losa::set_cuda_error(e__, #expr);                          \
      return LOSA_ERR_CUDA;                                        \
    }                                                              \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- entry points of the kernel translation units (host launchers) -------------------

size_t select_workspace_bytes(int64_t rows, int nKb);
int launch_select(int rows, int nKb, const float* mass, double tau, int fixed_count,
                  int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws, int* status,
                  cudaStream_t st);  // fixed_count > 0: keep that many blocks per row instead;
                                     // status: device-visible word that receives device-side errors
int launch_row_recall(int rows, int nKb, const float* mass, const int32_t* offsets,
                      const int32_t* kv_idx, double* retained, double* total, cudaStream_t st);
size_t select_noalloc_workspace_limit();
int launch_select_noalloc(int rows, int nKb, const float* mass, double tau, int32_t* offsets,
                          int32_t* kv_idx, int64_t kv_capacity, int32_t* device_status,
                          cudaStream_t st);
int launch_validate_csr(int rows, int nKb, const int32_t* offsets, const int32_t* kv_idx,
                        cudaStream_t st);

enum AttnMode { kDense = 0, kSparse = 1, kMass = 2, kFused = 3 };  // kFused: dense O and mass

size_t attn_workspace_bytes(AttnMode mode, const Geometry& g, int n_prob = 1);
void arm_stalled_launch(uint32_t polls);  // the next attention launch publishes no work (diagnostic)
int attn_work_slots(AttnMode mode, const Geometry& g, int sms);
int launch_attn(AttnMode mode, const Geometry& g, const void* q, const void* k, const void* v,
                const int32_t* offsets, const int32_t* kv_idx, void* o, int o_dtype, float* mass,
                float* lse, void* ws, cudaStream_t st, int n_prob = 1,
                const losa_layer_t* layers = nullptr);

}  // namespace losa
