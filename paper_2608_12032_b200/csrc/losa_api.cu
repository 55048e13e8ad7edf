// C ABI of liblosa: argument validation, workspace sizing, status word, launch dispatch.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "losa_common.cuh"

namespace losa {

namespace {
thread_local char g_cuda_error[256] = "";
std::mutex g_state_mutex;
DeviceState g_state[kMaxDevices];
std::atomic<int> g_state_ready[kMaxDevices];  // 0 = not created, 1 = ready
std::atomic<int> g_device_ok[kMaxDevices];    // 0 = not asked, 1 = sm_100, -1 = anything else
}  // namespace

const char* set_cuda_error(cudaError_t e, const char* what) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return g_cuda_error;
}

int check_device() {
  int dev = 0;
  LOSA_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LOSA_ERR_UNSUPPORTED;
  int ok = g_device_ok[dev].load(std::memory_order_acquire);
  if (ok == 0) {
    int major = 0;
    LOSA_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    ok = (major == 10) ? 1 : -1;  // the kernels are built for sm_100a only
    g_device_ok[dev].store(ok, std::memory_order_release);
  }
  if (ok < 0) {
    snprintf(g_cuda_error, sizeof(g_cuda_error),
             "device %d is not an sm_100 GPU: liblosa holds sm_100a kernels only", dev);
    return LOSA_ERR_UNSUPPORTED;
  }
  return LOSA_OK;
}

const DeviceState* device_state(int* rc) {
  int dev = 0;
  *rc = check_device();
  if (*rc != LOSA_OK) return nullptr;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    *rc = LOSA_ERR_CUDA;
    return nullptr;
  }
  if (g_state_ready[dev].load(std::memory_order_acquire)) return &g_state[dev];
  std::lock_guard<std::mutex> lock(g_state_mutex);
  if (g_state_ready[dev].load(std::memory_order_acquire)) return &g_state[dev];
  DeviceState st{};
  cudaError_t e = cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) {
    int* h = nullptr;
    e = cudaHostAlloc(reinterpret_cast<void**>(&h), 64, cudaHostAllocMapped | cudaHostAllocPortable);
    if (e == cudaSuccess) {
      *h = 0;
      e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&st.status_dev), h, 0);
      if (e != cudaSuccess) cudaFreeHost(h);
      st.status_host = h;
    }
  }
  if (e != cudaSuccess || st.sm_count <= 0) {
    set_cuda_error(e, "per-device state (SM count, status word)");
    *rc = LOSA_ERR_CUDA;
    return nullptr;
  }
  g_state[dev] = st;
  g_state_ready[dev].store(1, std::memory_order_release);
  return &g_state[dev];
}

int make_geometry(const losa_problem_t* p, Geometry* g) {
  if (!p) return LOSA_ERR_INVALID_ARG;
  if (p->B <= 0 || p->H <= 0 || p->N <= 0) return LOSA_ERR_INVALID_ARG;
  if (!(p->D == 64 || p->D == 128)) return LOSA_ERR_UNSUPPORTED;
  // query blocks of 64 or 128 rows; key blocks of 32, 64 or 128 rows, gathered into 128-key tiles
  if (!((p->R == 64 && p->C == 64) || (p->R == 128 && (p->C == 128 || p->C == 64 || p->C == 32))))
    return LOSA_ERR_UNSUPPORTED;
  if ((int64_t)(p->N + p->C - 1) / p->C >= 0xffff) return LOSA_ERR_UNSUPPORTED;  // 16-bit block index in the tile list
  if (p->sn < p->D || p->sh <= 0 || p->sb <= 0) return LOSA_ERR_INVALID_ARG;
  if ((p->sn % 8) || (p->sh % 8) || (p->sb % 8)) return LOSA_ERR_INVALID_ARG;
  if (!(p->scale >= 0.0f) || isinf(p->scale)) return LOSA_ERR_INVALID_ARG;
  g->B = p->B;
  g->H = p->H;
  g->N = p->N;
  g->D = p->D;
  g->R = p->R;
  g->C = p->C;
  g->nQb = (p->N + p->R - 1) / p->R;
  g->nKb = (p->N + p->C - 1) / p->C;
  g->nQt = (p->N + 127) / 128;
  g->nPairs = (g->nQt + 1) / 2;
  g->sb = p->sb;
  g->sh = p->sh;
  g->sn = p->sn;
  g->scale = (p->scale > 0.0f) ? p->scale : 1.0f / sqrtf((float)p->D);
  const int64_t rows = (int64_t)g->B * g->H * g->nQb;
  if (rows * g->nKb > INT32_MAX || (int64_t)g->B * g->H * g->nPairs > INT32_MAX)
    return LOSA_ERR_UNSUPPORTED;
  return LOSA_OK;
}

}  // namespace losa

using namespace losa;

extern "C" {

size_t losa_workspace_bytes(int op, const losa_problem_t* p) {
  if (!p) return 0;
  if (op == LOSA_OP_SELECT) {
    if (p->B <= 0 || p->H <= 0 || p->N <= 0 || p->R <= 0 || p->C <= 0) return 0;
    const int64_t nQb = (p->N + p->R - 1) / p->R, nKb = (p->N + p->C - 1) / p->C;
    return select_workspace_bytes((int64_t)p->B * p->H * nQb, (int)nKb);
  }
  Geometry g;
  if (make_geometry(p, &g) != LOSA_OK) return 0;
  switch (op) {
    case LOSA_OP_BLOCK_MASS: return attn_workspace_bytes(kMass, g);
    case LOSA_OP_SPARSE_ATTN: return attn_workspace_bytes(kSparse, g);
    case LOSA_OP_ATTN: return attn_workspace_bytes(kDense, g);
    case LOSA_OP_ATTN_MASS: return attn_workspace_bytes(kFused, g);
  }
  return 0;
}

int32_t losa_work_slots(int op, const losa_problem_t* p) {
  Geometry g;
  if (!p || make_geometry(p, &g) != LOSA_OK) return 0;
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return 0;
  switch (op) {
    case LOSA_OP_BLOCK_MASS: return attn_work_slots(kMass, g, dev->sm_count);
    case LOSA_OP_SPARSE_ATTN: return attn_work_slots(kSparse, g, dev->sm_count);
    case LOSA_OP_ATTN: return attn_work_slots(kDense, g, dev->sm_count);
    case LOSA_OP_ATTN_MASS: return attn_work_slots(kFused, g, dev->sm_count);
  }
  return 0;
}

int losa_block_mass(const losa_problem_t* p, const void* q, const void* k, float* mass, float* lse,
                    void* ws, size_t ws_bytes, void* cuda_stream) {
  Geometry g;
  int rc = make_geometry(p, &g);
  if (rc != LOSA_OK) return rc;
  if (!q || !k || !mass || !aligned16(q) || !aligned16(k) || !aligned16(mass))
    return LOSA_ERR_INVALID_ARG;
  const size_t need = attn_workspace_bytes(kMass, g);
  if (need > 0 && (!ws || ws_bytes < need)) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  return launch_attn(kMass, g, q, k, nullptr, nullptr, nullptr, nullptr, 0, mass, lse, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

int losa_select(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass, double tau,
                int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws, size_t ws_bytes,
                void* cuda_stream) {
  if (B <= 0 || H <= 0 || nQb <= 0 || nKb <= 0) return LOSA_ERR_INVALID_ARG;
  if (!(tau > 0.0) || !(tau <= 1.0)) return LOSA_ERR_INVALID_ARG;  // also rejects NaN
  if (!mass || !offsets || !kv_idx || kv_capacity < 0) return LOSA_ERR_INVALID_ARG;
  const int64_t rows = (int64_t)B * H * nQb;
  if (rows * nKb > INT32_MAX) return LOSA_ERR_UNSUPPORTED;
  if (nKb > LOSA_SELECT_MAX_KEY_BLOCKS) return LOSA_ERR_UNSUPPORTED;  // one row is sorted in shared memory
  const size_t need = select_workspace_bytes(rows, nKb);
  if (!ws || ws_bytes < need) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return rc;
  return launch_select((int)rows, nKb, mass, tau, 0, offsets, kv_idx, kv_capacity, ws,
                       dev->status_dev, static_cast<cudaStream_t>(cuda_stream));
}

int losa_select_topk(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass, int32_t k,
                     int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  if (B <= 0 || H <= 0 || nQb <= 0 || nKb <= 0) return LOSA_ERR_INVALID_ARG;
  if (k < 1 || k > nKb) return LOSA_ERR_INVALID_ARG;
  if (!mass || !offsets || !kv_idx || kv_capacity < 0) return LOSA_ERR_INVALID_ARG;
  const int64_t rows = (int64_t)B * H * nQb;
  if (rows * nKb > INT32_MAX || nKb > LOSA_SELECT_MAX_KEY_BLOCKS) return LOSA_ERR_UNSUPPORTED;
  const size_t need = select_workspace_bytes(rows, nKb);
  if (!ws || ws_bytes < need) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return rc;
  return launch_select((int)rows, nKb, mass, 0.5, k, offsets, kv_idx, kv_capacity, ws,
                       dev->status_dev, static_cast<cudaStream_t>(cuda_stream));
}

int losa_row_recall(int32_t rows, int32_t nKb, const float* mass, const int32_t* offsets,
                    const int32_t* kv_idx, double* retained, double* total, void* cuda_stream) {
  if (rows <= 0 || nKb <= 0 || !mass || !offsets || !kv_idx || !retained || !total)
    return LOSA_ERR_INVALID_ARG;
  return launch_row_recall(rows, nKb, mass, offsets, kv_idx, retained, total,
                           static_cast<cudaStream_t>(cuda_stream));
}

int losa_select_noalloc(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass,
                        double tau, int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity,
                        int32_t* device_status, void* cuda_stream) {
  if (B <= 0 || H <= 0 || nQb <= 0 || nKb <= 0) return LOSA_ERR_INVALID_ARG;
  if (!(tau > 0.0) || !(tau <= 1.0)) return LOSA_ERR_INVALID_ARG;
  if (!mass || !offsets || !kv_idx || kv_capacity < 0) return LOSA_ERR_INVALID_ARG;
  const int64_t rows = (int64_t)B * H * nQb;
  if (rows * nKb > INT32_MAX || nKb > LOSA_SELECT_MAX_KEY_BLOCKS) return LOSA_ERR_UNSUPPORTED;
  const size_t need = select_workspace_bytes(rows, nKb);
  if (need > select_noalloc_workspace_limit()) {
    snprintf(g_cuda_error, sizeof(g_cuda_error),
             "losa_select_noalloc: this mass matrix needs %zu bytes of scratch, the built-in "
             "array holds %zu; use losa_select with caller-provided workspace",
             need, select_noalloc_workspace_limit());
    return LOSA_ERR_WORKSPACE;
  }
  const int rc = check_device();  // (asks for an attribute; allocates nothing)
  if (rc != LOSA_OK) return rc;
  return launch_select_noalloc((int)rows, nKb, mass, tau, offsets, kv_idx, kv_capacity,
                               device_status, static_cast<cudaStream_t>(cuda_stream));
}

static int check_attn_args(const losa_problem_t* p, Geometry* g, const void* q, const void* k,
                           const void* v, const void* o, int o_dtype) {
  int rc = make_geometry(p, g);
  if (rc != LOSA_OK) return rc;
  if (!q || !k || !v || !o) return LOSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LOSA_ERR_INVALID_ARG;
  if (o_dtype != LOSA_DTYPE_BF16 && o_dtype != LOSA_DTYPE_F32) return LOSA_ERR_UNSUPPORTED;
  return LOSA_OK;
}

int losa_sparse_attn(const losa_problem_t* p, const void* q, const void* k, const void* v,
                     const int32_t* offsets, const int32_t* kv_idx, void* o, int o_dtype, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  Geometry g;
  int rc = check_attn_args(p, &g, q, k, v, o, o_dtype);
  if (rc != LOSA_OK) return rc;
  if (!offsets || !kv_idx) return LOSA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < attn_workspace_bytes(kSparse, g)) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  return launch_attn(kSparse, g, q, k, v, offsets, kv_idx, o, o_dtype, nullptr, nullptr, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

size_t losa_workspace_bytes_batched(int op, const losa_problem_t* p, int32_t n_layers) {
  Geometry g;
  if (op != LOSA_OP_SPARSE_ATTN || n_layers < 1 || n_layers > LOSA_MAX_BATCHED_LAYERS) return 0;
  if (make_geometry(p, &g) != LOSA_OK) return 0;
  if ((int64_t)n_layers * g.B * g.H * g.nPairs > (int64_t)0x00ffffff) return 0;
  return attn_workspace_bytes(kSparse, g, n_layers);
}

int losa_sparse_attn_batched(const losa_problem_t* p, int32_t n_layers, const losa_layer_t* layers,
                             int o_dtype, void* ws, size_t ws_bytes, void* cuda_stream) {
  Geometry g;
  if (n_layers < 1 || n_layers > LOSA_MAX_BATCHED_LAYERS || !layers) return LOSA_ERR_INVALID_ARG;
  for (int i = 0; i < n_layers; ++i) {
    const int rc = check_attn_args(p, &g, layers[i].q, layers[i].k, layers[i].v, layers[i].o, o_dtype);
    if (rc != LOSA_OK) return rc;
    if (!layers[i].offsets || !layers[i].kv_idx) return LOSA_ERR_INVALID_ARG;
  }
  if (!ws || ws_bytes < attn_workspace_bytes(kSparse, g, n_layers)) return LOSA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 127u) return LOSA_ERR_INVALID_ARG;
  if (n_layers == 1)
    return launch_attn(kSparse, g, layers[0].q, layers[0].k, layers[0].v, layers[0].offsets,
                       layers[0].kv_idx, layers[0].o, o_dtype, nullptr, nullptr, ws,
                       static_cast<cudaStream_t>(cuda_stream));
  return launch_attn(kSparse, g, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, o_dtype, nullptr,
                     nullptr, ws, static_cast<cudaStream_t>(cuda_stream), n_layers, layers);
}

int losa_attn(const losa_problem_t* p, const void* q, const void* k, const void* v, void* o,
              int o_dtype, void* ws, size_t ws_bytes, void* cuda_stream) {
  Geometry g;
  int rc = check_attn_args(p, &g, q, k, v, o, o_dtype);
  if (rc != LOSA_OK) return rc;
  if (!ws || ws_bytes < attn_workspace_bytes(kDense, g)) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  return launch_attn(kDense, g, q, k, v, nullptr, nullptr, o, o_dtype, nullptr, nullptr, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

int losa_attn_mass(const losa_problem_t* p, const void* q, const void* k, const void* v, void* o,
                   int o_dtype, float* mass, float* lse, void* ws, size_t ws_bytes,
                   void* cuda_stream) {
  Geometry g;
  int rc = check_attn_args(p, &g, q, k, v, o, o_dtype);
  if (rc != LOSA_OK) return rc;
  if (!mass || !aligned16(mass)) return LOSA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < attn_workspace_bytes(kFused, g)) return LOSA_ERR_WORKSPACE;
  if (!aligned16(ws)) return LOSA_ERR_INVALID_ARG;
  return launch_attn(kFused, g, q, k, v, nullptr, nullptr, o, o_dtype, mass, lse, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

int losa_validate_csr(int32_t rows, int32_t nKb, const int32_t* offsets, const int32_t* kv_idx,
                      void* cuda_stream) {
  if (rows <= 0 || nKb <= 0 || !offsets || !kv_idx) return LOSA_ERR_INVALID_ARG;
  return launch_validate_csr(rows, nKb, offsets, kv_idx, static_cast<cudaStream_t>(cuda_stream));
}

int losa_async_status(void* cuda_stream) {
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) {
    set_cuda_error(e, "cudaStreamSynchronize");
    return LOSA_ERR_CUDA;
  }
  // the word of the current device (the stream's device, by the calling convention); a device
  // that never launched anything has none
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOSA_ERR_CUDA;
  if (!g_state_ready[dev].load(std::memory_order_acquire)) return LOSA_OK;
  int* h = g_state[dev].status_host;
  return __atomic_exchange_n(h, 0, __ATOMIC_ACQ_REL);
}

int losa_debug_stall_next_launch(uint32_t polls) {
  if (polls == 0u || polls > (1u << 16)) return LOSA_ERR_INVALID_ARG;
  arm_stalled_launch(polls);
  return LOSA_OK;
}

const char* losa_status_string(int status) {
  switch (status) {
    case LOSA_OK: return "LOSA_OK";
    case LOSA_ERR_INVALID_ARG: return "LOSA_ERR_INVALID_ARG";
    case LOSA_ERR_UNSUPPORTED: return "LOSA_ERR_UNSUPPORTED";
    case LOSA_ERR_WORKSPACE: return "LOSA_ERR_WORKSPACE";
    case LOSA_ERR_CAPACITY: return "LOSA_ERR_CAPACITY";
    case LOSA_ERR_CUDA: return "LOSA_ERR_CUDA";
    case LOSA_ERR_TIMEOUT: return "LOSA_ERR_TIMEOUT";
    case LOSA_ERR_BAD_INDEX: return "LOSA_ERR_BAD_INDEX";
    case LOSA_ERR_BAD_MASS: return "LOSA_ERR_BAD_MASS";
    case LOSA_ERR_INTERNAL: return "LOSA_ERR_INTERNAL";
  }
  return "LOSA_ERR_UNKNOWN";
}

const char* losa_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"
