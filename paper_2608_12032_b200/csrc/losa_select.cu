// losa_select: retained-mass selection (Eq. 3) and CSR validation.
//
// Three small launches over a [rows, nKb] fp32 mass matrix:
//   1. select_rows_warp_kernel  rows of at most 1024 blocks: one warp per row, the row in
//                           registers, the threshold value found bit by bit with masked
//                           fixed-point sums (no sort); the kept set is written as a bitmap
//                           over block indices plus its size.
//      select_rows_kernel   longer rows: one CTA per
//                           row, sort (mass descending, index ascending) as 64-bit integer
//                           keys in shared memory, fp64 prefix sum along the sorted order,
//                           shortest prefix reaching tau; same outputs.
//   2. scan_counts_kernel   exclusive prefix of the per-row sizes -> offsets.
//   3. expand_rows_kernel   one warp per row: bitmap -> ascending block indices.
// Each mass element is read once and each kept index written once; the bitmap adds 1/16
// of the mass bytes.  The result is deterministic (no floating-point atomics).
#include <limits.h>

#include "losa_common.cuh"

namespace losa {
namespace {

constexpr int kSelThreads = 256;
constexpr unsigned long long kPadKey = ~0ull;

__device__ __forceinline__ double key_mass(unsigned long long key) {
  return (double)__uint_as_float(~(uint32_t)(key >> 32));
}

__global__ void __launch_bounds__(kSelThreads)
select_rows_kernel(const float* __restrict__ mass, int nKb, int n2, double tau, int fixed_count,
                   int32_t* __restrict__ counts, uint32_t* __restrict__ bitmaps, int* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(keys + n2);
  __shared__ double warp_total[kSelThreads / 32];
  __shared__ int first_pos;
  __shared__ double row_total;

  const int tid = threadIdx.x;
  const int64_t row = blockIdx.x;
  const int words = (nKb + 31) >> 5;
  const float* mrow = mass + row * nKb;

  bool bad = false;
  for (int i = tid; i < n2; i += kSelThreads) {
    unsigned long long key = kPadKey;
    if (i < nKb) {
      float m = mrow[i];
      if (!(m >= 0.0f) || m > 8.0f) {  // negative, NaN, or far beyond any mass
        bad = true;
        m = 0.0f;
      }
      // mass >= 0, so its IEEE bits order like the value; -0 becomes +0
      const uint32_t bits = (m == 0.0f) ? 0u : __float_as_uint(m);
      key = ((unsigned long long)(~bits) << 32) | (uint32_t)i;
    }
    keys[i] = key;
  }
  for (int w = tid; w < words; w += kSelThreads) bitmap[w] = 0u;
  if (tid == 0) first_pos = INT_MAX;
  if (bad) report_error(status, LOSA_ERR_BAD_MASS);
  __syncthreads();

  // bitonic sort, ascending keys = descending mass, ties by ascending block index; every thread
  // owns compare-exchange pairs (i, i | j), so no thread idles
  for (int k = 2; k <= n2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int pr = tid; pr < (n2 >> 1); pr += kSelThreads) {
        const int i = ((pr & ~(j - 1)) << 1) | (pr & (j - 1));
        const int ixj = i | j;
        const unsigned long long a = keys[i], b = keys[ixj];
        const bool up = ((i & k) == 0);
        if ((a > b) == up) {
          keys[i] = b;
          keys[ixj] = a;
        }
      }
      __syncthreads();
    }
  }

  // fp64 prefix sum along the sorted order: per-thread chunk, then a block scan of chunk sums
  const int chunk = (n2 + kSelThreads - 1) / kSelThreads;
  const int lo = min(tid * chunk, n2), hi = min(lo + chunk, n2);
  double local = 0.0;
  for (int i = lo; i < hi; ++i) local += key_mass(keys[i]);
  double incl = local;
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += up;
  }
  if (lane == 31) warp_total[warp] = incl;
  __syncthreads();
  double base = 0.0;
  for (int w = 0; w < warp; ++w) base += warp_total[w];
  double acc = base + (incl - local);
  for (int i = lo; i < hi; ++i) {
    acc += key_mass(keys[i]);
    if (acc >= tau) {
      atomicMin(&first_pos, i + 1);
      break;
    }
  }
  if (tid == kSelThreads - 1) row_total = base + incl;
  __syncthreads();
  int s = first_pos;
  if (tau >= 1.0 || s > nKb) s = nKb;
  // same rule as the warp-per-row kernel: a row whose masses add up to more than 8 is reported and
  // keeps every block
  if (row_total > 8.0) {
    s = nKb;
    if (tid == 0) report_error(status, LOSA_ERR_BAD_MASS);
  }
  if (fixed_count > 0) s = min(fixed_count, nKb);  // fixed-ratio rule: the k heaviest blocks

  for (int i = lo; i < hi; ++i) {
    if (i < s) {
      const uint32_t idx = (uint32_t)keys[i];
      atomicOr(&bitmap[idx >> 5], 1u << (idx & 31));
    }
  }
  __syncthreads();
  for (int w = tid; w < words; w += kSelThreads) bitmaps[row * words + w] = bitmap[w];
  if (tid == 0) counts[row] = s;
}

// Rows of at most 1024 blocks: one WARP per row, no sort.  The kept set of Eq. 3 is "every block
// heavier than v*, plus the lowest-indexed blocks equal to v* until the sum reaches tau", where v*
// is the largest value v with sum(mass >= v) >= tau.  Non-negative floats order like their bit
// patterns, so v* is found bit by bit (31 steps), each step one masked sum over the row, which
// the warp holds in registers (lane l owns blocks l, l + 32, ...).  The sums are taken in 2^-60
// fixed point: integer addition is exact and order-independent, so the result is deterministic
// and differs from a sequential fp64 sum by less than 1e-15 (masses below 2^-37 lose low bits).
// The kept set comes out as one ballot per 32 blocks - the bitmap word - and its size.
template <int K>  // blocks per lane
__global__ void __launch_bounds__(128)
select_rows_warp_kernel(const float* __restrict__ mass, int rows, int nKb, double tau, int fixed_count,
                        int32_t* __restrict__ counts, uint32_t* __restrict__ bitmaps, int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int words = (nKb + 31) >> 5;
  const float* mrow = mass + row * nKb;
  uint32_t bits[K];
  unsigned long long fx[K];
  bool bad = false;
  float row_sum = 0.0f;
#pragma unroll
  for (int k = 0; k < K; ++k) {
    const int i = k * 32 + lane;
    float m = (i < nKb) ? mrow[i] : 0.0f;
    if (!(m >= 0.0f) || m > 8.0f) {  // negative, NaN, or far beyond any mass
      bad = true;
      m = 0.0f;
    }
    bits[k] = (m == 0.0f) ? 0u : __float_as_uint(m);  // -0 becomes +0
    // the weight that is summed: the mass in 2^-60 fixed point (exact product), or 1 per existing
    // block for the fixed-ratio rule, which counts; blocks past the row's end weigh nothing
    if (fixed_count > 0) fx[k] = (i < nKb) ? 1ull : 0ull;
    else fx[k] = (unsigned long long)((double)m * 1152921504606846976.0);
    row_sum += m;
  }
  // The fixed-point sums below hold at most 16: a row whose masses add up to more than 8 (a mass
  // row sums to 1) is reported, and keeps every block, instead of wrapping silently.
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) row_sum += __shfl_xor_sync(0xffffffffu, row_sum, d);
  if (fixed_count <= 0 && row_sum > 8.0f) {
    bad = true;
#pragma unroll
    for (int k = 0; k < K; ++k) fx[k] = 0ull;
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) report_error(status, LOSA_ERR_BAD_MASS);

  // sum (or count, for the fixed-ratio rule) of the blocks with bits >= v, over the whole row
  auto measure_ge = [&](uint32_t v) -> unsigned long long {
    unsigned long long a0 = 0ull, a1 = 0ull;
#pragma unroll
    for (int k = 0; k < K; k += 2) {
      a0 += (bits[k] >= v) ? fx[k] : 0ull;
      a1 += (bits[k + 1] >= v) ? fx[k + 1] : 0ull;
    }
    const unsigned long long a = a0 + a1;
    // warp sum of 64-bit values as three integer reductions of 22-bit limbs (one instruction each)
    const unsigned r0 = __reduce_add_sync(0xffffffffu, (unsigned)(a & 0x3fffffull));
    const unsigned r1 = __reduce_add_sync(0xffffffffu, (unsigned)((a >> 22) & 0x3fffffull));
    const unsigned r2 = __reduce_add_sync(0xffffffffu, (unsigned)(a >> 44));
    return (unsigned long long)r0 + ((unsigned long long)r1 << 22) + ((unsigned long long)r2 << 44);
  };

  const unsigned long long target =
      (fixed_count > 0) ? (unsigned long long)min(fixed_count, nKb)
                        : (unsigned long long)(fmin(tau, 1.0) * 1152921504606846976.0);
  int s = nKb, need = 0;
  uint32_t v = 0u;  // kept: bits > v, and the first `need` (by index) with bits == v
  const bool all = (fixed_count <= 0 && tau >= 1.0) || measure_ge(0u) < target;  // never reaches tau
  if (!all) {
    for (int b = 30; b >= 0; --b) {
      const uint32_t cand = v | (1u << b);
      if (measure_ge(cand) >= target) v = cand;
    }
    unsigned long long gt = 0ull;
    int n_gt = 0, n_eq = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
      const bool valid = (k * 32 + lane) < nKb;
      if (valid && bits[k] > v) {
        gt += fx[k];
        ++n_gt;
      }
      if (valid && bits[k] == v) ++n_eq;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      gt += __shfl_xor_sync(0xffffffffu, gt, d);
      n_gt += __shfl_xor_sync(0xffffffffu, n_gt, d);
      n_eq += __shfl_xor_sync(0xffffffffu, n_eq, d);
    }
    unsigned long long need64;
    if (fixed_count > 0) {
      need64 = target - gt;
    } else {
      const unsigned long long fv = (unsigned long long)((double)__uint_as_float(v) * 1152921504606846976.0);
      need64 = (fv == 0ull) ? (unsigned long long)n_eq : (target - gt + fv - 1ull) / fv;
    }
    need = (int)min(need64, (unsigned long long)n_eq);
    s = n_gt + need;
  }
  int seen = 0;  // ties at lower indices
#pragma unroll
  for (int k = 0; k < K; ++k) {
    const bool valid = (k * 32 + lane) < nKb;
    const bool eq = valid && !all && bits[k] == v;
    const uint32_t eqm = __ballot_sync(0xffffffffu, eq);
    const int rank = seen + __popc(eqm & ((1u << lane) - 1u));
    const bool keep = valid && (all || bits[k] > v || (eq && rank < need));
    seen += __popc(eqm);
    const uint32_t word = __ballot_sync(0xffffffffu, keep);
    if (lane == 0 && k < words) bitmaps[row * words + k] = word;
  }
  if (lane == 0) counts[row] = s;
}

__global__ void __launch_bounds__(1024)
scan_counts_kernel(const int32_t* __restrict__ counts, int rows, int32_t* __restrict__ offsets,
                   int64_t kv_capacity, int* status) {
  __shared__ int warp_total[32];
  __shared__ int carry_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < rows; base += 1024) {
    const int i = base + tid;
    const int c = (i < rows) ? counts[i] : 0;
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += up;
    }
    if (lane == 31) warp_total[warp] = incl;
    __syncthreads();
    int wbase = 0;
    for (int w = 0; w < warp; ++w) wbase += warp_total[w];
    const int carry = carry_s;
    if (i < rows) offsets[i] = carry + wbase + incl - c;
    __syncthreads();
    if (tid == 1023) carry_s = carry + wbase + incl;
    __syncthreads();
  }
  if (tid == 0) {
    offsets[rows] = carry_s;
    if ((int64_t)carry_s > kv_capacity) report_error(status, LOSA_ERR_CAPACITY);
  }
}

__global__ void __launch_bounds__(256)
expand_rows_kernel(const uint32_t* __restrict__ bitmaps, const int32_t* __restrict__ offsets,
                   int rows, int nKb, int32_t* __restrict__ kv_idx, int64_t kv_capacity) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int words = (nKb + 31) >> 5;
  int64_t pos0 = offsets[row];
  for (int w0 = 0; w0 < words; w0 += 32) {
    const int w = w0 + lane;
    uint32_t word = (w < words) ? bitmaps[row * words + w] : 0u;
    const int cnt = __popc(word);
    int incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += up;
    }
    int64_t pos = pos0 + incl - cnt;
    while (word) {
      const int b = __ffs(word) - 1;
      word &= word - 1;
      if (pos < kv_capacity) kv_idx[pos] = w * 32 + b;
      ++pos;
    }
    pos0 += __shfl_sync(0xffffffffu, incl, 31);
  }
}

__global__ void __launch_bounds__(256)
validate_csr_kernel(int rows, int nKb, const int32_t* __restrict__ offsets,
                    const int32_t* __restrict__ kv_idx, int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int32_t b = offsets[row], e = offsets[row + 1];
  const int32_t nnz = offsets[rows];  // every read below stays inside [0, nnz)
  bool bad = (row == 0 && b != 0) || e <= b || (e - b) > nKb || b < 0 || e > nnz;
  if (!bad) {
    for (int p = b + lane; p < e; p += 32) {
      const int32_t j = kv_idx[p];
      if (j < 0 || j >= nKb) bad = true;
      if (p > b && kv_idx[p - 1] >= j) bad = true;
    }
  }
  if (bad) report_error(status, LOSA_ERR_BAD_INDEX);
}

// Retained and total mass of every row under a CSR pattern (Eq. 2 before the outer sums): one
// warp per row, fp64 partial sums per lane, shuffle tree.
__global__ void __launch_bounds__(256)
row_recall_kernel(const float* __restrict__ mass, int rows, int nKb,
                  const int32_t* __restrict__ offsets, const int32_t* __restrict__ kv_idx,
                  double* __restrict__ retained, double* __restrict__ total, int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float* mrow = mass + row * nKb;
  double tot = 0.0, ret = 0.0;
  for (int j = lane; j < nKb; j += 32) tot += (double)mrow[j];
  const int32_t b = offsets[row], e = offsets[row + 1];
  bool bad = false;
  for (int p = b + lane; p < e; p += 32) {
    const int32_t j = kv_idx[p];
    if (j < 0 || j >= nKb) bad = true;  // skipped, never used as an address
    else ret += (double)mrow[j];
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    tot += __shfl_xor_sync(0xffffffffu, tot, d);
    ret += __shfl_xor_sync(0xffffffffu, ret, d);
  }
  if (bad) report_error(status, LOSA_ERR_BAD_INDEX);
  if (lane == 0) {
    retained[row] = ret;
    total[row] = tot;
  }
}

int next_pow2(int x) {
  int n = 32;
  while (n < x) n <<= 1;
  return n;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

size_t select_workspace_bytes(int64_t rows, int nKb) {
  const size_t words = (size_t)(nKb + 31) / 32;
  return align_up((size_t)rows * sizeof(int32_t), 256) + (size_t)rows * words * sizeof(uint32_t);
}

int launch_select(int rows, int nKb, const float* mass, double tau, int fixed_count,
                  int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws, int* status,
                  cudaStream_t st) {
  int32_t* counts = static_cast<int32_t*>(ws);
  uint32_t* bitmaps = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) +
                                                  align_up((size_t)rows * sizeof(int32_t), 256));
  if (nKb <= 1024) {
    // one warp per row, the row in registers, no sort
    const int ctas = (rows + 3) / 4;
    if (nKb <= 256)
      select_rows_warp_kernel<8><<<ctas, 128, 0, st>>>(mass, rows, nKb, tau, fixed_count, counts, bitmaps, status);
    else if (nKb <= 512)
      select_rows_warp_kernel<16><<<ctas, 128, 0, st>>>(mass, rows, nKb, tau, fixed_count, counts, bitmaps, status);
    else
      select_rows_warp_kernel<32><<<ctas, 128, 0, st>>>(mass, rows, nKb, tau, fixed_count, counts, bitmaps, status);
  } else {
    const int n2 = next_pow2(nKb);
    const int words = (nKb + 31) / 32;
    const size_t smem = (size_t)n2 * 8 + (size_t)words * 4;
    // (a function attribute belongs to the current device: set on every call, it costs nothing)
    if (smem > 48 * 1024) {
      LOSA_CUDA_TRY(cudaFuncSetAttribute(select_rows_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    select_rows_kernel<<<rows, kSelThreads, smem, st>>>(mass, nKb, n2, tau, fixed_count, counts, bitmaps,
                                                        status);
  }
  scan_counts_kernel<<<1, 1024, 0, st>>>(counts, rows, offsets, kv_capacity, status);
  const int warps_per_cta = 8;
  expand_rows_kernel<<<(rows + warps_per_cta - 1) / warps_per_cta, warps_per_cta * 32, 0, st>>>(
      bitmaps, offsets, rows, nKb, kv_idx, kv_capacity);
  LOSA_CUDA_TRY(cudaGetLastError());
  return LOSA_OK;
}

// ---- allocation-free variant ----------------------------------------------------------
// Scratch for losa_select_noalloc lives in the library image: one array per GPU that loads
// the library, held until the process exits.  The first 256 bytes hold the status word of
// the last call, the rest is the counts + bitmaps workspace.
constexpr size_t kStaticStatusBytes = 256;
static __device__ __align__(256) unsigned char g_select_scratch[LOSA_SELECT_NOALLOC_MAX_SCRATCH];

namespace {
unsigned char* g_scratch_addr[kMaxDevices] = {};  // device address of g_select_scratch, per device
}  // namespace

size_t select_noalloc_workspace_limit() {
  return (size_t)LOSA_SELECT_NOALLOC_MAX_SCRATCH - kStaticStatusBytes;
}

int launch_select_noalloc(int rows, int nKb, const float* mass, double tau, int32_t* offsets,
                          int32_t* kv_idx, int64_t kv_capacity, int32_t* device_status,
                          cudaStream_t st) {
  int dev = 0;
  LOSA_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LOSA_ERR_UNSUPPORTED;
  if (!g_scratch_addr[dev]) {
    // In host code the array's name is only a handle; the device address must be asked for,
    // once per device, with that device current.
    unsigned char* ptr = nullptr;
    LOSA_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_select_scratch));
    g_scratch_addr[dev] = ptr;
  }
  unsigned char* base = g_scratch_addr[dev];
  int* status = reinterpret_cast<int*>(base);
  unsigned char* ws = base + kStaticStatusBytes;
  // the array keeps the previous call's contents: the status word must start at zero; counts
  // and bitmaps are fully rewritten by the first kernel before anything reads them
  LOSA_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), st));
  // the same kernels, dispatch and workspace layout as losa_select
  const int rc = launch_select(rows, nKb, mass, tau, 0, offsets, kv_idx, kv_capacity, ws, status, st);
  if (rc != LOSA_OK) return rc;
  if (device_status)
    LOSA_CUDA_TRY(cudaMemcpyAsync(device_status, status, sizeof(int), cudaMemcpyDeviceToDevice, st));
  return LOSA_OK;
}

int launch_row_recall(int rows, int nKb, const float* mass, const int32_t* offsets,
                      const int32_t* kv_idx, double* retained, double* total, cudaStream_t st) {
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return rc;
  int* status = dev->status_dev;
  row_recall_kernel<<<(rows + 7) / 8, 256, 0, st>>>(mass, rows, nKb, offsets, kv_idx, retained,
                                                    total, status);
  LOSA_CUDA_TRY(cudaGetLastError());
  return LOSA_OK;
}

int launch_validate_csr(int rows, int nKb, const int32_t* offsets, const int32_t* kv_idx,
                        cudaStream_t st) {
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return rc;
  int* status = dev->status_dev;
  validate_csr_kernel<<<(rows + 7) / 8, 256, 0, st>>>(rows, nKb, offsets, kv_idx, status);
  LOSA_CUDA_TRY(cudaGetLastError());
  return LOSA_OK;
}

}  // namespace losa
