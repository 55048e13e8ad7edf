/*
 * liblosa — LoSA's attention hot path for NVIDIA B200 (sm_100a), C ABI.
 *
 * LoSA ("Near-Lossless Sparse Attention", Methodology section) measures the
 * exact block attention mass of one dense attention step, keeps for every
 * (head, query block) the smallest set of key/value blocks whose mass reaches
 * a threshold tau, and reuses those frozen block indices in a block-sparse
 * attention forward at every later step.  This library is that path:
 *
 *     losa_block_mass   Eq. 1   q, k            -> mass[B, H, nQb, nKb]
 *     losa_select       Eq. 3   mass, tau       -> CSR (offsets, kv_idx)
 *     losa_sparse_attn  Eq. 4   q, k, v, CSR    -> o
 *     losa_attn         dense softmax attention (the warm-up steps and the
 *                       denominator of the sparse-versus-dense ratio)
 *     losa_attn_mass    dense attention + block mass in one pass (the construction step)
 *
 * Conventions shared by every call
 * --------------------------------
 *  - All tensor pointers are DEVICE pointers on the current CUDA device,
 *    16-byte aligned.  The caller owns every buffer, including workspace;
 *    the library allocates no device memory per call (per device it keeps
 *    one small pinned status word and the SM count, created on the device's
 *    first call).  Several devices may be driven from one process, each
 *    call with its device current; a device that is not an sm_100 GPU gets
 *    LOSA_ERR_UNSUPPORTED.
 *  - q, k, v, o are [B, H, N, D] with element strides (sb, sh, sn) and D
 *    contiguous; strides must be multiples of 8 elements.  q, k, v are bf16.
 *    N is the number of VALID tokens and need not be a multiple of the block
 *    sizes: the last query/key block is short, tokens >= N do not exist (they
 *    enter no softmax and no mass) and rows >= N of o are never written.
 *  - nQb = ceil(N / R), nKb = ceil(N / C).  A "row" is one (b, h, i) query
 *    block, numbered (b*H + h)*nQb + i.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t; NULL = default
 *    stream) and return without synchronising.  The return value reports
 *    errors found on the host before any launch.  Errors found on the device
 *    (a bounded wait that expired, a bad block index, a negative mass, a CSR
 *    that overflowed its capacity) are recorded in the device's status word,
 *    which losa_async_status() returns and clears.  The word is shared by
 *    every stream and host thread that uses the device: it holds the first
 *    error since it was last cleared, whichever call raised it.  No kernel
 *    ever traps, asserts or waits without a bound.
 *  - Supported shapes: D in {64, 128}; (R, C) in {(64, 64), (128, 128), (128, 64), (128, 32)}
 *    (the last is the block geometry the paper runs with); fewer than 65535 key blocks for the
 *    attention and mass calls, at most LOSA_SELECT_MAX_KEY_BLOCKS (8192) per row for the
 *    selection calls (a longer row gets LOSA_ERR_UNSUPPORTED): with C = 32 the whole chain
 *    mass -> select -> sparse attention therefore reaches 262144 tokens.
 */
#ifndef LOSA_H_
#define LOSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  LOSA_OK = 0,
  LOSA_ERR_INVALID_ARG = -1, /* null / misaligned pointer, bad size, tau outside (0, 1]      */
  LOSA_ERR_UNSUPPORTED = -2, /* D, R, C, dtype or device not supported                       */
  LOSA_ERR_WORKSPACE = -3,   /* workspace smaller than losa_workspace_bytes()                */
  LOSA_ERR_CAPACITY = -4,    /* CSR longer than kv_capacity (device-side)                    */
  LOSA_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed                            */
  LOSA_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired (device-side)             */
  LOSA_ERR_BAD_INDEX = -7,   /* kv_idx / offsets out of range or not ascending (device-side) */
  LOSA_ERR_BAD_MASS = -8,    /* losa_select saw a negative, NaN or > 8 mass, or a row whose
                                masses add up to more than 8 (device-side)                   */
  LOSA_ERR_INTERNAL = -9     /* checked build only (-DLOSA_CHECKED=1): a kernel computed an index
                                outside its buffer; the access was skipped (device-side)     */
};

enum {
  LOSA_OP_BLOCK_MASS = 0,
  LOSA_OP_SELECT = 1,
  LOSA_OP_SPARSE_ATTN = 2,
  LOSA_OP_ATTN = 3,
  LOSA_OP_ATTN_MASS = 4
};

enum { LOSA_DTYPE_BF16 = 0, LOSA_DTYPE_F32 = 1 };

/* Longest mass row (key blocks) the selection calls accept. */
#define LOSA_SELECT_MAX_KEY_BLOCKS 8192

typedef struct {
  int32_t B, H, N, D; /* batch, heads, VALID tokens, head dimension                     */
  int32_t R, C;       /* query / key-value block size: (64,64), (128,128), (128,64), (128,32) */
  int64_t sb, sh, sn; /* element strides of batch, head, token (D is contiguous)        */
  float scale;        /* softmax scale; 0 selects 1/sqrt(D) as in A = softmax(QK^T/sqrt d) */
} losa_problem_t;

/* Bytes of caller-provided device workspace an operation needs for this problem
 * (LOSA_OP_*).  For LOSA_OP_SELECT only B, H, N, R, C are read.  Returns 0 for an invalid
 * problem.  Host-only: touches no GPU. */
size_t losa_workspace_bytes(int op, const losa_problem_t* p);

/* Exact block attention mass of one dense attention step (Eq. 1).
 * For every row (b, h, i) and key block j:
 *     mass[b,h,i,j] = (1/|B^Q_i|) * sum_{q in B^Q_i} sum_{k in B^K_j} A(q,k),
 *     A = row-wise softmax(q k^T * scale) over the N valid keys,
 * i.e. the paper's M(i,j) divided by the number of valid rows of query block i, so
 * that each row of `mass` sums to 1 and Eq. 3's threshold theta*R becomes tau.
 * One pass over Q K^T: every row keeps a running sum of exponentials against a reference
 * score (the row's maximum over its first key tile; rows whose later scores outgrow the
 * fp32 range around it are recomputed with a running maximum by a second launch on the same
 * stream); the per-key-block sums are taken in the same pass and normalised by the row's
 * final sum at the end.
 *   q, k    bf16 [B,H,N,D] (strides from p)
 *   mass    f32  [B,H,nQb,nKb] contiguous, fully overwritten
 *   lse     f32  [B,H,N] contiguous or NULL: natural-log sum-exp of each row's scaled scores
 *   ws      >= losa_workspace_bytes(LOSA_OP_BLOCK_MASS, p) bytes, contents undefined after */
int losa_block_mass(const losa_problem_t* p, const void* q, const void* k, float* mass,
                    float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/* Retained-mass selection (Eq. 3).  For every row r = (b, h, i): sort the nKb masses in
 * decreasing order (equal masses: lower block index first), accumulate them in fp64 and
 * keep the shortest prefix whose sum is >= tau; tau >= 1 keeps every block, and so does a
 * row whose sum never reaches tau.  Each row keeps at least one block.
 *   mass        f32 [rows, nKb], rows = B*H*nQb, nKb <= LOSA_SELECT_MAX_KEY_BLOCKS; values in
 *               [0, 8] and row sums <= 8 (a mass row sums to 1), else LOSA_ERR_BAD_MASS is
 *               recorded: a bad value counts as 0, a row with a bad sum keeps every block
 *   tau         in (0, 1]
 *   offsets     i32 [rows + 1]: exclusive prefix of the per-row counts; offsets[rows] = nnz
 *   kv_idx      i32 [kv_capacity]: kept block indices, row after row, ascending in a row
 *   kv_capacity rows*nKb always suffices; if nnz exceeds it nothing past the capacity is
 *               written and the status word becomes LOSA_ERR_CAPACITY (offsets stay exact)
 *   ws          >= losa_workspace_bytes(LOSA_OP_SELECT, p) bytes                          */
int losa_select(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass, double tau,
                int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws,
                size_t ws_bytes, void* cuda_stream);

/* Fixed-ratio selection, the rule the paper's ablation compares Eq. 3 with ("Retained mass versus
 * fixed-ratio top-k selection"): every row keeps its k heaviest blocks (equal masses: lower block
 * index first), 1 <= k <= nKb.  Same outputs, workspace and error behaviour as losa_select;
 * offsets[r] = r * k. */
int losa_select_topk(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass, int32_t k,
                     int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity, void* ws,
                     size_t ws_bytes, void* cuda_stream);

/* Retained and total block mass of every row under a CSR pattern: the numerator and denominator
 * of Recall (Eq. 2) before the sums over heads and query blocks, accumulated in fp64.
 * Recall = sum(retained) / sum(total); Coverage is offsets[rows] / (rows * nKb).
 *   mass f32 [rows, nKb];  retained, total  f64 [rows] (device).  A block index outside
 *   [0, nKb) is skipped and reported as LOSA_ERR_BAD_INDEX.  Needs no workspace. */
int losa_row_recall(int32_t rows, int32_t nKb, const float* mass, const int32_t* offsets,
                    const int32_t* kv_idx, double* retained, double* total, void* cuda_stream);

/* Bytes of the scratch array built into the library for losa_select_noalloc (per GPU). */
#define LOSA_SELECT_NOALLOC_MAX_SCRATCH (4u * 1024u * 1024u)

/* losa_select for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of losa_select, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits or unaffordable - inside a
 * latency-critical serving loop whose memory was carved up at start-up, under a framework
 * whose allocator owns every byte of the device, or in a plugin that is handed its tensors
 * and nothing else.  Such callers cannot supply the workspace losa_select asks for.  Here the
 * workspace is a fixed array inside the library image instead: LOSA_SELECT_NOALLOC_MAX_SCRATCH
 * bytes on every GPU that loads the library, held until the process exits.  The call performs
 * no cudaMalloc, cudaFree, cudaHostAlloc or other allocating call, and unlike the other entry
 * points it does not touch the library's pinned status word (creating that allocates).
 *
 * Same kernels, arguments and results as losa_select, except:
 *   - no workspace arguments.  The problem must fit the array: 256-byte-rounded 4*rows
 *     plus 4*rows*ceil(nKb/32) bytes, plus 256, at most LOSA_SELECT_NOALLOC_MAX_SCRATCH
 *     (all five benchmark shapes fit); otherwise LOSA_ERR_WORKSPACE is returned, nothing is
 *     launched, and losa_last_cuda_error() says how many bytes were needed.
 *   - device-side errors (LOSA_ERR_CAPACITY, LOSA_ERR_BAD_MASS) are not visible through
 *     losa_async_status().  If device_status is not NULL it must point to an int32 in device
 *     memory; the call writes LOSA_OK or the error code there, in stream order.
 *   - the first call on each device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - every call on a device shares the one array, which still holds the previous call's
 *     contents.  The call clears what has to start at zero itself, so back-to-back calls on
 *     one stream are fine; calls that can overlap on the GPU (different streams, different
 *     host threads) race on the array and must be serialised by the caller. */
int losa_select_noalloc(int32_t B, int32_t H, int32_t nQb, int32_t nKb, const float* mass,
                        double tau, int32_t* offsets, int32_t* kv_idx, int64_t kv_capacity,
                        int32_t* device_status, void* cuda_stream);

/* Block-sparse attention with a frozen pattern (Eq. 4).  Every valid query row q of query
 * block i attends to the valid keys of the blocks kv_idx[offsets[r] .. offsets[r+1]) only;
 * the softmax denominator runs over those keys only:
 *     o(q) = sum_{k in K(q)} softmax_{K(q)}(q k^T * scale) v(k).
 * The CSR must satisfy losa_validate_csr(); a block index outside [0, nKb) is skipped and
 * reported as LOSA_ERR_BAD_INDEX, never dereferenced.
 *   q, k, v  bf16 [B,H,N,D];  o  [B,H,N,D] with the same strides, bf16 or f32 (o_dtype)
 *   ws       >= losa_workspace_bytes(LOSA_OP_SPARSE_ATTN, p) bytes (about 21 MB at D = 128
 *            plus the work units' tile lists: the counter the persistent CTAs draw work
 *            items from, the partial results of the last work items, which are processed in
 *            parts and merged by a second kernel on the same stream, and the list of work
 *            units that a fallback launch recomputes because their scores outgrew the
 *            reference of their first tile); not shared between calls that may run
 *            concurrently; contents undefined afterwards.  The result does not depend on
 *            timing: the same call on the same GPU gives the same bits.
 * The output is normalised by the sum of the bf16-rounded weights the tensor core multiplies
 * with V, so every output row is a weighted mean of value rows (exact for a row that a
 * single key dominates).                                                                 */
int losa_sparse_attn(const losa_problem_t* p, const void* q, const void* k, const void* v,
                     const int32_t* offsets, const int32_t* kv_idx, void* o, int o_dtype,
                     void* ws, size_t ws_bytes, void* cuda_stream);

/* One problem of a batched launch: its tensors, its own frozen pattern, its output.  All
 * problems of a launch share the shape, strides and block geometry of one losa_problem_t. */
typedef struct {
  const void* q;          /* bf16 [B,H,N,D] */
  const void* k;
  const void* v;
  const int32_t* offsets; /* i32 [B*H*nQb + 1]: this problem's CSR */
  const int32_t* kv_idx;
  void* o;                /* [B,H,N,D], bf16 or f32 */
} losa_layer_t;

#define LOSA_MAX_BATCHED_LAYERS 64

/* losa_sparse_attn (Eq. 4) for several problems in ONE persistent launch.  The paper keeps the
 * pattern separately for each layer, head and query block and for the two guidance branches
 * ("One-Time Pattern Construction"); the batch dimension B carries branches inside a call, this
 * call carries whole problems that each have their own tensors and CSR - layers whose inputs
 * are all available, or independent requests of one shape.  The persistent CTAs draw work
 * items across all problems from one counter, so that small problems share one launch (a
 * call on a 2048-token layer is bound by launch latency, not by work) and only the last wave
 * of the whole batch, not of every problem, runs partly filled.  Each problem's result is bit
 * for bit that of its own losa_sparse_attn call as long as neither launch cuts the work
 * items of its last wave into parts (which items are cut depends on the total count).
 *   layers   HOST array of n_layers entries (1 .. LOSA_MAX_BATCHED_LAYERS), device pointers
 *            inside, 16-byte aligned; read before the call returns
 *   ws       >= losa_workspace_bytes_batched(LOSA_OP_SPARSE_ATTN, p, n_layers) bytes,
 *            128-byte aligned */
int losa_sparse_attn_batched(const losa_problem_t* p, int32_t n_layers, const losa_layer_t* layers,
                             int o_dtype, void* ws, size_t ws_bytes, void* cuda_stream);

/* Workspace of a batched call (op: LOSA_OP_SPARSE_ATTN); 0 for an invalid problem or count. */
size_t losa_workspace_bytes_batched(int op, const losa_problem_t* p, int32_t n_layers);

/* How many work slots (persistent CTAs, or pairs of CTAs where the kernel pairs them) a call
 * of kind `op` (a LOSA_OP_* attention call) occupies on the current device.  A call's work items -
 * pairs of 128-row query tiles per (batch, head) - are spread over these slots, and the items of
 * a last, partly filled wave are cut into parts and merged; callers that compare results bit for
 * bit across calls of different sizes need this number.  0 for an invalid problem or op.
 * (On a device that cannot hold a pair of CTAs the paired kernels fall back to single CTAs; the
 * number returned does not know that.) */
int32_t losa_work_slots(int op, const losa_problem_t* p);

/* Dense softmax attention o = softmax(q k^T * scale) v over the N valid keys: the paper's
 * dense steps up to the construction step, and this library's own dense baseline.
 * Same tensors and workspace rule as losa_sparse_attn, without the CSR. */
int losa_attn(const losa_problem_t* p, const void* q, const void* k, const void* v, void* o,
              int o_dtype, void* ws, size_t ws_bytes, void* cuda_stream);

/* The construction step as one kernel: dense attention that also accumulates the exact block
 * masses (the paper's Implementation paragraph builds the pattern inside the dense attention of
 * step t0, with a kernel of its own that sums the block masses on the way).  Results are those of
 * losa_attn (o) and losa_block_mass (mass, optional lse) on the same inputs, from one pass over
 * Q K^T.
 *   ws   >= losa_workspace_bytes(LOSA_OP_ATTN_MASS, p) bytes                               */
int losa_attn_mass(const losa_problem_t* p, const void* q, const void* k, const void* v, void* o,
                   int o_dtype, float* mass, float* lse, void* ws, size_t ws_bytes,
                   void* cuda_stream);

/* Checks a CSR on the device: offsets[0] == 0, offsets non-decreasing with every row
 * holding between 1 and nKb entries (Eq. 3 keeps at least one block), indices in
 * [0, nKb) and strictly ascending inside a row.  A violation sets the status word to
 * LOSA_ERR_BAD_INDEX.  Needs no workspace. */
int losa_validate_csr(int32_t rows, int32_t nKb, const int32_t* offsets, const int32_t* kv_idx,
                      void* cuda_stream);

/* Synchronises `cuda_stream`, then returns and clears the device-side status word
 * (LOSA_OK or the first device-side LOSA_ERR_* recorded since the last call). */
int losa_async_status(void* cuda_stream);

/* Diagnostic for tests of the time-out path.  (The paper has no counterpart.)  Every wait inside
 * the attention kernels is bounded; this call makes the bound observable without harming the
 * GPU.  It arms ONE launch: the next losa_attn, losa_sparse_attn, losa_block_mass or
 * losa_attn_mass of this process runs its kernel with the role that publishes the work
 * (the tile lists) publishing nothing, and with every device-side wait limited to `polls` polls
 * (1 .. 65536; a few milliseconds) instead of about a second.  No copy and no tensor-core
 * instruction is issued in that launch; every role's first wait runs out, the CTAs leave through
 * the common teardown that frees tensor memory, and the status word becomes LOSA_ERR_TIMEOUT.
 * The outputs of that call are undefined.  The launch after it is an ordinary one. */
int losa_debug_stall_next_launch(uint32_t polls);

/* Static, human-readable name of a status code. */
const char* losa_status_string(int status);

/* Text of the last host-side CUDA error seen by this thread's calls ("" if none). */
const char* losa_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LOSA_H_ */
