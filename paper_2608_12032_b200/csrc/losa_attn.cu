// Attention kernels of liblosa for sm_100a: dense attention, block-sparse attention over a
// frozen CSR pattern (Eq. 4), the exact block-mass pass (Eq. 1) and the fused construction step,
// as ONE warp-specialised persistent kernel template with two thread layouts.
//
// Warps 0-3 are utility warps: warp 0 is the TMA producer, which streams the query tiles and the
// K / V tiles named by the tile list into 128B-swizzled shared-memory rings (a K/V tile is 128
// keys: 128 / C key blocks, one copy per block and 64-column slab); warps 1 and 2 (one elected
// thread each) issue the tcgen05 MMAs: S = Q K^T from shared memory into TMEM, O += P V with P
// read from TMEM (bf16, written over S) and V from shared memory as the MN-major operand; warp 3
// publishes the tile list every other warp follows (sparse mode: streamed from lists that
// build_tile_lists_kernel made before the launch).  The softmax warps follow: two warpgroups, one
// 128-row query tile each and one thread per query row (mass pass, fused step, fallback), or four
// warpgroups with two threads per query row (dense and sparse forward); they take their registers
// from the utility warpgroup.
//
// A work item is a pair of consecutive query tiles of one (batch, head) - of one problem, in a
// batched launch.  The key blocks the pair visits are the union of the index lists of its query
// blocks (two lists, four when R = 64), so a K/V tile needed by both tiles is loaded once, and
// MMAs are issued only for the query tiles that list one of its blocks.  The items of the last,
// partly filled wave of the persistent grid are cut into parts of their lists, merged by
// merge_parts_kernel.
//
// One S = Q K^T covers a whole K/V tile (128-wide MMAs).  At head dimension 128 TMEM holds exactly
// S and O of both query tiles, P overwrites S, and per query tile the steps S -> softmax ->
// O += P V -> next S form a serial chain; the two tiles run that chain half a period apart, one
// issuer each, under a lock that keeps their bursts of MMAs from interleaving.  At head dimension
// 64 a third S buffer fits and the tiles take the three buffers in turn (one issuer for all
// S = Q K^T, one for all O += P V).  No mode keeps a running maximum on its common path: the
// exponentials are taken against a reference that moves only when a tile's row sums leave the safe
// range (one thread per row), or never within a work unit (two threads per row; units whose scores
// outgrow it are recomputed by a second launch of the one-thread-per-row kernel).
//
// Every wait is bounded; a wait that expires raises the CTA's abort flag, records
// LOSA_ERR_TIMEOUT, and all roles leave through the common teardown that frees TMEM.
//
// The dense and sparse forward and the fused step at head dimension 128 with 128-row query blocks and
// key blocks of 64 or 128 keys run in a second kernel, losa_pair_kernel (losa_attn_pair.cuh, included below): pairs
// of CTAs that multiply together (tcgen05.mma.cta_group::2), one query tile and three S buffers per
// CTA.  This kernel serves every other shape and mode and the fallback launch of all of them.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <atomic>
#include <cstddef>
#include <vector>

#include "losa_common.cuh"
#include "losa_ptx.cuh"

namespace losa {
namespace {

#ifndef LOSA_USE_PAIR
#define LOSA_USE_PAIR 1
#endif
#ifndef LOSA_PAIR_FUSED
#define LOSA_PAIR_FUSED 1
#endif
#ifndef LOSA_PAIR_MASS
#define LOSA_PAIR_MASS 1
#endif
#ifndef LOSA_PAIR_MIN_C
#define LOSA_PAIR_MIN_C 32
#endif

std::atomic<uint32_t> g_stall_polls{0u};  // > 0: the next attention launch is a diagnostic one

// Thread layout.  Warps 0-3 are the utility warpgroup (TMA, 2 MMA issuers, scheduler); the softmax
// warps follow.  Two layouts:
//   one thread per query row (SPLIT = false): 2 softmax warpgroups, one per query tile, each thread
//     holding a whole 128-column S row.  Used by the mass pass and the fused construction step,
//     and as the fallback of the attention-only modes.
//   two threads per query row (SPLIT = true): 4 softmax warpgroups, two per query tile, each
//     thread holding 64 columns.  A warp's ex2 instructions occupy it for 8 issue cycles each and
//     its other instructions do not overlap them (measured on the loop alone: 1301 cycles per
//     128-column row with one warp per scheduler partition, 1130 with two), so a query tile's
//     softmax needs two warps per partition to keep the special-function unit busy; the two warps
//     never talk to each other on the common path (see the softmax role).
template <bool SPLIT>
struct Lay {
  static constexpr int kSoftmaxWarps = SPLIT ? 16 : 8;
  static constexpr int kThreads = 128 + 32 * kSoftmaxWarps;
  static constexpr int kRegsSoftmax = SPLIT ? 104 : 216;
  static constexpr int kRegsUtility = SPLIT ? 64 : 72;
  static constexpr int kRegsAtLaunch = SPLIT ? 96 : 168;
  // setmaxnreg only moves registers inside the CTA's launch allocation: the increase waits until
  // the decrease has released enough, so the totals must balance or the increase never returns.
  static_assert(128 * kRegsUtility + 32 * kSoftmaxWarps * kRegsSoftmax <= kThreads * kRegsAtLaunch,
                "register reallocation exceeds the CTA's launch allocation");
  static_assert(kThreads * kRegsAtLaunch <= 65536, "launch allocation exceeds the register file");
};
// The utility warps take the LOWEST warp ids.  When several warps of a scheduler partition are
// ready, the hardware favours the lower (older) ids; a softmax warp in an arithmetic-dense
// stretch is ready every cycle, and with the MMA issuer behind it in that order each of the
// issuer's instructions waited ~10x longer (measured), which put the issuer on the critical path.
constexpr int kProducerWarp = 0, kIssuerWarp = 1, kSchedulerWarp = 3;  // issuers: warps 1 and 2
constexpr int kTmemCols = 512;
// Tile list ring: the scheduler warp writes one 32-bit entry per work item header, per K/V tile
// and one end marker; every other warp reads all of them in order.
constexpr size_t kCounterBytes = 256;  // head of the workspace: the work-item counter
constexpr size_t kRowstatBytes = (size_t)kMaxPersistentCtas * 2 * 128 * sizeof(float2);
constexpr size_t kPartMlBytes = kRowstatBytes;  // same shape: [slot][2][128] float2
constexpr int kTlChunks = 4;
constexpr uint32_t kTlItem = 1u << 28, kTlEnd = 2u << 28;  // entry type in bits 31:28 (0 = tile)
// An item header carries the work item in bits 23:0 and, for a unit that covers only part of the
// item's key range, the part index in bits 26:24 and a flag in bit 27.
constexpr uint32_t kTlItemMask = 0x00ffffffu, kTlPartial = 1u << 27;
// A K/V tile is a group of 128 / C consecutive tile entries (key block index in bits 15:0,
// membership bits from bit 16); the last group of an item is padded with this entry: no member,
// and a block index whose rows lie past the end of the tensor (the copy engine fills zeros).
constexpr uint32_t kTlPad = 0xffffu;
constexpr int kMaxParts = 8;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;
constexpr float kSafeRowSum = 1.099511627776e12f;  // 2^40: a tile's row sum beyond this re-centres the reference
// two threads per row: a tile's half-row sum beyond 2^60 (or NaN) sends the work unit to the fallback
constexpr float kSplitSafeSum = 1.152921504606846976e18f;

template <int D, int R, int C_, int MODE, int KT, bool ROT = false>
struct Cfg {
  static constexpr int kC = C_;                       // keys per key block
  static constexpr int kT = KT;                       // keys per K/V tile: one S = Q K^T per tile
  static constexpr int kG = kT / kC;                  // key blocks gathered into one K/V tile
  static constexpr int kQBT = 128 / R;                // query blocks per 128-row tile
  static constexpr int kNB = 2 * kQBT;                // query blocks per work item
  static constexpr int kDH = D / 64;                  // 64-element slabs along D
  static constexpr int kQSlab = 128 * 128;            // bytes of a [128][64] bf16 slab
  static constexpr int kQBytes = kDH * kQSlab;        // one query tile
  static constexpr int kKVSlab = kT * 128;            // bytes of a [128][64] bf16 slab
  static constexpr int kKVBytes = kDH * kKVSlab;      // one K (or V) tile
  static constexpr int kBoxBytes = kC * 128;          // one key block of a slab (a TMA box)
  static constexpr bool kHasV = (MODE != kMass);
  static constexpr bool kWantMass = (MODE == kMass || MODE == kFused);
  static constexpr int kW = kT;                       // columns of S
  // TMEM (512 columns): with an O accumulator, per query tile one S of 128 columns (P in place)
  // and O; the mass pass has no O and double-buffers S instead.
  static constexpr int kNS = kHasV ? 1 : 2;           // S buffers per query tile
  static constexpr int kSStride = kHasV ? 128 : 256;  // TMEM columns between the tiles' S areas
  static constexpr int kRingBudget = (kHasV ? 160 : 128) * 1024;  // K + V rings
  // a V tile stays in use about one tile longer than a K tile (its product is issued after the
  // tile's softmax), so V gets the deeper ring
  // (rotating score buffers, head dimension 64: O += P V trails S = Q K^T by up to three steps, so
  // a V tile is held that much longer while a K tile goes back at once: 7 V and 4 K stages of 16 KB)
  static constexpr int kNV = ROT ? 7 : kHasV ? ((kKVBytes >= 32768) ? 3 : 4) : 0;
  static constexpr int kNK0 = (kRingBudget - kNV * kKVBytes) / kKVBytes;
  static constexpr int kNK = ROT ? 4 : kNK0 > 6 ? 6 : kNK0;
  static constexpr uint32_t kIdescQK = ptx::idesc_bf16_f32(128, kW, false, false);
  static constexpr uint32_t kIdescPV = ptx::idesc_bf16_f32(128, D, false, true);
};

// One entry per problem of a batched launch (several layers or requests of one shape in one
// persistent launch): the problem's tensor maps, its output and its own CSR pattern.  The table
// lives in the workspace and is written by the host before the launch.
struct alignas(128) ProblemEntry {
  CUtensorMap map_q, map_k, map_v;
  CUtensorMap map_kh;  // K with boxes of at most 64 keys (the CTA-pair kernel copies half a K tile per CTA)
  // boxes that span several key blocks, for K/V tiles whose key blocks are consecutive (C < 128)
  CUtensorMap map_k64, map_k128, map_v128;
  void* o;
  const int32_t* offsets;
  const int32_t* kv_idx;
};

struct Params {
  int B, H, N, nQb, nKb, nQt, nPairs, nWork;
  // Batched launch: work items run over nProb problems, item w belongs to problem
  // w / (B * H * nPairs); `problems` is null for a single problem, whose maps are kernel
  // parameters and whose o / offsets / kv_idx are the fields below.
  int nProb;
  const ProblemEntry* problems;
  // Work units: items [0, split_first) whole, items [split_first, nWork) in split_parts parts of
  // their key-block lists each (the last, partly filled wave of the persistent grid is cut finer).
  int nUnits, split_first, split_parts;
  // Sparse mode: the merged tile lists of all units, built by build_tile_lists_kernel before the
  // attention kernel: unit u owns tl_entries[u * tl_cap ...], tl_count[u] of them (padded to whole tiles).
  uint32_t* tl_entries;
  int32_t* tl_count;
  int tl_cap;
  float* part_o;    // [slot][2][128][D] unnormalised O of a partial unit, slot = (item - split_first) * parts + part
  float2* part_ml;  // [slot][2][128] (reference max, row sum) of a partial unit
  const int32_t* offsets;
  const int32_t* kv_idx;
  void* o;
  int o_f32;
  int64_t sb, sh, sn;
  float* mass;
  float* lse;
  int* work_counter;  // zeroed before the launch; CTAs draw work items from it
  float2* rowstat;  // mass modes: [grid][2][128] final (max, 1/sum) of every row of the item
                    // (fused step, two threads per row: [grid][2][2][128] the halves' row sums)
  float* rowinv;    // fused step, two threads per row: [grid][2][128] 1 / (row sum) of every row
  float2* table;  // mass modes: [grid][2][nKb][128] (sum of p, reference max) per row and key tile
  float scale_log2;
  int* status;
  // Work units whose scores outgrew the fixed reference of the two-threads-per-row kernel: it
  // appends them here, and a second launch (one thread per row, moving reference) recomputes them.
  int* redo_count;
  int* redo_list;
  int redo;             // this launch processes redo_list[0 .. *redo_count) instead of all units
  // extents of the buffers the kernels index into (elements), for the checked build
  long long cap_part_rows, cap_table_floats, cap_mass, cap_lse, cap_units;
  uint32_t wait_polls;  // bound of every device-side wait, in polls (ptx::kWaitPolls)
  int stall;            // diagnostic launch: the scheduler publishes nothing, so that every wait runs out
};

template <int NK, int NV, bool SPLIT, bool ROT>
struct Control {
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[NK], k_empty[NK];
  uint64_t v_full[NV > 0 ? NV : 1], v_empty[NV > 0 ? NV : 1];
  uint64_t s_full[2][2], s_free[2][2];  // per query tile and S buffer: written by the MMAs / read out
  uint64_t p_ready[2];                  // per query tile: P is in TMEM
  uint64_t o_done[2], o_free[2];  // per item: all products done / O read out
  uint64_t wg_bar[2];
  uint64_t tl_full[kTlChunks], tl_empty[kTlChunks];  // tile list ring, per 32-entry chunk
  uint32_t tl[kTlChunks * 32];
  uint64_t drain;
  uint32_t tmem_base;
  uint32_t mma_lock;  // held while a burst of MMAs is issued
  int abort_flag;
  // two threads per row: the pair's barrier per (query tile, lane quarter), the row sums the second
  // half hands to the first at the end of an item (two sets, used in turn), and the last work unit
  // this CTA sent to the fallback
  uint64_t pair_bar[SPLIT ? 8 : 1];
  float xch[SPLIT ? 2 * 2 * 128 : 1];
  int ovf_unit;
  // head dimension 64, two threads per row: three score buffers used in turn by both query tiles.
  // One barrier per (query tile, buffer): a barrier's phases then follow one query tile's own
  // sequence of tiles, so that its warps are never more than one phase away from it (they may be
  // whole work units ahead of, or behind, the other query tile's warps).
  uint64_t rot_s_full[ROT ? 6 : 1], rot_p_ready[ROT ? 6 : 1];
  uint64_t pv_done[ROT ? 3 : 1];  // per buffer: the product that read its P has run
};

// Checked build (-DLOSA_CHECKED=1, a substitute for a memory checker): every index the kernels
// compute into the workspace, the masses or the log-sum-exp is compared with the extent of its
// buffer; one that falls outside is recorded as LOSA_ERR_INTERNAL and the access is skipped (or
// redirected to element 0 of the same buffer).  The ordinary build compiles the checks away.
#ifndef LOSA_CHECKED
#define LOSA_CHECKED 0
#endif
#if LOSA_CHECKED
#define LOSA_IN_RANGE(idx, extent) \
  (((unsigned long long)(idx) < (unsigned long long)(extent)) || (report_error(p.status, LOSA_ERR_INTERNAL), false))
#else
#define LOSA_IN_RANGE(idx, extent) true
#endif

#define LOSA_WAIT_RELAXED(bar, parity)                                   \
  do {                                                                   \
    if (!ptx::mbar_wait_relaxed((bar), (parity), &ctl->abort_flag, p.wait_polls)) {    \
      ctl->abort_flag = 1;                                               \
      report_error(p.status, LOSA_ERR_TIMEOUT);                          \
      goto teardown;                                                     \
    }                                                                    \
  } while (0)

#define LOSA_WAIT(bar, parity)                                   \
  do {                                                           \
    if (!ptx::mbar_wait((bar), (parity), &ctl->abort_flag, p.wait_polls)) {    \
      ctl->abort_flag = 1;                                       \
      report_error(p.status, LOSA_ERR_TIMEOUT);                  \
      goto teardown;                                             \
    }                                                            \
  } while (0)

// Next entry of the tile list (whole warp): waits for the chunk when entering it and hands it
// back to the scheduler after its last entry.  `te` is the warp's running entry counter.
#define LOSA_TL_NEXT(ent)                                                            \
  do {                                                                               \
    const uint32_t c_ = (te >> 5) & (kTlChunks - 1);                                 \
    if ((te & 31) == 0) LOSA_WAIT(&ctl->tl_full[c_], (te / (kTlChunks * 32)) & 1);   \
    (ent) = *reinterpret_cast<volatile uint32_t*>(&ctl->tl[te & (kTlChunks * 32 - 1)]); \
    if ((te & 31) == 31) {                                                           \
      __syncwarp();                                                                  \
      if (lane == 0) ptx::mbar_arrive(&ctl->tl_empty[c_]);                           \
    }                                                                                \
    ++te;                                                                            \
  } while (0)

// Next K/V tile of the tile list: its kG entries into grp[]; `more` is false (and grp[0] holds the
// entry) when the item ends instead.
#define LOSA_TL_NEXT_TILE(grp, more)                            \
  do {                                                          \
    LOSA_TL_NEXT((grp)[0]);                                     \
    (more) = ((grp)[0] >> 28) == 0;                             \
    if (more) {                                                 \
      _Pragma("unroll") for (int g_ = 1; g_ < kG; ++g_) LOSA_TL_NEXT((grp)[g_]); \
    }                                                           \
  } while (0)

// Scheduler side: append n <= 32 entries at once, lane i holding entry i (whole warp).
#define LOSA_TL_PUT_BULK(ent, n)                                                      \
  do {                                                                                \
    const uint32_t first_ = te, last_ = te + (uint32_t)(n) - 1;                       \
    if ((first_ & 31) == 0)                                                           \
      LOSA_WAIT_RELAXED(&ctl->tl_empty[(first_ >> 5) & (kTlChunks - 1)],              \
                        ((first_ / (kTlChunks * 32)) & 1) ^ 1);                       \
    if ((last_ >> 5) != (first_ >> 5))                                                \
      LOSA_WAIT_RELAXED(&ctl->tl_empty[(last_ >> 5) & (kTlChunks - 1)],               \
                        ((last_ / (kTlChunks * 32)) & 1) ^ 1);                        \
    if (lane < (n)) ctl->tl[(first_ + lane) & (kTlChunks * 32 - 1)] = (ent);          \
    __syncwarp();                                                                     \
    if (lane == 0) {                                                                  \
      if ((last_ >> 5) != (first_ >> 5))                                              \
        ptx::mbar_arrive(&ctl->tl_full[(first_ >> 5) & (kTlChunks - 1)]);             \
      if ((last_ & 31) == 31) ptx::mbar_arrive(&ctl->tl_full[(last_ >> 5) & (kTlChunks - 1)]); \
    }                                                                                 \
    te += (uint32_t)(n);                                                              \
  } while (0)

// Scheduler side: append one entry (whole warp; lane 0 writes).
#define LOSA_TL_PUT(ent)                                                             \
  do {                                                                               \
    const uint32_t c_ = (te >> 5) & (kTlChunks - 1);                                 \
    if ((te & 31) == 0)                                                              \
      LOSA_WAIT_RELAXED(&ctl->tl_empty[c_], ((te / (kTlChunks * 32)) & 1) ^ 1);      \
    if (lane == 0) ctl->tl[te & (kTlChunks * 32 - 1)] = (ent);                       \
    if ((te & 31) == 31) {                                                           \
      __syncwarp();                                                                  \
      if (lane == 0) ptx::mbar_arrive(&ctl->tl_full[c_]);                            \
    }                                                                                \
    ++te;                                                                            \
  } while (0)

template <int D, int R, int C_, int MODE, int KT, bool SPLIT>
__global__ void __launch_bounds__(Lay<SPLIT>::kThreads, 1)
losa_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_kw,
                 const __grid_constant__ CUtensorMap map_vw, const Params p) {
  using C = Cfg<D, R, C_, MODE, KT, SPLIT && D == 64 && MODE != kMass>;
  using L = Lay<SPLIT>;
  using Ctl = Control<C::kNK, C::kNV, SPLIT, SPLIT && D == 64 && MODE != kMass>;
  // Head dimension 64 leaves 128 tensor-memory columns unused (O takes 64 per query tile), enough
  // for a third score buffer.  The two query tiles then take the three buffers in turn, in the
  // order in which their S = Q K^T are issued, so that the S of a query tile's next key tile is
  // computed while its current one is still being exponentiated: the softmax warps never wait for
  // the tensor core.  One issuer warp issues every S = Q K^T of the CTA in that fixed order, the
  // other every O += P V; a buffer is written again only after the product that read its P has
  // completed (a barrier between the two issuers).
  constexpr bool kRot = SPLIT && D == 64 && C::kHasV;
  constexpr int kC = C::kC, kG = C::kG, kQBT = C::kQBT, kNB = C::kNB, kW = C::kW, kNS = C::kNS;
  constexpr uint32_t kSStride = C::kSStride, kNVs = C::kNV > 0 ? C::kNV : 1;
  constexpr uint32_t kQMask = (1u << kQBT) - 1u;
  // The mass pass is bound by the special-function unit (16 exponentials per clock and SM): every
  // fourth group of four exponentials computes two of them with a polynomial on the FMA pipe
  // instead (12.5 % of all; measured 4.92 -> 4.63 ms at the Wan shape; a quarter or half of them
  // is slower, 5.6 and 5.8 ms: the loop turns issue-bound).  Not in the attention modes, which
  // wait on the chain of their steps, not on that unit (tried twice, slower each time).
  constexpr int kPolyEvery = (MODE == kMass) ? 4 : 0;
#ifndef LOSA_SPLIT_POLY
#define LOSA_SPLIT_POLY 1
#endif
#ifndef LOSA_SPLIT_POLY_OF
#define LOSA_SPLIT_POLY_OF 8
#endif
  // Two threads per row, head dimension 64, modes with an attention output: one group of four
  // scores in every eight (12.5 %) takes its exponentials from a polynomial on the FMA pipe.
  // Measured at the CogVideoX shape: dense 5.57 -> 4.95 ms, sparse 4.96 -> 4.54 ms (6.25 % gives
  // 5.02 / 4.58, 18.75 % 5.13 / 4.62, 25 % 5.35 / 4.81, 50 % 6.26 / 5.55), fused step 6.52 -> 6.38.
  // At head dimension 128 the fused step gets 3 % slower with it, and has none.
  constexpr int kSplitPoly = (SPLIT && C::kHasV && D == 64) ? LOSA_SPLIT_POLY : 0;
  constexpr int kSplitPolyOf = LOSA_SPLIT_POLY_OF;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // (the swizzled tiles need 1024-byte alignment; the one-thread-per-row layout has room for the
  // slack, the other relies on the declared alignment and checks it)
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  if (SPLIT && smem != smem_raw) {
    if (threadIdx.x == 0) report_error(p.status, LOSA_ERR_CUDA);
    return;
  }
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + 2 * C::kQBytes;
  uint8_t* sV = sK + C::kNK * C::kKVBytes;
  Ctl* ctl = reinterpret_cast<Ctl*>(sV + C::kNV * C::kKVBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ctl->q_full[i], 1);
      ptx::mbar_init(&ctl->q_empty[i], 1);
      for (int u = 0; u < 2; ++u) {
        ptx::mbar_init(&ctl->s_full[i][u], 1);
        ptx::mbar_init(&ctl->s_free[i][u], L::kSoftmaxWarps / 2);  // one elected arrival per softmax warp
      }
      ptx::mbar_init(&ctl->p_ready[i], L::kSoftmaxWarps / 2);  // one elected arrival per softmax warp
      ptx::mbar_init(&ctl->o_done[i], 1);
      ptx::mbar_init(&ctl->o_free[i], 128);  // the threads that read O out
      ptx::mbar_init(&ctl->wg_bar[i], 16 * L::kSoftmaxWarps);  // all softmax threads of a query tile
    }
    for (int i = 0; i < C::kNK; ++i) {
      ptx::mbar_init(&ctl->k_full[i], 1);
      ptx::mbar_init(&ctl->k_empty[i], 2);  // one arrival per query tile
    }
    for (int i = 0; i < C::kNV; ++i) {
      ptx::mbar_init(&ctl->v_full[i], 1);
      ptx::mbar_init(&ctl->v_empty[i], 2);
    }
    for (int i = 0; i < kTlChunks; ++i) {
      ptx::mbar_init(&ctl->tl_full[i], 1);
      // readers of the tile list: producer, 2 MMA issuers, the softmax warps
      ptx::mbar_init(&ctl->tl_empty[i], 3 + L::kSoftmaxWarps);
    }
    if (SPLIT) {
      for (int i = 0; i < 8; ++i) ptx::mbar_init(&ctl->pair_bar[i], 2);
      ctl->ovf_unit = -1;
    }
    if (kRot) {
      for (int i = 0; i < 3; ++i) ptx::mbar_init(&ctl->pv_done[i], 1);
      for (int i = 0; i < 6; ++i) {
        ptx::mbar_init(&ctl->rot_s_full[i], 1);
        ptx::mbar_init(&ctl->rot_p_ready[i], L::kSoftmaxWarps / 2);
      }
    }
    ptx::mbar_init(&ctl->drain, 2);  // the MMA issuers arrive on the abort path
    ctl->mma_lock = 0;
    ctl->abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == kIssuerWarp) {
    ptx::tmem_alloc(&ctl->tmem_base, kTmemCols);
    ptx::tmem_relinquish_alloc_permit();
  }
  if (warp == kProducerWarp && lane == 0) {
    ptx::prefetch_tensormap(&map_q);
    ptx::prefetch_tensormap(&map_k);
    if (C::kHasV) ptx::prefetch_tensormap(&map_v);
    if (kG > 2) {
      ptx::prefetch_tensormap(&map_kw);
      if (C::kHasV) ptx::prefetch_tensormap(&map_vw);
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  // The softmax warpgroups hold a whole S row per thread: the utility warpgroup gives registers
  // up and the softmax warpgroups take them.
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(L::kRegsUtility));
  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ TMA producer
    // (the whole warp walks the tile list; lane 0 alone issues the copies)
    {
      uint32_t nq[2] = {0, 0}, nk = 0, nv = 0, te = 0, ent;
      LOSA_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        const int w = (int)(ent & kTlItemMask);
        const int pbh = w / p.nPairs, pr = w % p.nPairs;
        const int bh = pbh % (p.B * p.H);
        const int b = bh / p.H, h = bh % p.H;
        const CUtensorMap *mq = &map_q, *mk = &map_k, *mv = &map_v, *mkw = &map_kw, *mvw = &map_vw;
        if (p.problems != nullptr) {
          const ProblemEntry* pe = p.problems + pbh / (p.B * p.H);
          mq = &pe->map_q;
          mk = &pe->map_k;
          mv = &pe->map_v;
          mkw = &pe->map_k128;
          mvw = &pe->map_v128;
        }
#pragma unroll
        for (int qt = 0; qt < 2; ++qt) {
          const int T = 2 * pr + qt;
          if (T < p.nQt) {
            LOSA_WAIT_RELAXED(&ctl->q_empty[qt], (nq[qt] & 1) ^ 1);
            if (lane == 0) {
              ptx::mbar_arrive_expect_tx(&ctl->q_full[qt], C::kQBytes);
#pragma unroll
              for (int s = 0; s < C::kDH; ++s)
                ptx::tma_load_4d(sQ + qt * C::kQBytes + s * C::kQSlab, mq, &ctl->q_full[qt],
                                 s * 64, T * 128, h, b);
            }
            ++nq[qt];
          }
        }
        for (;;) {
          uint32_t grp[kG];
          bool more;
          LOSA_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          // a tile gathers kG key blocks: block g of the group goes to rows g * C ... of the stage
          // (a padding entry names rows past the end of the tensor, which are filled with zeros)
          const uint32_t ks = nk % C::kNK;
          LOSA_WAIT_RELAXED(&ctl->k_empty[ks], ((nk / C::kNK) & 1) ^ 1);
          // one copy per (key block, slab), issued by as many lanes at once: a single thread
          // issuing 8 or 16 small copies per tile cannot keep up with the tile rate
          if (lane == 0) ptx::mbar_arrive_expect_tx(&ctl->k_full[ks], C::kKVBytes);
          __syncwarp();
          // (32-key blocks: a tile whose four key blocks are consecutive is one copy per slab - two
          // thirds of the sparse tiles on the workload's pattern, all of them in the dense modes;
          // dense forward 5.70 -> 5.51 ms, fused step 8.38 -> 8.01 ms.  With 64-key blocks one 16 KB
          // copy instead of two of 8 KB measured 5 % SLOWER in the dense forward, so they stay apart.)
          bool wide = kG > 2;
#pragma unroll
          for (int gg = 1; gg < kG; ++gg) wide = wide && (grp[gg] & 0xffffu) == (grp[0] & 0xffffu) + gg;
          if (wide) {
            if (lane < C::kDH)
              ptx::tma_load_4d(sK + ks * C::kKVBytes + lane * C::kKVSlab, mkw, &ctl->k_full[ks], lane * 64,
                               (int)(grp[0] & 0xffffu) * kC, h, b);
          } else if (lane < kG * C::kDH) {
            const int g = lane / C::kDH, s = lane % C::kDH;
            uint32_t eg = grp[0];
#pragma unroll
            for (int gg = 1; gg < kG; ++gg)
              if (g == gg) eg = grp[gg];
            const int jg = (int)(eg & 0xffffu);
            const int r0 = (jg == (int)kTlPad) ? p.nKb * kC : jg * kC;
            ptx::tma_load_4d(sK + ks * C::kKVBytes + s * C::kKVSlab + g * C::kBoxBytes, mk,
                             &ctl->k_full[ks], s * 64, r0, h, b);
          }
          ++nk;
          if (C::kHasV) {
            const uint32_t vs = nv % kNVs;
            LOSA_WAIT_RELAXED(&ctl->v_empty[vs], ((nv / kNVs) & 1) ^ 1);
            if (lane == 0) ptx::mbar_arrive_expect_tx(&ctl->v_full[vs], C::kKVBytes);
            __syncwarp();
            if (wide) {
              if (lane < C::kDH)
                ptx::tma_load_4d(sV + vs * C::kKVBytes + lane * C::kKVSlab, mvw, &ctl->v_full[vs], lane * 64,
                                 (int)(grp[0] & 0xffffu) * kC, h, b);
            } else if (lane < kG * C::kDH) {
              const int g = lane / C::kDH, s = lane % C::kDH;
              uint32_t eg = grp[0];
#pragma unroll
              for (int gg = 1; gg < kG; ++gg)
                if (g == gg) eg = grp[gg];
              const int jg = (int)(eg & 0xffffu);
              const int r0 = (jg == (int)kTlPad) ? p.nKb * kC : jg * kC;
              ptx::tma_load_4d(sV + vs * C::kKVBytes + s * C::kKVSlab + g * C::kBoxBytes, mv,
                               &ctl->v_full[vs], s * 64, r0, h, b);
            }
            ++nv;
          }
        }
      }
    }
  } else if (kRot && warp == kIssuerWarp) {
    // ------------------------------------------------------------------ rotating score buffers: the S = Q K^T issuer
    // For every K/V tile of the list, for each query tile that lists it (query tile 0 first): the
    // next score, number k, goes into buffer k % 3.  That buffer still holds the P of score
    // k - 3 until its O += P V has run, which the other issuer warp signals (pv_done).
    {
      const bool leader = ptx::elect_one();
      constexpr uint32_t kDescHi = ptx::smem_desc_hi_sw128(1024);
      const uint32_t k_lo = ptx::smem_desc_lo(ptx::smem_u32(sK), 16);
      const uint32_t q_lo = ptx::smem_desc_lo(ptx::smem_u32(sQ), 16);
      uint32_t nq[2] = {0, 0}, nt = 0, te = 0, ent, kq = 0;
      LOSA_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        bool q_ready[2] = {false, false};
        const int pr_ = (int)(ent & kTlItemMask) % p.nPairs;
        for (;;) {
          uint32_t grp[kG];
          bool more;
          LOSA_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          uint32_t memb = 0;
#pragma unroll
          for (int g = 0; g < kG; ++g) memb |= (grp[g] >> 16) & 0xfu;
          const uint32_t ks = nt % C::kNK, kph = (nt / C::kNK) & 1;
          LOSA_WAIT(&ctl->k_full[ks], kph);
#pragma unroll
          for (int qt = 0; qt < 2; ++qt) {
            if (((memb >> (qt * kQBT)) & kQMask) != 0) {
              if (!q_ready[qt]) {
                LOSA_WAIT(&ctl->q_full[qt], nq[qt] & 1);
                ++nq[qt];
                q_ready[qt] = true;
              }
              const uint32_t b = kq % 3u;
              if (kq >= 3u) LOSA_WAIT(&ctl->pv_done[b], (kq / 3u - 1u) & 1);
              ptx::tc_fence_after_sync();
              if (leader) {
                const uint32_t qd0 = q_lo + qt * (C::kQBytes >> 4), kd0 = k_lo + ks * (C::kKVBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                  ptx::mma_ss_lo(tmem_base + b * 128, qd0 + (((kk >> 2) * C::kQSlab + (kk & 3) * 32) >> 4),
                                 kd0 + (((kk >> 2) * C::kKVSlab + (kk & 3) * 32) >> 4), kDescHi,
                                 C::kIdescQK, kk > 0 ? 1u : 0u);
                ptx::mma_commit(&ctl->rot_s_full[qt * 3 + b]);
                ptx::mma_commit(&ctl->k_empty[ks]);
              }
              ++kq;
            } else {
              if (leader) ptx::mbar_arrive(&ctl->k_empty[ks]);
            }
          }
          ++nt;
        }
#pragma unroll
        for (int qt = 0; qt < 2; ++qt) {
          if (q_ready[qt]) {
            if (leader) ptx::mma_commit(&ctl->q_empty[qt]);
          } else if (2 * pr_ + qt < p.nQt) {
            // no key tile of this unit was listed by the query tile: its buffer goes back unused
            LOSA_WAIT(&ctl->q_full[qt], nq[qt] & 1);
            ++nq[qt];
            if (leader) ptx::mbar_arrive(&ctl->q_empty[qt]);
          }
        }
      }
    }
  } else if (kRot && warp == kIssuerWarp + 1) {
    // ------------------------------------------------------------------ rotating score buffers: the O += P V issuer
    // Walks the same list in the same order; product k reads P from buffer k % 3 once the softmax
    // warps of its query tile have packed it.
    {
      const bool leader = ptx::elect_one();
      constexpr uint32_t kDescHi = ptx::smem_desc_hi_sw128(1024);
      const uint32_t v_lo = ptx::smem_desc_lo(ptx::smem_u32(sV), C::kKVSlab);
      uint32_t nof[2] = {0, 0}, uses[6] = {0, 0, 0, 0, 0, 0}, nt = 0, te = 0, ent, kp = 0;
      LOSA_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        uint32_t pv_item[2] = {0, 0};
        for (;;) {
          uint32_t grp[kG];
          bool more;
          LOSA_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          uint32_t memb = 0;
#pragma unroll
          for (int g = 0; g < kG; ++g) memb |= (grp[g] >> 16) & 0xfu;
          const uint32_t vs = nt % kNVs, vph = (nt / kNVs) & 1;
          LOSA_WAIT(&ctl->v_full[vs], vph);
#pragma unroll
          for (int qt = 0; qt < 2; ++qt) {
            if (((memb >> (qt * kQBT)) & kQMask) != 0) {
              const uint32_t b = kp % 3u;
              if (pv_item[qt] == 0 && nof[qt] > 0) LOSA_WAIT(&ctl->o_free[qt], (nof[qt] - 1) & 1);
              LOSA_WAIT(&ctl->rot_p_ready[qt * 3 + b], uses[qt * 3 + b] & 1);
              ++uses[qt * 3 + b];
              ptx::tc_fence_after_sync();
              if (leader) {
                const uint32_t tP = tmem_base + b * 128, tO = tmem_base + 384 + qt * 64;
                const uint32_t vd0 = v_lo + vs * (C::kKVBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < kW / 16; ++kk)
                  ptx::mma_ts_lo(tO, tP + (kk & 3) * 8 + (kk >> 2) * 64, vd0 + kk * (2048 >> 4), kDescHi,
                                 C::kIdescPV, (kk > 0 || pv_item[qt] > 0) ? 1u : 0u);
                ptx::mma_commit(&ctl->pv_done[b]);
                ptx::mma_commit(&ctl->v_empty[vs]);
              }
              ++pv_item[qt];
              ++kp;
            } else {
              if (leader) ptx::mbar_arrive(&ctl->v_empty[vs]);
            }
          }
          ++nt;
        }
#pragma unroll
        for (int qt = 0; qt < 2; ++qt) {
          if (pv_item[qt] > 0) {
            if (leader) ptx::mma_commit(&ctl->o_done[qt]);  // every product of the item is done
            ++nof[qt];
          }
        }
      }
    }
  } else if (warp == kIssuerWarp || warp == kIssuerWarp + 1) {
    // ------------------------------------------------------------------ MMA issuers
    // One warp per query tile (lane 0 issues).  Per key tile that the query tile lists it runs
    //   S = Q K^T  ->  (softmax warps turn S into P, in place)  ->  O += P V
    // and only then S of the next key tile, because P lives in the columns of S.  That chain is
    // serial per query tile; the two query tiles run it half a period apart, so that one tile's
    // MMAs execute while the other tile's softmax runs and the two warpgroups do not compete
    // for the exponential unit.  The half-period offset is kept by a lock: a burst (O += P V
    // of one key tile, then S of the next) is issued whole, never interleaved with the other
    // tile's burst - interleaved bursts finish together and lock the tiles in step.
    // The mass pass has no P and no O: there S is double-buffered and handed back by the
    // softmax warps as soon as it is read.
    {
      const int qt = warp - kIssuerWarp;
      // The leader comes from elect.sync rather than from a lane test: the compiler then knows that
      // a single thread runs the issue code and keeps the MMA operands in uniform registers, which
      // halves the cost of issuing an MMA (measured: 27 instead of 55-65 cycles per instruction).
      const bool leader = ptx::elect_one();
      uint32_t nq = 0, nt = 0, nsub = 0, nof = 0, te = 0, ent;
      constexpr uint32_t kDescHi = ptx::smem_desc_hi_sw128(1024);
      const uint32_t k_lo = ptx::smem_desc_lo(ptx::smem_u32(sK), 16);
      const uint32_t v_lo = ptx::smem_desc_lo(ptx::smem_u32(sV), C::kKVSlab);
      const uint32_t tS = tmem_base + qt * kSStride;
      const uint32_t tO = tmem_base + 256 + qt * 128;
      // Every descriptor is built before the waits, so that the MMAs issue back to back.  The
      // dense and sparse forward keep only the low words in registers (the high word is the same
      // constant for every operand): 24 whole descriptors do not fit this warp's 72 registers
      // and spilled, which cost 4 % of the forward.  The mass pass has half as many operands,
      // and it and the fused mode were measured 3 % faster with whole descriptors.
      constexpr bool kLoDesc = (C::kHasV && !C::kWantMass) || SPLIT;
      uint32_t qd[D / 16];
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk)
        qd[kk] = ptx::smem_desc_lo(ptx::smem_u32(sQ), 16) + qt * (C::kQBytes >> 4) +
                 (((kk >> 2) * C::kQSlab + (kk & 3) * 32) >> 4);
      uint64_t qd64[D / 16];
      if (!kLoDesc) {
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) qd64[kk] = ptx::desc64(qd[kk], kDescHi);
      }

      LOSA_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        bool q_ready = false, pend = false;
        uint32_t pend_vs = 0, pend_vph = 0, pv_item = 0;
        // the producer loads this query tile for every item in which the tile exists
        const bool q_loaded = 2 * ((int)(ent & kTlItemMask) % p.nPairs) + qt < p.nQt;
        for (;;) {
          uint32_t grp[kG];
          bool more;
          LOSA_TL_NEXT_TILE(grp, more);
          if (!more) ent = grp[0];
          // the query tile takes part in a K/V tile if any of its query blocks lists any of the
          // tile's key blocks
          uint32_t memb = 0;
          if (more) {
#pragma unroll
            for (int g = 0; g < kG; ++g) memb |= (grp[g] >> 16) & 0xfu;
          }
          const uint32_t ks = nt % C::kNK, kph = (nt / C::kNK) & 1;
          const uint32_t vs = nt % kNVs, vph = (nt / kNVs) & 1;
          const bool member = more && ((memb >> (qt * kQBT)) & kQMask) != 0;
          const uint32_t buf = nsub % kNS;
          uint32_t kd[D / 16], vd[kW / 16];
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            kd[kk] = k_lo + ks * (C::kKVBytes >> 4) + (((kk >> 2) * C::kKVSlab + (kk & 3) * 32) >> 4);
#pragma unroll
          for (int kk = 0; kk < kW / 16; ++kk)
            vd[kk] = v_lo + pend_vs * (C::kKVBytes >> 4) + kk * (2048 >> 4);
          uint64_t kd64[D / 16], vd64[kW / 16];
          if (!kLoDesc) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) kd64[kk] = ptx::desc64(kd[kk], kDescHi);
            if (C::kHasV) {
#pragma unroll
              for (int kk = 0; kk < kW / 16; ++kk) vd64[kk] = ptx::desc64(vd[kk], kDescHi);
            }
          }
          // operands first, the softmax hand-over last: it is the wait that ends latest
          if (more) LOSA_WAIT(&ctl->k_full[ks], kph);
          if (member) {
            if (!q_ready) {
              LOSA_WAIT(&ctl->q_full[qt], nq & 1);
              ++nq;
              q_ready = true;
            }
            // mass pass: the S buffer is free once the softmax warps have read its last content
            if (!C::kHasV && nsub >= (uint32_t)kNS)
              LOSA_WAIT(&ctl->s_free[qt][buf], ((nsub / kNS) - 1) & 1);
          }
          if (C::kHasV && pend) {
            LOSA_WAIT(&ctl->v_full[pend_vs], pend_vph);
            if (pv_item == 0 && nof > 0) LOSA_WAIT(&ctl->o_free[qt], (nof - 1) & 1);
            LOSA_WAIT(&ctl->p_ready[qt], (nsub - 1) & 1);
          }
          if ((C::kHasV && pend) || member) {
            // ---- one burst, under the lock
            if (leader) {
              uint32_t it = 0;
              while (atomicCAS(&ctl->mma_lock, 0u, 1u) != 0u) {
                if (++it > (1u << 22) || ctl->abort_flag) break;  // bounded; a later wait reports it
                __nanosleep(32);
              }
            }
            __syncwarp();
            ptx::tc_fence_after_sync();
            if (leader) {
              if (C::kHasV && pend) {
                // O += P V for the previous key tile of this query tile
                if (kLoDesc) {
                  // (two threads per row: each half packs its P over the head of its own 64 score
                  // columns, so the second half of the keys reads its operand from column 64 on)
                  ptx::mma_ts_lo(tO, tS, vd[0], kDescHi, C::kIdescPV, pv_item > 0 ? 1u : 0u);
#pragma unroll
                  for (int kk = 1; kk < kW / 16; ++kk)
                    ptx::mma_ts_lo(tO, tS + (SPLIT ? (kk & 3) * 8 + (kk >> 2) * 64 : kk * 8), vd[kk],
                                   kDescHi, C::kIdescPV, 1u);
                } else {
                  ptx::mma_ts_d(tO, tS, vd64[0], C::kIdescPV, pv_item > 0 ? 1u : 0u);
#pragma unroll
                  for (int kk = 1; kk < kW / 16; ++kk)
                    ptx::mma_ts_d(tO, tS + kk * 8, vd64[kk], C::kIdescPV, 1u);
                }
              }
              if (member) {
                if (kLoDesc) {
                  ptx::mma_ss_lo(tS + buf * 128, qd[0], kd[0], kDescHi, C::kIdescQK, 0u);
#pragma unroll
                  for (int kk = 1; kk < D / 16; ++kk)
                    ptx::mma_ss_lo(tS + buf * 128, qd[kk], kd[kk], kDescHi, C::kIdescQK, 1u);
                } else {
                  ptx::mma_ss_d(tS + buf * 128, qd64[0], kd64[0], C::kIdescQK, 0u);
#pragma unroll
                  for (int kk = 1; kk < D / 16; ++kk)
                    ptx::mma_ss_d(tS + buf * 128, qd64[kk], kd64[kk], C::kIdescQK, 1u);
                }
                // completes after every MMA issued so far, the tile's last O += P V included
                ptx::mma_commit(&ctl->s_full[qt][buf]);
              }
              // the lock orders the issue of bursts, not data: a plain store releases it
              *reinterpret_cast<volatile uint32_t*>(&ctl->mma_lock) = 0u;
              // stages go back when the MMAs that read them have completed
              if (C::kHasV && pend) ptx::mma_commit(&ctl->v_empty[pend_vs]);
              if (member) ptx::mma_commit(&ctl->k_empty[ks]);
            }
          }
          if (C::kHasV && pend) {
            ++pv_item;
            pend = false;
          }
          if (!more) break;
          if (member) {
            ++nsub;
            pend = C::kHasV;
            pend_vs = vs;
            pend_vph = vph;
          } else {
            // the copies must have landed before a stage is handed back
            if (leader) ptx::mbar_arrive(&ctl->k_empty[ks]);
            if (C::kHasV) {
              LOSA_WAIT(&ctl->v_full[vs], vph);
              if (leader) ptx::mbar_arrive(&ctl->v_empty[vs]);
            }
          }
          ++nt;
        }
        if (C::kHasV && pv_item > 0) {
          if (leader) ptx::mma_commit(&ctl->o_done[qt]);  // every product of the item is done
          ++nof;
        }
        if (q_ready) {
          if (leader) ptx::mma_commit(&ctl->q_empty[qt]);
        } else if (q_loaded) {
          // no key tile of this unit was listed by the query tile (a part of a short list can be
          // empty): the query tile was loaded all the same and its buffer has to be handed back
          LOSA_WAIT(&ctl->q_full[qt], nq & 1);
          ++nq;
          if (leader) ptx::mbar_arrive(&ctl->q_empty[qt]);
        }
      }
    }
  } else if (warp == kSchedulerWarp) {
    // ------------------------------------------------------------------ scheduler
    // Walks the block-index lists of this CTA's work items and publishes, per item, a header
    // and the ascending merge of its tiles; nobody else touches the CSR.
    uint32_t te = 0;
    for (;;) {
      // (diagnostic launch, see losa_debug_stall_next_launch: no tile list is ever published, no
      // copy and no MMA is issued, and every other role's first wait runs out)
      if (p.stall) break;
      // work items are drawn from a global counter, in head-major order, so that a CTA that
      // finishes early takes the next item instead of idling at the end of the launch
      int w = 0;
      if (lane == 0) {
        w = atomicAdd(p.work_counter, 1);
        // fallback launch: the units the two-threads-per-row kernel could not finish
        if (p.redo) w = (w < *p.redo_count) ? p.redo_list[w] : p.nUnits;
      }
      w = __shfl_sync(0xffffffffu, w, 0);
      if (w >= p.nUnits) break;
      // units past split_first are parts of the key range of the last items
      int part = 0, parts = 1;
      uint32_t flags = 0;
      if (w >= p.split_first) {
        const int r = w - p.split_first;
        parts = p.split_parts;
        part = r % parts;
        w = p.split_first + r / parts;
        flags = kTlPartial | ((uint32_t)part << 24);
      }
      const int unit = (flags != 0) ? p.split_first + (w - p.split_first) * parts + part : w;
      const int pr = w % p.nPairs;
      LOSA_TL_PUT(kTlItem | flags | (uint32_t)w);
      if (MODE == kSparse) {
        // the unit's merged tile list was built before the launch: stream it into the ring,
        // 32 entries per step, so that this warp takes next to no issue slots from the softmax
        // warps of its scheduler partition
        const int cnt = LOSA_IN_RANGE(unit, p.cap_units) ? min(__ldg(p.tl_count + unit), p.tl_cap) : 0;
        const uint32_t* src = p.tl_entries + (int64_t)unit * p.tl_cap;
        for (int base = 0; base < cnt; base += 32) {
          const int n = min(32, cnt - base);
          const uint32_t e = (lane < n) ? __ldg(src + base + lane) : 0u;
          LOSA_TL_PUT_BULK(e, n);
        }
        continue;
      }
      // dense modes: every key block of the unit's share of the key range, listed by every query
      // block of the item that exists; K/V tiles are groups of kG entries, the last group is padded
      uint32_t memb = 0;
#pragma unroll
      for (int n = 0; n < kNB; ++n)
        if (2 * pr * kQBT + n < p.nQb) memb |= 1u << n;
      const int jlo = (int)(((int64_t)p.nKb * part) / parts);
      const int jhi = (int)(((int64_t)p.nKb * (part + 1)) / parts);
      const int cnt = (jhi - jlo + kG - 1) / kG * kG;
      for (int base = 0; base < cnt; base += 32) {
        const int n = min(32, cnt - base);
        const int j = jlo + base + lane;
        const uint32_t e = (j < jhi) ? ((uint32_t)j | (memb << 16)) : kTlPad;
        LOSA_TL_PUT_BULK(e, n);
      }
    }
    if (!p.stall) {
      LOSA_TL_PUT(kTlEnd);
      if ((te & 31) != 0) {  // publish the last, partly filled chunk
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl->tl_full[((te - 1) >> 5) & (kTlChunks - 1)]);
      }
    }
  }
  } else if constexpr (!SPLIT) {
    // ------------------------------------------------------------------ softmax warpgroups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(L::kRegsSoftmax));
    const int qt = (warp >> 2) - 1, wl = warp & 3;  // TMEM lanes 32 * (warp % 4) .. + 31
    const int row = wl * 32 + lane;
    const uint32_t lane_base = (uint32_t)(wl * 32) << 16;
    const uint32_t tS = tmem_base + lane_base + qt * kSStride;  // P overwrites its first kW/2 columns
    const uint32_t tO = tmem_base + lane_base + 256 + qt * 128;
    const int sub = (R == 64) ? (wl >> 1) : 0;
    const int my_bit = qt * kQBT + sub;
    uint32_t nsub = 0, nwg = 0, nod = 0;      // nsub: key tiles of this query tile so far
    uint32_t te = 0, ent;

    LOSA_TL_NEXT(ent);
    while ((ent >> 28) == 1) {
      const int w = (int)(ent & kTlItemMask);
      const bool partial = (ent & kTlPartial) != 0;
      const int part = (int)((ent >> 24) & 7u);
      const int pbh = w / p.nPairs, pr = w % p.nPairs;
      const int bh = pbh % (p.B * p.H);
      const int b = bh / p.H, h = bh % p.H;
      void* const o_base = (p.problems != nullptr) ? p.problems[pbh / (p.B * p.H)].o : p.o;
      const int T = 2 * pr + qt;
      const int grow = T * 128 + row;
      // l: row sum of the exponentials; in the attention-only modes of their bf16 roundings (what
      // the output is normalised by); the fused mode keeps both, the roundings' sum in lr
      float m_ref = -INFINITY, l = 0.f, lr = 0.f;
      bool have_ref = false;  // this warp's rows have a reference maximum (after their first tile)
      uint32_t pv_item = 0;
      float2* tab = nullptr;
      if (C::kWantMass)
        tab = p.table + ((int64_t)blockIdx.x * 2 + qt) * (int64_t)p.nKb * 128 + row;
      for (;;) {
        uint32_t grp[kG];
        bool more;
        LOSA_TL_NEXT_TILE(grp, more);
        if (!more) {
          ent = grp[0];
          break;
        }
        // vc[g]: how many keys of key block g of the tile this row attends to: all that exist, if
        // the row's query block lists the block, none otherwise (nor for a padding entry)
        uint32_t memb = 0;
        int vc[kG];
        bool mine = false, full = true, ragged = false;
#pragma unroll
        for (int g = 0; g < kG; ++g) {
          memb |= (grp[g] >> 16) & 0xfu;
          const int jg = (int)(grp[g] & 0xffffu);
          vc[g] = ((grp[g] >> (16 + my_bit)) & 1u) ? min(kC, p.N - jg * kC) : 0;
          mine = mine || vc[g] > 0;
          full = full && vc[g] == kC;
          ragged = ragged || (vc[g] > 0 && vc[g] < kC);  // the sequence's last, short key block
        }
        if (((memb >> (qt * kQBT)) & kQMask) == 0) continue;
        const uint32_t buf = nsub % kNS;
        const uint32_t tSb = tS + buf * 128;
        // S of this key tile is complete, and so is every earlier product into O
        LOSA_WAIT(&ctl->s_full[qt][buf], (nsub / kNS) & 1);
        ptx::tc_fence_after_sync();
        uint32_t sr[kW];
        // On the common path (a reference exists, no key of the tile is missing) only the first
        // 32 columns are waited for here; the rest arrive while those are exponentiated.
        const bool stream = C::kHasV && mine && have_ref && !ragged;
        if (mine) {
          ptx::tmem_ld32(tSb, &sr[0]);
          if (stream) ptx::tmem_wait_ld();
#pragma unroll
          for (int c0 = 32; c0 < kW; c0 += 32) ptx::tmem_ld32(tSb + c0, &sr[c0]);
          if (!stream) ptx::tmem_wait_ld();
        }
        if (!C::kHasV) {
          // mass pass: S is in registers (and stays there: no P is packed over it), hand the
          // buffer back
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl->s_free[qt][buf]);
        }
        if (mine) {
          // p = 2^(s * scale_log2 - m_ref) with a reference m_ref that is NOT the running maximum:
          // the result o = sum(p v) / sum(p) does not depend on it, it only has to keep p inside
          // the fp32 / bf16 range.  So the common path computes no row maximum at all: it
          // exponentiates against the reference it has and looks at the tile's row sums; only if a
          // sum left the safe range (> 2^40, inf or NaN; or there is no reference yet, in the
          // first tile of an item) does the warp compute the maximum, move the reference, rescale
          // O and the row sum, and exponentiate the tile again.  P is therefore stored only after
          // that test (S stays intact in TMEM for the second pass).
          float2 acc[kG][2];  // row sums per key block (the mass pass needs them apart), two chains each
          // The output is normalised by the sum of the weights the tensor core actually multiplies
          // with V - P as rounded to bf16 - not by the sum of the unrounded exponentials: then
          // o = sum(p~ v) / sum(p~) is a weighted mean of V whatever the rounding does, exact for a
          // row that one key dominates (with the unrounded sum such a row is off by up to 2^-8 |v|,
          // because the reference is not the row maximum and the dominant p is not a power of two).
          // The masses keep the unrounded sums.
          float2 racc[2];
          float gsum[kG], tsum = 0.f, rsum = 0.f;
          // (All rows of a warp belong to one query block and have seen the same tiles, so
          // whether a reference exists is known per warp without a vote.  In the mass pass the
          // scores stay in registers - no P is packed over them - so its second pass needs no
          // reload and the S buffer can be handed back right after the first read.  With several
          // key blocks per tile the mass pass keeps the running maximum: measured slower without
          // it, 6.1 against 5.6 ms at the CogVideoX shape, while 128-key blocks gain 3 %.)
          bool recentre = !have_ref || (!C::kHasV && kG > 1);
          have_ref = true;
#pragma unroll 1
          for (int pass = 0; pass < 2; ++pass) {
            // Key blocks the row's query block does not list must give p = 0: on the common path
            // that costs nothing, their columns simply get -inf instead of -m_ref as the addend
            // of the scaling FMA (straight-line code over all 128 columns; skipping blocks with
            // branches was measured 0.9 k cycles per tile slower at C = 32).  Scores are set to
            // -inf column by column only where single keys do not exist (>= N, in the sequence's
            // last key block) and on the re-centring pass, whose maximum must not see them.
            if (ragged || (recentre && !full)) {
#pragma unroll
              for (int c = 0; c < kW; ++c)
                if ((c % kC) >= vc[c / kC]) sr[c] = 0xff800000u;
            }
            if (recentre) {
              float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
              float mx2 = __uint_as_float(sr[2]), mx3 = __uint_as_float(sr[3]);
#pragma unroll
              for (int c = 4; c + 8 <= kW; c += 8) {
                mx0 = ptx::max3(mx0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
                mx1 = ptx::max3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
                mx2 = ptx::max3(mx2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
                mx3 = ptx::max3(mx3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
              }
              mx0 = ptx::max3(mx0, __uint_as_float(sr[kW - 4]), __uint_as_float(sr[kW - 3]));
              mx1 = ptx::max3(mx1, __uint_as_float(sr[kW - 2]), __uint_as_float(sr[kW - 1]));
              const float m_new =
                  fmaxf(m_ref, fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2);
              // rows whose reference is close enough keep it
              const bool need = m_new > m_ref + kRescaleThreshold;
              const float alpha = need ? ptx::ex2_approx(m_ref - m_new) : 1.f;
              if (need) m_ref = m_new;
              l *= alpha;
              lr *= alpha;
              if (C::kHasV && pv_item > 0) {
                // (every earlier product into O is complete: s_full covers them)
                const float2 a2 = make_float2(alpha, alpha);
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                  uint32_t r[32];
                  ptx::tmem_ld32(tO + c0, r);
                  ptx::tmem_wait_ld();
#pragma unroll
                  for (int c = 0; c < 32; c += 2) {
                    const float2 v = ptx::mul2(
                        make_float2(__uint_as_float(r[c]), __uint_as_float(r[c + 1])), a2);
                    r[c] = __float_as_uint(v.x);
                    r[c + 1] = __float_as_uint(v.y);
                  }
                  ptx::tmem_st32(tO + c0, r);
                }
              }
            }
            // two columns per instruction; the bf16 pairs overwrite the low half of the registers
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
            float2 nm2[kG];
#pragma unroll
            for (int g = 0; g < kG; ++g) {
              const float a = (vc[g] > 0) ? -m_ref : -INFINITY;
              nm2[g] = make_float2(a, a);
              acc[g][0] = acc[g][1] = make_float2(0.f, 0.f);
            }
            racc[0] = racc[1] = make_float2(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < kW; c += 4) {
              if (C::kHasV && c == 32) ptx::tmem_wait_ld();  // (nothing is in flight on a second pass)
              float2 x0 = ptx::fma2(
                  make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, nm2[c / kC]);
              float2 x1 = ptx::fma2(
                  make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sc2, nm2[c / kC]);
              x0.x = ptx::ex2_approx(x0.x);
              x0.y = ptx::ex2_approx(x0.y);
              if (kPolyEvery > 0 && ((c >> 2) % (kPolyEvery > 0 ? kPolyEvery : 1)) == 0) {
                x1 = ptx::ex2_poly2(x1);  // mass pass: a share of the exponentials on the FMA pipe
              } else {
                x1.x = ptx::ex2_approx(x1.x);
                x1.y = ptx::ex2_approx(x1.y);
              }
              if (C::kWantMass) {
                acc[c / kC][0] = ptx::add2(acc[c / kC][0], x0);
                acc[c / kC][1] = ptx::add2(acc[c / kC][1], x1);
              }
              if (C::kHasV) {
                const uint32_t u0 = ptx::pack_bf16x2(x0.x, x0.y), u1 = ptx::pack_bf16x2(x1.x, x1.y);
                sr[c >> 1] = u0;
                sr[(c >> 1) + 1] = u1;
                ptx::add_bf16x2(racc[0], u0);
                ptx::add_bf16x2(racc[1], u1);
              }
            }
            tsum = 0.f;
            if (C::kWantMass) {
#pragma unroll
              for (int g = 0; g < kG; ++g) {
                gsum[g] = (acc[g][0].x + acc[g][0].y) + (acc[g][1].x + acc[g][1].y);
                tsum += gsum[g];
              }
            }
            if (C::kHasV) {
              rsum = (racc[0].x + racc[0].y) + (racc[1].x + racc[1].y);
              if (!C::kWantMass) tsum = rsum;
            }
            // after a pass with a fresh maximum every p is at most 2^8
            if (recentre || !__any_sync(0xffffffffu, !(tsum <= kSafeRowSum))) break;
            recentre = true;
            if (C::kHasV) {  // the bf16 pairs of P overwrote the low half of the registers
#pragma unroll
              for (int c0 = 0; c0 < kW; c0 += 32) ptx::tmem_ld32(tSb + c0, &sr[c0]);
              ptx::tmem_wait_ld();
            }
          }
          l += tsum;
          if (C::kHasV && C::kWantMass) lr += rsum;
          if (C::kHasV) {
#pragma unroll
            for (int c0 = 0; c0 < kW / 2; c0 += 32) ptx::tmem_st32(tSb + c0, &sr[c0]);
          }
          if (C::kWantMass) {
            // one table entry per key block
#pragma unroll
            for (int g = 0; g < kG; ++g) {
              if (vc[g] > 0) {
                tab[(int64_t)(grp[g] & 0xffffu) * 128] = make_float2(gsum[g], m_ref);
              }
            }
          }
        } else if (C::kHasV) {
          // this part of the 128-row tile lists none of the tile's key blocks: P = 0
          uint32_t z[32];
#pragma unroll
          for (int c = 0; c < 32; ++c) z[c] = 0u;
#pragma unroll
          for (int c0 = 0; c0 < kW / 2; c0 += 32) ptx::tmem_st32(tSb + c0, z);
        }
        if (C::kHasV) {
          ptx::tmem_wait_st();
          ++pv_item;
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl->p_ready[qt]);
        }
        ++nsub;
      }

      if (C::kHasV) {
        // ---- epilogue: O / l -> global
        if (T < p.nQt) {
          const bool valid = grow < p.N;
          const float lo = C::kWantMass ? lr : l;
          const float inv = (lo > 0.f) ? 1.f / lo : 0.f;
          const int64_t off = (int64_t)b * p.sb + (int64_t)h * p.sh + (int64_t)grow * p.sn;
          const int64_t pslot =
              ((((int64_t)(w - p.split_first) * p.split_parts + part) * 2 + qt) * 128 + row);
          if (partial && LOSA_IN_RANGE(pslot, p.cap_part_rows)) p.part_ml[pslot] = make_float2(m_ref, l);
          if (pv_item > 0) {
            // o_done advances once per item, so its parity is unambiguous here (a product's own barrier may be
            // one, two or three phases from this warp's last look at it)
            LOSA_WAIT(&ctl->o_done[qt], nod & 1);
            ++nod;
            ptx::tc_fence_after_sync();
          }
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 32) {
            uint32_t r[32];
            if (pv_item > 0) {
              ptx::tmem_ld32(tO + c0, r);
              ptx::tmem_wait_ld();
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) r[c] = 0u;
            }
            if (partial) {
              // a part of the key range: unnormalised O, merged with the other parts afterwards
              float4* dst = reinterpret_cast<float4*>(p.part_o + (LOSA_IN_RANGE(pslot, p.cap_part_rows) ? pslot : 0) * D + c0);
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                dst[c >> 2] = make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                          __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
            } else if (valid) {
              if (p.o_f32) {
                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(o_base) + off + c0);
#pragma unroll
                for (int c = 0; c < 32; c += 4)
                  dst[c >> 2] = make_float4(__uint_as_float(r[c]) * inv, __uint_as_float(r[c + 1]) * inv,
                                            __uint_as_float(r[c + 2]) * inv,
                                            __uint_as_float(r[c + 3]) * inv);
              } else {
                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o_base) + off + c0);
#pragma unroll
                for (int c = 0; c < 32; c += 8) {
                  uint4 v;
                  v.x = ptx::pack_bf16x2(__uint_as_float(r[c]) * inv, __uint_as_float(r[c + 1]) * inv);
                  v.y = ptx::pack_bf16x2(__uint_as_float(r[c + 2]) * inv, __uint_as_float(r[c + 3]) * inv);
                  v.z = ptx::pack_bf16x2(__uint_as_float(r[c + 4]) * inv, __uint_as_float(r[c + 5]) * inv);
                  v.w = ptx::pack_bf16x2(__uint_as_float(r[c + 6]) * inv, __uint_as_float(r[c + 7]) * inv);
                  dst[c >> 3] = v;
                }
              }
            }
          }
          if (pv_item > 0) {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&ctl->o_free[qt]);
          }
        }
      }
      if (C::kWantMass) {
        // ---- epilogue of the mass pass: normalise the per-sub-tile sums by the final row
        // statistics and average them over the rows of each query block
        float2* rs = p.rowstat + ((int64_t)blockIdx.x * 2 + qt) * 128;
        if (T < p.nQt) {
          const bool valid = grow < p.N;
          rs[row] = make_float2(m_ref, (valid && l > 0.f) ? 1.f / l : 0.f);
          if (p.lse != nullptr && valid && LOSA_IN_RANGE((int64_t)bh * p.N + grow, p.cap_lse))
            p.lse[(int64_t)bh * p.N + grow] = (m_ref + log2f(l)) * kLn2;
        }
        ptx::mbar_arrive(&ctl->wg_bar[qt]);  // warpgroup sync with a bounded wait
        LOSA_WAIT(&ctl->wg_bar[qt], nwg & 1);
        ++nwg;
        if (T < p.nQt) {
          const float2* tb =
              p.table + ((int64_t)blockIdx.x * 2 + qt) * (int64_t)p.nKb * 128;
          float2 st[4];  // this lane's four rows
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) st[rr] = rs[rr * 32 + lane];
          for (int u = wl; u < p.nKb; u += 4) {
            float acc[kQBT];
#pragma unroll
            for (int q = 0; q < kQBT; ++q) acc[q] = 0.f;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
              const int r = rr * 32 + lane;
              const float2 tv = tb[(int64_t)u * 128 + r];
              const float wgt =
                  (st[rr].y > 0.f) ? tv.x * ptx::ex2_approx(tv.y - st[rr].x) * st[rr].y : 0.f;
              acc[(rr * 32) / R] += wgt;
            }
#pragma unroll
            for (int q = 0; q < kQBT; ++q) {
              float a = acc[q];
#pragma unroll
              for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
              const int g = T * kQBT + q;
              if (lane == 0 && g < p.nQb) {
                const int nvalid = min(R, p.N - g * R);
                {
                  const int64_t mi = ((int64_t)bh * p.nQb + g) * p.nKb + u;
                  if (LOSA_IN_RANGE(mi, p.cap_mass)) p.mass[mi] = a / (float)nvalid;
                }
              }
            }
          }
        }
        ptx::mbar_arrive(&ctl->wg_bar[qt]);
        LOSA_WAIT(&ctl->wg_bar[qt], nwg & 1);
        ++nwg;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps, two per row
    // Warps 4-11 serve query tile 0, warps 12-19 query tile 1; within a query tile the first
    // four warps (half 0) take key columns 0-63 of every S, the other four (half 1) columns
    // 64-127, each thread 64 columns of its row.  A pair of warps (same rows, the two halves)
    // shares a scheduler partition, so one warp's packing and summing fills the issue slots the
    // other's ex2 leaves empty.  On the common path the two never synchronise:
    //   * the reference the exponentials are taken against is the row maximum of the item's first
    //     tile, which each half computes for itself over all 128 columns, and it never moves;
    //   * each half packs its P over the head of its own score columns and keeps its own sum;
    //   * if a half's sum of a tile leaves the safe range (scores that rose 40 nats above the
    //     first tile), the whole work unit is handed to the fallback launch, whose one-thread-per-
    //     row kernel moves the reference; nothing here is rescaled.
    // At the end of an item half 1 hands its row sums to half 0, which normalises and writes O.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(L::kRegsSoftmax));
    const int sw = warp - 4;
    const int qt = sw >> 3, half = (sw >> 2) & 1, wl = sw & 3;  // TMEM lanes 32 * (warp % 4) .. + 31
    const int row = wl * 32 + lane;
    const uint32_t lane_base = (uint32_t)(wl * 32) << 16;
    // the row's 128 score columns, and this half's 64 of them (its P goes over their first 32);
    // with rotating buffers (head dimension 64) they change from tile to tile
    uint32_t tSrow = tmem_base + lane_base + qt * kSStride;
    uint32_t tS = tSrow + half * 64;
    const uint32_t tO = tmem_base + lane_base + (kRot ? 384 + qt * 64 : 256 + qt * 128);
    // fused construction step: this row's column of the CTA's table of per-block sums of the
    // unrounded exponentials, one float per row and 64-column half of a key tile when a key block
    // fills the tile (the halves' entries are added at the end), else one per row and key block
    float* const tabf = C::kWantMass ? reinterpret_cast<float*>(p.table) +
                                           ((int64_t)blockIdx.x * 2 + qt) * (int64_t)p.nKb * 256 + row
                                     : nullptr;
    uint32_t nwg = 0;
    uint32_t kq = 0;  // rotating buffers: scores issued so far, counted as the issuer counts them
    uint32_t uses[3] = {0, 0, 0};  // ... and how many of them, per buffer, were this query tile's
    const int sub = (R == 64) ? (wl >> 1) : 0;
    const int my_bit = qt * kQBT + sub;
    constexpr int kHB = (kG >= 2) ? kG / 2 : 1;   // key blocks of a half (a half block when C = 128)
    constexpr int kBW = 64 / kHB;                 // columns per such block
    uint64_t* const pair_bar = &ctl->pair_bar[qt * 4 + wl];
    uint32_t nsub = 0, nod = 0, npair = 0, nitem = 0, te = 0, ent;

    LOSA_TL_NEXT(ent);
    while ((ent >> 28) == 1) {
      const int w = (int)(ent & kTlItemMask);
      const bool partial = (ent & kTlPartial) != 0;
      const int part = (int)((ent >> 24) & 7u);
      const int pbh = w / p.nPairs, pr = w % p.nPairs;
      const int bh = pbh % (p.B * p.H);
      const int b = bh / p.H, h = bh % p.H;
      void* const o_base = (p.problems != nullptr) ? p.problems[pbh / (p.B * p.H)].o : p.o;
      const int T = 2 * pr + qt;
      const int grow = T * 128 + row;
      float m_ref = 0.f, l = 0.f, le = 0.f;  // le: row sum of the unrounded exponentials (masses, LSE)
      bool have_ref = false, ovf = false;
      uint32_t pv_item = 0;
      for (;;) {
        uint32_t grp[kG];
        bool more;
        LOSA_TL_NEXT_TILE(grp, more);
        if (!more) {
          ent = grp[0];
          break;
        }
        // hv[i]: how many columns of block i of this half the row attends to (a block is a key
        // block, or this half's 64 columns of a 128-key block)
        uint32_t memb = 0;
        int hv[kHB];
        bool mine = false, whole = true, pair_mine = false;
#pragma unroll
        for (int g = 0; g < kG; ++g) {
          memb |= (grp[g] >> 16) & 0xfu;
          pair_mine = pair_mine || ((grp[g] >> (16 + my_bit)) & 1u);
        }
#pragma unroll
        for (int i = 0; i < kHB; ++i) {
          const int g = (kG >= 2) ? half * kHB + i : 0;
          const int jg = (int)(grp[g] & 0xffffu);
          const int valid = ((grp[g] >> (16 + my_bit)) & 1u) ? min(kC, p.N - jg * kC) : 0;
          hv[i] = (kG >= 2) ? valid : max(0, min(64, valid - 64 * half));
          mine = mine || hv[i] > 0;
          whole = whole && hv[i] == kBW;
        }
        uint32_t rot_b = 0;
        if (kRot) {
          // the buffer follows from the tile's place in the issue order: per K/V tile, query tile 0
          // first, then query tile 1, each only if it lists the tile
          const bool m0 = (memb & kQMask) != 0, m1 = ((memb >> kQBT) & kQMask) != 0;
          const uint32_t kmine = kq + ((qt == 1 && m0) ? 1u : 0u);
          kq += (m0 ? 1u : 0u) + (m1 ? 1u : 0u);
          if (!(qt == 0 ? m0 : m1)) continue;
          rot_b = kmine % 3u;
          tSrow = tmem_base + lane_base + rot_b * 128;
          tS = tSrow + half * 64;
          const uint32_t par = (rot_b == 0 ? uses[0] : rot_b == 1 ? uses[1] : uses[2]) & 1;
          uses[0] += (rot_b == 0);
          uses[1] += (rot_b == 1);
          uses[2] += (rot_b == 2);
          LOSA_WAIT(&ctl->rot_s_full[qt * 3 + rot_b], par);
        } else {
          if (((memb >> (qt * kQBT)) & kQMask) == 0) continue;
          // S of this key tile is complete, and so is every earlier product into O
          // (the mass pass has two S buffers per query tile and no O)
          const uint32_t buf = nsub % kNS;
          if (!C::kHasV) {
            tSrow = tmem_base + lane_base + qt * kSStride + buf * 128;
            tS = tSrow + half * 64;
          }
          LOSA_WAIT(&ctl->s_full[qt][buf], (nsub / kNS) & 1);
        }
        ptx::tc_fence_after_sync();
        if (!have_ref && pair_mine) {
          // the item's first tile for this row: the reference is the maximum of the row's scores
          // over the keys it attends to, computed by both halves alike (no exchange)
          float mx = -INFINITY;
#pragma unroll
          for (int c0 = 0; c0 < kW; c0 += 32) {
            uint32_t r[32];
            ptx::tmem_ld32(tSrow + c0, r);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int cc = c0 + c;
              const int jg = (int)(grp[cc / kC] & 0xffffu);
              const int valid = ((grp[cc / kC] >> (16 + my_bit)) & 1u) ? min(kC, p.N - jg * kC) : 0;
              if ((cc % kC) < valid) mx = fmaxf(mx, __uint_as_float(r[c]));
            }
          }
          m_ref = mx * p.scale_log2;
          have_ref = true;
          // the other half reads the whole row too: nobody packs P over it before both are done
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(pair_bar);
          LOSA_WAIT(pair_bar, npair & 1);
          ++npair;
          ptx::tc_fence_after_sync();
        }
        uint32_t sr[64];
        if (mine) {
          ptx::tmem_ld32(tS, &sr[0]);
          if (whole) ptx::tmem_wait_ld();
          ptx::tmem_ld32(tS + 32, &sr[32]);
          if (!whole) {
            // keys that do not exist (>= N, in the sequence's last key block): -inf column by column
            ptx::tmem_wait_ld();
            bool ragged = false;
#pragma unroll
            for (int i = 0; i < kHB; ++i) ragged = ragged || (hv[i] > 0 && hv[i] < kBW);
            if (ragged) {
#pragma unroll
              for (int c = 0; c < 64; ++c)
                if ((c % kBW) >= hv[c / kBW]) sr[c] = 0xff800000u;
            }
          }
          if (!C::kHasV) {
            // mass pass: the scores are in registers and nothing is packed over them: the buffer goes back
            ptx::tmem_wait_ld();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->s_free[qt][nsub % kNS]);
          }
          // key blocks the row's query block does not list get -inf as the addend of the scaling FMA
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
          float2 nm2[kHB];
#pragma unroll
          for (int i = 0; i < kHB; ++i) {
            const float a = (hv[i] > 0) ? -m_ref : -INFINITY;
            nm2[i] = make_float2(a, a);
          }
          // The output is normalised by the sum of the weights the tensor core multiplies with V -
          // P as rounded to bf16 - so that o is a weighted mean of V whatever the rounding does.
          float2 racc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          float2 eacc[kHB];  // fused step: sums of the unrounded exponentials, per block of this half
#pragma unroll
          for (int i = 0; i < kHB; ++i) eacc[i] = make_float2(0.f, 0.f);
#pragma unroll
          for (int c = 0; c < 64; c += 4) {
            if (C::kHasV && whole && c == 32) ptx::tmem_wait_ld();
            float2 x0 = ptx::fma2(
                make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2, nm2[c / kBW]);
            float2 x1 = ptx::fma2(
                make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sc2, nm2[c / kBW]);
            if (kSplitPoly > 0 && (c >> 2) % kSplitPolyOf < kSplitPoly) {
              x0 = ptx::ex2_poly2(x0);
              x1 = ptx::ex2_poly2(x1);
            } else {
              x0.x = ptx::ex2_approx(x0.x);
              x0.y = ptx::ex2_approx(x0.y);
              x1.x = ptx::ex2_approx(x1.x);
              x1.y = ptx::ex2_approx(x1.y);
            }
            if (C::kHasV) {
              const uint32_t u0 = ptx::pack_bf16x2(x0.x, x0.y), u1 = ptx::pack_bf16x2(x1.x, x1.y);
              sr[c >> 1] = u0;
              sr[(c >> 1) + 1] = u1;
              ptx::add_bf16x2(racc[0], u0);
              ptx::add_bf16x2(racc[1], u1);
            }
            if (C::kWantMass) eacc[c / kBW] = ptx::add2(eacc[c / kBW], ptx::add2(x0, x1));
          }
          float tsum = (racc[0].x + racc[0].y) + (racc[1].x + racc[1].y);
          if (!C::kHasV) {
#pragma unroll
            for (int i = 0; i < kHB; ++i) tsum += eacc[i].x + eacc[i].y;
          }
          ovf = ovf || __any_sync(0xffffffffu, !(tsum <= kSplitSafeSum));
          l += tsum;
          if (C::kHasV) ptx::tmem_st32(tS, &sr[0]);
          if (C::kWantMass) {
#pragma unroll
            for (int i = 0; i < kHB; ++i) {
              const float es = eacc[i].x + eacc[i].y;
              le += es;
              const int g = (kG >= 2) ? half * kHB + i : 0;
              const int64_t sb = (kG >= 2) ? (int64_t)(grp[g] & 0xffffu) : (int64_t)(grp[0] & 0xffffu) * 2 + half;
              if (hv[i] > 0 && LOSA_IN_RANGE(sb * 128 + row, p.cap_table_floats)) tabf[sb * 128] = es;
            }
          }
        } else {
          // this half of the row lists none of the tile's keys: P = 0
          if (C::kHasV) {
            uint32_t z[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) z[c] = 0u;
            ptx::tmem_st32(tS, z);
          } else {
            // mass pass: the buffer goes back untouched
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->s_free[qt][nsub % kNS]);
          }
          // (a key block that fills the tile but ends before this half: its entry of the table is 0)
          if (C::kWantMass && kG == 1 && pair_mine &&
              LOSA_IN_RANGE(((int64_t)(grp[0] & 0xffffu) * 2 + half) * 128 + row, p.cap_table_floats))
            tabf[((int64_t)(grp[0] & 0xffffu) * 2 + half) * 128] = 0.f;
        }
        if (C::kHasV) {
          ptx::tmem_wait_st();
          ++pv_item;
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(kRot ? &ctl->rot_p_ready[qt * 3 + rot_b] : &ctl->p_ready[qt]);
        }
        ++nsub;
      }

      // ---- end of the item: half 1 hands its row sums over, half 0 writes O / l
      // (two sets of slots, used by alternate items: half 1 may be an item ahead of half 0's read)
      float* const xset = ctl->xch + ((nitem & 1) * 2 + qt) * 128;
      // (fused step: both halves need both sums; they go through the workspace, two sets as well)
      float2* const gset = C::kWantMass ? p.rowstat + ((((int64_t)blockIdx.x * 2 + (nitem & 1)) * 2 + qt) * 2) * 128
                                        : nullptr;
      ++nitem;
      if (C::kWantMass) gset[half * 128 + row] = make_float2(le, l);
      else if (half == 1) xset[row] = l;
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(pair_bar);
      LOSA_WAIT(pair_bar, npair & 1);
      ++npair;
      if (C::kWantMass) {
        const float2 other = gset[(half ^ 1) * 128 + row];
        le += other.x;
        l += other.y;
      }
      if (ovf && lane == 0) {
        // (the pair's warps may both get here, and so may the other pairs: the unit is listed once)
        const int unit = partial ? p.split_first + (w - p.split_first) * p.split_parts + part : w;
        if (atomicExch(&ctl->ovf_unit, unit) != unit) {
          const int slot = atomicAdd(p.redo_count, 1);
          if (slot < p.nUnits) p.redo_list[slot] = unit;
        }
      }
      if (C::kHasV && half == 0 && T < p.nQt) {
        if (!C::kWantMass) l += xset[row];
        const bool valid = grow < p.N;
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
        const int64_t off = (int64_t)b * p.sb + (int64_t)h * p.sh + (int64_t)grow * p.sn;
        const int64_t pslot =
            ((((int64_t)(w - p.split_first) * p.split_parts + part) * 2 + qt) * 128 + row);
        if (partial && LOSA_IN_RANGE(pslot, p.cap_part_rows)) p.part_ml[pslot] = make_float2(m_ref, l);
        if (pv_item > 0) {
          LOSA_WAIT(&ctl->o_done[qt], nod & 1);
          ++nod;
          ptx::tc_fence_after_sync();
        }
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t r[32];
          if (pv_item > 0) {
            ptx::tmem_ld32(tO + c0, r);
            ptx::tmem_wait_ld();
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c) r[c] = 0u;
          }
          if (partial) {
            float4* dst = reinterpret_cast<float4*>(p.part_o + (LOSA_IN_RANGE(pslot, p.cap_part_rows) ? pslot : 0) * D + c0);
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              dst[c >> 2] = make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                        __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
          } else if (valid) {
            if (p.o_f32) {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(o_base) + off + c0);
#pragma unroll
              for (int c = 0; c < 32; c += 4)
                dst[c >> 2] = make_float4(__uint_as_float(r[c]) * inv, __uint_as_float(r[c + 1]) * inv,
                                          __uint_as_float(r[c + 2]) * inv,
                                          __uint_as_float(r[c + 3]) * inv);
            } else {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(o_base) + off + c0);
#pragma unroll
              for (int c = 0; c < 32; c += 8) {
                uint4 v;
                v.x = ptx::pack_bf16x2(__uint_as_float(r[c]) * inv, __uint_as_float(r[c + 1]) * inv);
                v.y = ptx::pack_bf16x2(__uint_as_float(r[c + 2]) * inv, __uint_as_float(r[c + 3]) * inv);
                v.z = ptx::pack_bf16x2(__uint_as_float(r[c + 4]) * inv, __uint_as_float(r[c + 5]) * inv);
                v.w = ptx::pack_bf16x2(__uint_as_float(r[c + 6]) * inv, __uint_as_float(r[c + 7]) * inv);
                dst[c >> 3] = v;
              }
            }
          }
        }
        if (pv_item > 0) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&ctl->o_free[qt]);
        }
      }
      if (C::kWantMass) {
        // ---- fused construction step: the block masses of this query tile.  The reference did not
        // move during the item, so a row's weight is 1 / (its sum of exponentials) and a mass is the
        // mean over the query block's rows of weight x (the row's sum over the key block).
        float* const inv_rows = p.rowinv + ((int64_t)blockIdx.x * 2 + qt) * 128;
        if (half == 0 && T < p.nQt) {
          const bool valid = grow < p.N;
          inv_rows[row] = (valid && le > 0.f) ? 1.f / le : 0.f;
          if (p.lse != nullptr && valid && LOSA_IN_RANGE((int64_t)bh * p.N + grow, p.cap_lse))
            p.lse[(int64_t)bh * p.N + grow] = (m_ref + log2f(le)) * kLn2;
        }
        ptx::mbar_arrive(&ctl->wg_bar[qt]);  // all eight warps of the query tile, with a bounded wait
        LOSA_WAIT(&ctl->wg_bar[qt], nwg & 1);
        ++nwg;
        if (T < p.nQt) {
          const float* tb = reinterpret_cast<const float*>(p.table) +
                            ((int64_t)blockIdx.x * 2 + qt) * (int64_t)p.nKb * 256;
          float iv[4];  // this lane's four rows
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) iv[rr] = inv_rows[rr * 32 + lane];
          for (int u = half * 4 + wl; u < p.nKb; u += 8) {
            float acc[kQBT];
#pragma unroll
            for (int q = 0; q < kQBT; ++q) acc[q] = 0.f;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
              const int r = rr * 32 + lane;
              float wgt = 0.f;
              if (iv[rr] > 0.f) {
                const float sum = (kG >= 2) ? tb[(int64_t)u * 128 + r]
                                            : tb[(int64_t)u * 256 + r] + tb[(int64_t)u * 256 + 128 + r];
                wgt = sum * iv[rr];
              }
              acc[(rr * 32) / R] += wgt;
            }
#pragma unroll
            for (int q = 0; q < kQBT; ++q) {
              float a2 = acc[q];
#pragma unroll
              for (int d = 16; d > 0; d >>= 1) a2 += __shfl_xor_sync(0xffffffffu, a2, d);
              const int g = T * kQBT + q;
              if (lane == 0 && g < p.nQb) {
                const int nvalid = min(R, p.N - g * R);
                {
                  const int64_t mi = ((int64_t)bh * p.nQb + g) * p.nKb + u;
                  if (LOSA_IN_RANGE(mi, p.cap_mass)) p.mass[mi] = a2 / (float)nvalid;
                }
              }
            }
          }
        }
        // (the table and the row weights are written again by the next item)
        ptx::mbar_arrive(&ctl->wg_bar[qt]);
        LOSA_WAIT(&ctl->wg_bar[qt], nwg & 1);
        ++nwg;
      }
    }
  }

teardown:
  if (ctl->abort_flag) {
    // Abort path: give MMAs and bulk copies still in flight a bounded time to land before
    // shared memory and TMEM are released.
    // (the same thread that issued the MMAs: the election is deterministic for a full warp)
    if ((warp == kIssuerWarp || warp == kIssuerWarp + 1) && ptx::elect_one()) {
      ptx::mma_commit(&ctl->drain);
      for (uint32_t it = 0; it < (1u << 16); ++it) {
        if (ptx::mbar_try_wait(&ctl->drain, 0)) break;
        __nanosleep(128);
      }
    }
    if (warp == kProducerWarp && lane == 0) {
      for (uint32_t it = 0; it < (1u << 10); ++it) __nanosleep(1024);
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == kIssuerWarp) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

#include "losa_attn_pair.cuh"

#undef LOSA_TL_PUT_BULK
#undef LOSA_TL_NEXT_TILE
#undef LOSA_TL_NEXT
#undef LOSA_TL_PUT
#undef LOSA_WAIT_RELAXED
#undef LOSA_WAIT

// Sparse mode, before the attention kernel: one warp per work unit merges the index lists of the
// unit's query blocks into its tile list (entry = key block index | membership bits << 16,
// padded to whole K/V tiles of G entries; for the order see below).  Every list becomes a bitmap in shared
// memory (coalesced reads, one atomicOr per index), the union's set bits are enumerated 32 words
// at a time with a warp scan.  Doing this ahead of the launch keeps the in-kernel scheduler warp,
// which shares a scheduler partition with two softmax warps and is favoured over them, nearly
// idle.  A unit that is a part of an item takes the same share, by position, of every list, so
// each (query block, key block) pair belongs to exactly one part.  Indices out of range are
// reported and skipped; an unsorted list still gives a valid tile list.
template <int NB, int G>
__global__ void __launch_bounds__(32) build_tile_lists_kernel(const Params p) {
  extern __shared__ uint32_t bm[];  // [NB][W] bitmaps
  const int lane = threadIdx.x, unit = blockIdx.x;
  int w = unit, part = 0, parts = 1;
  if (unit >= p.split_first) {
    const int r = unit - p.split_first;
    parts = p.split_parts;
    part = r % parts;
    w = p.split_first + r / parts;
  }
  const int pbh = w / p.nPairs, pr = w % p.nPairs;
  const int bh = pbh % (p.B * p.H);
  const int32_t* offsets = p.offsets;
  const int32_t* kv_idx = p.kv_idx;
  if (p.problems != nullptr) {
    const ProblemEntry* pe = p.problems + pbh / (p.B * p.H);
    offsets = pe->offsets;
    kv_idx = pe->kv_idx;
  }
  const int W = (p.nKb + 31) >> 5;
  for (int i = lane; i < NB * W; i += 32) bm[i] = 0u;
  __syncwarp();
  const int32_t nnz = __ldg(offsets + (int64_t)p.B * p.H * p.nQb);
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const int g = pr * NB + n;
    if (g >= p.nQb) continue;
    const int64_t row = (int64_t)bh * p.nQb + g;
    const int32_t b = __ldg(offsets + row), e = __ldg(offsets + row + 1);
    if (b < 0 || e < b || e > nnz || e - b > p.nKb) {
      report_error(p.status, LOSA_ERR_BAD_INDEX);
      continue;
    }
    const int b2 = b + (int)(((int64_t)(e - b) * part) / parts);
    const int e2 = b + (int)(((int64_t)(e - b) * (part + 1)) / parts);
    for (int i = b2 + lane; i < e2; i += 32) {
      const int v = __ldg(kv_idx + i);
      if ((unsigned)v < (unsigned)p.nKb) atomicOr(&bm[n * W + (v >> 5)], 1u << (v & 31));
      else report_error(p.status, LOSA_ERR_BAD_INDEX);  // skipped, never used as an address
    }
  }
  __syncwarp();
  // Order of the entries.  A key block that only ONE of the unit's two query tiles lists is
  // processed by that tile alone, at half the CTA's rate; two such blocks, one of each tile, can
  // be in flight at the same time (the tiles' chains are independent).  So the list holds first
  // the blocks both tiles list, then the single-tile blocks of tile 0 and tile 1 in alternation
  // (K/V tile by K/V tile; a class that does not fill its last K/V tile pads it), then what is
  // left of the longer class.  Within a class the blocks ascend.  Correctness does not depend on
  // the order of the key blocks.
  uint32_t* dst = p.tl_entries + (int64_t)unit * p.tl_cap;
  int nb = 0, na = 0, nbb = 0;  // both, tile 0 only, tile 1 only
  for (int w0 = 0; w0 < W; w0 += 32) {
    const int wi = w0 + lane;
    uint32_t ta = 0, tb = 0;
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const uint32_t m = (wi < W) ? bm[n * W + wi] : 0u;
      if (n < NB / 2) ta |= m; else tb |= m;
    }
    nb += __popc(ta & tb);
    na += __popc(ta & ~tb);
    nbb += __popc(tb & ~ta);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    nb += __shfl_xor_sync(0xffffffffu, nb, d);
    na += __shfl_xor_sync(0xffffffffu, na, d);
    nbb += __shfl_xor_sync(0xffffffffu, nbb, d);
  }
  const int s1 = (nb + G - 1) / G * G;                       // entries of the first section
  const int tA = (na + G - 1) / G, tB = (nbb + G - 1) / G;   // K/V tiles of the single-tile classes
  const int tmin = min(tA, tB);
  const int total = min(s1 + (tA + tB) * G, p.tl_cap);
  for (int i = lane; i < total; i += 32) dst[i] = kTlPad;
  __syncwarp();
  int rb = 0, ra = 0, rbb = 0;  // entries of each class emitted by earlier windows
  for (int w0 = 0; w0 < W; w0 += 32) {
    const int wi = w0 + lane;
    uint32_t m[NB], ta = 0, tb = 0;
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      m[n] = (wi < W) ? bm[n * W + wi] : 0u;
      if (n < NB / 2) ta |= m[n]; else tb |= m[n];
    }
    uint32_t cls[3] = {ta & tb, ta & ~tb, tb & ~ta};
    int incl[3], tot[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      incl[k] = __popc(cls[k]);
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl[k], d);
        if (lane >= d) incl[k] += t;
      }
      tot[k] = __shfl_sync(0xffffffffu, incl[k], 31);
    }
    const int base[3] = {rb, ra, rbb};
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      uint32_t u = cls[k];
      int r = base[k] + incl[k] - __popc(u);  // rank of this lane's first entry within its class
      while (u) {
        const int bit = __ffs(u) - 1;
        u &= u - 1;
        uint32_t memb = 0;
#pragma unroll
        for (int n = 0; n < NB; ++n) memb |= ((m[n] >> bit) & 1u) << n;
        int pos;
        if (k == 0) {
          pos = r;
        } else {
          const int t = r / G;  // K/V tile of the class
          const int slot = (t < tmin) ? 2 * t + (k - 1) : 2 * tmin + (t - tmin);
          pos = s1 + slot * G + r % G;
        }
        if (pos < p.tl_cap) dst[pos] = (uint32_t)(wi * 32 + bit) | (memb << 16);
        ++r;
      }
    }
    rb += tot[0];
    ra += tot[1];
    rbb += tot[2];
  }
  if (lane == 0) p.tl_count[unit] = total;
}

// Merge of the partial units: for every row of the split items, combine the parts' unnormalised
// O, reference maximum and row sum (the usual log-sum-exp merge) and write the attention output.
// grid = (split items, 2 query tiles x 8 row chunks), 4 warps; a warp takes 4 rows, its lanes the
// columns.
template <int D>
__global__ void __launch_bounds__(128) merge_parts_kernel(const Params p) {
  const int r = blockIdx.x, qt = blockIdx.y >> 3, chunk = blockIdx.y & 7;
  const int w = p.split_first + r;
  const int pbh = w / p.nPairs, pr = w % p.nPairs;
  const int T = 2 * pr + qt;
  if (T >= p.nQt) return;
  const int bh = pbh % (p.B * p.H);
  const int b = bh / p.H, h = bh % p.H;
  void* const o_base = (p.problems != nullptr) ? p.problems[pbh / (p.B * p.H)].o : p.o;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int parts = p.split_parts;
#pragma unroll
  for (int rr = 0; rr < 4; ++rr) {
    const int row = chunk * 16 + warp * 4 + rr;
    const int grow = T * 128 + row;
    if (grow >= p.N) break;
    float sc[kMaxParts];
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < kMaxParts; ++s) {
      sc[s] = 0.f;
      if (s < parts) {
        const float2 ml = p.part_ml[(((int64_t)r * parts + s) * 2 + qt) * 128 + row];
        if (ml.y > 0.f) m = fmaxf(m, ml.x);
      }
    }
    float L = 0.f;
#pragma unroll
    for (int s = 0; s < kMaxParts; ++s) {
      if (s < parts) {
        const float2 ml = p.part_ml[(((int64_t)r * parts + s) * 2 + qt) * 128 + row];
        if (ml.y > 0.f) {
          sc[s] = ptx::ex2_approx(ml.x - m);
          L += ml.y * sc[s];
        }
      }
    }
    const float inv = (L > 0.f) ? 1.f / L : 0.f;
    const int d = lane * 4;
    if (d < D) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < kMaxParts; ++s) {
        if (s < parts && sc[s] != 0.f) {
          const float4 v = *reinterpret_cast<const float4*>(
              p.part_o + ((((int64_t)r * parts + s) * 2 + qt) * 128 + row) * D + d);
          acc.x += v.x * sc[s];
          acc.y += v.y * sc[s];
          acc.z += v.z * sc[s];
          acc.w += v.w * sc[s];
        }
      }
      const int64_t off = (int64_t)b * p.sb + (int64_t)h * p.sh + (int64_t)grow * p.sn + d;
      if (p.o_f32) {
        *reinterpret_cast<float4*>(static_cast<float*>(o_base) + off) =
            make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
      } else {
        uint2 v;
        v.x = ptx::pack_bf16x2(acc.x * inv, acc.y * inv);
        v.y = ptx::pack_bf16x2(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(o_base) + off) = v;
      }
    }
  }
}

// ---------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 [B,H,N,D] tensor, box = [box_rows][64] with 128-byte swizzle; rows >= N read as zero.
int make_map(CUtensorMap* m, const void* base, const Geometry& g, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled entry point");
    return LOSA_ERR_CUDA;
  }
  const cuuint64_t dims[4] = {(cuuint64_t)g.D, (cuuint64_t)g.N, (cuuint64_t)g.H, (cuuint64_t)g.B};
  const cuuint64_t strides[3] = {(cuuint64_t)g.sn * 2, (cuuint64_t)g.sh * 2, (cuuint64_t)g.sb * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return LOSA_ERR_CUDA;
  }
  return LOSA_OK;
}

// Configures (once per device) and launches one layout of the attention kernel.
template <int D, int R, int C_, int MODE, int KT, bool SPLIT>
int launch_kernel(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mkw,
                  const CUtensorMap& mvw, const Params& prm, int grid, cudaStream_t st) {
  using C = Cfg<D, R, C_, MODE, KT, SPLIT && D == 64 && MODE != kMass>;
  using L = Lay<SPLIT>;
  using Ctl = Control<C::kNK, C::kNV, SPLIT, SPLIT && D == 64 && MODE != kMass>;
  // (one thread per row: 1024 bytes of slack to align the tiles; two threads per row: none left,
  // the kernel checks the alignment of its shared memory instead)
  const size_t smem = (SPLIT ? 0 : 1024) + 2 * C::kQBytes +
                      (size_t)(C::kNK + C::kNV) * C::kKVBytes + sizeof(Ctl);
  static_assert((SPLIT ? 0 : 1024) + 2 * C::kQBytes + (C::kNK + C::kNV) * C::kKVBytes + sizeof(Ctl) <= 227 * 1024,
                "shared memory of one CTA");
  auto kern = losa_attn_kernel<D, R, C_, MODE, KT, SPLIT>;
  // (function attributes belong to a device: one flag per device ordinal)
  static bool configured_on[kMaxDevices] = {};
  int dev = 0;
  LOSA_CUDA_TRY(cudaGetDevice(&dev));
  bool& configured = configured_on[dev];
  if (!configured) {
    // the in-kernel register reallocation must fit the registers the CTA is launched with
    cudaFuncAttributes attr;
    LOSA_CUDA_TRY(cudaFuncGetAttributes(&attr, kern));
    if (attr.numRegs * L::kThreads < 128 * L::kRegsUtility + 32 * L::kSoftmaxWarps * L::kRegsSoftmax) {
      set_cuda_error(cudaErrorLaunchOutOfResources, "register budget of losa_attn_kernel");
      return LOSA_ERR_UNSUPPORTED;
    }
    LOSA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  kern<<<grid, L::kThreads, smem, st>>>(mq, mk, mv, mkw, mvw, prm);
  LOSA_CUDA_TRY(cudaGetLastError());
  return LOSA_OK;
}

// Configures (once per device) and launches the CTA-pair kernel on `clusters` pairs; *max_clusters
// (if not null) receives how many pairs the device can hold at once.
template <int C_, int MODE>
int launch_pair(const CUtensorMap& mq, const CUtensorMap& mkh, const CUtensorMap& mv, const CUtensorMap& mk64,
                const CUtensorMap& mv128, const Params& prm, int clusters, cudaStream_t st, int* max_clusters) {
  using L = Lay<true>;
  constexpr size_t smem = kPairQBytes + (size_t)(kPairNK + kPairNV) * kPairStage + sizeof(PairControl);
  static_assert(smem <= 227 * 1024, "shared memory of one CTA");
  auto kern = losa_pair_kernel<C_, MODE>;
  static int max_on[kMaxDevices] = {};
  int dev = 0;
  LOSA_CUDA_TRY(cudaGetDevice(&dev));
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(L::kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_on[dev] == 0) {
    cudaFuncAttributes fa;
    LOSA_CUDA_TRY(cudaFuncGetAttributes(&fa, kern));
    if (fa.numRegs * L::kThreads < 128 * L::kRegsUtility + 32 * L::kSoftmaxWarps * L::kRegsSoftmax) {
      set_cuda_error(cudaErrorLaunchOutOfResources, "register budget of losa_pair_kernel");
      return LOSA_ERR_UNSUPPORTED;
    }
    LOSA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cfg.gridDim = dim3(2 * kMaxPersistentCtas, 1, 1);
    int n = 0;
    LOSA_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kern, &cfg));
    if (n < 1) {
      set_cuda_error(cudaErrorLaunchOutOfResources, "no resident CTA pair of losa_pair_kernel");
      return LOSA_ERR_UNSUPPORTED;
    }
    max_on[dev] = n;
  }
  if (max_clusters != nullptr) {
    *max_clusters = max_on[dev];
    return LOSA_OK;
  }
  cfg.gridDim = dim3(2 * clusters, 1, 1);
  LOSA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, mq, mkh, mv, mk64, mv128, prm));
  return LOSA_OK;
}

template <int D, int R, int C_, int MODE, int KT>
int launch_t(const Geometry& g, const void* q, const void* k, const void* v, Params prm, int sms,
             cudaStream_t st) {
  using C = Cfg<D, R, C_, MODE, KT>;
  CUtensorMap mq, mk, mv;
  int rc;
  if ((rc = make_map(&mq, q, g, 128)) != LOSA_OK) return rc;
  if ((rc = make_map(&mk, k, g, C::kC)) != LOSA_OK) return rc;
  if ((rc = make_map(&mv, C::kHasV ? v : k, g, C::kC)) != LOSA_OK) return rc;
  CUtensorMap mk128, mv128;  // boxes of a whole 128-key tile, for tiles of consecutive key blocks
  if ((rc = make_map(&mk128, k, g, 128)) != LOSA_OK) return rc;
  if ((rc = make_map(&mv128, C::kHasV ? v : k, g, 128)) != LOSA_OK) return rc;
  int ctas = min(sms, kMaxPersistentCtas);
  // Head dimension 128 with 128-row query blocks, modes with an attention output: pairs of CTAs,
  // one work item per pair at a time (see losa_attn_pair.cuh); the single-CTA kernels stay the
  // fallback.  (With 32-key blocks the pair kernel was slower than the single-CTA kernel until
  // tiles of consecutive key blocks were copied whole: dense forward 6.3 against 5.9 ms before,
  // 5.56 against 6.20 ms after.)  The mass pass alone runs on pairs only with 32-key blocks (5.65 -> 5.16
  // ms at the Wan shape; with 64- and 128-key blocks it measured the same or 2 % slower on pairs: the
  // exponential unit bounds it either way).
  constexpr bool kPairMode = LOSA_USE_PAIR && D == 128 && R == 128 && C_ >= LOSA_PAIR_MIN_C &&
                             (MODE == kDense || MODE == kSparse || (LOSA_PAIR_FUSED && MODE == kFused) ||
                              (LOSA_PAIR_MASS && MODE == kMass && C_ < 64));
  bool pair = false;  // (a device that cannot hold a pair of these CTAs runs the single-CTA kernel)
  CUtensorMap mkh, mk64;
  if constexpr (kPairMode) {
    if ((rc = make_map(&mkh, k, g, C::kC < 64 ? C::kC : 64)) != LOSA_OK) return rc;
    if ((rc = make_map(&mk64, k, g, 64)) != LOSA_OK) return rc;
    int fit = 0;
    if (launch_pair<C_, MODE>(mq, mkh, mv, mk64, mv128, prm, 0, st, &fit) == LOSA_OK && fit >= 1 && sms >= 2) {
      pair = true;
      ctas = min(min(sms / 2, fit), kMaxPersistentCtas);
    }
  }
  // The items of the last, partly filled wave of the persistent grid (all items, if there are
  // fewer than CTAs) are cut into parts of the key range, so that the wave ends after 1/parts of
  // an item; their partial results are merged by a second, small kernel.  Attention output
  // only: the mass epilogue needs a row's final statistics inside the kernel.
  prm.nUnits = prm.nWork;
  prm.split_first = prm.nWork;
  prm.split_parts = 1;
  constexpr bool kAttnOnly = (MODE == kDense || MODE == kSparse);
  constexpr bool kTwoPerRow = true;  // every mode runs with two threads per row; one per row is the fallback
  if (kAttnOnly) {
    const int rest = (prm.nWork < ctas) ? prm.nWork : prm.nWork % ctas;
    int parts = rest > 0 ? ctas / rest : 1;
    parts = min(min(parts, kMaxParts), prm.nKb);
    if (parts >= 2) {
      prm.split_first = prm.nWork - rest;
      prm.split_parts = parts;
      prm.nUnits = prm.split_first + rest * parts;
    }
  }
  const int grid = min(ctas, prm.nUnits);
  if (MODE == kSparse) {
    const size_t bm_bytes = (size_t)C::kNB * ((prm.nKb + 31) / 32) * sizeof(uint32_t);  // <= 32 KB
    build_tile_lists_kernel<C::kNB, C::kG><<<prm.nUnits, 32, bm_bytes, st>>>(prm);
    LOSA_CUDA_TRY(cudaGetLastError());
  }
  if constexpr (kTwoPerRow) {
    // The modes with an attention output run with two threads per query row and a reference that
    // never moves; the units whose scores outgrew it (none, on ordinary inputs) are listed, and a second
    // launch of the one-thread-per-row kernel, which returns at once when the list is empty,
    // recomputes them with a moving reference.
    prm.redo = 0;
    bool launched = false;
    if constexpr (kPairMode) {
      if (pair) {
        if ((rc = launch_pair<C_, MODE>(mq, mkh, mv, mk64, mv128, prm, grid, st, nullptr)) != LOSA_OK) return rc;
        launched = true;
      }
    }
    if (!launched) {
      if ((rc = launch_kernel<D, R, C_, MODE, KT, true>(mq, mk, mv, mk128, mv128, prm, grid, st)) != LOSA_OK) return rc;
    }
    if (!prm.stall) {
      prm.redo = 1;
      prm.work_counter += 2;  // its own counter (zeroed with the first)
      // (as many CTAs as SMs, whichever kernel ran first)
      const int rgrid = min(min(sms, kMaxPersistentCtas), prm.nUnits);
      if ((rc = launch_kernel<D, R, C_, MODE, KT, false>(mq, mk, mv, mk128, mv128, prm, rgrid, st)) != LOSA_OK) return rc;
    }
  } else {
    prm.redo = 0;
    if ((rc = launch_kernel<D, R, C_, MODE, KT, false>(mq, mk, mv, mk128, mv128, prm, grid, st)) != LOSA_OK) return rc;
  }
  if (prm.split_parts > 1) {
    merge_parts_kernel<D><<<dim3(prm.nWork - prm.split_first, 16), 128, 0, st>>>(prm);
    LOSA_CUDA_TRY(cudaGetLastError());
  }
  return LOSA_OK;
}

template <int MODE>
int dispatch(const Geometry& g, const void* q, const void* k, const void* v, const Params& prm,
             int sms, cudaStream_t st) {
  // K/V tiles of 128 keys everywhere (128 / C gathered key blocks, 128-wide MMAs)
#define LOSA_CASE(d, r, c) \
  if (g.D == d && g.R == r && g.C == c) return launch_t<d, r, c, MODE, 128>(g, q, k, v, prm, sms, st)
  LOSA_CASE(128, 128, 128);
  LOSA_CASE(64, 64, 64);
  LOSA_CASE(128, 128, 32);  // the paper's own block geometry
  LOSA_CASE(64, 128, 32);
  LOSA_CASE(128, 64, 64);
  LOSA_CASE(64, 128, 128);
  LOSA_CASE(128, 128, 64);
  LOSA_CASE(64, 128, 64);
#undef LOSA_CASE
  return LOSA_ERR_UNSUPPORTED;
}

}  // namespace


namespace {
size_t part_o_bytes(const Geometry& g) {
  return (size_t)kMaxPersistentCtas * 2 * 128 * (size_t)g.D * sizeof(float);
}
// the last wave's items are cut into at most one unit per CTA
int64_t max_units(const Geometry& g, int n_prob) {
  return (int64_t)n_prob * g.B * g.H * g.nPairs + kMaxPersistentCtas;
}
int tile_list_cap(const Geometry& g) { return (g.nKb + 16 + 31) / 32 * 32; }  // union <= nKb, + padding of three sections
size_t tl_count_bytes(const Geometry& g, int n_prob) {
  return ((size_t)max_units(g, n_prob) * sizeof(int32_t) + 255) / 256 * 256;
}
size_t tl_entries_bytes(const Geometry& g, int n_prob) {
  return ((size_t)max_units(g, n_prob) * tile_list_cap(g) * sizeof(uint32_t) + 255) / 256 * 256;
}
}  // namespace

void arm_stalled_launch(uint32_t polls) { g_stall_polls.store(polls); }

// Work slots (persistent CTAs, or pairs of CTAs) that a call of this kind occupies on a device
// with `sms` multiprocessors: the host rule of launch_t, for callers that want to know how the
// work items are spread (which of them the last wave cuts into parts).
int attn_work_slots(AttnMode mode, const Geometry& g, int sms) {
  const int ctas = sms < kMaxPersistentCtas ? sms : kMaxPersistentCtas;
  const bool pair = LOSA_USE_PAIR && g.D == 128 && g.R == 128 && g.C >= LOSA_PAIR_MIN_C &&
                    (mode == kDense || mode == kSparse || (LOSA_PAIR_FUSED && mode == kFused) ||
                     (LOSA_PAIR_MASS && mode == kMass && g.C < 64)) && sms >= 2;
  return pair ? ctas / 2 : ctas;
}

size_t attn_workspace_bytes(AttnMode mode, const Geometry& g, int n_prob) {
  // attention output: counter, then one slot per partial unit (at most one per CTA) holding the
  // rows' (max, sum) and unnormalised O of both query tiles
  if (mode == kDense || mode == kSparse) {
    size_t bytes = kCounterBytes + kPartMlBytes + part_o_bytes(g);
    // sparse: the units' merged tile lists (count per unit, then tl_cap entries per unit)
    if (mode == kSparse) bytes += tl_count_bytes(g, n_prob) + tl_entries_bytes(g, n_prob);
    // batched launch: the table of the problems' tensor maps and pointers
    if (n_prob > 1) bytes += (size_t)n_prob * sizeof(ProblemEntry);
    // the work units handed to the fallback launch (each CTA of a pair may list a unit)
    bytes += 2 * tl_count_bytes(g, n_prob);
    return bytes;
  }
  // counter, per-CTA row statistics (three times as many for the fused step with two threads per
  // row: two sets of the halves' row sums, and the rows' weights), per-CTA table of one entry per
  // row and key tile, and the fused step's list of units for the fallback launch
  return kCounterBytes + 5 * kRowstatBytes +
         (size_t)kMaxPersistentCtas * 2 * (size_t)g.nKb * 128 * sizeof(float2) + 2 * tl_count_bytes(g, 1);
}

// Batched launch (n_prob > 1, attention-only modes): `layers` is a host array of n_prob problems of
// the geometry g; q, k, v, offsets, kv_idx and o are then ignored.
int launch_attn(AttnMode mode, const Geometry& g, const void* q, const void* k, const void* v,
                const int32_t* offsets, const int32_t* kv_idx, void* o, int o_dtype, float* mass,
                float* lse, void* ws, cudaStream_t st, int n_prob, const losa_layer_t* layers) {
  Params prm;
  prm.B = g.B;
  prm.H = g.H;
  prm.N = g.N;
  prm.nQb = g.nQb;
  prm.nKb = g.nKb;
  prm.nQt = g.nQt;
  prm.nPairs = g.nPairs;
  if ((int64_t)n_prob * g.B * g.H * g.nPairs > (int64_t)kTlItemMask)
    return LOSA_ERR_UNSUPPORTED;  // the tile list's item headers hold 24 bits
  prm.nWork = n_prob * g.B * g.H * g.nPairs;
  prm.nProb = n_prob;
  prm.problems = nullptr;
  prm.offsets = offsets;
  prm.kv_idx = kv_idx;
  prm.o = o;
  prm.o_f32 = (o_dtype == LOSA_DTYPE_F32) ? 1 : 0;
  prm.sb = g.sb;
  prm.sh = g.sh;
  prm.sn = g.sn;
  prm.mass = mass;
  prm.lse = lse;
  // workspace: [0, 256) work counter, then (mass modes) per-CTA row statistics and tables
  prm.work_counter = static_cast<int*>(ws);
  prm.rowstat = reinterpret_cast<float2*>(static_cast<char*>(ws) + kCounterBytes);
  prm.table = reinterpret_cast<float2*>(static_cast<char*>(ws) + kCounterBytes +
                                        ((mode == kFused || mode == kMass) ? 5 : 0) * kRowstatBytes);
  prm.rowinv = reinterpret_cast<float*>(static_cast<char*>(ws) + kCounterBytes + 4 * kRowstatBytes);
  prm.part_ml = reinterpret_cast<float2*>(static_cast<char*>(ws) + kCounterBytes);
  prm.part_o = reinterpret_cast<float*>(static_cast<char*>(ws) + kCounterBytes + kPartMlBytes);
  {
    char* tl = static_cast<char*>(ws) + kCounterBytes + kPartMlBytes + part_o_bytes(g);
    prm.tl_count = reinterpret_cast<int32_t*>(tl);
    prm.tl_entries = reinterpret_cast<uint32_t*>(tl + tl_count_bytes(g, n_prob));
    prm.tl_cap = tile_list_cap(g);
    if (n_prob > 1) {
      // the problems' table, behind the tile lists (dense mode has none), written before the launch
      char* tab = tl + (mode == kSparse ? tl_count_bytes(g, n_prob) + tl_entries_bytes(g, n_prob) : 0);
      std::vector<ProblemEntry> host(n_prob);
      for (int i = 0; i < n_prob; ++i) {
        int rc;
        if ((rc = make_map(&host[i].map_q, layers[i].q, g, 128)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_k, layers[i].k, g, g.C)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_v, layers[i].v, g, g.C)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_kh, layers[i].k, g, g.C < 64 ? g.C : 64)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_k64, layers[i].k, g, 64)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_k128, layers[i].k, g, 128)) != LOSA_OK) return rc;
        if ((rc = make_map(&host[i].map_v128, layers[i].v, g, 128)) != LOSA_OK) return rc;
        host[i].o = layers[i].o;
        host[i].offsets = layers[i].offsets;
        host[i].kv_idx = layers[i].kv_idx;
      }
      // (a copy from pageable memory is staged before the call returns: `host` may go out of scope)
      LOSA_CUDA_TRY(cudaMemcpyAsync(tab, host.data(), (size_t)n_prob * sizeof(ProblemEntry),
                                    cudaMemcpyHostToDevice, st));
      prm.problems = reinterpret_cast<const ProblemEntry*>(tab);
      q = layers[0].q;  // the kernel's parameter maps are unused but must be valid
      k = layers[0].k;
      v = layers[0].v;
    }
    // counter block: [0] work counter, [1] length of the fallback list, [2] the fallback launch's counter
    prm.redo_count = prm.work_counter + 1;
    prm.redo_list = reinterpret_cast<int*>(
        tl + (mode == kSparse ? tl_count_bytes(g, n_prob) + tl_entries_bytes(g, n_prob) : 0) +
        (n_prob > 1 ? (size_t)n_prob * sizeof(ProblemEntry) : 0));
    if (mode == kFused || mode == kMass)  // behind the table
      prm.redo_list = reinterpret_cast<int*>(reinterpret_cast<char*>(prm.table) +
                                             (size_t)kMaxPersistentCtas * 2 * (size_t)g.nKb * 128 * sizeof(float2));
  }
  prm.cap_part_rows = (long long)kMaxPersistentCtas * 2 * 128;
  prm.cap_table_floats = (long long)g.nKb * 256;
  prm.cap_mass = (long long)g.B * g.H * g.nQb * g.nKb;
  prm.cap_lse = (long long)g.B * g.H * g.N;
  prm.cap_units = (long long)max_units(g, n_prob);
  prm.scale_log2 = g.scale * kLog2e;
  int rc = LOSA_OK;
  const DeviceState* dev = device_state(&rc);
  if (!dev) return rc;
  prm.status = dev->status_dev;
  const int sms = dev->sm_count;
  // one-shot diagnostic armed by losa_debug_stall_next_launch()
  const uint32_t stall_polls = g_stall_polls.exchange(0u);
  prm.stall = stall_polls > 0u ? 1 : 0;
  prm.wait_polls = stall_polls > 0u ? stall_polls : ptx::kWaitPolls;
  LOSA_CUDA_TRY(cudaMemsetAsync(prm.work_counter, 0, 4 * sizeof(int), st));
  switch (mode) {
    case kDense: return dispatch<kDense>(g, q, k, v, prm, sms, st);
    case kSparse: return dispatch<kSparse>(g, q, k, v, prm, sms, st);
    case kMass: return dispatch<kMass>(g, q, k, v, prm, sms, st);
    case kFused: return dispatch<kFused>(g, q, k, v, prm, sms, st);
  }
  return LOSA_ERR_INVALID_ARG;
}

}  // namespace losa
