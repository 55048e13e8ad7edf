// Dense and block-sparse forward (Eq. 4) and the fused construction step (dense forward plus the
// block masses of Eq. 1) at head dimension 128 with 128-row query blocks, run by PAIRS of CTAs
// (clusters of two, one SM each).  Included by losa_attn.cu, inside its namespace.
//
// A work item is the same pair of consecutive query tiles as in the single-CTA kernel, but each
// CTA of the pair owns ONE of the two tiles, and the two SMs multiply together: every MMA is a
// tcgen05.mma.cta_group::2 over 256 rows (128 per CTA), issued by one thread of the first CTA,
// whose B operand is split between the two CTAs' shared memories - for S = Q K^T each CTA loads 64
// of the tile's 128 keys, for O += P V each loads the 64 head-dimension columns of V that it
// accumulates into.  A K/V tile is thus still fetched once for both query tiles, each SM reads
// 96 B per clock from shared memory instead of 128 (the limit), half as many MMAs are issued, and
// each CTA's tensor memory holds one O (128 columns) and THREE S buffers used in turn, so that the
// chain S -> softmax -> O += P V of one key tile overlaps the chains of the next two.
//
// Per CTA: warp 0 copies (its query tile, its half of every K and V tile), warp 3 of the first CTA
// publishes the tile list into both CTAs' rings, warps 1 and 2 of the first CTA issue every
// S = Q K^T and every O += P V of the pair, and 16 softmax warps turn S into P: two threads per query
// row (64 columns each), key tiles taken alternately by two groups of eight warps, so that each
// group has two tile periods for one tile.  The exponentials are taken against a reference that
// never moves within a work unit (the row maximum over the first key tile the row attends to,
// handed from the group that meets that tile to the other); units whose scores outgrow it are
// listed for the fallback launch, as in the single-CTA kernel.  A key tile that only one of the
// two query tiles lists is multiplied for both and masked to P = 0 for the other.
//
// Barriers that both CTAs feed (operands landed, P written, O read out, tile-list chunk consumed)
// live in the first CTA; barriers that the MMAs' completion feeds in both CTAs are reached with a
// commit to both.  Every wait is bounded; on the way out both CTAs meet at the cluster's barrier,
// so that neither leaves while the other may still signal into its shared memory.

constexpr int kPairNK = 4, kPairNV = 7;      // K and V stages of 16 KB per CTA
constexpr int kPairStage = 16384;
constexpr int kPairQBytes = 32768;

struct PairControl {
  uint64_t q_full, q_empty;
  uint64_t k_full[kPairNK], k_empty[kPairNK];
  uint64_t v_full[kPairNV], v_empty[kPairNV];
  uint64_t s_full[3], p_ready[3], pv_done[3];  // per score buffer
  uint64_t o_done, o_free;
  uint64_t tl_full[kTlChunks], tl_empty[kTlChunks];
  uint64_t pair_bar[8];    // per (group, lane quarter): the two halves of a row
  uint64_t ref_full[2], ref_empty[2];
  uint64_t item_bar;       // all softmax warps of the CTA, at the end of an item
  uint64_t fold_bar;       // ... and after the fused step's masses are folded out of the table
  uint64_t drain;
  alignas(16) uint32_t tl[kTlChunks * 32];  // (read in groups of up to four entries with one vector load)
  float ref[2][128];       // the rows' reference, from the group that met the first tile to the other
  float xch[2][8][128];    // the rows' partial sums at the end of an item (two sets, used in turn):
                           // four of the rounded weights, four of the unrounded exponentials (fused step)
  uint32_t tmem_base;
  int abort_flag;
  int ovf_unit;
};

#define PAIR_WAIT_CL(bar, parity)                                                          \
  do {                                                                                     \
    if (!ptx::mbar_wait_cluster((bar), (parity), &ctl->abort_flag, p.wait_polls)) {        \
      ctl->abort_flag = 1;                                                                 \
      report_error(p.status, LOSA_ERR_TIMEOUT);                                            \
      goto teardown;                                                                       \
    }                                                                                      \
  } while (0)

// The pair kernel's tile list is made of GROUPS of kG = 128 / C entries, each aligned to its size:
// a K/V tile's key blocks, or an item header / end marker followed by filler.  A group is read
// with one vector load (whole warp); a consumed chunk of 32 entries is handed back to the
// scheduler of the first CTA.
#define PAIR_TL_NEXT_TILE(grp, more)                                                       \
  do {                                                                                     \
    const uint32_t c_ = (te >> 5) & (kTlChunks - 1);                                       \
    if ((te & 31) == 0) PAIR_WAIT_CL(&ctl->tl_full[c_], (te / (kTlChunks * 32)) & 1);      \
    ptx::ld_shared_volatile_vec<kG>(&ctl->tl[te & (kTlChunks * 32 - 1)], (grp));           \
    if ((te & 31) == 32 - kG) {                                                            \
      __syncwarp();                                                                        \
      if (lane == 0) ptx::mbar_arrive_cluster(tl_empty0 + 8u * c_);                        \
    }                                                                                      \
    te += kG;                                                                              \
    (more) = ((grp)[0] >> 28) == 0;                                                        \
  } while (0)

// ... the first group of the list or of an item: its header
#define PAIR_TL_NEXT(ent)                                                                  \
  do {                                                                                     \
    uint32_t hdr_[kG];                                                                     \
    bool more_;                                                                            \
    PAIR_TL_NEXT_TILE(hdr_, more_);                                                        \
    (void)more_;                                                                           \
    (ent) = hdr_[0];                                                                       \
  } while (0)

// Scheduler of the first CTA: publish a chunk in both CTAs.
#define PAIR_TL_PUBLISH(chunk)                                                             \
  do {                                                                                     \
    ptx::mbar_arrive(&ctl->tl_full[(chunk)]);                                              \
    ptx::mbar_arrive_cluster(tl_full1 + 8u * (chunk));                                     \
  } while (0)

// ... append n <= 32 entries at once, lane i holding entry i (whole warp)
#define PAIR_TL_PUT_BULK(ent, n)                                                           \
  do {                                                                                     \
    const uint32_t first_ = te, last_ = te + (uint32_t)(n) - 1;                            \
    if ((first_ & 31) == 0)                                                                \
      LOSA_WAIT_RELAXED(&ctl->tl_empty[(first_ >> 5) & (kTlChunks - 1)],                \
                           ((first_ / (kTlChunks * 32)) & 1) ^ 1);                         \
    if ((last_ >> 5) != (first_ >> 5))                                                     \
      LOSA_WAIT_RELAXED(&ctl->tl_empty[(last_ >> 5) & (kTlChunks - 1)],                 \
                           ((last_ / (kTlChunks * 32)) & 1) ^ 1);                          \
    if (lane < (n)) {                                                                      \
      const uint32_t i_ = (first_ + lane) & (kTlChunks * 32 - 1);                          \
      ctl->tl[i_] = (ent);                                                                 \
      ptx::st_cluster_u32(tl1 + 4u * i_, (ent));                                           \
    }                                                                                      \
    ptx::fence_acq_rel_cluster();                                                          \
    __syncwarp();                                                                          \
    if (lane == 0) {                                                                       \
      if ((last_ >> 5) != (first_ >> 5)) PAIR_TL_PUBLISH((first_ >> 5) & (kTlChunks - 1)); \
      if ((last_ & 31) == 31) PAIR_TL_PUBLISH((last_ >> 5) & (kTlChunks - 1));             \
    }                                                                                      \
    te += (uint32_t)(n);                                                                   \
  } while (0)

// ... append an item header or the end marker: a group of its own, filled up with padding entries
#define PAIR_TL_PUT(ent)                                                                   \
  do {                                                                                     \
    const uint32_t e_ = (lane == 0) ? (uint32_t)(ent) : kTlPad;                            \
    PAIR_TL_PUT_BULK(e_, kG);                                                              \
  } while (0)

template <int C_, int MODE>
__global__ void __launch_bounds__(Lay<true>::kThreads, 1)
losa_pair_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_kw,
                 const __grid_constant__ CUtensorMap map_vw, const Params p) {
  using L = Lay<true>;
  constexpr int D = 128, R = 128;
  constexpr int kC = C_, kG = 128 / C_, kW = 128;
  constexpr int kKBox = (C_ < 64) ? C_ : 64;  // key rows per copy of this CTA's half of a K tile
  constexpr int kKCopies = 64 / kKBox;        // ... and copies per 64-column slab
  constexpr uint32_t kIdescQK = ptx::idesc_bf16_f32(256, 128, false, false);
  constexpr uint32_t kIdescPV = ptx::idesc_bf16_f32(256, 128, false, true);
  using Ctl = PairControl;
  constexpr bool kWantMass = (MODE == kFused || MODE == kMass);  // the block masses (Eq. 1) are wanted
  // the mass pass alone has no V, no P and no O: its score buffers go back as soon as they are read
  constexpr bool kHasV = (MODE != kMass);
  static_assert(offsetof(PairControl, tl) % 16 == 0, "the tile list is read with 16-byte loads");

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* const sQ = smem_raw;
  uint8_t* const sK = sQ + kPairQBytes;
  uint8_t* const sV = sK + kPairNK * kPairStage;
  Ctl* const ctl = reinterpret_cast<Ctl*>(sV + kPairNV * kPairStage);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();  // 0: the CTA that issues the MMAs; also the query tile of the pair
  // (the swizzled tiles rely on the declared alignment of the dynamic shared memory)
  const bool misaligned = (ptx::smem_u32(smem_raw) & 1023u) != 0;

  // shared::cluster addresses of the first CTA's barriers that both CTAs arrive on, and of the
  // second CTA's copy of the tile list (used by the first CTA's scheduler)
  const uint32_t q_full0 = ptx::mapa(ptx::smem_u32(&ctl->q_full), 0);
  const uint32_t k_full0 = ptx::mapa(ptx::smem_u32(&ctl->k_full[0]), 0);
  const uint32_t v_full0 = ptx::mapa(ptx::smem_u32(&ctl->v_full[0]), 0);
  const uint32_t p_ready0 = ptx::mapa(ptx::smem_u32(&ctl->p_ready[0]), 0);
  const uint32_t o_free0 = ptx::mapa(ptx::smem_u32(&ctl->o_free), 0);
  const uint32_t tl_empty0 = ptx::mapa(ptx::smem_u32(&ctl->tl_empty[0]), 0);
  const uint32_t tl_full1 = ptx::mapa(ptx::smem_u32(&ctl->tl_full[0]), 1);
  const uint32_t tl1 = ptx::mapa(ptx::smem_u32(&ctl->tl[0]), 1);
  const uint32_t abort_peer = ptx::mapa(ptx::smem_u32(&ctl->abort_flag), rank ^ 1u);

  if (threadIdx.x == 0) {
    ptx::mbar_init(&ctl->q_full, 2);   // one arrival (with its byte count) per CTA's producer
    ptx::mbar_init(&ctl->q_empty, 1);
    for (int i = 0; i < kPairNK; ++i) {
      ptx::mbar_init(&ctl->k_full[i], 2);
      ptx::mbar_init(&ctl->k_empty[i], 1);
    }
    for (int i = 0; i < kPairNV; ++i) {
      ptx::mbar_init(&ctl->v_full[i], 2);
      ptx::mbar_init(&ctl->v_empty[i], 1);
    }
    for (int i = 0; i < 3; ++i) {
      ptx::mbar_init(&ctl->s_full[i], 1);
      ptx::mbar_init(&ctl->p_ready[i], 16);  // the eight warps of a group, in both CTAs
      ptx::mbar_init(&ctl->pv_done[i], 1);
    }
    ptx::mbar_init(&ctl->o_done, 1);
    ptx::mbar_init(&ctl->o_free, 32);  // every softmax warp of both CTAs reads a quarter of its rows' O
    for (int i = 0; i < kTlChunks; ++i) {
      ptx::mbar_init(&ctl->tl_full[i], 1);
      // readers: first CTA producer, two issuers, 16 softmax warps; second CTA producer, 16 softmax warps
      ptx::mbar_init(&ctl->tl_empty[i], 19 + 17);
    }
    for (int i = 0; i < 8; ++i) ptx::mbar_init(&ctl->pair_bar[i], 2);
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&ctl->ref_full[i], 4);   // the first halves' warps of the group that sets it
      ptx::mbar_init(&ctl->ref_empty[i], 8);  // the warps of the other group
    }
    ptx::mbar_init(&ctl->item_bar, 16);
    ptx::mbar_init(&ctl->fold_bar, 16);
    ptx::mbar_init(&ctl->drain, 2);
    ctl->abort_flag = 0;
    ctl->ovf_unit = -1;
    ptx::fence_barrier_init();
  }
  if (warp == kIssuerWarp) {
    // (one warp of each CTA of the pair)
    ptx::tmem_alloc2(&ctl->tmem_base, kTmemCols);
    ptx::tmem_relinquish_alloc_permit2();
  }
  if (warp == kProducerWarp && lane == 0) {
    ptx::prefetch_tensormap(&map_q);
    ptx::prefetch_tensormap(&map_k);
    ptx::prefetch_tensormap(&map_v);
    if (kG > 2) {
      ptx::prefetch_tensormap(&map_kw);
      ptx::prefetch_tensormap(&map_vw);
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();  // both CTAs' barriers are initialised before either signals the other
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;
  {
    // the MMAs address both CTAs' tensor memory with one address
    const uint32_t other = ptx::ld_cluster_u32(ptx::mapa(ptx::smem_u32(&ctl->tmem_base), rank ^ 1u));
    if (misaligned || other != tmem_base) {
      if (threadIdx.x == 0) {
        ctl->abort_flag = 1;
        report_error(p.status, LOSA_ERR_CUDA);
      }
    }
  }
  __syncthreads();

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(L::kRegsUtility));
    if (ctl->abort_flag) goto teardown;
    if (warp == kProducerWarp) {
      // ------------------------------------------------------------------ TMA producer (both CTAs)
      uint32_t nq = 0, nk = 0, nv = 0, te = 0, ent;
      PAIR_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        const int w = (int)(ent & kTlItemMask);
        const int pbh = w / p.nPairs, pr = w % p.nPairs;
        const int bh = pbh % (p.B * p.H);
        const int b = bh / p.H, h = bh % p.H;
        // (map_kw: K in boxes of 64 keys, map_vw: V in boxes of 128 keys, for consecutive key blocks)
        const CUtensorMap *mq = &map_q, *mk = &map_k, *mv = &map_v, *mkw = &map_kw, *mvw = &map_vw;
        if (p.problems != nullptr) {
          const ProblemEntry* pe = p.problems + pbh / (p.B * p.H);
          mq = &pe->map_q;
          mk = &pe->map_kh;
          mv = &pe->map_v;
          mkw = &pe->map_k64;
          mvw = &pe->map_v128;
        }
        // this CTA's query tile (rows past the end of the sequence are filled with zeros)
        const int T = 2 * pr + (int)rank;
        LOSA_WAIT_RELAXED(&ctl->q_empty, (nq & 1) ^ 1);
        if (lane == 0) {
          ptx::mbar_arrive_expect_tx_cluster(q_full0, kPairQBytes);
          ptx::tma_load_4d_pair(sQ, mq, q_full0, 0, T * 128, h, b);
          ptx::tma_load_4d_pair(sQ + 16384, mq, q_full0, 64, T * 128, h, b);
        }
        ++nq;
        for (;;) {
          uint32_t grp[kG];
          bool more;
          PAIR_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          // K: keys 64 * rank ... + 63 of the tile, all 128 head-dimension columns (two slabs)
          const uint32_t ks = nk % kPairNK;
          LOSA_WAIT_RELAXED(&ctl->k_empty[ks], ((nk / kPairNK) & 1) ^ 1);
          if (lane == 0) ptx::mbar_arrive_expect_tx_cluster(k_full0 + 8u * ks, kPairStage);
          __syncwarp();
          // 32-key blocks: this CTA's two key blocks, if consecutive, are one copy per slab
          bool wide_k = false;
          uint32_t first_k = grp[0];
          if constexpr (kKCopies == 2) {
            const uint32_t e0 = (rank == 0) ? grp[0] : grp[kG / 2], e1 = (rank == 0) ? grp[1] : grp[kG / 2 + 1];
            wide_k = (e1 & 0xffffu) == (e0 & 0xffffu) + 1u;
            first_k = e0;
          }
          if (wide_k) {
            if (lane < 2)
              ptx::tma_load_4d_pair(sK + ks * kPairStage + lane * 8192, mkw, k_full0 + 8u * ks, lane * 64,
                                    (int)(first_k & 0xffffu) * kC, h, b);
          } else if (lane < 2 * kKCopies) {
            const int i = lane >> 1, s = lane & 1;
            const int keyoff = 64 * (int)rank + i * kKBox;  // within the tile
            const int g = keyoff / kC, inb = keyoff % kC;
            uint32_t eg = grp[0];
#pragma unroll
            for (int gg = 1; gg < kG; ++gg)
              if (g == gg) eg = grp[gg];
            const int jg = (int)(eg & 0xffffu);
            const int r0 = (jg == (int)kTlPad) ? p.nKb * kC : jg * kC + inb;
            ptx::tma_load_4d_pair(sK + ks * kPairStage + s * 8192 + i * kKBox * 128, mk, k_full0 + 8u * ks,
                                  s * 64, r0, h, b);
          }
          ++nk;
          if (!kHasV) continue;
          // V: all 128 keys of the tile, head-dimension columns 64 * rank ... + 63 (one slab)
          const uint32_t vs = nv % kPairNV;
          LOSA_WAIT_RELAXED(&ctl->v_empty[vs], ((nv / kPairNV) & 1) ^ 1);
          if (lane == 0) ptx::mbar_arrive_expect_tx_cluster(v_full0 + 8u * vs, kPairStage);
          __syncwarp();
          bool wide_v = kG > 2;
#pragma unroll
          for (int gg = 1; gg < kG; ++gg) wide_v = wide_v && (grp[gg] & 0xffffu) == (grp[0] & 0xffffu) + gg;
          if (wide_v) {
            if (lane == 0)
              ptx::tma_load_4d_pair(sV + vs * kPairStage, mvw, v_full0 + 8u * vs, (int)rank * 64,
                                    (int)(grp[0] & 0xffffu) * kC, h, b);
          } else if (lane < kG) {
            uint32_t eg = grp[0];
#pragma unroll
            for (int gg = 1; gg < kG; ++gg)
              if (lane == gg) eg = grp[gg];
            const int jg = (int)(eg & 0xffffu);
            const int r0 = (jg == (int)kTlPad) ? p.nKb * kC : jg * kC;
            ptx::tma_load_4d_pair(sV + vs * kPairStage + lane * kC * 128, mv, v_full0 + 8u * vs,
                                  (int)rank * 64, r0, h, b);
          }
          ++nv;
        }
      }
    } else if (warp == kIssuerWarp && rank == 0) {
      // ------------------------------------------------------------------ S = Q K^T of the pair
      // Score k of the launch goes into buffer k % 3, which holds the P of score k - 3 until the
      // product that reads it has run (pv_done, from the other issuer).
      const bool leader = ptx::elect_one();
      constexpr uint32_t kDescHi = ptx::smem_desc_hi_sw128(1024);
      const uint32_t k_lo = ptx::smem_desc_lo(ptx::smem_u32(sK), 16);
      uint32_t qd[D / 16];
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk)
        qd[kk] = ptx::smem_desc_lo(ptx::smem_u32(sQ), 16) + (((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
      uint32_t nq = 0, nt = 0, te = 0, ent;
      PAIR_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        bool q_ready = false;
        for (;;) {
          uint32_t grp[kG];
          bool more;
          PAIR_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          const uint32_t ks = nt % kPairNK;
          LOSA_WAIT(&ctl->k_full[ks], (nt / kPairNK) & 1);
          if (!q_ready) {
            LOSA_WAIT(&ctl->q_full, nq & 1);
            ++nq;
            q_ready = true;
          }
          const uint32_t bsel = nt % 3u;
          if (nt >= 3u) {
            // (mass pass: the softmax warps of both CTAs hand the buffer back once it is in registers)
            if (kHasV) LOSA_WAIT(&ctl->pv_done[bsel], (nt / 3u - 1u) & 1);
            else LOSA_WAIT(&ctl->p_ready[bsel], (nt / 3u - 1u) & 1);
          }
          ptx::tc_fence_after_sync();
          if (leader) {
            const uint32_t kd0 = k_lo + ks * (kPairStage >> 4);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
              ptx::mma2_ss_lo(tmem_base + bsel * 128, qd[kk], kd0 + (((kk >> 2) * 8192 + (kk & 3) * 32) >> 4),
                              kDescHi, kIdescQK, kk > 0 ? 1u : 0u);
            ptx::mma2_commit_both(&ctl->s_full[bsel]);
            ptx::mma2_commit_both(&ctl->k_empty[ks]);
          }
          ++nt;
        }
        if (!q_ready) {
          // a unit without key tiles: the query tiles were loaded all the same
          LOSA_WAIT(&ctl->q_full, nq & 1);
          ++nq;
        }
        if (leader) ptx::mma2_commit_both(&ctl->q_empty);
      }
    } else if (warp == kIssuerWarp + 1 && rank == 0) {
      // ------------------------------------------------------------------ O += P V of the pair
      const bool leader = ptx::elect_one();
      constexpr uint32_t kDescHi = ptx::smem_desc_hi_sw128(1024);
      const uint32_t v_lo = ptx::smem_desc_lo(ptx::smem_u32(sV), kPairStage);
      const uint32_t tO = tmem_base + 384;
      uint32_t nof = 0, nt = 0, te = 0, ent;
      PAIR_TL_NEXT(ent);
      while ((ent >> 28) == 1) {
        uint32_t pv_item = 0;
        for (;;) {
          uint32_t grp[kG];
          bool more;
          PAIR_TL_NEXT_TILE(grp, more);
          if (!more) {
            ent = grp[0];
            break;
          }
          if (!kHasV) continue;  // (mass pass: this warp only hands the list's chunks back)
          const uint32_t vs = nt % kPairNV;
          LOSA_WAIT(&ctl->v_full[vs], (nt / kPairNV) & 1);
          const uint32_t bsel = nt % 3u;
          if (pv_item == 0 && nof > 0) LOSA_WAIT(&ctl->o_free, (nof - 1) & 1);
          LOSA_WAIT(&ctl->p_ready[bsel], (nt / 3u) & 1);
          ptx::tc_fence_after_sync();
          if (leader) {
            const uint32_t tP = tmem_base + bsel * 128;
            const uint32_t vd0 = v_lo + vs * (kPairStage >> 4);
            // (each half of a row packs its P over the head of its own 64 score columns)
#pragma unroll
            for (int kk = 0; kk < kW / 16; ++kk)
              ptx::mma2_ts_lo(tO, tP + (kk & 3) * 8 + (kk >> 2) * 64, vd0 + kk * (2048 >> 4), kDescHi, kIdescPV,
                              (kk > 0 || pv_item > 0) ? 1u : 0u);
            ptx::mma2_commit(&ctl->pv_done[bsel]);
            ptx::mma2_commit_both(&ctl->v_empty[vs]);
          }
          ++pv_item;
          ++nt;
        }
        if (pv_item > 0) {
          if (leader) ptx::mma2_commit_both(&ctl->o_done);  // every product of the item is done
          ++nof;
        }
      }
    } else if (warp == kSchedulerWarp && rank == 0) {
      // ------------------------------------------------------------------ scheduler of the pair
      uint32_t te = 0;
      for (;;) {
        if (p.stall) break;  // diagnostic launch: nothing is published and every wait runs out
        int w = 0;
        if (lane == 0) w = atomicAdd(p.work_counter, 1);
        w = __shfl_sync(0xffffffffu, w, 0);
        if (w >= p.nUnits) break;
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
        PAIR_TL_PUT(kTlItem | flags | (uint32_t)w);
        if (MODE == kSparse) {
          const int cnt = LOSA_IN_RANGE(unit, p.cap_units) ? min(__ldg(p.tl_count + unit), p.tl_cap) : 0;
          const uint32_t* src = p.tl_entries + (int64_t)unit * p.tl_cap;
          for (int base = 0; base < cnt; base += 32) {
            const int n = min(32, cnt - base);
            const uint32_t e = (lane < n) ? __ldg(src + base + lane) : 0u;
            PAIR_TL_PUT_BULK(e, n);
          }
          continue;
        }
        uint32_t memb = 0;
#pragma unroll
        for (int n = 0; n < 2; ++n)
          if (2 * pr + n < p.nQb) memb |= 1u << n;
        const int jlo = (int)(((int64_t)p.nKb * part) / parts);
        const int jhi = (int)(((int64_t)p.nKb * (part + 1)) / parts);
        const int cnt = (jhi - jlo + kG - 1) / kG * kG;
        for (int base = 0; base < cnt; base += 32) {
          const int n = min(32, cnt - base);
          const int j = jlo + base + lane;
          const uint32_t e = (j < jhi) ? ((uint32_t)j | (memb << 16)) : kTlPad;
          PAIR_TL_PUT_BULK(e, n);
        }
      }
      if (!p.stall) {
        PAIR_TL_PUT(kTlEnd);
        if ((te & 31) != 0) {  // publish the last, partly filled chunk
          __syncwarp();
          if (lane == 0) PAIR_TL_PUBLISH(((te - 1) >> 5) & (kTlChunks - 1));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (both CTAs)
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(L::kRegsSoftmax));
    if (ctl->abort_flag) goto teardown;
    const int sw = warp - 4;
    const int grpi = sw >> 3, half = (sw >> 2) & 1, wl = sw & 3;  // group: which key tiles (even / odd)
    const int row = wl * 32 + lane;
    const uint32_t lane_base = (uint32_t)(wl * 32) << 16;
    const uint32_t tO = tmem_base + lane_base + 384;
    const int my_bit = (int)rank;
    constexpr int kHB = (kG >= 2) ? kG / 2 : 1;  // key blocks of a half (a half block when C = 128)
    constexpr int kBW = 64 / kHB;                // columns per such block
    uint64_t* const pair_bar = &ctl->pair_bar[grpi * 4 + wl];
    const int quarter = grpi * 2 + half;         // which 32 columns of O this thread writes out
    uint32_t kq = 0, nod = 0, npair = 0, nitem = 0, nref = 0, nfold = 0, te = 0, ent;
    // fused step: this row's column of the CTA's table of per-block sums of the unrounded
    // exponentials (one float per row and 64-column half of a key tile when a key block fills the
    // tile, else one per row and key block)
    float* const tabf = kWantMass ? reinterpret_cast<float*>(p.table) +
                                        (int64_t)blockIdx.x * 2 * (int64_t)p.nKb * 256 + row
                                  : nullptr;

    PAIR_TL_NEXT(ent);
    while ((ent >> 28) == 1) {
      const int w = (int)(ent & kTlItemMask);
      const bool partial = (ent & kTlPartial) != 0;
      const int part = (int)((ent >> 24) & 7u);
      const int pbh = w / p.nPairs, pr = w % p.nPairs;
      const int bh = pbh % (p.B * p.H);
      const int b = bh / p.H, h = bh % p.H;
      void* const o_base = (p.problems != nullptr) ? p.problems[pbh / (p.B * p.H)].o : p.o;
      const int T = 2 * pr + (int)rank;
      const int grow = T * 128 + row;
      float m_ref = 0.f, l = 0.f, le = 0.f;  // le: row sum of the unrounded exponentials (masses, LSE)
      // the reference of the item: set by the group that meets the first key tile this query tile
      // lists, taken over by the other group at its own first such tile (or dropped at the item's end)
      bool item_ref = false, have_ref = false, ref_mine = false, ovf = false;
      uint32_t pv_item = 0;
      for (;;) {
        uint32_t grp[kG];
        bool more;
        PAIR_TL_NEXT_TILE(grp, more);
        if (!more) {
          ent = grp[0];
          break;
        }
        bool member = false;
#pragma unroll
        for (int g = 0; g < kG; ++g) member = member || ((grp[g] >> (16 + my_bit)) & 1u);
        const bool first_member = member && !item_ref;
        if (first_member) {
          item_ref = true;
          ref_mine = ((int)(kq & 1u) == grpi);
        }
        const uint32_t bsel = kq % 3u, sph = (kq / 3u) & 1u;
        const bool my_tile = ((int)(kq & 1u) == grpi);
        ++kq;
        ++pv_item;
        if (!my_tile) continue;
        // hv[i]: how many columns of block i of this half the row attends to
        int hv[kHB];
        bool mine = false, whole = true;
#pragma unroll
        for (int i = 0; i < kHB; ++i) {
          const int g = (kG >= 2) ? half * kHB + i : 0;
          const int jg = (int)(grp[g] & 0xffffu);
          const int valid = ((grp[g] >> (16 + my_bit)) & 1u) ? min(kC, p.N - jg * kC) : 0;
          hv[i] = (kG >= 2) ? valid : max(0, min(64, valid - 64 * half));
          mine = mine || hv[i] > 0;
          whole = whole && hv[i] == kBW;
        }
        const uint32_t tSrow = tmem_base + lane_base + bsel * 128;
        const uint32_t tS = tSrow + half * 64;
        LOSA_WAIT(&ctl->s_full[bsel], sph);
        ptx::tc_fence_after_sync();
        if (member && !have_ref) {
          const uint32_t rs = nref & 1u;
          if (first_member) {
            // the row's maximum over the keys it attends to in this tile, computed by both halves
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
            // the other half reads the whole row too: nobody packs P over it before both are done
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(pair_bar);
            LOSA_WAIT(pair_bar, npair & 1);
            ++npair;
            ptx::tc_fence_after_sync();
            if (half == 0) {
              // (the slot's last readers, two items with a reference ago, are done with it)
              if (nref >= 2u) LOSA_WAIT(&ctl->ref_empty[rs], ((nref >> 1) - 1u) & 1);
              ctl->ref[rs][row] = m_ref;
              __syncwarp();
              if (lane == 0) ptx::mbar_arrive(&ctl->ref_full[rs]);
            }
          } else {
            LOSA_WAIT(&ctl->ref_full[rs], (nref >> 1) & 1);
            m_ref = ctl->ref[rs][row];
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->ref_empty[rs]);
          }
          have_ref = true;
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
          if (!kHasV) {
            // mass pass: the scores are in registers and nothing is packed over them
            ptx::tmem_wait_ld();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(p_ready0 + 8u * bsel);
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
            if (kHasV && whole && c == 32) ptx::tmem_wait_ld();
            float2 x0 = ptx::fma2(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sc2,
                                  nm2[c / kBW]);
            float2 x1 = ptx::fma2(make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sc2,
                                  nm2[c / kBW]);
            // (a share of these on the FMA pipe, as at head dimension 64, measured -1 % at 12.5 %
            // and +5 % at 25 % here: none)
            x0.x = ptx::ex2_approx(x0.x);
            x0.y = ptx::ex2_approx(x0.y);
            x1.x = ptx::ex2_approx(x1.x);
            x1.y = ptx::ex2_approx(x1.y);
            if (kHasV) {
              const uint32_t u0 = ptx::pack_bf16x2(x0.x, x0.y), u1 = ptx::pack_bf16x2(x1.x, x1.y);
              sr[c >> 1] = u0;
              sr[(c >> 1) + 1] = u1;
              ptx::add_bf16x2(racc[0], u0);
              ptx::add_bf16x2(racc[1], u1);
            }
            if (kWantMass) eacc[c / kBW] = ptx::add2(eacc[c / kBW], ptx::add2(x0, x1));
          }
          float tsum = (racc[0].x + racc[0].y) + (racc[1].x + racc[1].y);
          if (!kHasV) {
#pragma unroll
            for (int i = 0; i < kHB; ++i) tsum += eacc[i].x + eacc[i].y;
          }
          ovf = ovf || __any_sync(0xffffffffu, !(tsum <= kSplitSafeSum));
          l += tsum;
          if (kHasV) ptx::tmem_st32(tS, &sr[0]);
          if (kWantMass) {
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
          if (kHasV) {
            uint32_t z[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) z[c] = 0u;
            ptx::tmem_st32(tS, z);
          } else {
            // mass pass: the buffer goes back untouched
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(p_ready0 + 8u * bsel);
          }
          // (a key block that fills the tile but ends before this half: its entry of the table is 0)
          if (kWantMass && kG == 1 && member &&
              LOSA_IN_RANGE(((int64_t)(grp[0] & 0xffffu) * 2 + half) * 128 + row, p.cap_table_floats))
            tabf[((int64_t)(grp[0] & 0xffffu) * 2 + half) * 128] = 0.f;
        }
        if (kHasV) {
          ptx::tmem_wait_st();
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(p_ready0 + 8u * bsel);
        }
      }

      // ---- end of the item
      if (item_ref) {
        if (!ref_mine && !have_ref) {
          // this group met none of the tiles the query tile lists: it takes the reference here
          // (a partial unit records it) and hands the slot back
          const uint32_t rs = nref & 1u;
          LOSA_WAIT(&ctl->ref_full[rs], (nref >> 1) & 1);
          m_ref = ctl->ref[rs][row];
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl->ref_empty[rs]);
        }
        ++nref;
      }
      // the four partial sums of a row (two groups, two halves) meet in shared memory
      float* const xset = &ctl->xch[nitem & 1][0][0];
      xset[quarter * 128 + row] = l;
      if (kWantMass) xset[(4 + quarter) * 128 + row] = le;
      if (ovf && lane == 0) {
        const int unit = partial ? p.split_first + (w - p.split_first) * p.split_parts + part : w;
        if (atomicExch(&ctl->ovf_unit, unit) != unit) {
          const int slot = atomicAdd(p.redo_count, 1);
          if (slot < 2 * p.nUnits) p.redo_list[slot] = unit;  // (each CTA of the pair may list it)
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&ctl->item_bar);
      LOSA_WAIT(&ctl->item_bar, nitem & 1);
      ++nitem;
      l = (xset[row] + xset[128 + row]) + (xset[256 + row] + xset[384 + row]);
      if (kHasV) {
        // every thread writes out a quarter (32 columns) of its row of O
        const bool valid = (T < p.nQt) && grow < p.N;
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
        const int64_t off = (int64_t)b * p.sb + (int64_t)h * p.sh + (int64_t)grow * p.sn;
        const int64_t pslot = ((((int64_t)(w - p.split_first) * p.split_parts + part) * 2 + (int)rank) * 128 + row);
        if (partial && quarter == 0 && T < p.nQt && LOSA_IN_RANGE(pslot, p.cap_part_rows)) p.part_ml[pslot] = make_float2(m_ref, l);
        const int c0 = quarter * 32;
        uint32_t r[32];
        if (pv_item > 0) {
          LOSA_WAIT(&ctl->o_done, nod & 1);
          ++nod;
          ptx::tc_fence_after_sync();
          ptx::tmem_ld32(tO + c0, r);
          ptx::tmem_wait_ld();
          // (O is in registers: the next item's first product may overwrite it)
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(o_free0);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) r[c] = 0u;
        }
        if (partial) {
          if (T < p.nQt) {
            float4* dst = reinterpret_cast<float4*>(p.part_o + (LOSA_IN_RANGE(pslot, p.cap_part_rows) ? pslot : 0) * D + c0);
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              dst[c >> 2] = make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                        __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
          }
        } else if (valid) {
          if (p.o_f32) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(o_base) + off + c0);
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              dst[c >> 2] = make_float4(__uint_as_float(r[c]) * inv, __uint_as_float(r[c + 1]) * inv,
                                        __uint_as_float(r[c + 2]) * inv, __uint_as_float(r[c + 3]) * inv);
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
      if (kWantMass) {
        // ---- fused construction step: the block masses of this CTA's query tile (Eq. 1).  The
        // reference did not move during the item, so a row's weight is 1 / (its sum of unrounded
        // exponentials) and a mass is the mean over the query block's rows of weight x (the row's
        // sum over the key block).  The table was written by this CTA's softmax threads before the
        // item's barrier; all 16 warps fold it, key block by key block.
        if (quarter == 0 && T < p.nQt && grow < p.N && p.lse != nullptr &&
            LOSA_IN_RANGE((int64_t)bh * p.N + grow, p.cap_lse)) {
          const float le_row = (xset[512 + row] + xset[640 + row]) + (xset[768 + row] + xset[896 + row]);
          p.lse[(int64_t)bh * p.N + grow] = (m_ref + log2f(le_row)) * kLn2;
        }
        if (T < p.nQt) {
          const float* tb = reinterpret_cast<const float*>(p.table) + (int64_t)blockIdx.x * 2 * (int64_t)p.nKb * 256;
          float iv[4];  // this lane's four rows
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) {
            const int r = rr * 32 + lane;
            const float le_r = (xset[512 + r] + xset[640 + r]) + (xset[768 + r] + xset[896 + r]);
            iv[rr] = (T * 128 + r < p.N && le_r > 0.f) ? 1.f / le_r : 0.f;
          }
          const int nvalid = min(R, p.N - T * R);
          for (int u = sw; u < p.nKb; u += 16) {
            float acc = 0.f;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
              const int r = rr * 32 + lane;
              if (iv[rr] > 0.f) {
                const float sum = (kG >= 2) ? tb[(int64_t)u * 128 + r]
                                            : tb[(int64_t)u * 256 + r] + tb[(int64_t)u * 256 + 128 + r];
                acc += sum * iv[rr];
              }
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
            const int64_t mi = ((int64_t)bh * p.nQb + T) * p.nKb + u;
            if (lane == 0 && LOSA_IN_RANGE(mi, p.cap_mass)) p.mass[mi] = acc / (float)nvalid;
          }
        }
        // (the table is written again by the next item)
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl->fold_bar);
        LOSA_WAIT(&ctl->fold_bar, nfold & 1);
        ++nfold;
      }
    }
  }

teardown:
  if (ctl->abort_flag) {
    // the other CTA's waits give up at their next look at the flag
    if (lane == 0) ptx::st_cluster_u32(abort_peer, 1u);
    // give MMAs and bulk copies still in flight a bounded time to land before shared memory and
    // tensor memory are released
    if (rank == 0 && (warp == kIssuerWarp || warp == kIssuerWarp + 1) && ptx::elect_one()) {
      ptx::mma2_commit(&ctl->drain);
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
  // neither CTA leaves, or frees its tensor memory, while the other may still signal into it
  ptx::cluster_sync();
  if (warp == kIssuerWarp) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc2(tmem_base, kTmemCols);
  }
}

#undef PAIR_TL_PUT
#undef PAIR_TL_PUT_BULK
#undef PAIR_TL_PUBLISH
#undef PAIR_TL_NEXT_TILE
#undef PAIR_TL_NEXT
#undef PAIR_WAIT_CL
