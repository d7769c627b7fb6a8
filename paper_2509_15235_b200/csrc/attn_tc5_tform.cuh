// Transposed form of the TMA + tcgen05 attention kernel, for units of at most 64 query rows (G*N <= 64: the
// multi-head workloads).  Included by attn_tc5.cu (same helpers, schedule and parameters).
//
// A 128-lane tensor-core product wastes half its height on 64 rows, so here the roles of rows and tokens are
// swapped: S^T = K Q^T puts the step's 128 tokens on the TMEM lanes and the 64 rows on the columns (N = 64:
// half the instruction time), and O^T = V^T P^T accumulates [128 head-dim lanes x 64 row columns].  Both
// products take both operands from shared memory: K and V stages as they come from TMA (V^T is the V stage
// read MN-major), Q as a 64-row K-major tile, and P^T (bf16) written by the softmax threads into a swizzled
// [token][row] tile.
//
// Softmax without row reductions.  A thread owns one token (lane) and 32 of the 64 rows (columns), so a row's
// maximum and sum would cross lanes.  Instead every row keeps a reference m_ref: P = exp2(scale*s - m_ref) is
// elementwise, and each thread adds its own P values into 32 private partial sums that are reduced over the
// lanes once per segment.  The reference only has to be within 2^60 above the true maximum's neighbourhood to
// be exact in fp32/bf16 arithmetic (both share the 8-bit exponent), so it moves rarely: a thread that meets an
// allowed score more than 2^60 above the reference raises a flag; all softmax threads meet once per step
// (off the critical path, behind the exponentials) and, if the flag is up, take the slow path together: row
// maxima of the tile by shuffles and shared memory, new reference, O^T and the partial sums rescaled, the
// step's P recomputed.  The first step of a segment always takes it, which anchors the reference at a true
// tile maximum (so nothing that matters can underflow).
//
// Roles (12 warps) and barriers follow the row-major kernel: producer (K ring 3 stages, V ring 2), S^T issuer,
// PV issuer, schedule warp, 8 softmax warps (warps w and w+4 share the 32 lanes of a TMEM quarter and split
// the 64 row columns).  Epilogue: O^T goes through shared memory as [row][128] fp32 (the P tiles are idle by
// then), from where it is written out, parked as a partial, or pulled by the cluster peers.

constexpr int T_NSK = 3, T_NSV = 2;
constexpr int T_ROWS = 64;                                      // rows of a unit (the N of both products)
constexpr int T_Q_HALF = T_ROWS * 128;                          // one d-half of the Q tile
constexpr int T_P_BYTES = STEP * 128;                           // one P^T tile: 128 tokens x 64 rows bf16
constexpr int T_SMEM_K = 0;
constexpr int T_SMEM_V = T_SMEM_K + T_NSK * STAGE_BYTES;
constexpr int T_SMEM_Q = T_SMEM_V + T_NSV * STAGE_BYTES;
constexpr int T_SMEM_P = T_SMEM_Q + 2 * T_Q_HALF;               // two P^T tiles; in the epilogue [64 rows][128] fp32
constexpr int T_SMEM_CM = T_SMEM_P + 2 * T_P_BYTES;             // 128 x uint64: rows that may see tree token t
constexpr int T_SMEM_RM = T_SMEM_CM + 1024;                     // 64 x 2 x uint64 row masks (staging)
constexpr int T_SMEM_RED = T_SMEM_RM + 1024;                    // [2][4][32] floats: per-warp row maxima / sums
constexpr int T_SMEM_STAT = T_SMEM_RED + 1024;                  // 64 x float2 (m, l) of the segment
constexpr int T_SMEM_FLAG = T_SMEM_STAT + 512;                  // 2 ints: step index + 1 of the last raised flag
constexpr int T_SMEM_BAR = T_SMEM_FLAG + 64;
constexpr int T_SMEM_SCHED = T_SMEM_BAR + BAR_BYTES;
constexpr int T_SMEM_TOTAL = T_SMEM_SCHED + (int)sizeof(Sched);
static_assert(T_SMEM_TOTAL <= 232448, "over the 227 KB a CTA may have");
constexpr uint32_t T_TMEM_COLS = 256;
constexpr uint32_t T_COL_S = 0, T_COL_O = 128;                  // S^T[0] 0..63, S^T[1] 64..127, O^T 128..191
constexpr float kGapT = 60.0f;                                  // log2 units an allowed score may exceed the reference by

enum { TB_KFULL = 0, TB_KEMPTY = TB_KFULL + T_NSK, TB_VFULL = TB_KEMPTY + T_NSK, TB_VEMPTY = TB_VFULL + T_NSV,
       TB_SFULL = TB_VEMPTY + T_NSV, TB_SFREE = TB_SFULL + 2, TB_PFULL = TB_SFREE + 2, TB_PVDONE = TB_PFULL + 2,
       TB_QFULL = TB_PVDONE + 2, TB_ALLX = TB_QFULL + 1, TB_GRP = TB_ALLX + 1, TB_COUNT = TB_GRP + 2 };
static_assert(TB_COUNT * 8 + 16 <= BAR_BYTES, "barrier block too small");

// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 128, N = 64; a_mn / b_mn = 1 for MN-major operands.
__host__ __device__ constexpr uint32_t instr_desc_t(int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((64u >> 3) << 17) | ((128u >> 4) << 24);
}

template <bool CL>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc5t_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const Tc5Params p) {
    extern __shared__ __align__(1024) unsigned char sm[];
    TRACE_MISC(0);
    TL_START(p.trace_idx, 0);
    CTA_T(0);
    const uint32_t base = smem_u32(sm);
    if (base & 1023u) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)VISPEC_E_UNSUPPORTED);
        return;
    }
    const uint32_t bars = base + T_SMEM_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + T_SMEM_BAR + TB_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + T_SMEM_BAR + TB_COUNT * 8 + 8);
    Sched& sched = *reinterpret_cast<Sched*>(sm + T_SMEM_SCHED);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int G = p.Hq / p.Hkv, N = p.N, W = (N + 63) >> 6;
    const int rows_total = G * N;                          // <= 64

    if (tid == 0) {
        for (int i = 0; i < T_NSK; ++i) { mbar_init(bar(TB_KFULL + i), 1); mbar_init(bar(TB_KEMPTY + i), 1); }
        for (int i = 0; i < T_NSV; ++i) { mbar_init(bar(TB_VFULL + i), 1); mbar_init(bar(TB_VEMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            // (the softmax warps arrive once per warp: lane 0, after the warp has met)
            mbar_init(bar(TB_SFULL + i), 1); mbar_init(bar(TB_SFREE + i), kSmx / 32);
            mbar_init(bar(TB_PFULL + i), kSmx / 32); mbar_init(bar(TB_PVDONE + i), 1);
            mbar_init(bar(TB_GRP + i), 4);
        }
        mbar_init(bar(TB_QFULL), kSmx / 32);
        mbar_init(bar(TB_ALLX), kSmx / 32);
        *abort_flag = 0;
        reinterpret_cast<volatile int*>(sm + T_SMEM_FLAG)[0] = 0;
        reinterpret_cast<volatile int*>(sm + T_SMEM_FLAG)[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(T_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == 3) sched_build(sched, p, lane);
    pdl_launch_dependents();
    if (!p.early) pdl_wait();
    TRACE_MISC(1);
    tc_fence_before();
    __syncthreads();
    if (CL) cluster_sync_all();          // every CTA is up before a peer can read its shared memory
    tc_fence_after();
    TRACE_MISC(2);

    const int T = sched.base[p.B];
    const int geff = CL ? (int)gridDim.x : (T > 0 ? sched_ctas(T, sched.units, (int)gridDim.x, p.min_steps) : 0);
    const bool active = cta < geff;
    const int lo = (!CL && active) ? cta_lo(cta, T, geff) : 0, hi = (!CL && active) ? cta_lo(cta + 1, T, geff) : 0;
    const uint32_t tmem = *tmem_slot;
    const int ck = CL ? (int)cluster_size() : 1, cr = CL ? (int)cluster_ctarank() : 0;
    Seg cl_seg = {};
    if (CL) {
        const int upb = p.Hkv * p.n_mblocks;
        const int unit = cta / ck, b = unit / upb, uib = unit - b * upb;
        cl_seg.b = b; cl_seg.kvh = uib / p.n_mblocks; cl_seg.mblock = uib - cl_seg.kvh * p.n_mblocks;
        cl_seg.steps = sched.steps[b]; cl_seg.S = sched.len[b];
        cl_seg.st0 = (cr * cl_seg.steps) / ck;
        cl_seg.n = ((cr + 1) * cl_seg.steps) / ck - cl_seg.st0;
        cl_seg.slot = -1;
    }
    auto make_iter = [&]() {
        SegIter it; it.s = &sched; it.B = p.B; it.n_mblocks = p.n_mblocks; it.g = lo; it.lo = lo; it.hi = hi; it.cta = cta;
        it.cl = CL; it.cl_done = false; it.cl_seg = cl_seg;
        return it;
    };

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0 && active) {
            const uint64_t pol = l2_evict_first_policy();
            bool waited = !p.early;
            int it = 0, nk = 0, nv = 0;
            bool ok = true;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                const int bh = sg.b * p.Hkv + sg.kvh;
                for (int t = 0; t < sg.n; ++t, ++it) {
                    const int tok = (sg.st0 + t) * STEP;
                    if (!waited && tok + STEP > sg.S) { pdl_wait(); waited = true; }   // the tree's rows come from the preceding kernel
                    const int sk = it % T_NSK, sv = it % T_NSV;
                    if (!mbar_wait(bar(TB_KEMPTY + sk), ((it / T_NSK) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(bar(TB_KFULL + sk), STAGE_BYTES);
                    tma_load_3d(base + T_SMEM_K + sk * STAGE_BYTES, &k_map, bar(TB_KFULL + sk), 0, tok, bh, pol);
                    tma_load_3d(base + T_SMEM_K + sk * STAGE_BYTES + HALF_BYTES, &k_map, bar(TB_KFULL + sk), 64, tok, bh, pol);
                    ++nk;
                    if (!mbar_wait(bar(TB_VEMPTY + sv), ((it / T_NSV) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(bar(TB_VFULL + sv), STAGE_BYTES);
                    tma_load_3d(base + T_SMEM_V + sv * STAGE_BYTES, &v_map, bar(TB_VFULL + sv), 0, tok, bh, pol);
                    tma_load_3d(base + T_SMEM_V + sv * STAGE_BYTES + HALF_BYTES, &v_map, bar(TB_VFULL + sv), 64, tok, bh, pol);
                    ++nv;
                }
            }
            if (*abort_flag) {
                volatile int never = 0;
                for (int u = max(0, nk - T_NSK); u < nk; ++u) mbar_wait(bar(TB_KFULL + u % T_NSK), (u / T_NSK) & 1, &never);
                for (int u = max(0, nv - T_NSV); u < nv; ++u) mbar_wait(bar(TB_VFULL + u % T_NSV), (u / T_NSV) & 1, &never);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= issuer of S^T = K Q^T (A = K stage, B = Q tile, both K-major) =================
        if (lane == 0 && active) {
            constexpr uint32_t IDESC = instr_desc_t(0, 0);
            constexpr uint32_t DESC_HI = desc_hi(1024);
            bool ok = true;
            int it = 0, seg = 0;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                if (!mbar_wait(bar(TB_QFULL), seg & 1, abort_flag)) { ok = false; break; }
                for (int t = 0; t < sg.n && ok; ++t, ++it) {
                    const int bs = it & 1, sk = it % T_NSK;
                    TRACE(1, it, 0);
                    if (!mbar_wait(bar(TB_KFULL + sk), (it / T_NSK) & 1, abort_flag)) { ok = false; break; }
                    TRACE(1, it, 1);
                    if (it >= 2 && !mbar_wait(bar(TB_SFREE + bs), ((it >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t kb = desc_lo(base + T_SMEM_K + sk * STAGE_BYTES, 16);
                    const uint32_t qb = desc_lo(base + T_SMEM_Q, 16);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {       // 16 d-columns per instruction
                        const uint32_t koff = ((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4;
                        const uint32_t qoff = ((ks >> 2) * T_Q_HALF + (ks & 3) * 32) >> 4;
                        tc_mma_ss(tmem + T_COL_S + bs * 64, kb + koff, DESC_HI, qb + qoff, DESC_HI, IDESC, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(TB_KEMPTY + sk));
                    tc_commit(bar(TB_SFULL + bs));
                    TRACE(1, it, 2);
                }
                ++seg;
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ================= issuer of O^T += V^T P^T (A = V stage read MN-major, B = P^T tile MN-major) =================
        if (lane == 0 && active) {
            constexpr uint32_t IDESC = instr_desc_t(1, 1);
            constexpr uint32_t DESC_HI = desc_hi(1024);
            bool ok = true;
            int u = 0;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                for (int t = 0; t < sg.n; ++t, ++u) {
                    const int bu = u & 1, sv = u % T_NSV;
                    TRACE(1, u, 3);
                    if (!mbar_wait(bar(TB_PFULL + bu), (u >> 1) & 1, abort_flag)) { ok = false; break; }
                    TRACE(1, u, 4);
                    if (!mbar_wait(bar(TB_VFULL + sv), (u / T_NSV) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t vb = desc_lo(base + T_SMEM_V + sv * STAGE_BYTES, HALF_BYTES);
                    const uint32_t pb = desc_lo(base + T_SMEM_P + bu * T_P_BYTES, 16);
#pragma unroll
                    for (int ks = 0; ks < STEP / 16; ++ks)      // 16 tokens per instruction: 2 KB of the V stage and of P^T
                        tc_mma_ss(tmem + T_COL_O, vb + ks * 128, DESC_HI, pb + ks * 128, DESC_HI, IDESC,
                                  (t > 0 || ks > 0) ? 1u : 0u);   // the first product of a segment starts a fresh O^T
                    tc_commit(bar(TB_VEMPTY + sv));
                    tc_commit(bar(TB_PVDONE + bu));
                    TRACE(1, u, 6);
                }
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ================= softmax: thread <-> (token of the step, 32 of the 64 rows) =================
        const int sp = warp & 3;                              // TMEM lane quarter
        const int ch = (warp - 4) >> 2;                       // which 32 rows (columns of S^T and O^T)
        const int tl = sp * 32 + lane;                        // TMEM lane: token of a step / head-dim index of O^T
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sp) << 16);
        const int st = tid - 128;                             // 0..255
        uint64_t* colmask = reinterpret_cast<uint64_t*>(sm + T_SMEM_CM);
        uint64_t* rowmask = reinterpret_cast<uint64_t*>(sm + T_SMEM_RM);
        float* red = reinterpret_cast<float*>(sm + T_SMEM_RED) + ch * 128;      // this group's [4 warps][32 rows]
        float2* stat = reinterpret_cast<float2*>(sm + T_SMEM_STAT);
        volatile int* flagv = reinterpret_cast<volatile int*>(sm + T_SMEM_FLAG);
        float* pbuf = reinterpret_cast<float*>(sm + T_SMEM_P);                    // epilogue: [64 rows][128]
        int ax = 0, gx = 0;                                   // phases used of the all-softmax and the group barrier
        // One arrival per warp: 256 threads arriving one by one on the same barrier word would serialise.
        auto warp_arrive = [&](uint32_t b) {
            __syncwarp();
            if (lane == 0) mbar_arrive(b);
        };
        auto all_sync = [&]() -> bool {
            warp_arrive(bar(TB_ALLX));
            const bool r = mbar_wait_warp(bar(TB_ALLX), ax & 1, abort_flag);
            ++ax;
            return r;
        };
        auto grp_sync = [&]() -> bool {                       // the 128 threads that share this thread's rows
            warp_arrive(bar(TB_GRP + ch));
            const bool r = mbar_wait_warp(bar(TB_GRP + ch), gx & 1, abort_flag);
            ++gx;
            return r;
        };
        pdl_wait();                                           // q, tree_mask and every output come after the preceding kernel
        TRACE_MISC(4);

        // rejected sequences (kv_len < 0 or kv_len + N > S_max): zero output, -inf lse, status word
        {
            bool any_bad = false;
            for (int b = 0; b < p.B; ++b) {
                const int S = sched.len[b];
                if (S >= 0 && S + N <= p.S_max) continue;
                any_bad = true;
                const int vecs = N * p.Hq * (D / 8);
                uint4* o = reinterpret_cast<uint4*>(p.out + (size_t)b * N * p.Hq * D);
                for (int i = cta * kSmx + st; i < vecs; i += (int)gridDim.x * kSmx) o[i] = make_uint4(0, 0, 0, 0);
                if (p.lse)
                    for (int i = cta * kSmx + st; i < N * p.Hq; i += (int)gridDim.x * kSmx) p.lse[(size_t)b * p.Hq * N + i] = -INFINITY;
            }
            if (any_bad && cta == 0 && st == 0) atomicCAS(p.status, 0, (int)VISPEC_E_RANGE);
        }

        if (active) {
            SegIter si = make_iter();
            Seg sg;
            int it = 0, seg = 0;
            bool ok = true;
            while (ok && si.next(sg)) {
                const int S = sg.S, total = S + N;
                // ---- segment set-up: Q tile (64 rows, K-major, swizzled like a K stage) and the row masks ----
                {
                    const int qc = st & 15;
                    uint4 v[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int row = (st >> 4) + 16 * k;
                        v[k] = make_uint4(0, 0, 0, 0);
                        if (row < rows_total) {
                            const int node = row / G, head = sg.kvh * G + row % G;
                            v[k] = *(reinterpret_cast<const uint4*>(p.q + (((size_t)sg.b * N + node) * p.Hq + head) * D) + qc);
                        }
                    }
                    uint64_t m0 = 0, m1 = 0;
                    if (st < T_ROWS && st < rows_total) {
                        const uint64_t* mrow = p.mask + ((size_t)sg.b * N + st / G) * W;
                        m0 = mrow[0];
                        if (W > 1) m1 = mrow[1];
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int r = (st >> 4) + 16 * k;
                        *reinterpret_cast<uint4*>(sm + T_SMEM_Q + (qc >> 3) * T_Q_HALF + r * 128 + (((qc & 7) ^ (r & 7)) << 4)) = v[k];
                    }
                    if (st < T_ROWS) { rowmask[2 * st] = m0; rowmask[2 * st + 1] = m1; }
                    fence_async_smem();
                    warp_arrive(bar(TB_QFULL));
                    if (!all_sync()) { ok = false; break; }
                    // tree token t may be seen by the rows whose mask has bit t (bits at or beyond N are no tokens)
                    if (st < 128) {
                        uint64_t cm = 0;
                        if (st < N) {
#pragma unroll 8
                            for (int r = 0; r < T_ROWS; ++r)
                                cm |= ((rowmask[2 * r + (st >> 6)] >> (st & 63)) & 1ull) << r;
                        }
                        colmask[st] = cm;
                    }
                    if (!all_sync()) { ok = false; break; }
                }
                TRACE_MISC(3);
                float mref[32], lsum[32];
#pragma unroll
                for (int r = 0; r < 32; ++r) { mref[r] = -INFINITY; lsum[r] = 0.f; }

                uint32_t anch = 0;                                     // rows whose reference is a real score bound
                for (int t = 0; t < sg.n; ++t, ++it) {
                    const int bs = it & 1;
                    const int tok0 = (sg.st0 + t) * STEP;
                    const int j = tok0 + tl;                                 // this thread's token
                    if (tid == 128) TRACE(2, it, 0);
                    if (!mbar_wait_warp(bar(TB_SFULL + bs), (it >> 1) & 1, abort_flag)) { ok = false; break; }
                    if (tid == 128) TRACE(2, it, 1);
                    tc_fence_after();
                    float x[32];                                             // scale * s, then shifted by the references
                    {
                        uint32_t sraw[32];
                        tmem_ld32(lane_addr + T_COL_S + bs * 64 + ch * 32, sraw);
                        tmem_wait_ld();
#pragma unroll
                        for (int r = 0; r < 32; ++r) x[r] = __uint_as_float(sraw[r]) * p.scale_log2;
                    }
                    // S^T[bs] may be overwritten by the product of step it+2
                    tc_fence_before();
                    warp_arrive(bar(TB_SFREE + bs));
                    // rows that may attend to this token (a token of the committed prefix is seen by every row)
                    uint32_t am = 0xffffffffu;
                    if (tok0 + STEP > S) am = j < S ? 0xffffffffu : (j < total ? (uint32_t)(colmask[j - S] >> (32 * ch)) : 0u);
                    const bool all_rows = __all_sync(0xffffffffu, am == 0xffffffffu);
                    if (t == 0) {
                        // First step of a segment: anchor every row's reference at its score against the step's first
                        // token when that token belongs to the committed prefix (every row sees it, so the row sum is
                        // at least 1 and nothing that matters can underflow); otherwise the slow path below finds the
                        // tile's row maxima.
                        const bool anchored = tok0 < S;
                        if (anchored && tl == 0) {
#pragma unroll
                            for (int r = 0; r < 32; ++r) red[r] = x[r];
                        }
                        if (!all_sync()) { ok = false; break; }
                        if (anchored) {
#pragma unroll
                            for (int r = 0; r < 32; ++r) mref[r] = red[r];
                            anch = 0xffffffffu;
                        } else {
#pragma unroll
                            for (int r = 0; r < 32; ++r) mref[r] = 0.f;         // provisional
                            anch = 0u;
                        }
                    }
                    // shifted scores; does an allowed one overshoot its reference, or meet a provisional one?
                    float xmax;
                    {
                        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        if (all_rows) {
#pragma unroll
                            for (int r = 0; r < 32; ++r) { x[r] -= mref[r]; mx[r & 3] = fmaxf(mx[r & 3], x[r]); }
                        } else {
#pragma unroll
                            for (int r = 0; r < 32; ++r) {
                                x[r] = ((am >> r) & 1u) ? x[r] - mref[r] : -INFINITY;        // exp2(-inf) = 0
                                mx[r & 3] = fmaxf(mx[r & 3], x[r]);
                            }
                        }
                        xmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                    }
                    if (xmax > kGapT || (am & ~anch) != 0u) flagv[bs] = it + 1;
                    if (tid == 128) TRACE(2, it, 2);
                    warp_arrive(bar(TB_ALLX));
                    // exponentials against the current references (thrown away if the flag turns out to be up)
                    float e[32];
                    uint32_t pd[16];
#pragma unroll
                    for (int r = 0; r < 32; ++r) e[r] = exp2f(x[r]);
#pragma unroll
                    for (int c = 0; c < 16; ++c) pd[c] = pack_bf16(e[2 * c], e[2 * c + 1]);
                    if (tid == 128) TRACE(2, it, 3);
                    // P^T[bs] is free once the PV product of step it-2 has completed
                    if (it >= 2) {
                        if (!mbar_wait_warp(bar(TB_PVDONE + bs), ((it >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    }
                    unsigned char* prow = sm + T_SMEM_P + bs * T_P_BYTES + tl * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4*>(prow + (((ch * 4 + c) ^ (tl & 7)) << 4)) = make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
                    bool fail = false;
                    if (tok0 + STEP > total) {
                        // last step of the sequence: V rows past the last key may hold anything and meet weight-0
                        // entries of P^T in the product: clear them (thread r of the first 128 clears row r)
                        const int sv = it % T_NSV;
                        fail = !mbar_wait(bar(TB_VFULL + sv), (it / T_NSV) & 1, abort_flag);
                        if (!fail && ch == 0 && j >= total) {
                            unsigned char* vrow = sm + T_SMEM_V + sv * STAGE_BYTES + tl * 128;
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                                *reinterpret_cast<uint4*>(vrow + HALF_BYTES + c * 16) = make_uint4(0, 0, 0, 0);
                            }
                        }
                    }
                    if (__any_sync(0xffffffffu, fail)) { ok = false; break; }
                    if (tid == 128) TRACE(2, it, 4);
                    // has anybody raised the flag for this step?
                    if (!mbar_wait_warp(bar(TB_ALLX), ax & 1, abort_flag)) { ok = false; break; }
                    ++ax;
                    if (tid == 128) TRACE(2, it, 5);
                    if (flagv[bs] == it + 1) {
                        // ---- slow path, all softmax threads together: row maxima of this tile, new references,
                        // O^T and the partial sums rescaled, P recomputed.  The references are finite here, so the
                        // scaled scores come back as x + m_ref. ----
                        float y[32];
#pragma unroll
                        for (int r = 0; r < 32; ++r) {
                            y[r] = ((am >> r) & 1u) ? x[r] + mref[r] : -INFINITY;
                            float v = y[r];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
                            if (lane == r) red[sp * 32 + r] = v;
                        }
                        if (!grp_sync()) { ok = false; break; }
                        float alpha[32];
#pragma unroll
                        for (int r = 0; r < 32; ++r) {
                            const float tm = fmaxf(fmaxf(red[r], red[32 + r]), fmaxf(red[64 + r], red[96 + r]));
                            alpha[r] = 1.f;
                            if (tm > -INFINITY) {
                                if ((anch >> r) & 1u) {
                                    const float nm = fmaxf(mref[r], tm);
                                    alpha[r] = exp2f(mref[r] - nm);
                                    mref[r] = nm;
                                } else {
                                    mref[r] = tm;           // nothing has been accumulated for this row yet
                                    anch |= 1u << r;
                                }
                            }
                            lsum[r] *= alpha[r];
                        }
                        if (t > 0) {
                            // O^T was last written by the PV product of step it-1; this thread rescales its lane's 32 columns
                            if (!mbar_wait_warp(bar(TB_PVDONE + (bs ^ 1)), ((it - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            uint32_t o[32];
                            tmem_ld32(lane_addr + T_COL_O + ch * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int r = 0; r < 32; ++r) o[r] = __float_as_uint(__uint_as_float(o[r]) * alpha[r]);
                            tmem_st32(lane_addr + T_COL_O + ch * 32, o);
                            tmem_wait_st();
                            tc_fence_before();
                        }
#pragma unroll
                        for (int r = 0; r < 32; ++r) { x[r] = y[r] - mref[r]; e[r] = exp2f(x[r]); }
#pragma unroll
                        for (int c = 0; c < 16; ++c) pd[c] = pack_bf16(e[2 * c], e[2 * c + 1]);
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(prow + (((ch * 4 + c) ^ (tl & 7)) << 4)) = make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
                        // a second meeting: the per-warp maxima may be overwritten (by the anchor of a later
                        // segment) only after everybody has read them
                        if (!grp_sync()) { ok = false; break; }
                    }
                    if (tid == 128) TRACE(2, it, 6);
#pragma unroll
                    for (int r = 0; r < 32; ++r) lsum[r] += e[r];
                    fence_async_smem();
                    warp_arrive(bar(TB_PFULL + bs));
                }
                if (!ok) break;

                // ---- segment epilogue ----
                TRACE_MISC(5);
                if (sg.n > 0) ok = mbar_wait_warp(bar(TB_PVDONE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                TRACE_MISC(6);
                // row sums over the 128 lanes: shuffles within the warp, the four warps of the group through shared memory
#pragma unroll
                for (int r = 0; r < 32; ++r) {
                    float v = lsum[r];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (lane == r) red[sp * 32 + r] = v;
                }
                // O^T -> [row][128] fp32 in the (idle) P tiles: lane <-> head-dim index, conflict-free
                {
                    uint32_t o[32];
                    if (sg.n > 0) { tmem_ld32(lane_addr + T_COL_O + ch * 32, o); tmem_wait_ld(); }
#pragma unroll
                    for (int r = 0; r < 32; ++r) pbuf[(ch * 32 + r) * 128 + tl] = sg.n > 0 ? __uint_as_float(o[r]) : 0.f;
                }
                if (!grp_sync()) { ok = false; break; }
                if (sp == 0) {
                    // lane r of the group's first warp owns row 32 ch + r; every thread holds the same references
                    float mine = -INFINITY;
#pragma unroll
                    for (int r = 0; r < 32; ++r) mine = (lane == r) ? mref[r] : mine;
                    const float l = red[lane] + red[32 + lane] + red[64 + lane] + red[96 + lane];
                    stat[ch * 32 + lane] = make_float2(l > 0.f ? mine : -INFINITY, l);
                }
                if (!all_sync()) { ok = false; break; }
                TRACE_MISC(10);
                if (!CL) {
                    // write the unit out (a whole unit) or park it as a partial (in the merge kernel's layout)
                    const bool final_out = sg.slot < 0;
                    for (int item = st; item < T_ROWS * 32; item += kSmx) {
                        const int row = item >> 5, c4 = item & 31;
                        if (row >= rows_total) continue;
                        const float4 v = *reinterpret_cast<const float4*>(pbuf + row * 128 + c4 * 4);
                        const float2 ml = stat[row];
                        if (final_out) {
                            const float inv = ml.y > 0.f ? 1.f / ml.y : 0.f;
                            const int node = row / G, head = sg.kvh * G + row % G;
                            *reinterpret_cast<uint2*>(p.out + (((size_t)sg.b * N + node) * p.Hq + head) * D + c4 * 4) =
                                make_uint2(pack_bf16(v.x * inv, v.y * inv), pack_bf16(v.z * inv, v.w * inv));
                            if (c4 == 0 && p.lse)
                                p.lse[((size_t)sg.b * p.Hq + head) * N + node] = ml.y > 0.f ? (ml.x + log2f(ml.y)) * 0.6931471805599453f : -INFINITY;
                        } else {
                            p.part_o[((size_t)sg.slot * 32 + c4) * T_ROWS + row] = v;
                            if (c4 == 0) p.part_ml[(size_t)sg.slot * T_ROWS + row] = ml;
                        }
                    }
                    // the P tiles and the statistics are reused by the next segment
                    if (!all_sync()) { ok = false; break; }
                }
                tc_fence_before();        // the next segment's first product overwrites O^T
                TRACE_MISC(12);
                ++seg;
            }
        }
    }

    if (CL) {
        // ---- cluster exchange: every CTA of the unit has parked its partial ([row][128] fp32 and (m, l) per row) in
        // its own shared memory.  All threads of the cluster meet at the hardware cluster barrier; then rank r
        // merges rows [r*rp, (r+1)*rp) of all k partials through distributed shared memory and writes them out. ----
        __syncwarp();
        cluster_sync_all();
        TRACE_MISC(13);
        if (warp >= 4 && !*abort_flag) {
            const int rp = (T_ROWS + ck - 1) / ck;
            const int row0 = cr * rp;
            const int nrows = min(rp, T_ROWS - row0);
            const uint32_t pbuf_a = base + T_SMEM_P, pst_a = base + T_SMEM_STAT;
            auto merge_items = [&](auto km_tag, auto it_tag) {
                constexpr int KM = decltype(km_tag)::value, IT = decltype(it_tag)::value;
                for (int item0 = tid - 128; item0 < nrows * 32; item0 += kSmx * IT) {
                    float2 ml[IT][KM];
                    float4 pv[IT][KM];
                    int c4s[IT], rows[IT];
#pragma unroll
                    for (int e = 0; e < IT; ++e) {
                        const int item = item0 + e * kSmx;
                        const int lr = row0 + item / 32, c4 = item & 31;      // a row's 32 column quads are contiguous
                        c4s[e] = c4;
                        rows[e] = (item < nrows * 32) ? lr : rows_total;
#pragma unroll
                        for (int j = 0; j < KM; ++j) {
                            ml[e][j] = make_float2(-INFINITY, 0.f);
                            pv[e][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (j < ck && rows[e] < rows_total) {
                                ml[e][j] = dsmem_ld2(dsmem_addr(pst_a + lr * 8, (uint32_t)j));
                                pv[e][j] = dsmem_ld4(dsmem_addr(pbuf_a + (lr * 32 + c4) * 16, (uint32_t)j));
                            }
                        }
                    }
#pragma unroll
                    for (int e = 0; e < IT; ++e) {
                        if (rows[e] >= rows_total) continue;
                        float mm = -INFINITY;
#pragma unroll
                        for (int j = 0; j < KM; ++j) mm = fmaxf(mm, ml[e][j].x);
                        const float m_fin = (mm == -INFINITY) ? 0.f : mm;
                        float ll = 0.f;
                        float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int j = 0; j < KM; ++j) {
                            const float w = exp2f(ml[e][j].x - m_fin);          // 0 for an empty or absent part
                            ll += ml[e][j].y * w;
                            a4.x += w * pv[e][j].x; a4.y += w * pv[e][j].y; a4.z += w * pv[e][j].z; a4.w += w * pv[e][j].w;
                        }
                        const float inv2 = ll > 0.f ? 1.f / ll : 0.f;
                        const int nd = rows[e] / G, hd = cl_seg.kvh * G + rows[e] % G;
                        *reinterpret_cast<uint2*>(p.out + (((size_t)cl_seg.b * N + nd) * p.Hq + hd) * D + c4s[e] * 4) =
                            make_uint2(pack_bf16(a4.x * inv2, a4.y * inv2), pack_bf16(a4.z * inv2, a4.w * inv2));
                        if (c4s[e] == 0 && p.lse)
                            p.lse[((size_t)cl_seg.b * p.Hq + hd) * N + nd] = ll > 0.f ? (mm + log2f(ll)) * 0.6931471805599453f : -INFINITY;
                    }
                }
            };
            if (ck <= 4) merge_items(std::integral_constant<int, 4>{}, std::integral_constant<int, 2>{});
            else merge_items(std::integral_constant<int, 8>{}, std::integral_constant<int, 1>{});
        }
        TRACE_MISC(14);
    }

    // ---- tear-down: everyone meets, TMEM goes back ----
    TRACE_MISC(8);
    tc_fence_before();
    __syncthreads();
    // Cluster form: nobody leaves while a peer may still read its shared memory.  Every CTA gets here (all its
    // other waits are bounded), so this hardware barrier ends.
    if (CL) cluster_sync_all();
    TRACE_MISC(9);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(T_TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicCAS(p.status, 0, (int)VISPEC_E_TIMEOUT);
    TL_END(p.trace_idx, 1);
    CTA_T(1);
}
