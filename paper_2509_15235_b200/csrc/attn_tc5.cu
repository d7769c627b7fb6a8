// Tree-verification attention for sm_100a: TMA-staged K/V tiles, tcgen05 tensor-core products with
// TMEM accumulators, fp32 online softmax (Eq. 1 restricted to prefix + ancestors).
//
// Shape served: D = 128 and G*N <= 64 query rows per kv head (the multi-head workloads: one head's
// whole tree fits one 64-row tile).  Everything else goes to the generic kernel.
//
// One CTA works on one (sequence, kv head, KV range).  Its 6 warps are specialised:
//   warp 0   TMA producer: K and V rings of 128-token stages (two 64-token tiles each)
//   warp 1   tensor-core issuer: S = Q K^T and O += P V as tcgen05.mma (M = 64), owns TMEM
//   warps 2-5  softmax: one thread per (query row, tile parity)
// A 64-row accumulator only occupies TMEM lanes 0-15 of each 32-lane quarter, so two tile streams are
// interleaved: even tiles of the range accumulate in lanes 0-15 (+32q), odd tiles in lanes 16-31
// (+32q).  Each softmax thread then owns one TMEM lane = one query row of one stream: row maximum, sum and
// rescale are thread-local, no shuffles.  The two streams are merged once, in the epilogue.
// The running maximum is only moved when a tile exceeds it by more than 2^8 (the accumulators stay exact
// either way because O and l share the reference), so O is re-scaled in TMEM rarely.
// Every wait on an mbarrier is bounded; on a timeout the CTA records VISPEC_E_TIMEOUT, drains its own
// copies, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "vispec_internal.h"

namespace vispec {

cudaError_t launch_attn_combine64(const AttnArgs& a, int n_split, int n_mblocks, cudaStream_t st);

namespace {

constexpr int D = 128;
constexpr int TILE = 64;                       // tokens per tile
constexpr int STEP = 2 * TILE;                 // tokens per pipeline step (one tile per stream)
constexpr int HALF_BYTES = STEP * 128;         // one d-half (64 columns) of a stage: 128 rows x 128 B
constexpr int STAGE_BYTES = 2 * HALF_BYTES;    // 32 KB
constexpr int NSK = 2, NSV = 3;
constexpr int kThreads = 192;
constexpr int Q_BYTES = 64 * D * 2;            // 16 KB
constexpr int P_TILE_BYTES = 64 * TILE * 2;    // 8 KB: 64 rows x 64 tokens bf16
constexpr int SMEM_Q = 0;
constexpr int SMEM_P = SMEM_Q + Q_BYTES;                       // [2 buffers][2 streams]
constexpr int SMEM_K = SMEM_P + 4 * P_TILE_BYTES;
constexpr int SMEM_V = SMEM_K + NSK * STAGE_BYTES;
constexpr int SMEM_BAR = SMEM_V + NSV * STAGE_BYTES;
constexpr int SMEM_TOTAL = SMEM_BAR + 256;
constexpr int SMEM_ALLOC = SMEM_TOTAL + 1024;                  // slack to align the base to 1024 B
constexpr uint32_t TMEM_COLS = 256;                            // S[0] 0..63, S[1] 64..127, O 128..255
constexpr uint32_t COL_O = 128;
constexpr float kRescaleGap = 8.0f;                            // log2 units
constexpr long long kWaitCycles = 1500000000LL;                // ~0.8 s at 1.9 GHz

// ---- barrier indices ----
enum { B_KFULL = 0, B_KEMPTY = B_KFULL + NSK, B_VFULL = B_KEMPTY + NSK, B_VEMPTY = B_VFULL + NSV,
       B_SFULL = B_VEMPTY + NSV, B_SFREE = B_SFULL + 2, B_PFULL = B_SFREE + 2, B_PFREE = B_PFULL + 2,
       B_COUNT = B_PFREE + 2 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the completion of the phase with parity `parity`.  Returns false after ~kWaitCycles
// or as soon as another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63) == 63) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitCycles) { *abort_flag = 1; return false; }
        }
    }
}
// Same, with a warp-uniform result (every lane of a converged warp calls it): the warp-collective
// tcgen05.ld/st that follow must never be reached by only part of a warp.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One tcgen05.mma (cta_group::1, kind::f16).  The 64-bit shared-memory descriptors are passed as 32-bit
// halves: the high half is a per-operand constant, the low half carries the address, so that the issuing
// thread spends one add per operand and instruction.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                       uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 bit, 32 consecutive columns: thread i of the warp receives lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format), split in halves.  Low: start address and leading byte
// offset, both in 16-byte units.  High: stride byte offset (16-byte units), descriptor version 1 (bit 46),
// 128-byte swizzle (value 2 in bits 61-63).  Tile bases are 1024-byte aligned (base offset 0).
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr >> 4) & 0x3FFFu) | ((lbo_bytes >> 4) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) {
    return (sbo_bytes >> 4) | (1u << 14) | (2u << 29);
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, M = 64, N = n; b_mn = 1 if B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((64u >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

#ifdef VISPEC_TC5_TRACE
// Debug build only: CTA (0,0) logs clock64() stamps per role and step: g_trace[role][step][slot].
__device__ long long g_trace[3][64][8];
#define TRACE(role, step, slot) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (step) < 64) g_trace[role][step][slot] = clock64(); } while (0)
#else
#define TRACE(role, step, slot) do {} while (0)
#endif

struct Tc5Params {
    const __nv_bfloat16* q; const int32_t* kv_len; const uint64_t* mask;
    __nv_bfloat16* out; float* lse;
    float* part_o; float* part_ml;        // [unit][split][64][D], [unit][split][64][2]
    int B, N, Hq, Hkv, S_max, n_split;
    float scale_log2;
    int* status;
};

__global__ void __launch_bounds__(kThreads, 1)
attn_tc5_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const Tc5Params p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    const uint32_t bars = base + SMEM_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + SMEM_BAR + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + SMEM_BAR + B_COUNT * 8 + 8);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, unit = blockIdx.y;
    const int b = unit / p.Hkv, kvh = unit % p.Hkv;
    const int G = p.Hq / p.Hkv, N = p.N, W = (N + 63) >> 6;
    const int rows_total = G * N;

    const int S = p.kv_len[b];
    const bool seq_ok = (S >= 0 && S + N <= p.S_max);
    if (!seq_ok && tid == 0 && split == 0) atomicCAS(p.status, 0, (int)VISPEC_E_RANGE);
    const int total = seq_ok ? S + N : 0;
    const int steps_total = (total + STEP - 1) / STEP;
    const int sps = (steps_total + p.n_split - 1) / p.n_split;
    const int step_begin = min(split * sps, steps_total);
    const int nsteps = min(step_begin + sps, steps_total) - step_begin;
    const int tok_begin = step_begin * STEP;

    // ---- set-up: barriers, Q tile (swizzled K-major: two d-halves of 64 rows x 128 B), TMEM ----
    if (tid == 0) {
        for (int i = 0; i < NSK; ++i) { mbar_init(bar(B_KFULL + i), 1); mbar_init(bar(B_KEMPTY + i), 1); }
        for (int i = 0; i < NSV; ++i) { mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_SFULL + i), 1); mbar_init(bar(B_SFREE + i), 128);
            mbar_init(bar(B_PFULL + i), 128); mbar_init(bar(B_PFREE + i), 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (nsteps > 0) {
        for (int idx = tid; idx < 64 * 16; idx += kThreads) {
            const int r = idx >> 4, c = idx & 15;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r < rows_total) {
                const int i = r / G, g = r % G;
                val = *reinterpret_cast<const uint4*>(p.q + (((size_t)b * N + i) * p.Hq + kvh * G + g) * D + c * 8);
            }
            *reinterpret_cast<uint4*>(sm + SMEM_Q + (c >> 3) * 8192 + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = val;
        }
        fence_async_smem();
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // per-row epilogue state lives in the softmax threads; declared here so the tail code sees it
    const int sp = warp & 3;                       // TMEM lane quarter this warp may access
    const int par = lane >> 4;                     // which tile stream this thread serves
    const int row = sp * 16 + (lane & 15);         // query row of the 64-row tile
    float m_ref = -INFINITY, l_run = 0.f;
    bool has_o = false;

    if (nsteps > 0) {
        const uint32_t tmem = *tmem_slot;
        if (warp == 0) {
            // ================= TMA producer =================
            if (lane == 0) {
                int issued = 0;
                for (int t = 0; t < nsteps; ++t) {
                    const int tok = tok_begin + t * STEP;
                    const int sk = t % NSK, sv = t % NSV;
                    TRACE(0, t, 0);
                    if (!mbar_wait(bar(B_KEMPTY + sk), ((t / NSK) & 1) ^ 1, abort_flag)) break;
                    TRACE(0, t, 1);
                    mbar_expect_tx(bar(B_KFULL + sk), STAGE_BYTES);
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES, &k_map, bar(B_KFULL + sk), 0, tok, unit);
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES + HALF_BYTES, &k_map, bar(B_KFULL + sk), 64, tok, unit);
                    if (!mbar_wait(bar(B_VEMPTY + sv), ((t / NSV) & 1) ^ 1, abort_flag)) { issued = -(t + 1); break; }
                    TRACE(0, t, 2);
                    mbar_expect_tx(bar(B_VFULL + sv), STAGE_BYTES);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES, &v_map, bar(B_VFULL + sv), 0, tok, unit);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + HALF_BYTES, &v_map, bar(B_VFULL + sv), 64, tok, unit);
                    issued = t + 1;
                }
                if (*abort_flag) {
                    // drain: wait (bounded, fresh timer) until every copy this thread issued has landed
                    volatile int never = 0;
                    const int nk = issued < 0 ? -issued : issued, nv = issued < 0 ? -issued - 1 : issued;
                    for (int u = max(0, nk - NSK); u < nk; ++u) mbar_wait(bar(B_KFULL + u % NSK), (u / NSK) & 1, &never);
                    for (int u = max(0, nv - NSV); u < nv; ++u) mbar_wait(bar(B_VFULL + u % NSV), (u / NSV) & 1, &never);
                }
            }
            __syncwarp();
        } else if (warp == 1) {
            // ================= tensor-core issuer =================
            if (lane == 0) {
                constexpr uint32_t IDESC_S = instr_desc(TILE, 0);      // 64 x 64, K-major B (K tile)
                constexpr uint32_t IDESC_O = instr_desc(D, 1);         // 64 x 128, MN-major B (V tile)
                constexpr uint32_t DESC_HI = desc_hi(1024);            // 8 rows x 128 B between row groups, everywhere
                const uint32_t q_lo = desc_lo(base + SMEM_Q, 16);
                auto tile_valid = [&](int t, int s) { return tok_begin + t * STEP + s * TILE < total; };
                auto issue_pv = [&](int u) -> bool {
                    const int bu = u & 1, sv = u % NSV;
                    TRACE(1, u, 3);
                    if (!mbar_wait(bar(B_PFULL + bu), (u >> 1) & 1, abort_flag)) return false;
                    TRACE(1, u, 4);
                    if (!mbar_wait(bar(B_VFULL + sv), (u / NSV) & 1, abort_flag)) return false;
                    TRACE(1, u, 5);
                    tc_fence_after();
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        if (!tile_valid(u, s)) continue;
                        const uint32_t pa = desc_lo(base + SMEM_P + (bu * 2 + s) * P_TILE_BYTES, 16);
                        const uint32_t vb = desc_lo(base + SMEM_V + sv * STAGE_BYTES + s * (TILE * 128), HALF_BYTES);
#pragma unroll
                        for (int ks = 0; ks < TILE / 16; ++ks)      // address steps are in 16-byte units
                            tc_mma(tmem + ((uint32_t)(16 * s) << 16) + COL_O, pa + ks * 2, DESC_HI, vb + ks * 128, DESC_HI,
                                   IDESC_O, (u > 0 || ks > 0) ? 1u : 0u);
                    }
                    tc_commit(bar(B_VEMPTY + sv));
                    tc_commit(bar(B_PFREE + bu));
                    TRACE(1, u, 6);
                    return true;
                };
                bool ok = true;
                for (int t = 0; t < nsteps && ok; ++t) {
                    const int bs = t & 1, sk = t % NSK;
                    TRACE(1, t, 0);
                    if (!mbar_wait(bar(B_KFULL + sk), (t / NSK) & 1, abort_flag)) { ok = false; break; }
                    TRACE(1, t, 1);
                    if (t >= 2 && !mbar_wait(bar(B_SFREE + bs), ((t >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        if (!tile_valid(t, s)) continue;
                        const uint32_t kb = desc_lo(base + SMEM_K + sk * STAGE_BYTES + s * (TILE * 128), 16);
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            const uint32_t off = ((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4;   // K stage: d-halves 16 KB apart
                            const uint32_t qoff = ((ks >> 2) * 8192 + (ks & 3) * 32) >> 4;        // Q: d-halves 8 KB apart
                            tc_mma(tmem + ((uint32_t)(16 * s) << 16) + bs * TILE, q_lo + qoff, DESC_HI, kb + off, DESC_HI,
                                   IDESC_S, ks > 0 ? 1u : 0u);
                        }
                    }
                    tc_commit(bar(B_KEMPTY + sk));
                    tc_commit(bar(B_SFULL + bs));
                    TRACE(1, t, 2);
                    if (t >= 1) ok = issue_pv(t - 1);
                }
                if (ok) issue_pv(nsteps - 1);
            }
            __syncwarp();
        } else {
            // ================= softmax: one thread per (row, stream) =================
            uint64_t mk0 = 0, mk1 = 0;
            if (row < rows_total) {
                const uint64_t* mrow = p.mask + ((size_t)b * N + row / G) * W;
                mk0 = mrow[0];
                if (W > 1) mk1 = mrow[1];
            }
            const uint32_t lane_addr = tmem + ((uint32_t)(32 * sp) << 16);
            bool ok = true;
            for (int t = 0; t < nsteps; ++t) {
                const int bs = t & 1;
                if (tid == 64) TRACE(2, t, 0);
                if (!mbar_wait_warp(bar(B_SFULL + bs), (t >> 1) & 1, abort_flag)) { ok = false; break; }
                if (tid == 64) TRACE(2, t, 1);
                tc_fence_after();
                uint32_t sraw[2][32];
                tmem_ld32(lane_addr + bs * TILE, sraw[0]);
                tmem_ld32(lane_addr + bs * TILE + 32, sraw[1]);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(B_SFREE + bs));
                if (tid == 64) TRACE(2, t, 2);

                const int j0 = tok_begin + t * STEP + par * TILE;       // first token of this thread's tile
                const bool valid = j0 < total;
                float x[64];
                float tmax = -INFINITY;
                if (valid) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) x[c] = __uint_as_float(sraw[c >> 5][c & 31]) * p.scale_log2;
                    if (j0 + TILE > S) {
                        // tile reaches past the committed prefix: ancestor bits for tree rows, nothing beyond them
                        const int t0 = j0 - S;                           // tree index of column 0 (may be negative)
#pragma unroll
                        for (int c = 0; c < 64; ++c) {
                            const int tt = t0 + c;
                            bool allow = true;
                            if (tt >= 0) allow = (tt < N) && ((tt < 64 ? (mk0 >> tt) : (mk1 >> (tt - 64))) & 1ull);
                            if (!allow) x[c] = -INFINITY;
                        }
                    }
                    float mx[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) mx[c] = x[c];
#pragma unroll
                    for (int c = 8; c < 64; ++c) mx[c & 7] = fmaxf(mx[c & 7], x[c]);
                    tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                }
                // move the reference maximum only when the tile exceeds it by more than the gap
                float alpha = 1.f;
                bool rescale = false;
                if (valid && tmax > m_ref + kRescaleGap) {          // also true on the first finite tile (m_ref = -inf)
                    alpha = exp2f(m_ref - tmax);                     // 0 when m_ref = -inf
                    m_ref = tmax;
                    l_run *= alpha;
                    rescale = has_o;
                }
                if (__any_sync(0xffffffffu, rescale)) {
                    // O of this stream was last written by the PV product of step t-1
                    if (!mbar_wait_warp(bar(B_PFREE + (bs ^ 1)), ((t - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[32];
                        tmem_ld32(lane_addr + COL_O + ch * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        tmem_st32(lane_addr + COL_O + ch * 32, o);
                    }
                    tmem_wait_st();
                }
                if (tid == 64) TRACE(2, t, 3);
                if (t >= 2 && !mbar_wait_warp(bar(B_PFREE + bs), ((t >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                if (tid == 64) TRACE(2, t, 4);
                bool fail = false;
                if (valid) {
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    float sum = 0.f;
                    unsigned char* prow = sm + SMEM_P + (bs * 2 + par) * P_TILE_BYTES + row * 128;
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        float e[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) { e[k] = exp2f(x[ch * 8 + k] - m_use); sum += e[k]; }
                        *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) =
                            make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7]));
                    }
                    l_run += sum;
                    has_o = true;
                    if (j0 + TILE > total) {
                        // rows of the V tile past the last key may hold anything: clear them before the product
                        const int sv = t % NSV;
                        fail = !mbar_wait(bar(B_VFULL + sv), (t / NSV) & 1, abort_flag);
                        const int r = sp * 16 + (lane & 15);           // 64 threads of this stream, one V row each
                        if (!fail && j0 + r >= total) {
                            unsigned char* vrow = sm + SMEM_V + sv * STAGE_BYTES + par * (TILE * 128) + r * 128;
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                                *reinterpret_cast<uint4*>(vrow + HALF_BYTES + c * 16) = make_uint4(0, 0, 0, 0);
                            }
                        }
                    }
                }
                if (__any_sync(0xffffffffu, fail)) { ok = false; break; }
                if (tid == 64) TRACE(2, t, 5);
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar(B_PFULL + bs));
                if (tid == 64) TRACE(2, t, 6);
            }
            // ---- epilogue: wait for the last product, merge the two streams, write out ----
            if (ok) ok = mbar_wait_warp(bar(B_PFREE + ((nsteps - 1) & 1)), ((nsteps - 1) >> 1) & 1, abort_flag);
            if (ok) {
                tc_fence_after();
                const float m_other = __shfl_xor_sync(0xffffffffu, m_ref, 16);
                const float l_other = __shfl_xor_sync(0xffffffffu, l_run, 16);
                const float m_all = fmaxf(m_ref, m_other);
                const float m_fin = (m_all == -INFINITY) ? 0.f : m_all;
                const float w_me = has_o ? exp2f(m_ref - m_fin) : 0.f;
                const float w_other = exp2f(m_other - m_fin);           // 0 when the other stream saw nothing
                const float l_all = l_run * w_me + l_other * w_other;
                const bool final_out = (p.n_split == 1);
                const float inv = final_out ? (l_all > 0.f ? 1.f / l_all : 0.f) : 1.f;
                const int i = row / G, g = row % G, head = kvh * G + g;
                const size_t slot = ((size_t)unit * p.n_split + split) * 64 + row;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t o[32];
                    tmem_ld32(lane_addr + COL_O + ch * 32, o);
                    tmem_wait_ld();
                    float mine[16];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float v = has_o ? __uint_as_float(o[c]) * w_me : 0.f;
                        const float sum = v + __shfl_xor_sync(0xffffffffu, v, 16);
                        if ((c >> 4) == par) mine[c & 15] = sum * inv;     // stream-0 lanes keep columns 0-15 of the chunk
                    }
                    if (row < rows_total) {
                        const int col = ch * 32 + par * 16;
                        if (final_out) {
                            __nv_bfloat16* dst = p.out + (((size_t)b * N + i) * p.Hq + head) * D + col;
                            *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16(mine[0], mine[1]), pack_bf16(mine[2], mine[3]),
                                                                        pack_bf16(mine[4], mine[5]), pack_bf16(mine[6], mine[7]));
                            *reinterpret_cast<uint4*>(dst + 8) = make_uint4(pack_bf16(mine[8], mine[9]), pack_bf16(mine[10], mine[11]),
                                                                            pack_bf16(mine[12], mine[13]), pack_bf16(mine[14], mine[15]));
                        } else {
                            float* dst = p.part_o + slot * D + col;
#pragma unroll
                            for (int c = 0; c < 16; c += 4)
                                *reinterpret_cast<float4*>(dst + c) = make_float4(mine[c], mine[c + 1], mine[c + 2], mine[c + 3]);
                        }
                    }
                }
                if (par == 0 && row < rows_total) {
                    if (final_out) {
                        if (p.lse) p.lse[((size_t)b * p.Hq + head) * N + i] =
                            l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                    } else {
                        *reinterpret_cast<float2*>(p.part_ml + slot * 2) = make_float2(m_all, l_all);
                    }
                }
                tc_fence_before();
            }
        }
    } else if (p.n_split > 1 || !seq_ok || total == 0) {
        // nothing to attend to in this range: an empty partial, or a zero output for an empty / rejected sequence
        for (int idx = tid; idx < 64 * (D / 4); idx += kThreads) {
            const int r = idx / (D / 4), c4 = idx % (D / 4);
            if (r >= rows_total) continue;
            if (p.n_split > 1) {
                const size_t slot = ((size_t)unit * p.n_split + split) * 64 + r;
                *reinterpret_cast<float4*>(p.part_o + slot * D + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                if (c4 == 0) *reinterpret_cast<float2*>(p.part_ml + slot * 2) = make_float2(-INFINITY, 0.f);
            } else {
                const int i = r / G, g = r % G, head = kvh * G + g;
                *reinterpret_cast<uint2*>(p.out + (((size_t)b * N + i) * p.Hq + head) * D + c4 * 4) = make_uint2(0, 0);
                if (c4 == 0 && p.lse) p.lse[((size_t)b * p.Hq + head) * N + i] = -INFINITY;
            }
        }
    }

    // ---- tear-down: everyone meets, TMEM goes back ----
    __syncthreads();
    if (nsteps > 0) {
        if (warp == 1) {
            tc_fence_after();
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(TMEM_COLS) : "memory");
        }
        if (tid == 0 && *abort_flag) atomicCAS(p.status, 0, (int)VISPEC_E_TIMEOUT);
    }
}

}  // namespace

#ifdef VISPEC_TC5_TRACE
extern "C" int vispec_debug_read_trace(long long* host) {
    return cudaMemcpyFromSymbol(host, g_trace, sizeof(g_trace)) == cudaSuccess ? 0 : -1;
}
#endif

bool attn_tc5_supports(const AttnArgs& a) {
    return a.D == 128 && (a.Hq / a.Hkv) * a.N <= 64 && a.k_map && a.v_map && a.B > 0;
}

cudaError_t init_attn_tc5() {
    return cudaFuncSetAttribute(attn_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ALLOC);
}

cudaError_t launch_attn_tc5(const AttnArgs& a, cudaStream_t st, int* n_launches) {
    *n_launches = 0;
    const int units = a.B * a.Hkv;
    const int max_steps = (a.S_max + STEP - 1) / STEP;
    int n_split = a.sm_count / units;
    if (n_split < 1) n_split = 1;
    if (n_split > max_steps) n_split = max_steps;
    const size_t half_slot = slot_bytes(a.D) / 2;
    while (n_split > 1 && kCounterBytes + (size_t)units * n_split * half_slot > a.ws_bytes) --n_split;

    Tc5Params p;
    p.q = (const __nv_bfloat16*)a.q; p.kv_len = a.kv_len; p.mask = a.mask;
    p.out = (__nv_bfloat16*)a.out; p.lse = a.lse;
    unsigned char* ws = (unsigned char*)a.ws + kCounterBytes;
    p.part_o = (float*)ws;
    p.part_ml = (float*)(ws + (size_t)units * n_split * 64 * a.D * 4);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max; p.n_split = n_split;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.status = a.status;
    dim3 grid(n_split, units);
    attn_tc5_kernel<<<grid, kThreads, SMEM_ALLOC, st>>>(*a.k_map, *a.v_map, p);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    ++*n_launches;
    if (n_split > 1) {
        err = launch_attn_combine64(a, n_split, 1, st);
        if (err != cudaSuccess) return err;
        ++*n_launches;
    }
    return cudaSuccess;
}

}  // namespace vispec
