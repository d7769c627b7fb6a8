// Tree-verification attention for sm_100a (D = 128): TMA-staged K/V tiles, tcgen05 tensor-core products
// with every accumulator AND both A operands in TMEM, fp32 online softmax (Eq. 1 restricted to prefix +
// ancestors).
//
// One CTA works on one (sequence, kv head, block of query rows, KV range).  Its 6 warps are specialised:
//   warp 0     TMA producer: K ring and V ring of 128-token stages (32 KB each, 128-byte swizzle)
//   warp 1     tensor-core issuer (one thread): S = Q K^T and O += P V as 128x128x16 tcgen05.mma, owns TMEM
//   warps 2-5  softmax: thread <-> TMEM lane, i.e. one thread per accumulator row, no shuffles
// TMEM map (512 columns x 128 lanes): S[0] 0..127, S[1] 128..255, O 256..383, Q 384..447.
// Q (bf16, packed two per column) is written to TMEM once by the softmax threads and is the A operand of
// every S product; P (bf16) overwrites the first 64 columns of the S buffer it came from and is the A
// operand of the PV product, so neither Q nor P ever touches shared memory: all of it goes to the rings.
//
// Two row layouts share the code:
//   FULL  (G*N > 64):  lane r holds query row r of the block; a thread handles all 128 tokens of a step.
//   PAIR  (G*N <= 64): the <= 64 query rows are duplicated, lanes 0-63 take tokens 0-63 of each step and
//                      lanes 64-127 tokens 64-127 (P is block-diagonal); the two halves keep independent
//                      softmax states and are merged once in the epilogue.  All 128 threads stay busy and
//                      the tensor core runs full-height instructions, which cost less than two 64-row ones.
// The running maximum is only moved when a tile exceeds it by more than 2^8 (O and l share the reference, so
// the result is exact either way); O is therefore re-scaled in TMEM rarely.
// Every wait on an mbarrier is bounded; on a timeout the CTA records VISPEC_E_TIMEOUT, drains its own
// copies, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "vispec_internal.h"

namespace vispec {

cudaError_t launch_attn_combine(const AttnArgs& a, int n_split, int n_mblocks, int rows_per_block, cudaStream_t st);

namespace {

constexpr int D = 128;
constexpr int STEP = 128;                      // tokens per pipeline step = rows of one K or V stage
constexpr int HALF_BYTES = STEP * 128;         // one d-half (64 columns) of a stage: 128 rows x 128 B
constexpr int STAGE_BYTES = 2 * HALF_BYTES;    // 32 KB
constexpr int NSK = 3, NSV = 4;
constexpr int kThreads = 192;
constexpr int SMEM_K = 0;
constexpr int SMEM_V = SMEM_K + NSK * STAGE_BYTES;
constexpr int SMEM_BAR = SMEM_V + NSV * STAGE_BYTES;
constexpr int SMEM_TOTAL = SMEM_BAR + 256;
constexpr int SMEM_ALLOC = SMEM_TOTAL + 1024;                  // slack to align the base to 1024 B
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_S = 0, COL_O = 256, COL_Q = 384;
constexpr float kRescaleGap = 8.0f;                            // log2 units
constexpr long long kWaitCycles = 1500000000LL;                // ~0.8 s at 1.9 GHz

enum { B_KFULL = 0, B_KEMPTY = B_KFULL + NSK, B_VFULL = B_KEMPTY + NSK, B_VEMPTY = B_VFULL + NSV,
       B_SFULL = B_VEMPTY + NSV, B_PFULL = B_SFULL + 2, B_PVDONE = B_PFULL + 2,
       B_XSTAT = B_PVDONE + 2, B_XWGT = B_XSTAT + 1, B_XCH = B_XWGT + 1, B_COUNT = B_XCH + 4 };
static_assert(B_COUNT * 8 + 16 <= 256, "barrier block too small");

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
// One tcgen05.mma (cta_group::1, kind::f16) with the A operand in TMEM and B described in shared memory.
// The 64-bit descriptor is passed as 32-bit halves: the high half is constant, the low half carries the address.
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 bit, 32 consecutive columns: thread i of the warp accesses lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
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
// Instruction descriptor, kind::f16: D fp32, A and B bf16, A K-major, M = 128, N = 128; b_mn = 1 if B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

#ifdef VISPEC_TC5_TRACE
// Debug build only: CTA (0,0) logs clock64() stamps per role and step: g_trace[role][step][slot].
__device__ long long g_trace[3][64][8];
__device__ long long g_trace_misc[16];
#define TRACE(role, step, slot) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (step) < 64) g_trace[role][step][slot] = clock64(); } while (0)
#define TRACE_MISC(slot) do { if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 64) g_trace_misc[slot] = clock64(); } while (0)
#else
#define TRACE(role, step, slot) do {} while (0)
#define TRACE_MISC(slot) do {} while (0)
#endif

struct Tc5Params {
    const __nv_bfloat16* q; const int32_t* kv_len; const uint64_t* mask;
    __nv_bfloat16* out; float* lse;
    float* part_o; float* part_ml;        // [unit][split][ROWS][D], [unit][split][ROWS][2]
    int B, N, Hq, Hkv, S_max, n_split, n_mblocks;
    float scale_log2;
    int* status;
};

template <bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc5_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const Tc5Params p) {
    constexpr int ROWS = PAIR ? 64 : 128;      // distinct query rows per CTA
    constexpr int NCOL = PAIR ? 64 : 128;      // tokens of a step one thread handles
    extern __shared__ unsigned char smem_raw[];
    TRACE_MISC(0);
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    const uint32_t bars = base + SMEM_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + SMEM_BAR + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + SMEM_BAR + B_COUNT * 8 + 8);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, unit = blockIdx.y;
    const int mblock = unit % p.n_mblocks, bh = unit / p.n_mblocks;       // bh = sequence * Hkv + kv head
    const int b = bh / p.Hkv, kvh = bh % p.Hkv;
    const int G = p.Hq / p.Hkv, N = p.N, W = (N + 63) >> 6;
    const int rows_total = G * N;

    const int S = p.kv_len[b];
    const bool seq_ok = (S >= 0 && S + N <= p.S_max);
    if (!seq_ok && tid == 0 && split == 0 && mblock == 0) atomicCAS(p.status, 0, (int)VISPEC_E_RANGE);
    const int total = seq_ok ? S + N : 0;
    const int steps_total = (total + STEP - 1) / STEP;
    const int sps = (steps_total + p.n_split - 1) / p.n_split;
    const int step_begin = min(split * sps, steps_total);
    const int nsteps = min(step_begin + sps, steps_total) - step_begin;
    const int tok_begin = step_begin * STEP;

    // row handled by this thread if it is a softmax thread (warps 2..5 cover the four TMEM lane quarters)
    const int sp = warp & 3;
    const int tl = sp * 32 + lane;                       // TMEM lane
    const int half = PAIR ? (tl >> 6) : 0;               // PAIR: which 64 tokens of each step
    const int lrow = PAIR ? (tl & 63) : tl;              // row within the block
    const int row = mblock * 128 + lrow;                 // query row within the kv head's G*N rows
    const bool row_ok = row < rows_total;
    const int node = row_ok ? row / G : 0, head = kvh * G + (row_ok ? row % G : 0);

    if (tid == 0) {
        for (int i = 0; i < NSK; ++i) { mbar_init(bar(B_KFULL + i), 1); mbar_init(bar(B_KEMPTY + i), 1); }
        for (int i = 0; i < NSV; ++i) { mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_SFULL + i), 1); mbar_init(bar(B_PFULL + i), 128); mbar_init(bar(B_PVDONE + i), 1);
        }
        for (int i = B_XSTAT; i < B_COUNT; ++i) mbar_init(bar(i), 64);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (nsteps > 0 && warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    TRACE_MISC(1);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    TRACE_MISC(2);

    float m_ref = -INFINITY, l_run = 0.f;
    bool has_o = false;

    if (nsteps > 0) {
        const uint32_t tmem = *tmem_slot;
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sp) << 16);
        // ---- Q -> TMEM: each softmax thread packs its row (bf16 pairs) into columns COL_Q..COL_Q+63 ----
        if (warp >= 2) {
            uint32_t qreg[64];
            if (row_ok) {
                const uint4* src = reinterpret_cast<const uint4*>(p.q + (((size_t)b * N + node) * p.Hq + head) * D);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint4 v4 = src[c];
                    qreg[4 * c] = v4.x; qreg[4 * c + 1] = v4.y; qreg[4 * c + 2] = v4.z; qreg[4 * c + 3] = v4.w;
                }
            } else {
#pragma unroll
                for (int c = 0; c < 64; ++c) qreg[c] = 0u;
            }
            tmem_st32(lane_addr + COL_Q, qreg);
            tmem_st32(lane_addr + COL_Q + 32, qreg + 32);
            tmem_wait_st();
        }
        TRACE_MISC(3);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        TRACE_MISC(4);

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
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES, &k_map, bar(B_KFULL + sk), 0, tok, bh);
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES + HALF_BYTES, &k_map, bar(B_KFULL + sk), 64, tok, bh);
                    if (!mbar_wait(bar(B_VEMPTY + sv), ((t / NSV) & 1) ^ 1, abort_flag)) { issued = -(t + 1); break; }
                    TRACE(0, t, 2);
                    mbar_expect_tx(bar(B_VFULL + sv), STAGE_BYTES);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES, &v_map, bar(B_VFULL + sv), 0, tok, bh);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + HALF_BYTES, &v_map, bar(B_VFULL + sv), 64, tok, bh);
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
                constexpr uint32_t IDESC_S = instr_desc(0);            // B = K stage, K-major
                constexpr uint32_t IDESC_O = instr_desc(1);            // B = V stage, MN-major
                constexpr uint32_t DESC_HI = desc_hi(1024);            // 8 rows x 128 B between row groups, everywhere
                auto issue_pv = [&](int u) -> bool {
                    const int bu = u & 1, sv = u % NSV;
                    TRACE(1, u, 3);
                    if (!mbar_wait(bar(B_PFULL + bu), (u >> 1) & 1, abort_flag)) return false;
                    TRACE(1, u, 4);
                    if (!mbar_wait(bar(B_VFULL + sv), (u / NSV) & 1, abort_flag)) return false;
                    TRACE(1, u, 5);
                    tc_fence_after();
                    const uint32_t vb = desc_lo(base + SMEM_V + sv * STAGE_BYTES, HALF_BYTES);
#pragma unroll
                    for (int ks = 0; ks < STEP / 16; ++ks)      // 16 tokens per instruction: 8 P columns, 16 V rows (2 KB)
                        tc_mma_ts(tmem + COL_O, tmem + COL_S + bu * 128 + ks * 8, vb + ks * 128, DESC_HI, IDESC_O,
                                  (u > 0 || ks > 0) ? 1u : 0u);
                    tc_commit(bar(B_VEMPTY + sv));
                    tc_commit(bar(B_PVDONE + bu));
                    TRACE(1, u, 6);
                    return true;
                };
                bool ok = true;
                for (int t = 0; t < nsteps && ok; ++t) {
                    const int bs = t & 1, sk = t % NSK;
                    TRACE(1, t, 0);
                    if (!mbar_wait(bar(B_KFULL + sk), (t / NSK) & 1, abort_flag)) { ok = false; break; }
                    TRACE(1, t, 1);
                    // S[bs] (and the P that aliases it) is free once the PV product of step t-2 has completed
                    if (t >= 2 && !mbar_wait(bar(B_PVDONE + bs), ((t >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t kb = desc_lo(base + SMEM_K + sk * STAGE_BYTES, 16);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)         // 16 d-columns per instruction: 8 Q columns, 32 B of each K row
                        tc_mma_ts(tmem + COL_S + bs * 128, tmem + COL_Q + ks * 8,
                                  kb + (((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4), DESC_HI, IDESC_S, ks > 0 ? 1u : 0u);
                    tc_commit(bar(B_KEMPTY + sk));
                    tc_commit(bar(B_SFULL + bs));
                    TRACE(1, t, 2);
                    if (t >= 1) ok = issue_pv(t - 1);
                }
                if (ok) issue_pv(nsteps - 1);
            }
            __syncwarp();
        } else {
            // ================= softmax: one thread per accumulator row =================
            uint64_t mk0 = 0, mk1 = 0;
            if (row_ok) {
                const uint64_t* mrow = p.mask + ((size_t)b * N + node) * W;
                mk0 = mrow[0];
                if (W > 1) mk1 = mrow[1];
            }
            bool ok = true;
            for (int t = 0; t < nsteps; ++t) {
                const int bs = t & 1;
                if (tid == 64) TRACE(2, t, 0);
                if (!mbar_wait_warp(bar(B_SFULL + bs), (t >> 1) & 1, abort_flag)) { ok = false; break; }
                if (tid == 64) TRACE(2, t, 1);
                tc_fence_after();
                uint32_t sraw[NCOL];
#pragma unroll
                for (int ch = 0; ch < NCOL / 32; ++ch) tmem_ld32(lane_addr + COL_S + bs * 128 + half * 64 + ch * 32, sraw + ch * 32);
                tmem_wait_ld();
                if (tid == 64) TRACE(2, t, 2);

                const int j0 = tok_begin + t * STEP + half * 64;        // first token this thread looks at
                const bool valid = j0 < total;
                float tmax = -INFINITY;
                if (valid) {
#pragma unroll
                    for (int c = 0; c < NCOL; ++c) sraw[c] = __float_as_uint(__uint_as_float(sraw[c]) * p.scale_log2);
                    if (j0 + NCOL > S) {
                        // reaches past the committed prefix: ancestor bits for tree rows, nothing beyond them
                        const int t0 = j0 - S;                           // tree index of column 0 (may be negative)
#pragma unroll
                        for (int c = 0; c < NCOL; ++c) {
                            const int tt = t0 + c;
                            bool allow = true;
                            if (tt >= 0) allow = (tt < N) && ((tt < 64 ? (mk0 >> tt) : (mk1 >> (tt - 64))) & 1ull);
                            if (!allow) sraw[c] = 0xff800000u;          // -inf
                        }
                    }
                    float mx[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) mx[c] = __uint_as_float(sraw[c]);
#pragma unroll
                    for (int c = 8; c < NCOL; ++c) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(sraw[c]));
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
                    // O was last written by the PV product of step t-1
                    if (!mbar_wait_warp(bar(B_PVDONE + (bs ^ 1)), ((t - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
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
                }
                if (tid == 64) TRACE(2, t, 3);
                // P = exp2(x - m_ref) as bf16 pairs into the first 64 columns of S[bs] (column c holds tokens 2c, 2c+1)
                uint32_t pd[NCOL / 2];
                if (valid) {
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                    for (int c = 0; c < NCOL / 2; ++c) {
                        const float e0 = exp2f(__uint_as_float(sraw[2 * c]) - m_use);
                        const float e1 = exp2f(__uint_as_float(sraw[2 * c + 1]) - m_use);
                        sum0 += e0; sum1 += e1;
                        pd[c] = pack_bf16(e0, e1);
                    }
                    l_run += sum0 + sum1;
                    has_o = true;
                } else {
#pragma unroll
                    for (int c = 0; c < NCOL / 2; ++c) pd[c] = 0u;
                }
                uint32_t pk[64];
                if (PAIR) {
                    // block-diagonal P: this row weighs only its own half's tokens, the other 32 columns are zero
#pragma unroll
                    for (int c = 0; c < 32; ++c) { pk[c] = half ? 0u : pd[c]; pk[32 + c] = half ? pd[c] : 0u; }
                } else {
#pragma unroll
                    for (int c = 0; c < 64; ++c) pk[c] = pd[c % (NCOL / 2)];
                }
                tmem_st32(lane_addr + COL_S + bs * 128, pk);
                tmem_st32(lane_addr + COL_S + bs * 128 + 32, pk + 32);
                bool fail = false;
                if (tok_begin + (t + 1) * STEP > total) {
                    // last step of the sequence: V rows past the last key may hold anything, and they meet
                    // weight-0 columns of P in the product: clear them (thread r clears row r of the stage)
                    const int sv = t % NSV;
                    fail = !mbar_wait(bar(B_VFULL + sv), (t / NSV) & 1, abort_flag);
                    if (!fail && tok_begin + t * STEP + tl >= total) {
                        unsigned char* vrow = sm + SMEM_V + sv * STAGE_BYTES + tl * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4*>(vrow + HALF_BYTES + c * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
                    fence_async_smem();
                }
                tmem_wait_st();
                if (__any_sync(0xffffffffu, fail)) { ok = false; break; }
                if (tid == 64) TRACE(2, t, 5);
                tc_fence_before();
                mbar_arrive(bar(B_PFULL + bs));
                if (tid == 64) TRACE(2, t, 6);
            }
            // ---- epilogue: wait for the last product, (PAIR) merge the two halves, write out ----
            TRACE_MISC(5);
            if (ok) ok = mbar_wait_warp(bar(B_PVDONE + ((nsteps - 1) & 1)), ((nsteps - 1) >> 1) & 1, abort_flag);
            TRACE_MISC(6);
            // The rings are idle now (all copies landed, every product that read them has completed), so the
            // K ring serves as the PAIR exchange area: [32 col4][64 rows] float4 (32 KB) followed by 64 float2.
            float4* xch = reinterpret_cast<float4*>(sm + SMEM_K);
            float2* xst = reinterpret_cast<float2*>(sm + SMEM_K + 32 * 64 * 16);
            float w_me = 1.f, m_all = m_ref, l_all = l_run;
            if (PAIR && ok) {
                // lanes 64-127 hand their statistics to lanes 0-63, which answer with the merge weight
                if (half == 1) {
                    xst[lrow] = make_float2(has_o ? m_ref : -INFINITY, l_run);
                    mbar_arrive(bar(B_XSTAT));
                    ok = mbar_wait(bar(B_XWGT), 0, abort_flag);
                    w_me = has_o ? xst[lrow].x : 0.f;
                } else {
                    ok = mbar_wait(bar(B_XSTAT), 0, abort_flag);
                    const float2 other = xst[lrow];
                    const float mm = has_o ? m_ref : -INFINITY;
                    m_all = fmaxf(mm, other.x);
                    const float m_fin = (m_all == -INFINITY) ? 0.f : m_all;
                    w_me = has_o ? exp2f(m_ref - m_fin) : 0.f;
                    const float w_other = exp2f(other.x - m_fin);       // 0 when the other half saw nothing
                    l_all = l_run * w_me + other.y * w_other;
                    xst[lrow] = make_float2(w_other, 0.f);
                    mbar_arrive(bar(B_XWGT));
                }
                ok = __all_sync(0xffffffffu, ok);
            }
            TRACE_MISC(7);
            if (ok) {
                tc_fence_after();
                const bool final_out = (p.n_split == 1);
                const float inv = final_out ? (l_all > 0.f ? 1.f / l_all : 0.f) : 1.f;
                const size_t slot = ((size_t)unit * p.n_split + split) * ROWS + lrow;
                __nv_bfloat16* orow = p.out + (((size_t)b * N + node) * p.Hq + head) * D;
                float* prow = p.part_o + slot * D;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t o[32];
                    tmem_ld32(lane_addr + COL_O + ch * 32, o);
                    tmem_wait_ld();
                    float v[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) v[c] = has_o ? __uint_as_float(o[c]) * w_me : 0.f;
                    bool got = true;
                    if (PAIR) {
                        if (half == 1) {
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4)
                                xch[(ch * 8 + c4) * 64 + lrow] = make_float4(v[4 * c4], v[4 * c4 + 1], v[4 * c4 + 2], v[4 * c4 + 3]);
                            mbar_arrive(bar(B_XCH + ch));
                        } else {
                            got = mbar_wait(bar(B_XCH + ch), 0, abort_flag);
                            if (got) {
#pragma unroll
                                for (int c4 = 0; c4 < 8; ++c4) {
                                    const float4 w = xch[(ch * 8 + c4) * 64 + lrow];
                                    v[4 * c4] += w.x; v[4 * c4 + 1] += w.y; v[4 * c4 + 2] += w.z; v[4 * c4 + 3] += w.w;
                                }
                            }
                        }
                    }
                    if (row_ok && half == 0 && got) {
                        if (final_out) {
#pragma unroll
                            for (int c8 = 0; c8 < 4; ++c8)
                                *reinterpret_cast<uint4*>(orow + ch * 32 + c8 * 8) =
                                    make_uint4(pack_bf16(v[8 * c8] * inv, v[8 * c8 + 1] * inv), pack_bf16(v[8 * c8 + 2] * inv, v[8 * c8 + 3] * inv),
                                               pack_bf16(v[8 * c8 + 4] * inv, v[8 * c8 + 5] * inv), pack_bf16(v[8 * c8 + 6] * inv, v[8 * c8 + 7] * inv));
                        } else {
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4)
                                *reinterpret_cast<float4*>(prow + ch * 32 + c4 * 4) = make_float4(v[4 * c4], v[4 * c4 + 1], v[4 * c4 + 2], v[4 * c4 + 3]);
                        }
                    }
                }
                if (row_ok && half == 0) {
                    if (final_out) {
                        if (p.lse) p.lse[((size_t)b * p.Hq + head) * N + node] =
                            l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                    } else {
                        *reinterpret_cast<float2*>(p.part_ml + slot * 2) = make_float2(l_all > 0.f ? m_all : -INFINITY, l_all);
                    }
                }
                tc_fence_before();
            }
        }
    } else if (p.n_split > 1 || total == 0) {
        // nothing to attend to in this range: an empty partial, or a zero output for an empty / rejected sequence
        for (int idx = tid; idx < ROWS * (D / 4); idx += kThreads) {
            const int r = idx / (D / 4), c4 = idx % (D / 4);
            const int gr = mblock * 128 + r;
            if (gr >= rows_total) continue;
            if (p.n_split > 1) {
                const size_t slot = ((size_t)unit * p.n_split + split) * ROWS + r;
                *reinterpret_cast<float4*>(p.part_o + slot * D + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                if (c4 == 0) *reinterpret_cast<float2*>(p.part_ml + slot * 2) = make_float2(-INFINITY, 0.f);
            } else {
                const int i = gr / G, hd = kvh * G + gr % G;
                *reinterpret_cast<uint2*>(p.out + (((size_t)b * N + i) * p.Hq + hd) * D + c4 * 4) = make_uint2(0, 0);
                if (c4 == 0 && p.lse) p.lse[((size_t)b * p.Hq + hd) * N + i] = -INFINITY;
            }
        }
    }

    // ---- tear-down: everyone meets, TMEM goes back ----
    TRACE_MISC(8);
    __syncthreads();
    TRACE_MISC(9);
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
extern "C" int vispec_debug_read_trace_misc(long long* host) {
    return cudaMemcpyFromSymbol(host, g_trace_misc, sizeof(g_trace_misc)) == cudaSuccess ? 0 : -1;
}
#endif

bool attn_tc5_supports(const AttnArgs& a) {
    return a.D == 128 && a.k_map && a.v_map && a.B > 0;
}

cudaError_t init_attn_tc5() {
    cudaError_t e = cudaFuncSetAttribute(attn_tc5_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ALLOC);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_tc5_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ALLOC);
}

cudaError_t launch_attn_tc5(const AttnArgs& a, cudaStream_t st, int* n_launches) {
    *n_launches = 0;
    const int rows_total = (a.Hq / a.Hkv) * a.N;
    const bool pair = rows_total <= 64;
    const int rows = pair ? 64 : 128;
    const int n_mblocks = pair ? 1 : (rows_total + 127) / 128;
    const int units = a.B * a.Hkv * n_mblocks;
    const int max_steps = (a.S_max + STEP - 1) / STEP;
    int n_split = a.sm_count / units;
    if (n_split < 1) n_split = 1;
    if (n_split > max_steps) n_split = max_steps;
    const size_t part_bytes = (size_t)rows * (a.D * 4 + 8);
    while (n_split > 1 && kCounterBytes + (size_t)units * n_split * part_bytes > a.ws_bytes) --n_split;

    Tc5Params p;
    p.q = (const __nv_bfloat16*)a.q; p.kv_len = a.kv_len; p.mask = a.mask;
    p.out = (__nv_bfloat16*)a.out; p.lse = a.lse;
    unsigned char* ws = (unsigned char*)a.ws + kCounterBytes;
    p.part_o = (float*)ws;
    p.part_ml = (float*)(ws + (size_t)units * n_split * rows * a.D * 4);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max; p.n_split = n_split; p.n_mblocks = n_mblocks;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.status = a.status;
    dim3 grid(n_split, units);
    if (pair) attn_tc5_kernel<true><<<grid, kThreads, SMEM_ALLOC, st>>>(*a.k_map, *a.v_map, p);
    else attn_tc5_kernel<false><<<grid, kThreads, SMEM_ALLOC, st>>>(*a.k_map, *a.v_map, p);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    ++*n_launches;
    if (n_split > 1) {
        err = launch_attn_combine(a, n_split, n_mblocks, rows, st);
        if (err != cudaSuccess) return err;
        ++*n_launches;
    }
    return cudaSuccess;
}

}  // namespace vispec
