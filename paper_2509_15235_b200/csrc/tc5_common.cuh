// Device helpers of the TMA + tcgen05 attention kernel: PTX wrappers, the work schedule every CTA derives from kv_len,
// the merge of split-KV partials, and the launch helper.  Included by the kernel's translation unit only.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

#include "vispec_internal.h"

namespace vispec {
namespace tc5 {

constexpr int D = 128;
constexpr int kMaxB = 32;                      // sequences per call these kernels take
constexpr float kRescaleGap = 8.0f;            // log2 units
constexpr long long kWaitCycles = 1500000000LL;   // ~0.8 s at 1.9 GHz

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
// Has the phase with parity `parity` completed?  One non-blocking test; its result can be left unused for a while.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for the completion of the phase with parity `parity`.  Returns false after ~limit cycles
// or as soon as another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit = kWaitCycles) {
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
            else if (now - t0 > limit) { *abort_flag = 1; return false; }
        }
    }
}
// The same wait for a barrier that threads of other CTAs of the cluster arrive on (acquire at cluster scope).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  long long limit = kWaitCycles) {
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63) == 63) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) { *abort_flag = 1; return false; }
        }
    }
}
// Same, with a warp-uniform result (every lane of a converged warp calls it): the warp-collective
// tcgen05.ld/st that follow must never be reached by only part of a warp.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
}
// The K/V tiles are read once per call: they are marked evict-first in L2 so that the stream does not push out
// what is read again soon (q, masks, partial results, the next kernels' operands).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(pol) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Thread-block cluster helpers (distributed shared memory).
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank)); return r;
}
__device__ __forceinline__ float4 dsmem_ld4(uint32_t a) {
    float4 v; asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory"); return v;
}
__device__ __forceinline__ float2 dsmem_ld2(uint32_t a) {
    float2 v; asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a) : "memory"); return v;
}
// The hardware cluster barrier in two halves: a warp arrives once and waits once per phase, all its lanes together
// (a wait taken by one lane and later by the other 31 never returns); the wait may sit anywhere later in the warp's
// path.  Relaxed arrival: what the peers must see, the initialised barriers, is published by fence.mbarrier_init.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
// One arrival on an mbarrier of another CTA of the cluster (address from dsmem_addr), ordered after this thread's
// earlier accesses at cluster scope.
__device__ __forceinline__ void mbar_arrive_peer(uint32_t peer_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(peer_bar) : "memory");
}
// Programmatic dependent launch: let the next kernel in the stream be scheduled / wait for the previous one.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
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
// The same with both operands described in shared memory.
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
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
// 128-bit shifts on (lo, hi) pairs; any shift count >= 0.
__device__ __forceinline__ void shr128(uint64_t lo, uint64_t hi, int s, uint64_t& rlo, uint64_t& rhi) {
    if (s >= 128) { rlo = 0; rhi = 0; }
    else if (s >= 64) { rlo = hi >> (s - 64); rhi = 0; }
    else if (s == 0) { rlo = lo; rhi = hi; }
    else { rlo = (lo >> s) | (hi << (64 - s)); rhi = hi >> s; }
}
__device__ __forceinline__ void shl128_fill(uint64_t lo, uint64_t hi, int s, uint64_t& rlo, uint64_t& rhi) {
    // shift left by s in (0, 128) and set the s vacated low bits
    if (s >= 64) { rlo = ~0ull; rhi = (lo << (s - 64)) | (s == 64 ? 0ull : ((1ull << (s - 64)) - 1)); }
    else { rlo = (lo << s) | ((1ull << s) - 1); rhi = (hi << s) | (lo >> (64 - s)); }
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct Tc5Params {
    const __nv_bfloat16* q; const int32_t* kv_len; const uint64_t* mask;
    __nv_bfloat16* out; float* lse;
    float4* part_o;            // [slot][32 col4][ROWS]: column-of-4 major, so that a warp's 32 rows are contiguous
    float2* part_ml;           // [slot][ROWS]: (m in log2 units or -inf, l)
    int B, N, Hq, Hkv, S_max, n_mblocks;
    int grid_attn;             // CTAs of the attention kernel (the merge kernel needs it for the schedule)
    int min_steps;             // a CTA is given at least this many steps (fewer CTAs work on small problems)
    int early;                 // stream committed-prefix tiles before waiting for the preceding kernel
    float scale_log2;
    int* status;
    int step;                  // cached tokens per pipeline step (rows of one K or V stage)
};

// The schedule every CTA (and the merge kernel) derives from kv_len.
struct Sched {
    int base[kMaxB + 1];   // first global step of sequence b; base[B] = T
    int steps[kMaxB];      // steps of one unit of sequence b (0: sequence rejected or empty)
    int len[kMaxB];        // committed length S of sequence b
    int units;             // units with at least one step
};

// ---- schedule ---------------------------------------------------------------------------------------
// Built by one full warp.  Reads kv_len only.
static __device__ void sched_build(Sched& s, const Tc5Params& p, int lane, int kv_first) {   // kv_first: kv_len[lane], fetched by the caller

    const int upb = p.Hkv * p.n_mblocks;        // units per sequence
    int carry = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
        const int b = b0 + lane;
        int st = 0, S = 0;
        if (b < p.B) {
            S = b0 == 0 ? kv_first : p.kv_len[b];
            const bool ok = (S >= 0 && S + p.N <= p.S_max);
            st = ok ? (S + p.N + p.step - 1) / p.step : 0;
            s.steps[b] = st;
            s.len[b] = S;
        }
        int x = st * upb;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (b < p.B) s.base[b] = carry + x - st * upb;
        carry += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) s.base[p.B] = carry;
    __syncwarp();
    int live = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
        const int b = b0 + lane;
        live += __popc(__ballot_sync(0xffffffffu, b < p.B && s.steps[b] > 0));
    }
    if (lane == 0) s.units = live * upb;
}
// Number of CTAs that get work: every CTA at least min_steps steps; a multiple of the unit count when
// the units are fewer than the CTAs (equally long units then never share a CTA).
__device__ __forceinline__ int sched_ctas(int T, int units, int grid, int min_steps) {
    int g = T / min_steps;
    g = g < 1 ? 1 : g;
    g = g < grid ? g : grid;
    if (units <= g) g = (g / units) * units;
    return g;
}
// (T * grid < 2^31 is checked on the host, so 32-bit arithmetic suffices)
__device__ __forceinline__ int cta_lo(int c, int T, int geff) { return (int)(((unsigned)c * (unsigned)T) / (unsigned)geff); }
// The CTA whose range holds global step g.
__device__ __forceinline__ int cta_of(int g, int T, int geff) {
    int c = (int)((((unsigned)g + 1u) * (unsigned)geff - 1u) / (unsigned)T);
    c = c > geff - 1 ? geff - 1 : c;
    while (cta_lo(c, T, geff) > g) --c;
    while (c + 1 < geff && cta_lo(c + 1, T, geff) <= g) ++c;
    return c;
}

struct Seg {
    int b, kvh, mblock, st0, n, steps, S, slot;    // slot < 0: the segment is a whole unit
};
struct SegIter {
    const Sched* s;
    int B, n_mblocks, g, lo, hi, cta;
    bool cl, cl_done;          // cluster schedule: exactly one segment (possibly empty), given in cl_seg
    Seg cl_seg;
    __device__ __forceinline__ bool next(Seg& o) {
        if (cl) {
            if (cl_done) return false;
            cl_done = true;
            o = cl_seg;
            return true;
        }
        if (g >= hi) return false;
        int l = 0, r = B;                               // first b with base[b] > g, minus one
        while (l < r) { const int m = (l + r) >> 1; if (s->base[m] <= g) l = m + 1; else r = m; }
        o.b = l - 1;
        o.steps = s->steps[o.b];
        o.S = s->len[o.b];
        const int rel = g - s->base[o.b];
        const int uib = rel / o.steps;
        o.st0 = rel - uib * o.steps;
        o.n = min(hi - g, o.steps - o.st0);
        o.kvh = uib / n_mblocks;
        o.mblock = uib - o.kvh * n_mblocks;
        const bool whole = (o.st0 == 0 && o.n == o.steps);
        o.slot = whole ? -1 : (g == lo ? 2 * cta : 2 * cta + 1);
        g += o.n;
        return true;
    }
};

// One (row, 16 output columns) of a unit: the partials of CTAs c0..c1 (slot 2c if the unit starts CTA c's range,
// else 2c + 1) folded into the final output.  Shared by the merge kernel and by the attention kernel's own merge.
template <int ROWS>
__device__ __forceinline__ void merge_row_cols(const float4* __restrict__ part_o, const float2* __restrict__ part_ml,
                                               __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int T, int geff,
                                               int ub, int c0, int c1, int b, int node, int head, int Hq, int N,
                                               int lrow, int cw) {
    auto slot_of = [&](int c) { return cta_lo(c, T, geff) >= ub ? 2 * c : 2 * c + 1; };
    // Segments are taken four at a time with every load of a group issued before the first use, so that a
    // group costs one memory round trip; groups are folded with the usual running-maximum rescale.
    float m_all = -INFINITY, l_all = 0.f;
    float4 acc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int cb = c0; cb <= c1; cb += 4) {
        float2 ml[4];
        float4 v[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = cb + j;
            ml[j] = make_float2(-INFINITY, 0.f);
#pragma unroll
            for (int k = 0; k < 4; ++k) v[j][k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c <= c1) {
                const int slot = slot_of(c);
                ml[j] = __ldcg(&part_ml[(size_t)slot * ROWS + lrow]);
                const float4* src = part_o + ((size_t)slot * 32 + cw * 4) * ROWS + lrow;
#pragma unroll
                for (int k = 0; k < 4; ++k) v[j][k] = __ldcg(src + (size_t)k * ROWS);
            }
        }
        float m_new = m_all;
#pragma unroll
        for (int j = 0; j < 4; ++j) m_new = fmaxf(m_new, ml[j].x);
        const float m_fin = (m_new == -INFINITY) ? 0.f : m_new;
        const float a = exp2f(m_all - m_fin);                 // 0 while nothing has been accumulated
        l_all *= a;
#pragma unroll
        for (int k = 0; k < 4; ++k) { acc[k].x *= a; acc[k].y *= a; acc[k].z *= a; acc[k].w *= a; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float w = exp2f(ml[j].x - m_fin);           // 0 for a segment that saw nothing (or is absent)
            l_all += ml[j].y * w;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[k].x += w * v[j][k].x; acc[k].y += w * v[j][k].y; acc[k].z += w * v[j][k].z; acc[k].w += w * v[j][k].w;
            }
        }
        m_all = m_new;
    }
    const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
    __nv_bfloat16* orow = out + (((size_t)b * N + node) * Hq + head) * D + cw * 16;
#pragma unroll
    for (int k = 0; k < 2; ++k)
        *reinterpret_cast<uint4*>(orow + k * 8) =
            make_uint4(pack_bf16(acc[2 * k].x * inv, acc[2 * k].y * inv), pack_bf16(acc[2 * k].z * inv, acc[2 * k].w * inv),
                       pack_bf16(acc[2 * k + 1].x * inv, acc[2 * k + 1].y * inv), pack_bf16(acc[2 * k + 1].z * inv, acc[2 * k + 1].w * inv));
    if (lse && cw == 0)
        lse[((size_t)b * Hq + head) * N + node] = l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
}

// One (row, 4 output columns) of a unit, the merge kernel's piece: sixteen segments at a time with every load issued
// before the first use (a unit cut over many CTAs - few sequences, long caches - is merged from dozens of partials,
// and a round of loads is a memory round trip).
template <int ROWS>
__device__ __forceinline__ void merge_row_c4(const float4* __restrict__ part_o, const float2* __restrict__ part_ml,
                                             __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int T, int geff,
                                             int ub, int c0, int c1, int b, int node, int head, int Hq, int N,
                                             int lrow, int c4) {
    auto slot_of = [&](int c) { return cta_lo(c, T, geff) >= ub ? 2 * c : 2 * c + 1; };
    float m_all = -INFINITY, l_all = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int cb = c0; cb <= c1; cb += 16) {
        float2 ml[16];
        float4 v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int c = cb + j;
            ml[j] = make_float2(-INFINITY, 0.f);
            v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c <= c1) {
                const int slot = slot_of(c);
                ml[j] = __ldcg(&part_ml[(size_t)slot * ROWS + lrow]);
                v[j] = __ldcg(part_o + ((size_t)slot * 32 + c4) * ROWS + lrow);
            }
        }
        float m_new = m_all;
#pragma unroll
        for (int j = 0; j < 16; ++j) m_new = fmaxf(m_new, ml[j].x);
        const float m_fin = (m_new == -INFINITY) ? 0.f : m_new;
        const float a = exp2f(m_all - m_fin);                 // 0 while nothing has been accumulated
        l_all *= a;
        acc.x *= a; acc.y *= a; acc.z *= a; acc.w *= a;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float w = exp2f(ml[j].x - m_fin);           // 0 for a segment that saw nothing (or is absent)
            l_all += ml[j].y * w;
            acc.x += w * v[j].x; acc.y += w * v[j].y; acc.z += w * v[j].z; acc.w += w * v[j].w;
        }
        m_all = m_new;
    }
    const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
    *reinterpret_cast<uint2*>(out + (((size_t)b * N + node) * Hq + head) * D + c4 * 4) =
        make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    if (lse && c4 == 0)
        lse[((size_t)b * Hq + head) * N + node] = l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
}

// The whole unit, by the softmax threads of the CTA that delivered the unit's last partial (thread st of nthreads).
// Not inlined: its accumulators stay out of the attention kernel's register budget.
struct MergeArgs { const float4* part_o; const float2* part_ml; __nv_bfloat16* out; float* lse; int Hq, G, N, rows_total; };
template <int ROWS>
__device__ __noinline__ void merge_unit(const MergeArgs m, int T, int geff, int ub, int c0, int c1, int b, int kvh,
                                        int mblock, int st, int nthreads) {
    for (int item = st; item < ROWS * 8; item += nthreads) {
        const int cw = item / ROWS, lrow = item - cw * ROWS;
        const int row = mblock * ROWS + lrow;
        if (row >= m.rows_total) continue;
        merge_row_cols<ROWS>(m.part_o, m.part_ml, m.out, m.lse, T, geff, ub, c0, c1, b, row / m.G, kvh * m.G + row % m.G,
                             m.Hq, m.N, lrow, cw);
    }
}

// pool [num_blocks][Hkv][page_rows][D] (tensor map (d, slot, block * Hkv + head)) or, token_major,
// [num_blocks][page_rows][Hkv][D] (tensor map (d, head, block * page_rows + slot));
// block_table[b][i] = pool block of logical slots [i * page_rows, (i + 1) * page_rows)
// Fourth kernel parameter of the instantiations with the fused rotary embedding (they serve contiguous caches, so it
// takes the place of PagedArgs; a larger common parameter block costs the other instantiations registers).
struct RopeArgs {
    const double2* rope_k;     // [B][N][D/2] (cos, sin) of positions * theta^(-2j/D), fp64: the k rows' rotation
    const float2* rope_q;      // the same angles in fp32: the q rows' rotation (q is only consumed, never written back)
    const __nv_bfloat16* k_new; const __nv_bfloat16* v_new;   // [B][N][Hkv][D] rows of the tree, to be placed at slots S + i
    __nv_bfloat16* k_cache; __nv_bfloat16* v_cache;            // [B][Hkv][S_max][D]
    int* unit_counters;        // as in PagedArgs
};
struct PagedArgs { const int32_t* block_table; int table_stride, page_rows, num_blocks, Hkv, N, token_major; int* status;
                   int* unit_counters; };   // even split: arrivals per unit (all zero between calls); nullptr: a merge kernel follows

// Merge of the partials of every unit that more than one CTA worked on, 4 warps per block, lane <-> row.  Two
// shapes: grid (unit, 2 * group of 32 rows + half of the columns), a warp sums 16 output columns over the unit's
// segments four at a time - for units cut into a few pieces; FINE: grid (unit, 8 * group of 32 rows + eighth of the
// columns), a warp sums 4 output columns sixteen segments at a time - for units cut over many CTAs (few sequences, long
// caches), where the rounds of loads are what the merge takes: qwen3b_S32768_N16_B1 (2 units over 148 CTAs) 42.7 ->
// 29.1 us per layer, qwen3b_S32768_N60_B1 34.8 -> 31.8; with many units of two partials the coarse shape is 3 % faster.
// The blocks are small so that they fit beside a resident attention CTA: they are launched early
// (programmatic dependent launch) and must not keep the next layer's attention CTAs off the SMs.
template <int ROWS, bool FINE = false>
__global__ void __launch_bounds__(128)
attn_tc5_merge_kernel(const Tc5Params p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    // The schedule, recomputed per thread from kv_len (which the attention kernel does not write) without
    // shared memory: beside a resident attention CTA an SM has no shared memory to spare.
    const int upb = p.Hkv * p.n_mblocks;
    const int unit = blockIdx.x, b = unit / upb, uib = unit - b * upb;
    int T = 0, live = 0, base_b = 0, steps = 0;
    for (int bb = 0; bb < p.B; ++bb) {
        const int S = p.kv_len[bb];
        const int st = (S >= 0 && S + p.N <= p.S_max) ? (S + p.N + p.step - 1) / p.step : 0;
        if (bb == b) { base_b = T; steps = st; }
        T += st * upb;
        live += st > 0 ? upb : 0;
    }
    pdl_wait();                                        // the partials are complete
    if (steps == 0) return;
    const int geff = sched_ctas(T, live, p.grid_attn, p.min_steps);
    const int ub = base_b + uib * steps, ue = ub + steps;
    const int c0 = cta_of(ub, T, geff), c1 = cta_of(ue - 1, T, geff);
    if (c0 == c1) return;                              // one CTA had the whole unit and wrote the output itself
    const int G = p.Hq / p.Hkv, N = p.N;
    const int kvh = uib / p.n_mblocks, mblock = uib - kvh * p.n_mblocks;
    const int lrow = (FINE ? blockIdx.y >> 3 : blockIdx.y >> 1) * 32 + lane;
    const int cw = FINE ? (blockIdx.y & 7) * 4 + warp : (blockIdx.y & 1) * 4 + warp;    // which 4 (FINE) or 16 output columns
    const int row = mblock * ROWS + lrow;
    if (row >= G * N) return;
    const int node = row / G, head = kvh * G + row % G;

    if (FINE) merge_row_c4<ROWS>(p.part_o, p.part_ml, p.out, p.lse, T, geff, ub, c0, c1, b, node, head, p.Hq, N, lrow, cw);
    else merge_row_cols<ROWS>(p.part_o, p.part_ml, p.out, p.lse, T, geff, ub, c0, c1, b, node, head, p.Hq, N, lrow, cw);
}

// Launch with programmatic stream serialisation and, when cluster > 0, thread-block clusters of that size.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (cluster > 0) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace tc5
}  // namespace vispec
