// Tree-verification attention for sm_100a (D = 128): TMA-staged K/V tiles, tcgen05 tensor-core products
// with fp32 accumulators in TMEM, fp32 online softmax (Eq. 1 restricted to prefix + ancestors), work split
// over the SMs.
//
// Work.  A *unit* is (sequence, kv head, block of <= 128 query rows, rows ordered node-major so that all heads
// and nodes of a head group share every K/V tile); it needs ceil((S+N)/128) *steps*, one per 128 cached
// tokens.  Two ways to spread the units over the CTAs (at most one CTA per SM):
//   cluster form     one thread-block cluster of k <= 8 CTAs per unit; the CTA of rank r takes the r-th of k
//                    equal parts of the unit's steps and parks its unnormalised partial (O, m, l) in its own
//                    shared memory; after a hardware cluster barrier rank r merges rows [r*rows/k, ...) of all
//                    k partials through distributed shared memory and writes them out.  One launch.
//   even split       all steps of all units, in the order (sequence, kv head, row block, step), form one line
//                    of T steps cut into equal ranges, one per CTA (the CTA count is a multiple of the unit
//                    count when the units are fewer than the SMs, so that equally long units are cut into
//                    whole CTAs).  A CTA runs a few *segments*: the tail of one unit, whole units, the head of
//                    another.  A segment that covers its whole unit writes the final bf16 output; any other
//                    writes a partial into one of the CTA's two slots (first segment -> slot 2c, a later one
//                    -> slot 2c+1) and a second, small kernel merges the partials of each unit.
// Both kernels derive the schedule from kv_len on the device, so the host never reads lengths.
//
// Inside a CTA the 12 warps are specialised:
//   warp 0     TMA producer: K ring and V ring of 128-token stages (3 x 32 KB each, 128-byte swizzle, evict-first
//              in L2); it runs ahead across segment boundaries
//   warp 1     issuer (one thread) of S = Q K^T as 128x128x16 tcgen05.mma; owns the TMEM allocation
//   warp 2     issuer (one thread) of O += P V; the two chains wait on different barriers, so each has its own
//              thread and neither's waits delay the other's instructions
//   warp 3     derives the schedule from kv_len; with at most 64 rows per unit (its lane 0; the whole warp on a paged
//              cache) and on pools of 16-row blocks it then produces the V ring, so that warp 0's K copies never
//              queue behind a wait for a V stage
//   warps 4-11 softmax: thread <-> TMEM lane; warps w and w+4 share the same 32 accumulator rows and each takes
//              half of a step's columns (the row maximum is exchanged through shared memory), so a row costs
//              no shuffles; they also load Q at the start of every segment and run the segment epilogue
// TMEM map (512 columns x 128 lanes): S[0] 0..127, S[1] 128..255, O 256..383, P[0] 384..447, P[1] 448..511.
// P (bf16, packed two per column) is the A operand of the PV product and never touches shared memory; Q
// sits in shared memory in the same swizzled K-major layout as a K stage.  S and P are double-buffered: S
// is released as soon as the softmax threads have read it, so the S product of step u+1 and the PV
// product of step u-1 run while step u is in the softmax.
//
// Two row layouts share the code:
//   FULL  (G*N > 64):  lane r holds query row r of the block.
//   PAIR  (G*N <= 64): the <= 64 query rows are duplicated, lanes 0-63 take tokens 0-63 of each step and
//                      lanes 64-127 tokens 64-127 (P is block-diagonal); the two halves keep independent
//                      softmax states and are merged once per segment through shared memory.
// The running maximum is only moved when a tile exceeds it by more than 2^8 (O and l share the reference, so
// the result is exact either way); O is therefore re-scaled in TMEM rarely.
//
// Programmatic dependent launch: every launch carries the programmatic stream serialisation attribute.  The
// attention kernel reads kv_len and (when early prefetch is on) streams K/V tiles that lie wholly inside the
// committed prefix before it waits for the preceding kernel; q, tree_mask, the tree's own K/V rows and every
// write come after that wait.
//
// Every wait on an mbarrier is bounded; on a timeout the CTA records VISPEC_E_TIMEOUT, drains its own
// copies, frees its TMEM and returns.  The cluster form's hardware cluster barriers (two; three phases with the
// fused rotary embedding, whose first is arrived at after set-up and waited for by whole warps before their first
// signal to a peer) are reached by every thread of every CTA of the cluster (all other waits being bounded), so
// they end.
//
// Fused rotary embedding (ROPE instantiations, cluster form, contiguous caches): each rank of a unit's cluster
// rotates and places its share of the unit's N tree rows beside its (rotating) Q load and tells every rank; the
// producers hold back the tiles that contain those slots until all ranks have told.
#include <cuda_bf16.h>
#include <cstdio>
#include <cstdlib>
#include <type_traits>

#include "tc5_common.cuh"

namespace vispec {

using namespace tc5;

namespace {

constexpr int STEP = 128;                      // tokens per pipeline step = rows of one K or V stage
constexpr int HALF_BYTES = STEP * 128;         // one d-half (64 columns) of a stage: 128 rows x 128 B
constexpr int STAGE_BYTES = 2 * HALF_BYTES;    // 32 KB
constexpr int NSK = 3, NSV = 3;
constexpr int kThreads = 384;                  // 12 warps: producer, two issuers, one spare, eight softmax
constexpr int kSmx = 256;                      // softmax threads
constexpr int SMEM_K = 0;
constexpr int SMEM_V = SMEM_K + NSK * STAGE_BYTES;
constexpr int SMEM_Q = SMEM_V + NSV * STAGE_BYTES;             // Q tile, 128 rows, laid out like a K stage; between
                                                               // segments it is the PAIR exchange [32 col4][64 rows] float4
constexpr int SMEM_XM = SMEM_Q + STAGE_BYTES;                  // 512 floats: tile maxima / row statistics exchanged between threads
constexpr int SMEM_BAR = SMEM_XM + 2048;
constexpr int BAR_BYTES = 256;
constexpr int SMEM_SCHED = SMEM_BAR + BAR_BYTES;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_S = 0, COL_O = 256, COL_P = 384;

enum { B_KFULL = 0, B_KEMPTY = B_KFULL + NSK, B_VFULL = B_KEMPTY + NSK, B_VEMPTY = B_VFULL + NSV,
       B_SFULL = B_VEMPTY + NSV, B_SFREE = B_SFULL + 2, B_PFULL = B_SFREE + 2, B_PVDONE = B_PFULL + 2,
       B_QFULL = B_PVDONE + 2, B_PAIRX = B_QFULL + 1, B_XCH = B_PAIRX + 4, B_XFREE = B_XCH + 1,
       B_SEGSYNC = B_XFREE + 1,
       B_ROWS = B_SEGSYNC + 1,      // fused rotary embedding: every rank of the cluster has put its share of the tree rows into the cache
       B_COUNT = B_ROWS + 1 };
static_assert(B_COUNT * 8 + 20 <= BAR_BYTES, "barrier block too small");

constexpr int SMEM_TABRING = SMEM_SCHED + ((int)sizeof(Sched) + 15) / 16 * 16;   // 8 steps x 8 block numbers (paged cache)
constexpr int SMEM_TOTAL = SMEM_TABRING + 256;
constexpr int SMEM_ALLOC = SMEM_TOTAL;                         // the base must come out 1024-byte aligned (checked)
static_assert(SMEM_ALLOC <= 232448, "over the 227 KB a CTA may have");






// ---- producer of a paged segment ---------------------------------------------------------------------
// Paged cache: a step's 128 slots are 128 / page_rows pool blocks, each its own box.  Run by the whole producer
// warp: lane j owns block j of every step - its table entry and its four copies (two d-halves of K and of V) -
// so that one instruction issues the copies of all the step's blocks; lane 0 alone waits for the free stage and
// posts the expected byte count.  The block numbers travel from the table to a small ring in shared memory by
// asynchronous 4-byte copies issued six steps ahead of their use: a plain load held in a register that long would
// share a scoreboard with the waits and copies in between and stall them for its whole latency.  Blocks that start
// at or past kv_len + N are not fetched: their table entries need not exist, and the rows they would fill are
// masked like any slot past the end.  Not inlined, so that it stays out of the kernel's register budget, and
// everything by value, so that the caller's counters stay in registers.  Returns steps issued in full | K-only
// step << 28 | a wait gave up << 29 | has waited for the preceding kernel << 30 (the same in every lane).
constexpr int kTabRing = 4, kTabAhead = 3;     // steps held in a ring / steps a copy is issued ahead (two rings of
                                               // 128 bytes: the K producer's and, where V has its own warp, the V producer's)
__device__ __noinline__ uint32_t produce_paged(const PagedArgs p, const CUtensorMap* k_map, const CUtensorMap* v_map,
                                               int b, int kvh, int st0, int n, int S, uint32_t base, uint32_t bars,
                                               uint32_t ring, volatile int* abort_flag, uint64_t pol, int it,
                                               bool waited, int lane, int which /* 0: K and V, 1: K only, 2: V only */) {
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    const int nsub = STEP / p.page_rows;
    const uint32_t sub_bytes = (uint32_t)p.page_rows * 128u;
    const int32_t* trow = p.block_table + (size_t)b * p.table_stride;
    const int total = S + p.N;
    const bool mine = lane < nsub;
    auto issue = [&](int t) {                  // one group per step and lane, empty where there is nothing to fetch
        const int blk = (st0 + t) * nsub + lane;
        if (mine && t < n && blk * p.page_rows < total)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(ring + 4u * (uint32_t)((t % kTabRing) * 8 + lane)), "l"(trow + blk) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int t = 0; t < kTabAhead; ++t) issue(t);
    uint32_t fail = 0;
    int t = 0;
    for (; t < n; ++t, ++it) {
        issue(t + kTabAhead);
        asm volatile("cp.async.wait_group %0;" ::"n"(kTabAhead) : "memory");     // this lane's entry of step t has landed
        const int tok = (st0 + t) * STEP;
        if (!waited && tok + STEP > S) { pdl_wait(); waited = true; }   // the tree's rows come from the preceding kernel
        const bool load = mine && tok + lane * p.page_rows < total;
        int c1 = 0, c2 = -p.page_rows;                                   // a box outside the pool: reads as zeros
        if (load) {
            int e;
            asm volatile("ld.shared.s32 %0, [%1];" : "=r"(e) : "r"(ring + 4u * (uint32_t)((t % kTabRing) * 8 + lane)) : "memory");
            if (e >= 0 && e < p.num_blocks) {
                c1 = p.token_major ? kvh : 0;
                c2 = p.token_major ? e * p.page_rows : e * p.Hkv + kvh;
            } else if (p.status) {
                atomicCAS(p.status, 0, VISPEC_E_RANGE);
            }
        }
        const uint32_t tx = (uint32_t)__popc(__ballot_sync(0xffffffffu, load)) * sub_bytes * 2u;
        const int sk = it % NSK, sv = it % NSV;
        bool w = true;
        if (which != 2) {
            if (lane == 0) {
                w = mbar_wait(bar(B_KEMPTY + sk), ((it / NSK) & 1) ^ 1, abort_flag);
                if (w) mbar_expect_tx(bar(B_KFULL + sk), tx);
            }
            w = __shfl_sync(0xffffffffu, w, 0);                          // the byte count is posted before any lane copies
            if (!w) { fail = 2u << 28; break; }
            if (load) {
                tma_load_3d(base + SMEM_K + sk * STAGE_BYTES + lane * sub_bytes, k_map, bar(B_KFULL + sk), 0, c1, c2, pol);
                tma_load_3d(base + SMEM_K + sk * STAGE_BYTES + HALF_BYTES + lane * sub_bytes, k_map, bar(B_KFULL + sk), 64, c1, c2, pol);
            }
        }
        if (which != 1) {
            if (lane == 0) {
                w = mbar_wait(bar(B_VEMPTY + sv), ((it / NSV) & 1) ^ 1, abort_flag);
                if (w) mbar_expect_tx(bar(B_VFULL + sv), tx);
            }
            w = __shfl_sync(0xffffffffu, w, 0);
            if (!w) { fail = (which == 2 ? 2u : 3u) << 28; break; }      // (V only: nothing of this step was issued)
            if (load) {
                tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + lane * sub_bytes, v_map, bar(B_VFULL + sv), 0, c1, c2, pol);
                tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + HALF_BYTES + lane * sub_bytes, v_map, bar(B_VFULL + sv), 64, c1, c2, pol);
            }
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");                     // nothing of this segment stays in flight
    return (uint32_t)t | fail | (waited ? 1u << 30 : 0u);
}

// ---- fused rotary embedding ---------------------------------------------------------------------------
// Eight pairs (x = element j of the lower half, y = element j + D/2) rotated by their angles: fp64 with one rounding
// to bf16 for the k rows that go to the cache, fp32 for q rows (consumed by the product, never stored).
__device__ __forceinline__ void rope8_f64(uint4& lo, uint4& hi, const double2* cs) {
    __nv_bfloat16* a = reinterpret_cast<__nv_bfloat16*>(&lo);
    __nv_bfloat16* b = reinterpret_cast<__nv_bfloat16*>(&hi);
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const double x = (double)__bfloat162float(a[t]), y = (double)__bfloat162float(b[t]);
        a[t] = __double2bfloat16(x * cs[t].x - y * cs[t].y);
        b[t] = __double2bfloat16(y * cs[t].x + x * cs[t].y);
    }
}
__device__ __forceinline__ void rope8_f32(uint4& lo, uint4& hi, const float2* cs) {
    __nv_bfloat16* a = reinterpret_cast<__nv_bfloat16*>(&lo);
    __nv_bfloat16* b = reinterpret_cast<__nv_bfloat16*>(&hi);
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const float x = __bfloat162float(a[t]), y = __bfloat162float(b[t]);
        a[t] = __float2bfloat16_rn(x * cs[t].x - y * cs[t].y);
        b[t] = __float2bfloat16_rn(y * cs[t].x + x * cs[t].y);
    }
}
// Prologue of a CTA with the fused rotary embedding (one function, so that both memory round trips overlap): the upper
// half of the softmax threads fetches this rank's share of the tree rows, tree index in [t_lo, t_hi), of (sequence b,
// kv head kvh): one item = (k row, pair of 16-byte chunks c and c + 8) with its eight fp64 (cos, sin) pairs, plus two
// 16-byte chunks of v rows; then every thread fetches its part of the Q tile (chunk pair (c, c + 8) of rows st/8,
// st/8 + 32, ... with eight fp32 pairs each); only then the k rows are rotated (fp64, one rounding: bit-compatible with the
// rotation kernel) and written to slots S + t of the cache with the v rows, and the Q rows are rotated (fp32: they feed
// the score product only) into the swizzled tile.  Shares of more than 16 rows take further passes after that.  Not
// inlined: its registers stay out of the step loop's budget and its code out of the step loop's way.
template <bool PAIR, int ROWS>
__device__ __noinline__ void rope_prologue(unsigned char* sm, const __nv_bfloat16* __restrict__ q, const RopeArgs p, int N_, int Hq,
                                           int Hkv_, int S_max_, int G, int rows_total, int b, int kvh, int mblock, int S,
                                           int t_lo, int t_hi, int st) {
    constexpr int HALF = kSmx / 2;
    const int ps = st - HALF;                     // >= 0: this thread places rows
    const size_t cache_row0 = ((size_t)b * Hkv_ + kvh) * S_max_ + S;
    const int nk = (t_hi - t_lo) * 8, nv = (t_hi - t_lo) * 16;
    auto k_src = [&](int i) { return reinterpret_cast<const uint4*>(p.k_new + (((size_t)b * N_ + t_lo + (i >> 3)) * Hkv_ + kvh) * D); };
    auto k_tab = [&](int i) { return p.rope_k + ((size_t)b * N_ + t_lo + (i >> 3)) * (D / 2) + 8 * (i & 7); };
    auto v_src = [&](int i) { return reinterpret_cast<const uint4*>(p.v_new + (((size_t)b * N_ + t_lo + (i >> 4)) * Hkv_ + kvh) * D) + (i & 15); };
    auto k_store = [&](int i, uint4& lo, uint4& hi, const double2* cs) {
        rope8_f64(lo, hi, cs);
        uint4* dst = reinterpret_cast<uint4*>(p.k_cache + (cache_row0 + t_lo + (i >> 3)) * D);
        dst[i & 7] = lo; dst[(i & 7) + 8] = hi;
    };
    auto v_store = [&](int i, const uint4& x) { reinterpret_cast<uint4*>(p.v_cache + (cache_row0 + t_lo + (i >> 4)) * D)[i & 15] = x; };

    // ---- tree rows, first pass (16 rows): loads
    uint4 klo = make_uint4(0, 0, 0, 0), khi = klo, vx[2];
    double2 cs[8];
    const bool has_k = ps >= 0 && ps < nk;
    if (has_k) {
        const uint4* src = k_src(ps);
        klo = src[ps & 7]; khi = src[(ps & 7) + 8];
        const double2* tab = k_tab(ps);
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = tab[j];
    }
#pragma unroll
    for (int u = 0; u < 2; ++u)
        if (ps >= 0 && ps + HALF * u < nv) vx[u] = *v_src(ps + HALF * u);
    // (with 128 rows per unit the Q tile alone takes 96 registers per thread: there the rows are finished first; timed in
    // one call on qwen7b: 18.7 against 20.1 us per layer of a step with both sets of loads in flight)
    auto finish_rows = [&]() {
        if (has_k) k_store(ps, klo, khi, cs);
#pragma unroll
        for (int u = 0; u < 2; ++u)
            if (ps >= 0 && ps + HALF * u < nv) v_store(ps + HALF * u, vx[u]);
    };
    if (!PAIR) finish_rows();

    // ---- Q tile: loads
    constexpr int PITEMS = ROWS * 8 / kSmx;
    const int c = st & 7;
    uint4 lo[PITEMS], hi[PITEMS];
    float4 tab[PITEMS][4];
#pragma unroll
    for (int k = 0; k < PITEMS; ++k) {
        const int row = mblock * ROWS + (st >> 3) + 32 * k;
        lo[k] = make_uint4(0, 0, 0, 0); hi[k] = lo[k];
#pragma unroll
        for (int j = 0; j < 4; ++j) tab[k][j] = make_float4(1.f, 0.f, 1.f, 0.f);
        if (row < rows_total) {
            const int node = row / G, head = kvh * G + row % G;
            const uint4* src = reinterpret_cast<const uint4*>(q + (((size_t)b * N_ + node) * Hq + head) * D);
            lo[k] = src[c]; hi[k] = src[c + 8];
            const float4* t4 = reinterpret_cast<const float4*>(p.rope_q + ((size_t)b * N_ + node) * (D / 2) + 8 * c);
#pragma unroll
            for (int j = 0; j < 4; ++j) tab[k][j] = t4[j];
        }
    }

    // ---- tree rows, first pass: rotate and store
    if (PAIR) finish_rows();

    // ---- Q tile: rotate into shared memory
#pragma unroll
    for (int k = 0; k < PITEMS; ++k) {
        const int r = (st >> 3) + 32 * k;
        rope8_f32(lo[k], hi[k], reinterpret_cast<const float2*>(tab[k]));
        unsigned char* dst = sm + SMEM_Q + r * 128 + ((c ^ (r & 7)) << 4);
        *reinterpret_cast<uint4*>(dst) = lo[k];
        *reinterpret_cast<uint4*>(dst + HALF_BYTES) = hi[k];
        if (PAIR) {
            *reinterpret_cast<uint4*>(dst + 64 * 128) = lo[k];
            *reinterpret_cast<uint4*>(dst + HALF_BYTES + 64 * 128) = hi[k];
        }
    }

    // ---- tree rows beyond the first 16 of the share
    if (ps >= 0) {
        for (int i = ps + HALF, j = ps + 2 * HALF; i < nk || j < nv; i += HALF, j += 2 * HALF) {
            const bool more_k = i < nk;
            if (more_k) {
                const uint4* src = k_src(i);
                klo = src[i & 7]; khi = src[(i & 7) + 8];
                const double2* tb = k_tab(i);
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) cs[jj] = tb[jj];
            }
#pragma unroll
            for (int u = 0; u < 2; ++u)
                if (j + HALF * u < nv) vx[u] = *v_src(j + HALF * u);
            if (more_k) k_store(i, klo, khi, cs);
#pragma unroll
            for (int u = 0; u < 2; ++u)
                if (j + HALF * u < nv) v_store(j + HALF * u, vx[u]);
        }
    }
}

// The softmax's exponentials are what the special-function pipe (16 lanes per SM) spends a step on; one in
// 2 * kPolyEvery of them is formed on the FMA pipe instead.  Timed in one call, none / 1 in 6 / 1 in 8 / 1 in 16:
// llava7b 17.33 / 17.12 / 17.15 / 17.24 us per layer, qwen7b 16.5 / 16.2 / 16.2 / 16.3, qwen3b_S8192_N60_B4 32.1 / 31.3 /
// 31.3 / 31.8; 1 in 4 and 1 in 2 were slower again (issue slots).
constexpr int kPolyEvery = 4;
// 2^x on the FMA pipe (x <= 120; anything at or below -126 comes out as a denormal, which the flush-to-zero arithmetic that
// follows reads as 0): nearest integer by the 1.5 * 2^23 trick, cubic on the remainder in [-0.5, 0.5] (relative error
// 8e-5, well inside the bf16 rounding of P), the integer added into the exponent field.
__device__ __forceinline__ float exp2_fma(float x) {
    x = fmaxf(x, -126.f);
    const float z = x + 12582912.f;
    const float f = x - (z - 12582912.f);
    float p = fmaf(f, 0.055088684f, 0.24260405f);
    p = fmaf(p, f, 0.69327623f);
    p = fmaf(p, f, 0.99992895f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(z) << 23));
}

// PAGED instantiations carry the paged producer; the others are compiled without it (its call sites cost the
// contiguous kernels registers they do not have to spare).
template <bool PAIR, bool CL, bool PAGED, bool ROPE = false>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc5_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const Tc5Params p,
                const std::conditional_t<ROPE, RopeArgs, PagedArgs> pa) {
    static_assert(!(ROPE && PAGED), "the fused rotary embedding serves contiguous caches");
    static_assert(!ROPE || CL, "the fused rotary embedding exists in the cluster form only (the even split goes through the rotation kernel)");
    constexpr int ROWS = PAIR ? 64 : 128;      // distinct query rows per CTA
    constexpr int NC = PAIR ? 32 : 64;         // tokens of a step one softmax thread handles (two threads per row)
    // The V ring can have a producer of its own, the spare warp (its lane 0; paged: all of it).  With at most 64 rows per
    // unit it always has; with 128 only for pools of 16-row blocks, where one warp issuing a step's 32 copies is what
    // holds the call back (larger blocks lose 1 % with two producers, like the contiguous cache).
    constexpr bool SPLIT_V = PAIR || PAGED;
    bool split_v = PAIR;
    if constexpr (PAGED && !PAIR) split_v = pa.page_rows <= 16;
    extern __shared__ __align__(1024) unsigned char sm[];
    // the schedule hangs on kv_len, and a CTA that starts after its predecessor kernel has ended hangs on the
    // schedule: the load goes out first
    int kv_first = 0;
    if (p.early && threadIdx.x >= 96 && threadIdx.x < 128 && (int)threadIdx.x - 96 < p.B) kv_first = p.kv_len[threadIdx.x - 96];
    const uint32_t base = smem_u32(sm);
    if (base & 1023u) {
        // the swizzled tiles need a 1024-byte aligned base; every CTA sees the same base, so all of them leave
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)VISPEC_E_UNSUPPORTED);
        return;
    }
    const uint32_t bars = base + SMEM_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + SMEM_BAR + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + SMEM_BAR + B_COUNT * 8 + 8);
    volatile int* seg_flag = abort_flag + 1;               // this CTA delivered the last partial of the unit just finished
    Sched& sched = *reinterpret_cast<Sched*>(sm + SMEM_SCHED);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int G = p.Hq / p.Hkv, N = p.N, W = (N + 63) >> 6;
    const int rows_total = G * N;

    if (tid == 0) {
        for (int i = 0; i < NSK; ++i) { mbar_init(bar(B_KFULL + i), 1); mbar_init(bar(B_KEMPTY + i), 1); }
        for (int i = 0; i < NSV; ++i) { mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_SFULL + i), 1); mbar_init(bar(B_SFREE + i), kSmx);
            mbar_init(bar(B_PFULL + i), kSmx); mbar_init(bar(B_PVDONE + i), 1);
        }
        for (int i = 0; i < 4; ++i) mbar_init(bar(B_PAIRX + i), 64);
        mbar_init(bar(B_QFULL), kSmx);
        mbar_init(bar(B_XCH), 128); mbar_init(bar(B_XFREE), 128);
        mbar_init(bar(B_SEGSYNC), kSmx);
        if (ROPE) mbar_init(bar(B_ROWS), cluster_size());
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    if (!p.early) {                                          // nothing is read before the preceding kernel has ended
        pdl_wait();
        if (warp == 3 && lane < p.B) kv_first = p.kv_len[lane];
    }
    if (warp == 3) sched_build(sched, p, lane, kv_first);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Fused rotary embedding: the ranks signal one another's barriers, which must exist by then.  Everybody arrives at
    // the cluster barrier here (relaxed: fence.mbarrier_init has published the barriers); a warp waits, as a whole,
    // where it first needs the guarantee.
    bool cl_waited = !ROPE;
    if (ROPE) cluster_arrive();

    // Schedule.  Cluster form: cluster <-> unit, the CTA of rank r takes the r-th of k equal parts of the
    // unit's steps (an empty part still takes part in the exchange).  Otherwise: equal ranges of the line of
    // all steps.
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
        if ((PAGED || lane == 0) && active) {        // paged: the whole warp, each lane one block of a step
            const uint64_t pol = l2_evict_first_policy();
            bool waited = !p.early;
            int it = 0, nk = 0, nv = 0;          // steps started; K / V stages issued
            bool ok = true;
            SegIter si = make_iter();
            Seg sg;
            if constexpr (PAGED) {
                while (ok && si.next(sg)) {
                    const uint32_t r = produce_paged(pa, &k_map, &v_map, sg.b, sg.kvh, sg.st0, sg.n, sg.S, base, bars, base + SMEM_TABRING, abort_flag, pol, it, waited, lane, split_v ? 1 : 0);
                    const int done = (int)(r & 0x0fffffffu);
                    it += done; nv += split_v ? 0 : done; nk += done + (int)((r >> 28) & 1u);
                    ok = !((r >> 29) & 1u);
                    waited = (r >> 30) & 1u;
                }
            }
            while (!PAGED && ok && si.next(sg)) {
                const int bh = sg.b * p.Hkv + sg.kvh;
                for (int t = 0; t < sg.n; ++t, ++it) {
                    const int tok = (sg.st0 + t) * STEP;
                    if (!waited && tok + STEP > sg.S) { pdl_wait(); waited = true; }   // the tree's rows come from the preceding kernel
                    if (ROPE && tok + STEP > sg.S) {
                        // the tile holds tree rows: every rank's share must be in the cache, and ordered before this copy
                        if (!mbar_wait_cluster(bar(B_ROWS), 0, abort_flag)) { ok = false; break; }
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                    const int sk = it % NSK;
                    if (!mbar_wait(bar(B_KEMPTY + sk), ((it / NSK) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(bar(B_KFULL + sk), STAGE_BYTES);
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES, &k_map, bar(B_KFULL + sk), 0, tok, bh, pol);
                    tma_load_3d(base + SMEM_K + sk * STAGE_BYTES + HALF_BYTES, &k_map, bar(B_KFULL + sk), 64, tok, bh, pol);
                    ++nk;
                    if constexpr (!SPLIT_V) {
                        const int sv = it % NSV;
                        if (!mbar_wait(bar(B_VEMPTY + sv), ((it / NSV) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(bar(B_VFULL + sv), STAGE_BYTES);
                        tma_load_3d(base + SMEM_V + sv * STAGE_BYTES, &v_map, bar(B_VFULL + sv), 0, tok, bh, pol);
                        tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + HALF_BYTES, &v_map, bar(B_VFULL + sv), 64, tok, bh, pol);
                        ++nv;
                    }
                }
            }
            if (*abort_flag && lane == 0) {
                // drain: wait (bounded, fresh timer) until every copy this warp issued has landed
                volatile int never = 0;
                for (int u = max(0, nk - NSK); u < nk; ++u) mbar_wait(bar(B_KFULL + u % NSK), (u / NSK) & 1, &never);
                for (int u = max(0, nv - NSV); u < nv; ++u) mbar_wait(bar(B_VFULL + u % NSV), (u / NSV) & 1, &never);
            }
        }
        __syncwarp();
    } else if (warp == 3) {
        // ================= TMA producer of the V ring (contiguous caches, rows <= 64) =================
        // A V stage is free only after the PV product of the step it held, a softmax later than the K stage of the
        // same step: one thread issuing both in order holds the K copies back behind every wait for a V stage.
        // Measured in one call, one thread against two: 17.70 -> 17.50 us per layer on llava7b, 17.11 -> 16.91 on
        // paper_tree, 71.4 -> 71.0 on llava13b_b4; with 128 rows per unit the two threads lose 1 % (16.43 -> 16.59 on
        // qwen7b, 63.3 -> 63.8 on qwen3b_S32768_N16_B8), so those keep the single producer.
        if constexpr (SPLIT_V && PAGED) {
            if (active && split_v) {
                const uint64_t pol = l2_evict_first_policy();
                bool waited = !p.early, ok = true;
                int it = 0;
                SegIter si = make_iter();
                Seg sg;
                while (ok && si.next(sg)) {
                    const uint32_t r = produce_paged(pa, &k_map, &v_map, sg.b, sg.kvh, sg.st0, sg.n, sg.S, base, bars, base + SMEM_TABRING + 128, abort_flag, pol, it, waited, lane, 2);
                    it += (int)(r & 0x0fffffffu);
                    ok = !((r >> 29) & 1u);
                    waited = (r >> 30) & 1u;
                }
                if (*abort_flag && lane == 0) {
                    volatile int never = 0;
                    for (int u = max(0, it - NSV); u < it; ++u) mbar_wait(bar(B_VFULL + u % NSV), (u / NSV) & 1, &never);
                }
            }
        } else if (SPLIT_V && lane == 0 && active) {
            const uint64_t pol = l2_evict_first_policy();
            bool waited = !p.early;
            int it = 0;
            bool ok = true;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                const int bh = sg.b * p.Hkv + sg.kvh;
                for (int t = 0; t < sg.n; ++t, ++it) {
                    const int tok = (sg.st0 + t) * STEP;
                    if (!waited && tok + STEP > sg.S) { pdl_wait(); waited = true; }
                    if (ROPE && tok + STEP > sg.S) {
                        if (!mbar_wait_cluster(bar(B_ROWS), 0, abort_flag)) { ok = false; break; }
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                    const int sv = it % NSV;
                    if (!mbar_wait(bar(B_VEMPTY + sv), ((it / NSV) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(bar(B_VFULL + sv), STAGE_BYTES);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES, &v_map, bar(B_VFULL + sv), 0, tok, bh, pol);
                    tma_load_3d(base + SMEM_V + sv * STAGE_BYTES + HALF_BYTES, &v_map, bar(B_VFULL + sv), 64, tok, bh, pol);
                }
            }
            if (*abort_flag) {
                volatile int never = 0;
                for (int u = max(0, it - NSV); u < it; ++u) mbar_wait(bar(B_VFULL + u % NSV), (u / NSV) & 1, &never);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= issuer of the S products =================
        if (lane == 0 && active) {
            constexpr uint32_t IDESC_S = instr_desc(0);            // B = K stage, K-major
            constexpr uint32_t DESC_HI = desc_hi(1024);            // 8 rows x 128 B between row groups, everywhere
            bool ok = true;
            int it = 0, seg = 0;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                if (!mbar_wait(bar(B_QFULL), seg & 1, abort_flag)) { ok = false; break; }
                for (int t = 0; t < sg.n && ok; ++t, ++it) {
                    const int bs = it & 1, sk = it % NSK;
                    if (!mbar_wait(bar(B_KFULL + sk), (it / NSK) & 1, abort_flag)) { ok = false; break; }
                    // S[bs] is free once the softmax threads have read the scores of step it-2 out of it
                    if (it >= 2 && !mbar_wait(bar(B_SFREE + bs), ((it >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t kb = desc_lo(base + SMEM_K + sk * STAGE_BYTES, 16);
                    const uint32_t qb = desc_lo(base + SMEM_Q, 16);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {       // 16 d-columns per instruction: 32 B of each Q and K row
                        const uint32_t koff = ((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4;
                        tc_mma_ss(tmem + COL_S + bs * 128, qb + koff, DESC_HI, kb + koff, DESC_HI, IDESC_S, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(B_KEMPTY + sk));
                    tc_commit(bar(B_SFULL + bs));
                }
                ++seg;
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ================= issuer of the PV products =================
        if (lane == 0 && active) {
            constexpr uint32_t IDESC_O = instr_desc(1);            // B = V stage, MN-major
            constexpr uint32_t DESC_HI = desc_hi(1024);
            bool ok = true;
            int u = 0;
            SegIter si = make_iter();
            Seg sg;
            while (ok && si.next(sg)) {
                for (int t = 0; t < sg.n; ++t, ++u) {
                    const int bu = u & 1, sv = u % NSV;
                    if (!mbar_wait(bar(B_PFULL + bu), (u >> 1) & 1, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(bar(B_VFULL + sv), (u / NSV) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t vb = desc_lo(base + SMEM_V + sv * STAGE_BYTES, HALF_BYTES);
#pragma unroll
                    for (int ks = 0; ks < STEP / 16; ++ks)      // 16 tokens per instruction: 8 P columns, 16 V rows (2 KB)
                        tc_mma_ts(tmem + COL_O, tmem + COL_P + bu * 64 + ks * 8, vb + ks * 128, DESC_HI, IDESC_O,
                                  (t > 0 || ks > 0) ? 1u : 0u);   // the first product of a segment starts a fresh O
                    tc_commit(bar(B_VEMPTY + sv));
                    tc_commit(bar(B_PVDONE + bu));
                }
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ================= softmax: two threads per accumulator row, each takes half of a step's columns =================
        const int sp = warp & 3;                              // TMEM lane quarter of this warp
        const int ch = (warp - 4) >> 2;                       // which half of the row's columns (and of the O columns)
        const int tl = sp * 32 + lane;                        // TMEM lane
        const int half = PAIR ? (tl >> 6) : 0;                // PAIR: which 64 tokens of each step the lane's row copy covers
        const int lrow = PAIR ? (tl & 63) : tl;               // row within the block
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sp) << 16);
        const int st = tid - 128;                             // 0..255
        float* xm = reinterpret_cast<float*>(sm + SMEM_XM);   // [2 step parities][2 column halves][128 lanes] tile maxima;
                                                              // in the epilogue: [0..255] l by (ch, lane), [256..383] m by lane
        int px = 0;                                           // phases of the pair barrier used so far
        int sx = 0;                                           // phases of the segment barrier used so far
        pdl_wait();                                           // q, tree_mask and every output come after the preceding kernel

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

        // Q of a segment -> shared memory, rows in the swizzled K-major layout of a K stage (PAIR: rows 64-127
        // repeat rows 0-63).  Thread t moves 16-byte chunk t%16 of rows t/16, t/16 + 16, ...
        auto load_q = [&](const Seg& sg, int seg) -> bool {
            if (PAIR && seg > 0) {
                // the tile doubles as the exchange area of the previous segment's epilogue
                if (!mbar_wait_warp(bar(B_XFREE), (seg - 1) & 1, abort_flag)) return false;
            }
            if constexpr (ROPE) {
                // the Q tile and, beside it, this rank's share of the unit's tree rows into the cache (a rejected
                // sequence, steps == 0, has no slots to write to: an empty share)
                const int t_lo = (cr * N) / ck;
                rope_prologue<PAIR, ROWS>(sm, p.q, pa, N, p.Hq, p.Hkv, p.S_max, G, rows_total, sg.b, sg.kvh, sg.mblock, sg.S,
                                          t_lo, sg.steps > 0 ? ((cr + 1) * N) / ck : t_lo, st);
                fence_async_smem();
                mbar_arrive(bar(B_QFULL));
                return true;
            }
            constexpr int ITEMS = ROWS * 16 / kSmx;
            const int qc = st & 15;
            uint4 v[ITEMS];
#pragma unroll
            for (int k = 0; k < ITEMS; ++k) {
                const int row = sg.mblock * ROWS + (st >> 4) + 16 * k;
                v[k] = make_uint4(0, 0, 0, 0);
                if (row < rows_total) {
                    const int node = row / G, head = sg.kvh * G + row % G;
                    v[k] = *(reinterpret_cast<const uint4*>(p.q + (((size_t)sg.b * N + node) * p.Hq + head) * D) + qc);
                }
            }
#pragma unroll
            for (int k = 0; k < ITEMS; ++k) {
                const int r = (st >> 4) + 16 * k;
                unsigned char* dst = sm + SMEM_Q + (qc >> 3) * HALF_BYTES + r * 128 + (((qc & 7) ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = v[k];
                if (PAIR) *reinterpret_cast<uint4*>(dst + 64 * 128) = v[k];
            }
            fence_async_smem();
            mbar_arrive(bar(B_QFULL));
            return true;
        };
        // Meeting of the two warps that share this warp's rows (bounded; warp-uniform result).
        auto pair_sync = [&]() -> bool {
            mbar_arrive(bar(B_PAIRX + sp));
            const bool r = mbar_wait_warp(bar(B_PAIRX + sp), px & 1, abort_flag);
            ++px;
            return r;
        };

        if (PAIR && active) {
            // block-diagonal P: a lane's row copy weighs only its own half's 64 tokens of a step; the columns of the
            // other half are zero in both P buffers for the whole call, and nobody else writes them
            uint32_t zero[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) zero[c] = 0u;
            tmem_st16(lane_addr + COL_P + (half ^ 1) * 32 + ch * 16, zero);
            tmem_st16(lane_addr + COL_P + 64 + (half ^ 1) * 32 + ch * 16, zero);
            tmem_wait_st();
        }
        if (active) {
            SegIter si = make_iter();
            Seg sg;
            int it = 0, seg = 0;
            bool ok = true;
            float4* xch = reinterpret_cast<float4*>(sm + SMEM_Q);
            while (ok && si.next(sg)) {
                // every S product of the previous segment has been consumed by now, so Q may be replaced
                if (!load_q(sg, seg)) { ok = false; break; }
                if constexpr (ROPE) {
                    // Each rank of the cluster has just put its share of the unit's N tree rows into the cache (beside its Q
                    // tile).  The ranks whose steps contain the rows (the last, at most the last two) hold those tiles back
                    // until every rank has said that its share is in global memory: fence, meeting of this CTA's softmax
                    // threads, then one arrival per rank on that rank's barrier.
                    __threadfence();                                          // the rows are in global memory ...
                    asm volatile("fence.proxy.async.global;" ::: "memory");   // ... and ordered before bulk copies that read them
                    mbar_arrive(bar(B_SEGSYNC));
                    if (!cl_waited) { cluster_wait(); cl_waited = true; }     // the peers' barriers exist
                    if (st < ck) {
                        if (!mbar_wait(bar(B_SEGSYNC), sx & 1, abort_flag)) { ok = false; }
                        else mbar_arrive_peer(dsmem_addr(bar(B_ROWS), (uint32_t)st));
                    }
                    ++sx;
                    if (__any_sync(0xffffffffu, !ok)) { ok = false; break; }
                }

                const int row = sg.mblock * ROWS + lrow;         // query row within the kv head's G*N rows
                const bool row_ok = row < rows_total;
                const int node = row_ok ? row / G : 0, head = sg.kvh * G + (row_ok ? row % G : 0);
                const int S = sg.S, total = S + N;
                uint64_t mk0 = 0, mk1 = 0;
                if (row_ok) {
                    const uint64_t* mrow = p.mask + ((size_t)sg.b * N + node) * W;
                    mk0 = mrow[0];
                    if (W > 1) mk1 = mrow[1];
                    // bits at or beyond N are not tree nodes
                    if (N < 64) mk0 &= (1ull << N) - 1;
                    if (N < 128) mk1 &= N > 64 ? (1ull << (N - 64)) - 1 : 0ull;
                }
                // m_ref and has_o are the same in both threads of a row; l_run covers this thread's columns only
                float m_ref = -INFINITY, l_run = 0.f;
                bool has_o = false;

                for (int t = 0; t < sg.n; ++t, ++it) {
                    const int bs = it & 1;
                    const int tok0 = (sg.st0 + t) * STEP;
                    if (!mbar_wait_warp(bar(B_SFULL + bs), (it >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    uint32_t sraw[NC];
#pragma unroll
                    for (int c = 0; c < NC / 32; ++c) tmem_ld32(lane_addr + COL_S + bs * 128 + half * 64 + ch * NC + c * 32, sraw + c * 32);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(bar(B_SFREE + bs));             // the S product of step it+2 may overwrite the buffer

                    const int jr = tok0 + half * 64;                        // first token of the row's part of the tile
                    const int j0 = jr + ch * NC;                            // first token this thread looks at
                    const bool row_valid = jr < total, valid = j0 < total;
                    float lmax = -INFINITY;
                    if (valid) {
                        if (j0 + NC > S) {
                            // reaches past the committed prefix: ancestor bits for tree rows, nothing beyond them
                            // bit c of a0: column c may be attended to (prefix column, or visible tree node)
                            const int t0 = j0 - S;                           // tree index of column 0 (may be negative)
                            uint64_t a0, a1;
                            if (t0 >= 0) shr128(mk0, mk1, t0, a0, a1); else shl128_fill(mk0, mk1, -t0, a0, a1);
#pragma unroll
                            for (int c = 0; c < NC; ++c)
                                if (!((a0 >> c) & 1ull)) sraw[c] = 0xff800000u;   // -inf
                        }
                        float mx[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) mx[c] = __uint_as_float(sraw[c]);
#pragma unroll
                        for (int c = 8; c < NC; ++c) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(sraw[c]));
                        // the scale is positive, so it commutes with the maximum
                        lmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7]))) * p.scale_log2;
                    }
                    // the row's maximum over the tile: the other thread of the row has the other columns
                    xm[(it & 1) * 256 + ch * 128 + tl] = lmax;
                    if (!pair_sync()) { ok = false; break; }
                    const float tmax = fmaxf(lmax, xm[(it & 1) * 256 + (ch ^ 1) * 128 + tl]);
                    // move the reference maximum only when the tile exceeds it by more than the gap
                    float alpha = 1.f;
                    bool rescale = false;
                    if (row_valid && tmax > m_ref + kRescaleGap) {      // also true on the first finite tile (m_ref = -inf)
                        alpha = exp2f(m_ref - tmax);                     // 0 when m_ref = -inf
                        m_ref = tmax;
                        l_run *= alpha;
                        rescale = has_o;
                    }
                    if (__any_sync(0xffffffffu, rescale)) {
                        // O was last written by the PV product of step it-1 (same segment: has_o is set); this thread
                        // rescales its half of the row's columns
                        if (!mbar_wait_warp(bar(B_PVDONE + (bs ^ 1)), ((it - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            tmem_ld32(lane_addr + COL_O + ch * 64 + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32(lane_addr + COL_O + ch * 64 + c * 32, o);
                        }
                    }
                    // P[bs] is free once the PV product of step it-2 has completed: as a rule it has, long ago, and one test
                    // issued here, ahead of the exponentials, says so without a wait after them
                    const bool p_free = it < 2 || mbar_test(bar(B_PVDONE + bs), ((it >> 1) - 1) & 1);
                    // P = exp2(scale * s - m_ref) as bf16 pairs (column c of P holds tokens 2c, 2c+1)
                    uint32_t pd[NC / 2];
                    if (valid) {
                        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                        for (int c = 0; c < NC / 2; ++c) {
                            const float e0 = exp2f(fmaf(__uint_as_float(sraw[2 * c]), p.scale_log2, -m_use));
                            const float x1 = fmaf(__uint_as_float(sraw[2 * c + 1]), p.scale_log2, -m_use);
                            const float e1 = (c % kPolyEvery == kPolyEvery - 1) ? exp2_fma(x1) : exp2f(x1);
                            sum0 += e0; sum1 += e1;
                            pd[c] = pack_bf16(e0, e1);
                        }
                        l_run += sum0 + sum1;
                    } else {
#pragma unroll
                        for (int c = 0; c < NC / 2; ++c) pd[c] = 0u;
                    }
                    if (row_valid) has_o = true;
                    if (it >= 2) {
                        if (!__all_sync(0xffffffffu, p_free) &&
                            !mbar_wait_warp(bar(B_PVDONE + bs), ((it >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                    }
                    if (PAIR) {
                        // block-diagonal P: the row weighs only its own half's tokens (the other 32 columns stay zero)
                        tmem_st16(lane_addr + COL_P + bs * 64 + half * 32 + ch * 16, pd);
                    } else {
                        tmem_st32(lane_addr + COL_P + bs * 64 + ch * 32, pd);
                    }
                    bool fail = false;
                    if (tok0 + STEP > total) {
                        // last step of the sequence: V rows past the last key may hold anything, and they meet
                        // weight-0 columns of P in the product: clear them (thread r of the first 128 clears row r)
                        const int sv = it % NSV;
                        fail = !mbar_wait(bar(B_VFULL + sv), (it / NSV) & 1, abort_flag);
                        if (!fail && ch == 0 && tok0 + tl >= total) {
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
                    tc_fence_before();
                    mbar_arrive(bar(B_PFULL + bs));
                }
                if (!ok) break;

                // ---- segment epilogue: wait for the last product, add up the row statistics, (PAIR) merge the two
                // halves, write out.  A thread owns columns [64 ch, 64 ch + 64) of its lane's accumulator row. ----
                if (sg.n > 0) ok = mbar_wait_warp(bar(B_PVDONE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // (the tile-maximum slots are idle: the other thread of the row read its last one before it arrived
                // for the last PV product)
                xm[ch * 128 + tl] = l_run;
                if (ch == 0) xm[256 + tl] = has_o ? m_ref : -INFINITY;
                if (!pair_sync()) { ok = false; break; }
                const float l_lane = xm[tl] + xm[128 + tl];                  // l of this lane's row copy
                float w_me = has_o ? 1.f : 0.f, w_other = 0.f, m_all = has_o ? m_ref : -INFINITY, l_all = l_lane;
                if (PAIR) {
                    if (half == 1) {
                        // hand the raw accumulator to the lane that owns the row (the Q tile is idle: every S product
                        // of the segment has completed); the statistics are in place already
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            tmem_ld32(lane_addr + COL_O + ch * 64 + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4)
                                xch[(ch * 16 + c * 8 + c4) * 64 + lrow] = make_float4(__uint_as_float(o[4 * c4]), __uint_as_float(o[4 * c4 + 1]),
                                                                                     __uint_as_float(o[4 * c4 + 2]), __uint_as_float(o[4 * c4 + 3]));
                        }
                        tc_fence_before();
                        mbar_arrive(bar(B_XCH));
                    } else {
                        ok = mbar_wait_warp(bar(B_XCH), seg & 1, abort_flag);
                        if (!ok) break;
                        const float m_o = xm[256 + 64 + tl], l_o = xm[64 + tl] + xm[128 + 64 + tl];
                        m_all = fmaxf(m_all, m_o);
                        const float m_fin = (m_all == -INFINITY) ? 0.f : m_all;
                        w_me = has_o ? exp2f(m_ref - m_fin) : 0.f;
                        w_other = exp2f(m_o - m_fin);                   // 0 when the other half saw nothing
                        l_all = l_lane * w_me + l_o * w_other;
                    }
                }
                // O is only defined once a product has run (an empty cluster part never ran one): select, never
                // multiply, where the weight is zero
                float4* pbuf = reinterpret_cast<float4*>(sm + SMEM_K);                       // cluster form: [32 col4][ROWS]
                float2* pst = reinterpret_cast<float2*>(sm + SMEM_K + 32 * ROWS * 16);       //               [ROWS] (m, l)
                if (half == 0) {
                    const bool final_out = !CL && sg.slot < 0;
                    const float inv = final_out ? (l_all > 0.f ? 1.f / l_all : 0.f) : 1.f;
                    __nv_bfloat16* orow = p.out + (((size_t)sg.b * N + node) * p.Hq + head) * D + ch * 64;
                    float4* prow = (CL ? pbuf : p.part_o + (size_t)(final_out ? 0 : sg.slot) * 32 * ROWS) + (size_t)ch * 16 * ROWS + lrow;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
                        tmem_ld32(lane_addr + COL_O + ch * 64 + c * 32, o);
                        tmem_wait_ld();
                        float v[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = has_o ? __uint_as_float(o[e]) * w_me : 0.f;
                        if (PAIR) {
                            if (w_other > 0.f) {
#pragma unroll
                                for (int c4 = 0; c4 < 8; ++c4) {
                                    const float4 w = xch[(ch * 16 + c * 8 + c4) * 64 + lrow];
                                    v[4 * c4] += w.x * w_other; v[4 * c4 + 1] += w.y * w_other;
                                    v[4 * c4 + 2] += w.z * w_other; v[4 * c4 + 3] += w.w * w_other;
                                }
                            }
                        }
                        if (final_out) {
                            if (row_ok) {
#pragma unroll
                                for (int c8 = 0; c8 < 4; ++c8)
                                    *reinterpret_cast<uint4*>(orow + c * 32 + c8 * 8) =
                                        make_uint4(pack_bf16(v[8 * c8] * inv, v[8 * c8 + 1] * inv), pack_bf16(v[8 * c8 + 2] * inv, v[8 * c8 + 3] * inv),
                                                   pack_bf16(v[8 * c8 + 4] * inv, v[8 * c8 + 5] * inv), pack_bf16(v[8 * c8 + 6] * inv, v[8 * c8 + 7] * inv));
                            }
                        } else if (CL || row_ok) {
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4)
                                prow[(size_t)(c * 8 + c4) * ROWS] = make_float4(v[4 * c4], v[4 * c4 + 1], v[4 * c4 + 2], v[4 * c4 + 3]);
                        }
                    }
                    if (ch == 0) {
                        const float2 stat = make_float2(l_all > 0.f ? m_all : -INFINITY, l_all);
                        if (CL) {
                            pst[lrow] = stat;
                        } else if (row_ok) {
                            if (final_out) {
                                if (p.lse) p.lse[((size_t)sg.b * p.Hq + head) * N + node] =
                                    l_all > 0.f ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                            } else {
                                p.part_ml[(size_t)sg.slot * ROWS + lrow] = stat;
                            }
                        }
                    }
                    if (PAIR) mbar_arrive(bar(B_XFREE));
                }
                if (PAIR && !CL && pa.unit_counters && sg.slot >= 0) {
                    // ---- even split without a merge kernel (rows <= 64 only: with 128 rows the merge kernel is faster): the CTA that delivers a unit's last partial merges the
                    // unit.  Nobody waits for another CTA: a fence, one atomic per segment, and the last arrival
                    // reads the others' partials (written before their fences) from L2. ----
                    __threadfence();
                    mbar_arrive(bar(B_SEGSYNC));                       // every softmax thread has written and fenced
                    if (!mbar_wait_warp(bar(B_SEGSYNC), sx & 1, abort_flag)) { ok = false; break; }
                    ++sx;
                    const int uib = sg.kvh * p.n_mblocks + sg.mblock;
                    const int ub = sched.base[sg.b] + uib * sg.steps;
                    const int c0 = cta_of(ub, T, geff), c1 = cta_of(ub + sg.steps - 1, T, geff);
                    if (st == 0) {
                        int* cnt = pa.unit_counters + (sg.b * p.Hkv * p.n_mblocks + uib);
                        const bool last = atomicAdd(cnt, 1) == c1 - c0;
                        if (last) *cnt = 0;                            // all zero again for the next call
                        *seg_flag = last ? 1 : 0;
                    }
                    mbar_arrive(bar(B_SEGSYNC));
                    if (!mbar_wait_warp(bar(B_SEGSYNC), sx & 1, abort_flag)) { ok = false; break; }
                    ++sx;
                    if (*seg_flag) {
                        __threadfence();
                        const MergeArgs ma = {p.part_o, p.part_ml, p.out, p.lse, p.Hq, G, N, rows_total};
                        merge_unit<ROWS>(ma, T, geff, ub, c0, c1, sg.b, sg.kvh, sg.mblock, st, kSmx);
                    }
                }

                tc_fence_before();        // the next segment's first product overwrites O
                ++seg;
            }
        }
    }

    if (CL) {
        // ---- cluster exchange: every CTA of the unit has parked its partial (O, m, l) in its own shared memory.
        // All threads of the cluster meet at the hardware cluster barrier (the warps that finished early wait
        // there without polling); then rank r merges rows [r*rp, (r+1)*rp) of all k partials through distributed
        // shared memory and writes them out. ----
        __syncwarp();
        if (!cl_waited) { cluster_wait(); cl_waited = true; }     // (fused rotary embedding: the start-up phase, warps 0-3)
        cluster_sync_all();
        if (warp == 1) {
            // every thread of the CTA is past its last tensor-memory access: give the columns back now, beside the
            // merge, instead of on the way out
            tc_fence_after();
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(TMEM_COLS) : "memory");
        }
        if (warp >= 4 && !*abort_flag) {
        const int rp = (ROWS + ck - 1) / ck;
        const int row0 = cr * rp;
        const int nrows = min(rp, ROWS - row0);
        const uint32_t pbuf_a = base + SMEM_K, pst_a = base + SMEM_K + 32 * ROWS * 16;
        // IT items (row, column quad) at a time per thread, all loads of all KM pieces issued before the first use
        auto merge_items = [&](auto km_tag, auto it_tag) {
            constexpr int KM = decltype(km_tag)::value, IT = decltype(it_tag)::value;
            for (int item0 = tid - 128; item0 < nrows * 32; item0 += kSmx * IT) {
                float2 ml[IT][KM];
                float4 pv[IT][KM];
                int c4s[IT], grows[IT];
#pragma unroll
                for (int e = 0; e < IT; ++e) {
                    const int item = item0 + e * kSmx;
                    const int c4 = item / nrows, lr = row0 + (item - c4 * nrows);
                    c4s[e] = c4;
                    grows[e] = (item < nrows * 32) ? cl_seg.mblock * ROWS + lr : rows_total;
#pragma unroll
                    for (int j = 0; j < KM; ++j) {
                        ml[e][j] = make_float2(-INFINITY, 0.f);
                        pv[e][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (j < ck && grows[e] < rows_total) {
                            ml[e][j] = dsmem_ld2(dsmem_addr(pst_a + lr * 8, (uint32_t)j));
                            pv[e][j] = dsmem_ld4(dsmem_addr(pbuf_a + (c4 * ROWS + lr) * 16, (uint32_t)j));
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < IT; ++e) {
                    if (grows[e] >= rows_total) continue;
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
                    const int nd = grows[e] / G, hd = cl_seg.kvh * G + grows[e] % G;
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
    }

    // ---- tear-down: everyone meets, TMEM goes back ----
    tc_fence_before();
    __syncthreads();
    // Cluster form: nobody leaves while a peer may still read its shared memory or signal its barriers.  Every
    // CTA gets here (all its other waits are bounded), so this hardware barrier ends.
    if (CL) cluster_sync_all();
    if (!CL && warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicCAS(p.status, 0, (int)VISPEC_E_TIMEOUT);
}



}  // namespace


static size_t tc5_partial_bytes(int grid, int rows) { return (size_t)2 * grid * rows * (D * 4 + 8); }

namespace {

// Streaming-read probe: the K/V rows one attention call reads, moved by the same TMA producer through the same
// rings on the even split of all steps over the CTAs, and nothing else (a second thread hands every stage
// straight back).  It measures what this way of streaming reaches on its own: the ceiling the attention kernel
// can approach.
__global__ void __launch_bounds__(64, 1)
stream_probe_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const Tc5Params p) {
    extern __shared__ __align__(1024) unsigned char sm[];
    const uint32_t base = smem_u32(sm);
    if (base & 1023u) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)VISPEC_E_UNSUPPORTED);
        return;
    }
    constexpr int NS = NSK + NSV;                              // stages: K and V of a step take consecutive ones
    const uint32_t bars = base + NS * STAGE_BYTES;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + NS * STAGE_BYTES + 2 * NS * 8);
    Sched& sched = *reinterpret_cast<Sched*>(sm + NS * STAGE_BYTES + 256);
    auto full = [&](int i) { return bars + 8u * (uint32_t)i; };
    auto empty = [&](int i) { return bars + 8u * (uint32_t)(NS + i); };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < NS; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) sched_build(sched, p, lane, lane < p.B ? p.kv_len[lane] : 0);
    pdl_launch_dependents();
    if (!p.early) pdl_wait();
    __syncthreads();
    const int T = sched.base[p.B];
    const int geff = T > 0 ? sched_ctas(T, sched.units, (int)gridDim.x, p.min_steps) : 0;
    const int cta = blockIdx.x;
    if (cta < geff && lane == 0) {
        const int lo = cta_lo(cta, T, geff), hi = cta_lo(cta + 1, T, geff);
        SegIter si; si.s = &sched; si.B = p.B; si.n_mblocks = p.n_mblocks; si.g = lo; si.lo = lo; si.hi = hi; si.cta = cta;
        si.cl = false; si.cl_done = false;
        Seg sg;
        int n = 0;                                             // stages handled so far
        if (warp == 0) {
            const uint64_t pol = l2_evict_first_policy();
            bool waited = !p.early, ok = true;
            while (ok && si.next(sg)) {
                const int bh = sg.b * p.Hkv + sg.kvh;
                for (int t = 0; t < sg.n && ok; ++t) {
                    const int tok = (sg.st0 + t) * STEP;
                    if (!waited && tok + STEP > sg.S) { pdl_wait(); waited = true; }
                    for (int kv = 0; kv < 2; ++kv, ++n) {
                        const int s = n % NS;
                        if (!mbar_wait(empty(s), ((n / NS) & 1) ^ 1, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(full(s), STAGE_BYTES);
                        tma_load_3d(base + s * STAGE_BYTES, kv ? &v_map : &k_map, full(s), 0, tok, bh, pol);
                        tma_load_3d(base + s * STAGE_BYTES + HALF_BYTES, kv ? &v_map : &k_map, full(s), 64, tok, bh, pol);
                    }
                }
            }
            if (*abort_flag) {
                volatile int never = 0;
                for (int u = max(0, n - NS); u < n; ++u) mbar_wait(full(u % NS), (u / NS) & 1, &never);
            }
        } else {
            bool ok = true;
            while (ok && si.next(sg))
                for (int t = 0; t < 2 * sg.n; ++t, ++n) {
                    if (!mbar_wait(full(n % NS), (n / NS) & 1, abort_flag)) { ok = false; break; }
                    mbar_arrive(empty(n % NS));
                }
        }
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) atomicCAS(p.status, 0, (int)VISPEC_E_TIMEOUT);
}

}  // namespace

// Largest number of co-resident clusters of each size (index: PAIR, cluster size), found once per device.
static int g_max_clusters[2][9];

static int query_max_clusters(bool pair, int k) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(k * 64); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = SMEM_ALLOC;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = k; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    cudaError_t e = pair ? cudaOccupancyMaxActiveClusters(&n, attn_tc5_kernel<true, true, false>, &cfg)
                         : cudaOccupancyMaxActiveClusters(&n, attn_tc5_kernel<false, true, false>, &cfg);
    if (e != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

// Cluster size for the cluster form, or 0 when the even split with partials in global memory serves better:
// one cluster per unit, all clusters co-resident.  `pair`: units of at most 64 rows in the duplicated-row layout,
// n_mblocks of them per kv head.  *est_us: the estimate of the form it returns.
static int tc5_cluster_size(const AttnArgs& a, bool pair, int n_mblocks, double* est_us = nullptr, bool clusters_if_possible = false) {
    const int units = a.B * a.Hkv * n_mblocks;
    if (est_us) *est_us = 1e30;
    if (a.tc5_path == 1 || a.tc5_path == 3) return 0;
    int best = 0;
    for (int k = 1; k <= 8; ++k)
        if (units * k <= a.sm_count && g_max_clusters[pair][k] >= units) best = k;
    if (best == 0) return 0;
    if (a.tc5_path == 2 || clusters_if_possible) return best;
    // Both forms, estimated in microseconds from what was measured over the workloads (the long-response sweep
    // cells, the 7B and 13B shapes): a fixed part (11 for the cluster form, 14 for the even split with its partials
    // and second phase), the steps of the busiest CTA at 1.2 per step or at the HBM share of that many CTAs (64 KB
    // per step at 5.2 TB/s over the cluster form's CTAs, 6.6 TB/s over the even split's; the row blocks of one kv
    // head read the same tiles, so only one in n_mblocks comes from HBM), and 0.25 per partial a unit is merged
    // from.  The host knows only the capacity S_max, not kv_len: the estimate is for full caches unless the caller
    // has given the length it expects (VISPEC_OPT_KV_LEN_HINT).
    const int slots = (a.kv_len_hint > 0 && a.kv_len_hint + a.N < a.S_max) ? a.kv_len_hint + a.N : a.S_max;
    const double steps = (double)((slots + STEP - 1) / STEP), T = steps * units;
    const double n_c = (double)units * best, per_c = (double)(((slots + STEP - 1) / STEP + best - 1) / best);
    const double est_c = 11.0 + per_c * fmax(1.2, n_c * 0.0125 / n_mblocks);
    const double n_e = fmin((double)a.sm_count, fmax(1.0, T / 2.0));
    // (merge: 0.25 per piece of a unit; from four pieces on the fine-grained merge kernel, 1 + 0.055 per piece)
    const double pieces = n_e / units;
    const double est_e = 14.0 + (T / n_e) * fmax(1.2, n_e * 0.00973 / n_mblocks) + (pieces >= 4.0 ? 1.0 + 0.055 * pieces : 0.25 * pieces);
    // (units of several row blocks per kv head in small clusters: measured over the sweep, the even split's steps come
    // out dearer than the estimate there - 54.8 against 52.6 us on qwen3b_S8192_N60_B8, 96.1 against 92.4 on
    // qwen3b_S16384_N128_B4 - so the clusters get a tenth of tolerance)
    const double tol = (n_mblocks > 1 && best <= 4) ? 1.1 : 1.0;
    if (est_us) *est_us = est_c <= tol * est_e ? est_c : est_e;
    return est_c <= tol * est_e ? best : 0;
}

// Row layout of a call.  At most 64 query rows per kv head: one unit of 64 rows, rows duplicated over the two lane
// halves.  More: blocks of 128 rows, lane = row - unless that leaves most of the GPU idle (few sequences and kv
// heads, rows just over 64: one cluster of at most 8 CTAs per unit is all the cluster form can use): then blocks of 64
// rows in the duplicated layout make twice the units, and a step of such a unit costs its softmax threads half the
// columns (measured per step and CTA: 0.9 against 1.4-1.8 us), at the price of every K/V tile crossing from L2 twice as
// often and half of each product computed for nothing.  Taken when both layouts would run as clusters and the
// estimate (steps of the busiest CTA at those rates) says a twentieth less or better.
struct Tc5Layout { bool pair; int rows, n_mblocks, ck; };
static Tc5Layout tc5_layout(const AttnArgs& a) {
    const int rows_total = (a.Hq / a.Hkv) * a.N;
    Tc5Layout full = {rows_total <= 64, rows_total <= 64 ? 64 : 128, rows_total <= 64 ? 1 : (rows_total + 127) / 128, 0};
    double est_full = 0.0;
    full.ck = tc5_cluster_size(a, full.pair, full.n_mblocks, &est_full);
    if (full.pair || a.tc5_path != 0) return full;
    Tc5Layout half = {true, 64, (rows_total + 63) / 64, 0};
    half.ck = tc5_cluster_size(a, true, half.n_mblocks, nullptr, true);     // (clusters or nothing: the even split gains nothing from smaller blocks)
    if (half.ck == 0) return full;
    const int slots = (a.kv_len_hint > 0 && a.kv_len_hint + a.N < a.S_max) ? a.kv_len_hint + a.N : a.S_max;
    const int steps = (slots + STEP - 1) / STEP;
    auto est = [&](const Tc5Layout& l, double step_us) {
        const double n_c = (double)a.B * a.Hkv * l.n_mblocks * l.ck;
        return 11.0 + (double)((steps + l.ck - 1) / l.ck) * fmax(step_us, n_c * 0.0125 / l.n_mblocks);
    };
    if (full.ck > 0) return est(half, 0.95) < 0.95 * est(full, full.n_mblocks > 1 ? 1.7 : 1.45) ? half : full;
    // 128-row blocks would go as an even split (its estimate: est_full); small clusters of 64-row blocks, whose fixed
    // part measures 8 rather than 11 us, against that
    return est(half, 0.95) - 3.0 < 0.95 * est_full ? half : full;
}

bool attn_tc5_supports(const AttnArgs& a) {
    if (!(a.D == 128 && a.k_map && a.v_map && a.B > 0 && a.B <= kMaxB)) return false;
    const int rows_total = (a.Hq / a.Hkv) * a.N;
    const int rows = rows_total <= 64 ? 64 : 128;
    const long long n_mblocks = (rows_total + 63) / 64;          // the most either layout makes
    const long long t_max = (long long)a.B * a.Hkv * n_mblocks * ((a.S_max + STEP - 1) / STEP);
    if (t_max * a.sm_count >= (1ll << 31)) return false;
    if (!(a.scale > 0.f)) return false;       // the kernel takes the maximum before scaling
    return kCounterBytes + tc5_partial_bytes(a.sm_count, rows) <= a.ws_bytes;
}

cudaError_t init_attn_tc5() {
    cudaError_t e = cudaSuccess;
    const void* kernels[8] = {(const void*)attn_tc5_kernel<true, false, false>, (const void*)attn_tc5_kernel<false, false, false>,
                              (const void*)attn_tc5_kernel<true, true, false>, (const void*)attn_tc5_kernel<false, true, false>,
                              (const void*)attn_tc5_kernel<true, false, true>, (const void*)attn_tc5_kernel<false, false, true>,
                              (const void*)attn_tc5_kernel<true, true, true>, (const void*)attn_tc5_kernel<false, true, true>};
    for (const void* k : kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ALLOC);
        if (e != cudaSuccess) return e;
    }
    const void* rope_kernels[2] = {(const void*)attn_tc5_kernel<true, true, false, true>, (const void*)attn_tc5_kernel<false, true, false, true>};
    for (const void* k : rope_kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_ALLOC);
        if (e != cudaSuccess) return e;
    }
    for (int k = 1; k <= 8; ++k) { g_max_clusters[0][k] = query_max_clusters(false, k); g_max_clusters[1][k] = query_max_clusters(true, k); }
    if (getenv("VISPEC_DEBUG")) for (int k = 1; k <= 8; ++k) fprintf(stderr, "vispec: cluster size %d: %d (rows > 64) / %d (rows <= 64) co-resident clusters\n", k, g_max_clusters[0][k], g_max_clusters[1][k]);
    // The merge blocks must be able to join an SM that an attention CTA has configured for maximum shared memory.
    const void* merge_kernels[4] = {(const void*)attn_tc5_merge_kernel<64>, (const void*)attn_tc5_merge_kernel<128>,
                                    (const void*)attn_tc5_merge_kernel<64, true>, (const void*)attn_tc5_merge_kernel<128, true>};
    for (const void* k : merge_kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool attn_tc5_uses_clusters(const AttnArgs& a) { return tc5_layout(a).ck > 0; }

cudaError_t launch_attn_tc5(const AttnArgs& a, cudaStream_t st, int* n_launches) {
    *n_launches = 0;
    const Tc5Layout lay = tc5_layout(a);
    const bool pair = lay.pair;
    const int rows = lay.rows, n_mblocks = lay.n_mblocks, ck = lay.ck;
    const int units = a.B * a.Hkv * n_mblocks;
    const long long t_max = (long long)units * ((a.S_max + STEP - 1) / STEP);
    const int grid = ck > 0 ? units * ck : (int)(t_max < a.sm_count ? t_max : a.sm_count);

    Tc5Params p = {};
    p.q = (const __nv_bfloat16*)a.q; p.kv_len = a.kv_len; p.mask = a.mask;
    p.out = (__nv_bfloat16*)a.out; p.lse = a.lse;
    unsigned char* ws = (unsigned char*)a.ws + kCounterBytes;
    p.part_o = (float4*)ws;
    p.part_ml = (float2*)(ws + (size_t)2 * grid * rows * D * 4);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max; p.n_mblocks = n_mblocks;
    p.grid_attn = grid; p.min_steps = 2; p.early = a.early_prefetch ? 1 : 0; p.step = STEP;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.status = a.status;
    cudaError_t err;
    const bool paged = a.page_rows != 0;
    // even split, at most 64 rows per unit: the arrival counters at the head of the workspace serve the in-kernel
    // merge (measured: 68.8 against 70.3 us per layer on llava13b_b4; with 128 rows it lost, 65.9 against 60.5 us on
    // qwen3b_S32768_N16_B8, so those, a grid with more units than counters, and split form 3 get the merge kernel)
    const bool own_merge = pair && ck == 0 && a.tc5_path != 3 && (size_t)units * sizeof(int) <= kCounterBytes;
    const PagedArgs pa = {a.block_table, a.table_stride, a.page_rows, a.num_blocks, a.Hkv, a.N, a.token_major, a.status,
                          own_merge ? (int*)a.ws : nullptr};
    auto launch_attn = [&](auto kernel, int cluster) {
        return launch_pdl(kernel, dim3(grid), dim3(kThreads), SMEM_ALLOC, st, cluster, *a.k_map, *a.v_map, p, pa);
    };
    if (a.rope_table) {
        // fused rotary embedding (contiguous caches): the table holds B*N*D/2 fp64 (cos, sin) pairs, then the same in fp32
        const size_t n = (size_t)a.B * a.N * (D / 2);
        const RopeArgs ra = {(const double2*)a.rope_table, (const float2*)((const double2*)a.rope_table + n),
                             (const __nv_bfloat16*)a.k_new, (const __nv_bfloat16*)a.v_new, (__nv_bfloat16*)a.k, (__nv_bfloat16*)a.v,
                             own_merge ? (int*)a.ws : nullptr};
        auto launch_rope = [&](auto kernel, int cluster) {
            return launch_pdl(kernel, dim3(grid), dim3(kThreads), SMEM_ALLOC, st, cluster, *a.k_map, *a.v_map, p, ra);
        };
        if (ck <= 0) return cudaErrorInvalidValue;        // cluster form only: the caller asks attn_tc5_uses_clusters first
        err = pair ? launch_rope(attn_tc5_kernel<true, true, false, true>, ck) : launch_rope(attn_tc5_kernel<false, true, false, true>, ck);
        if (err != cudaSuccess) return err;
        ++*n_launches;
        return cudaSuccess;
    }
    if (ck > 0) {
        // cluster form: the CTAs of a unit merge their partials through distributed shared memory; one launch
        err = paged ? (pair ? launch_attn(attn_tc5_kernel<true, true, true>, ck) : launch_attn(attn_tc5_kernel<false, true, true>, ck))
                    : (pair ? launch_attn(attn_tc5_kernel<true, true, false>, ck) : launch_attn(attn_tc5_kernel<false, true, false>, ck));
        if (err != cudaSuccess) return err;
        ++*n_launches;
        return cudaSuccess;
    }
    err = paged ? (pair ? launch_attn(attn_tc5_kernel<true, false, true>, 0) : launch_attn(attn_tc5_kernel<false, false, true>, 0))
                : (pair ? launch_attn(attn_tc5_kernel<true, false, false>, 0) : launch_attn(attn_tc5_kernel<false, false, false>, 0));
    if (err != cudaSuccess) return err;
    ++*n_launches;
    if (own_merge) return cudaSuccess;
    if (grid >= 4 * units)        // units cut into many pieces: the fine-grained merge
        err = pair ? launch_pdl(attn_tc5_merge_kernel<64, true>, dim3(units, 16), dim3(128), 0, st, 0, p)
                   : launch_pdl(attn_tc5_merge_kernel<128, true>, dim3(units, 32), dim3(128), 0, st, 0, p);
    else
        err = pair ? launch_pdl(attn_tc5_merge_kernel<64>, dim3(units, 4), dim3(128), 0, st, 0, p)
                   : launch_pdl(attn_tc5_merge_kernel<128>, dim3(units, 8), dim3(128), 0, st, 0, p);
    if (err != cudaSuccess) return err;
    ++*n_launches;
    return cudaSuccess;
}

namespace {

// The attention kernels' wait routine on a barrier that never completes: thread 0 runs out of its limit and raises the
// give-up flag; thread 32 waits on a second such barrier with the ordinary (long) limit and must be released by that
// flag.  Then the block reports VISPEC_E_TIMEOUT and leaves one arrival counter non-zero, as a call that gave up
// between a partial's arrival and the unit's merge would.
__global__ void __launch_bounds__(64)
bounded_wait_selftest_kernel(long long limit, int* status, int* counters) {
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ int flag;
    volatile int* abort_flag = &flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool gave_up = false;
    if (threadIdx.x == 0) gave_up = !mbar_wait(smem_u32(&bars[0]), 0, abort_flag, limit);
    if (threadIdx.x == 32) gave_up = !mbar_wait(smem_u32(&bars[1]), 0, abort_flag);
    const int n = __syncthreads_count(gave_up);
    if (threadIdx.x == 0 && n == 2 && *abort_flag) {
        atomicCAS(status, 0, (int)VISPEC_E_TIMEOUT);
        atomicAdd(counters, 1);
    }
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(long long limit, int* status, int* counters, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(limit, status, counters);
    return cudaGetLastError();
}

cudaError_t init_stream_probe() {
    return cudaFuncSetAttribute(stream_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (NSK + NSV) * STAGE_BYTES + 256 + (int)sizeof(Sched));
}

cudaError_t launch_stream_probe(const AttnArgs& a, cudaStream_t st) {
    const int rows_total = (a.Hq / a.Hkv) * a.N;
    const int n_mblocks = rows_total <= 64 ? 1 : (rows_total + 127) / 128;
    Tc5Params p = {};
    p.kv_len = a.kv_len;
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max;
    p.n_mblocks = 1;                                       // every K/V row once, whatever the number of row blocks
    (void)n_mblocks;
    const long long t_max = (long long)a.B * a.Hkv * ((a.S_max + STEP - 1) / STEP);
    const int grid = (int)(t_max < a.sm_count ? t_max : a.sm_count);
    p.grid_attn = grid; p.min_steps = 2; p.early = a.early_prefetch ? 1 : 0; p.step = STEP;
    p.status = a.status;
    return launch_pdl(stream_probe_kernel, dim3(grid), dim3(64), (size_t)((NSK + NSV) * STAGE_BYTES + 256 + sizeof(Sched)), st, 0,
                      *a.k_map, *a.v_map, p);
}

}  // namespace vispec
