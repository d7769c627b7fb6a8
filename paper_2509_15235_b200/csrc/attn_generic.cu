// Generic split-KV tree-verification attention (Eq. 1 restricted to prefix + ancestors) on
// warp-level tensor-core instructions (mma.sync m16n8k16, bf16 in, fp32 accumulate).
//
// It serves every supported shape (D = 64 or 128, any G, N <= 128) and is the path for shapes the
// TMA/tcgen05 kernel does not take.  Work unit: (sequence b, kv head, block of 64 query rows,
// KV split).  Query rows of one kv head are ordered node-major: row r = i * G + g  (node i, group
// member g, query head kvh*G + g), so all G heads and all N nodes of a head group share each K/V tile.
// Tiles of 64 cached tokens stream through a 2-stage cp.async ring; scores are masked with the node's
// ancestor bits only in tiles that reach past the committed prefix; softmax is the online fp32
// rescale; each split writes an unnormalised partial (O, m, l) and a second kernel merges them.
#include <cuda_bf16.h>

#include "vispec_internal.h"

namespace vispec {

namespace {

constexpr int BM = 64;       // query rows per CTA (4 warps x 16)
constexpr int BN = 64;       // cached tokens per tile
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled, nothing is read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte chunk `chunk` of row `row` in a tile whose rows are D*2 bytes, with the
// chunk index XOR-ed by the row so that 8 consecutive rows of one chunk column hit 8 bank groups.
template <int D> __device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

struct GenericParams {
    const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;
    const int32_t* kv_len; const uint64_t* mask;
    __nv_bfloat16* out; float* lse;
    float* part_o; float* part_ml;      // partials: [unit][split][BM][D], [unit][split][BM][2]
    int B, N, Hq, Hkv, S_max, n_split, n_mblocks;
    int bm;                             // rows per partial block (merge kernel only)
    float scale_log2;
    int* status;
};

template <int D>
__global__ void __launch_bounds__(kThreads)
attn_generic_kernel(const GenericParams p) {
    constexpr int CH = D / 8;                 // 16-byte chunks per row
    constexpr int KS = D / 16;                // k-steps of the QK^T product
    constexpr int TILE_BYTES = BN * D * 2;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sQ = smem;
    unsigned char* sK = smem + BM * D * 2;
    unsigned char* sV = sK + 2 * TILE_BYTES;

    const int split = blockIdx.x, mblk = blockIdx.y;
    const int b = blockIdx.z / p.Hkv, kvh = blockIdx.z % p.Hkv;
    const int G = p.Hq / p.Hkv, N = p.N, W = (N + 63) >> 6;
    const int rows_total = G * N;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit = (blockIdx.z * p.n_mblocks + mblk);

    int S = p.kv_len[b];
    const bool seq_ok = (S >= 0 && S + N <= p.S_max);
    if (!seq_ok) { if (tid == 0 && split == 0 && mblk == 0) atomicCAS(p.status, 0, (int)VISPEC_E_RANGE); S = 0; }
    const int total = seq_ok ? S + N : 0;                      // keys that exist for this sequence
    const int n_tiles = (total + BN - 1) / BN;
    const int tps = (n_tiles + p.n_split - 1) / p.n_split;
    const int t_begin = min(split * tps, n_tiles), t_end = min(t_begin + tps, n_tiles);

    // ---- Q tile -> shared (rows beyond G*N are zero) ----
    const int row_base = mblk * BM;
    for (int idx = tid; idx < BM * CH; idx += kThreads) {
        const int r = idx / CH, c = idx % CH;
        const int gr = row_base + r;
        const bool valid = gr < rows_total;
        const int i = valid ? gr / G : 0, g = valid ? gr % G : 0;
        const __nv_bfloat16* src = p.q + (((size_t)b * N + i) * p.Hq + kvh * G + g) * D + c * 8;
        cp_async16(smem_u32(sQ + tile_off<D>(r, c)), src, valid);
    }
    cp_async_commit();

    const __nv_bfloat16* kbase = p.k + ((size_t)b * p.Hkv + kvh) * (size_t)p.S_max * D;
    const __nv_bfloat16* vbase = p.v + ((size_t)b * p.Hkv + kvh) * (size_t)p.S_max * D;
    auto load_tile = [&](int t, int stage) {
        const int j0 = t * BN;
        for (int idx = tid; idx < BN * CH; idx += kThreads) {
            const int r = idx / CH, c = idx % CH;
            const bool valid = (j0 + r) < total;               // rows past S+N are zero-filled, never read
            const size_t goff = (size_t)(valid ? j0 + r : 0) * D + c * 8;
            const uint32_t so = tile_off<D>(r, c);
            cp_async16(smem_u32(sK + stage * TILE_BYTES + so), kbase + goff, valid);
            cp_async16(smem_u32(sV + stage * TILE_BYTES + so), vbase + goff, valid);
        }
    };
    if (t_begin < t_end) load_tile(t_begin, 0);
    cp_async_commit();

    // ---- per-thread row state: rows r0 = lane/4 and r0 + 8 of this warp's 16 ----
    const int lr0 = warp * 16 + (lane >> 2);
    uint64_t mk[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int gr = row_base + lr0 + h * 8;
        if (gr < rows_total) {
            const uint64_t* mrow = p.mask + ((size_t)b * N + gr / G) * W;
            mk[h][0] = mrow[0];
            if (W > 1) mk[h][1] = mrow[1];
        }
    }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

    cp_async_wait<1>();          // Q has landed (the first K/V tile may still be in flight)
    __syncthreads();
    uint32_t qf[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
        ldsm_x4(smem_u32(sQ + tile_off<D>(warp * 16 + (lane & 15), 2 * ks + (lane >> 4))),
                qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);

    for (int t = t_begin; t < t_end; ++t) {
        const int stage = (t - t_begin) & 1;
        if (t + 1 < t_end) load_tile(t + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const unsigned char* tK = sK + stage * TILE_BYTES;
        const unsigned char* tV = sV + stage * TILE_BYTES;

        // S = Q K^T : 16 rows x 64 tokens per warp
        float s[BN / 8][4];
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int jp = 0; jp < BN / 16; ++jp) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4(smem_u32(tK + tile_off<D>(jp * 16 + (lane & 7) + ((lane >> 4) << 3), 2 * ks + ((lane >> 3) & 1))),
                        b0, b1, b2, b3);
                mma_bf16(s[2 * jp], qf[ks], b0, b1);
                mma_bf16(s[2 * jp + 1], qf[ks], b2, b3);
            }
        }
        // scale into the log2 domain and mask.  Only tiles reaching past the prefix need the bit test.
        const int j0 = t * BN;
        const bool tail = (j0 + BN > S);
#pragma unroll
        for (int j = 0; j < BN / 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x = s[j][e] * p.scale_log2;
                if (tail) {
                    const int col = j0 + j * 8 + 2 * (lane & 3) + (e & 1);
                    const int tt = col - S;
                    bool allow = true;
                    if (tt >= 0) {
                        const int h = e >> 1;
                        allow = (tt < N) && ((tt < 64 ? (mk[h][0] >> tt) : (mk[h][1] >> (tt - 64))) & 1ull);
                    }
                    if (!allow) x = -INFINITY;
                }
                s[j][e] = x;
            }
        }
        // online softmax (rows live in quads of 4 lanes)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < BN / 8; ++j) mx = fmaxf(mx, fmaxf(s[j][2 * h], s[j][2 * h + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[h], mx);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;     // all-masked rows stay at zero mass
            const float alpha = exp2f(m_run[h] - m_use);                 // exp2(-inf) = 0 on first use
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < BN / 8; ++j) {
                const float p0 = exp2f(s[j][2 * h] - m_use), p1 = exp2f(s[j][2 * h + 1] - m_use);
                s[j][2 * h] = p0; s[j][2 * h + 1] = p1;
                sum += p0 + p1;
            }
            l_run[h] = l_run[h] * alpha + sum;
            m_run[h] = m_new;
#pragma unroll
            for (int j = 0; j < D / 8; ++j) { o[j][2 * h] *= alpha; o[j][2 * h + 1] *= alpha; }
        }
        // O += P V
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
            uint32_t a[4];
            a[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
            a[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
            a[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
            a[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
            for (int jp = 0; jp < D / 16; ++jp) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(smem_u32(tV + tile_off<D>(ks * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * jp + (lane >> 4))),
                          b0, b1, b2, b3);
                mma_bf16(o[2 * jp], a, b0, b1);
                mma_bf16(o[2 * jp + 1], a, b2, b3);
            }
        }
        __syncthreads();     // everyone is done with this stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- epilogue: quad-reduce the row sums, then either finish or park a partial ----
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
    const float LN2 = 0.6931471805599453f;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int lr = lr0 + h * 8;
        const int gr = row_base + lr;
        if (p.n_split == 1) {
            if (gr >= rows_total) continue;
            const int i = gr / G, g = gr % G, head = kvh * G + g;
            const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
            __nv_bfloat16* orow = p.out + (((size_t)b * N + i) * p.Hq + head) * D;
#pragma unroll
            for (int j = 0; j < D / 8; ++j)
                *reinterpret_cast<uint32_t*>(orow + j * 8 + 2 * (lane & 3)) =
                    pack_bf16(o[j][2 * h] * inv, o[j][2 * h + 1] * inv);
            if (p.lse && (lane & 3) == 0)
                p.lse[((size_t)b * p.Hq + head) * N + i] =
                    l_run[h] > 0.f ? (m_run[h] + log2f(l_run[h])) * LN2 : -INFINITY;
        } else {
            const size_t slot = ((size_t)unit * p.n_split + split) * BM + lr;
            float* po = p.part_o + slot * D;
#pragma unroll
            for (int j = 0; j < D / 8; ++j)
                *reinterpret_cast<float2*>(po + j * 8 + 2 * (lane & 3)) = make_float2(o[j][2 * h], o[j][2 * h + 1]);
            if ((lane & 3) == 0) *reinterpret_cast<float2*>(p.part_ml + slot * 2) = make_float2(m_run[h], l_run[h]);
        }
    }
}

// Merge of the split partials: one warp per output row (b, node, head).
template <int D>
__global__ void __launch_bounds__(128)
attn_generic_combine_kernel(const GenericParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.Hq / p.Hkv, N = p.N;
    const long row = (long)blockIdx.x * 4 + warp;                 // over B * N * Hq
    if (row >= (long)p.B * N * p.Hq) return;
    const int head = (int)(row % p.Hq), i = (int)((row / p.Hq) % N), b = (int)(row / ((long)p.Hq * N));
    const int kvh = head / G, g = head % G;
    const int gr = i * G + g, mblk = gr / p.bm, lr = gr % p.bm;
    const int unit = (b * p.Hkv + kvh) * p.n_mblocks + mblk;
    float m = -INFINITY;
    for (int s = 0; s < p.n_split; ++s)
        m = fmaxf(m, p.part_ml[(((size_t)unit * p.n_split + s) * p.bm + lr) * 2]);
    const float m_use = (m == -INFINITY) ? 0.f : m;
    constexpr int PER = D / 32;
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    float l = 0.f;
    for (int s = 0; s < p.n_split; ++s) {
        const size_t slot = ((size_t)unit * p.n_split + s) * p.bm + lr;
        const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + slot * 2);
        const float w = exp2f(ml.x - m_use);
        l += ml.y * w;
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] += w * p.part_o[slot * D + e * 32 + lane];
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    __nv_bfloat16* orow = p.out + (((size_t)b * N + i) * p.Hq + head) * D;
#pragma unroll
    for (int e = 0; e < PER; ++e) orow[e * 32 + lane] = __float2bfloat16_rn(acc[e] * inv);
    if (p.lse && lane == 0)
        p.lse[((size_t)b * p.Hq + head) * N + i] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

}  // namespace

// Merge of partials laid out as [unit][split][rows][D] + [unit][split][rows][2] behind the workspace header,
// unit = (sequence * Hkv + kv head) * n_mblocks + row block.  Also used by the TMA/tcgen05 kernel.
cudaError_t launch_attn_combine(const AttnArgs& a, int n_split, int n_mblocks, int rows_per_block, cudaStream_t st) {
    GenericParams p;
    p.q = nullptr; p.k = nullptr; p.v = nullptr; p.kv_len = a.kv_len; p.mask = a.mask;
    p.out = (__nv_bfloat16*)a.out; p.lse = a.lse;
    const size_t units = (size_t)a.B * a.Hkv * n_mblocks;
    unsigned char* ws = (unsigned char*)a.ws + kCounterBytes;
    p.part_o = (float*)ws;
    p.part_ml = (float*)(ws + units * n_split * rows_per_block * a.D * 4);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max;
    p.n_split = n_split; p.n_mblocks = n_mblocks; p.bm = rows_per_block; p.scale_log2 = 0.f; p.status = a.status;
    const long rows = (long)a.B * a.N * a.Hq;
    const int blocks = (int)((rows + 3) / 4);
    if (a.D == 128) attn_generic_combine_kernel<128><<<blocks, 128, 0, st>>>(p);
    else attn_generic_combine_kernel<64><<<blocks, 128, 0, st>>>(p);
    return cudaGetLastError();
}

// Per-device set-up: the D = 128 instance needs more than the default 48 KB of dynamic shared memory.
cudaError_t init_attn_generic() {
    return cudaFuncSetAttribute(attn_generic_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                BM * 128 * 2 + 4 * BN * 128 * 2);
}

cudaError_t launch_attn_generic(const AttnArgs& a, cudaStream_t st, int* n_launches) {
    *n_launches = 0;
    if (a.B == 0) return cudaSuccess;
    const int G = a.Hq / a.Hkv;
    const int n_mblocks = (G * a.N + BM - 1) / BM;
    const int units = a.B * a.Hkv * n_mblocks;
    const int max_tiles = (a.S_max + BN - 1) / BN;
    int n_split = (4 * a.sm_count + units - 1) / units;          // aim at ~4 CTAs per SM in flight
    n_split = n_split < 1 ? 1 : n_split;
    if (n_split > max_tiles) n_split = max_tiles;
    if (n_split > 32) n_split = 32;
    const size_t slot = slot_bytes(a.D);
    // the workspace holds at least (8*sm_count + units_max) half-slots of BM rows: always enough here
    while (n_split > 1 && kCounterBytes + (size_t)units * n_split * (slot / 2) > a.ws_bytes) --n_split;

    GenericParams p;
    p.q = (const __nv_bfloat16*)a.q; p.k = (const __nv_bfloat16*)a.k; p.v = (const __nv_bfloat16*)a.v;
    p.kv_len = a.kv_len; p.mask = a.mask; p.out = (__nv_bfloat16*)a.out; p.lse = a.lse;
    unsigned char* ws = (unsigned char*)a.ws + kCounterBytes;
    p.part_o = (float*)ws;
    p.part_ml = (float*)(ws + (size_t)units * n_split * BM * a.D * 4);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.S_max = a.S_max;
    p.n_split = n_split; p.n_mblocks = n_mblocks; p.bm = BM;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.status = a.status;

    dim3 grid(n_split, n_mblocks, a.B * a.Hkv);
    const size_t smem = (size_t)BM * a.D * 2 + 4 * (size_t)BN * a.D * 2;
    cudaError_t err;
    if (a.D == 128) attn_generic_kernel<128><<<grid, kThreads, smem, st>>>(p);
    else attn_generic_kernel<64><<<grid, kThreads, smem, st>>>(p);
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    ++*n_launches;
    if (n_split > 1) {
        const long rows = (long)a.B * a.N * a.Hq;
        const int blocks = (int)((rows + 3) / 4);
        if (a.D == 128) attn_generic_combine_kernel<128><<<blocks, 128, 0, st>>>(p);
        else attn_generic_combine_kernel<64><<<blocks, 128, 0, st>>>(p);
        err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        ++*n_launches;
    }
    return cudaSuccess;
}

}  // namespace vispec
