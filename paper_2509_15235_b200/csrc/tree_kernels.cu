// Integer kernels of the verification step: ancestor mask, greedy acceptance, KV commit.
// All three are latency-bound (a few KB of traffic); each is a single launch.
#include <cuda_bf16.h>

#include "vispec_internal.h"

namespace vispec {

__device__ __forceinline__ void record_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

// ------------------------------------------------------------------------------------------------
// Ancestor mask (tree of Sec. 3.1 / App. A).  One block per sequence, one thread per node: the
// thread follows its node's parent links and ORs the visited indices into a 128-bit set.
// A chain that meets an invalid link yields the self bit only and flags VISPEC_E_BAD_TREE.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
tree_mask_kernel(const int32_t* __restrict__ parents, int N, uint64_t* __restrict__ mask,
                 int32_t* __restrict__ depth, int* status) {
    __shared__ int32_t par[VISPEC_MAX_TREE_NODES];
    const int b = blockIdx.x, i = threadIdx.x;
    if (i < N) par[i] = parents[(size_t)b * N + i];
    __syncthreads();
    if (i >= N) return;
    const int W = (N + 63) >> 6;
    uint64_t m0 = 0, m1 = 0;
    bool ok = (par[0] == -1);
    int a = i, d = 0;
    while (ok) {
        if (a < 64) m0 |= 1ull << a; else m1 |= 1ull << (a - 64);
        if (a == 0) break;
        const int p = par[a];
        if (p < 0 || p >= a) { ok = false; break; }
        a = p;
        ++d;
    }
    if (!ok) {
        m0 = i < 64 ? 1ull << i : 0;
        m1 = i < 64 ? 0 : 1ull << (i - 64);
        d = 0;
        record_status(status, VISPEC_E_BAD_TREE);
    }
    uint64_t* row = mask + ((size_t)b * N + i) * W;
    row[0] = m0;
    if (W > 1) row[1] = m1;
    if (depth) depth[(size_t)b * N + i] = d;
}

cudaError_t launch_tree_mask(const int32_t* parents, int B, int N, uint64_t* mask, int32_t* depth,
                             int* status, cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    tree_mask_kernel<<<B, 128, 0, st>>>(parents, N, mask, depth, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Greedy acceptance (Sec. 3.1 at temperature 0).  One warp per sequence; lane l owns nodes
// l, l+32, l+64, l+96.  matched bits are gathered with ballots into a 128-bit set; a node is
// reachable iff its ancestor set minus the matched set is empty; the winner is the deepest
// reachable node (smallest index among equals), found with a shuffle max-reduction on the key
// depth*256 + (255 - index).
// ------------------------------------------------------------------------------------------------
// One warp decides one sequence.  par / tgt are shared-memory copies of the sequence's parents and target ids
// (filled by the caller, visible to the warp).  Returns (warp-uniform) the accepted length; `path_out[0..N)`
// (any memory the warp can write) receives the path padded with -1, `*bonus_out` the bonus token (lane 0).
__device__ int accept_warp(const int32_t* __restrict__ draft_row, const int32_t* par, const int32_t* tgt, int N,
                           int32_t* path_out, int32_t* bonus_out, int* status) {
    const int lane = threadIdx.x & 31;
    // validity of the whole tree (every link must point to an earlier node)
    bool tree_ok = true;
    for (int i = lane; i < N; i += 32) tree_ok &= (i == 0) ? (par[0] == -1) : (par[i] >= 0 && par[i] < i);
    tree_ok = __all_sync(0xffffffffu, tree_ok);

    uint32_t matched[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const int i = w * 32 + lane;
        bool m = false;
        if (tree_ok && i < N) m = (i == 0) || (draft_row[i] == tgt[par[i]]);
        matched[w] = __ballot_sync(0xffffffffu, m);
    }
    int best_key = -1;
    if (tree_ok) {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const int i = w * 32 + lane;
            if (i < N) {
                uint32_t anc[4] = {0, 0, 0, 0};
                int d = 0;
                for (int a = i; ; a = par[a]) { anc[a >> 5] |= 1u << (a & 31); if (a == 0) break; ++d; }
                const bool reach = ((anc[0] & ~matched[0]) | (anc[1] & ~matched[1]) |
                                    (anc[2] & ~matched[2]) | (anc[3] & ~matched[3])) == 0;
                if (reach) best_key = max(best_key, d * 256 + (255 - i));
            }
        }
    } else {
        if (lane == 0) { best_key = 255; record_status(status, VISPEC_E_BAD_TREE); }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) best_key = max(best_key, __shfl_xor_sync(0xffffffffu, best_key, off));
    const int best_depth = best_key >> 8;
    const int best = 255 - (best_key & 255);
    for (int k = lane; k < N; k += 32) if (k > best_depth) path_out[k] = -1;
    if (lane == 0) {
        int a = best;
        for (int k = best_depth; k >= 0; --k) { path_out[k] = a; a = (a == 0) ? 0 : par[a]; }
        *bonus_out = tgt[best];
    }
    return best_depth + 1;
}

__global__ void __launch_bounds__(32)
accept_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ target,
              const int32_t* __restrict__ parents, int N, int32_t* __restrict__ path,
              int32_t* __restrict__ accept_len, int32_t* __restrict__ bonus, int* status) {
    __shared__ int32_t par[VISPEC_MAX_TREE_NODES];
    __shared__ int32_t tgt[VISPEC_MAX_TREE_NODES];
    const int b = blockIdx.x, lane = threadIdx.x;
    const size_t base = (size_t)b * N;
    for (int i = lane; i < N; i += 32) { par[i] = parents[base + i]; tgt[i] = target[base + i]; }
    __syncwarp();
    const int len = accept_warp(draft + base, par, tgt, N, path + base, bonus + b, status);
    if (lane == 0) accept_len[b] = len;
}

cudaError_t launch_accept(const int32_t* draft, const int32_t* target, const int32_t* parents, int B,
                          int N, int32_t* path, int32_t* accept_len, int32_t* bonus, int* status,
                          cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    accept_kernel<<<B, 32, 0, st>>>(draft, target, parents, N, path, accept_len, bonus, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// KV commit (App. A, pre-allocated cache).  One block per (layer, sequence, kv head); rows are
// D*2 contiguous bytes and move as 16-byte vectors.  Entries are processed in passes of 16 path
// positions in increasing order: gather the pass into shared memory, barrier, scatter.  Because the
// path is strictly increasing with path[k] >= k, a pass writes only slots below every later pass's
// sources, so the result equals gather-everything-then-scatter.  Entries with path[k] == k are
// already in place and are skipped.
// ------------------------------------------------------------------------------------------------
constexpr int kCompactRows = 16;

// Where logical slot `slot` of (sequence b, kv head h) lives, in 16-byte vectors from the tensor's base.
// Contiguous cache [B,Hkv,S_max,D]: table == nullptr.  Paged pool [num_blocks,Hkv,page_rows,D], or
// [num_blocks,page_rows,Hkv,D] if token_major: through the block table; -1 if the table entry is outside the pool.
struct RowMap {
    const int32_t* table; int table_stride, page_rows, num_blocks, token_major;
    __device__ __forceinline__ long long at(int b, int h, int slot, int Hkv, int S_max, int chunks) const {
        if (!table) return (((long long)b * Hkv + h) * S_max + slot) * chunks;
        const int blk = table[(size_t)b * table_stride + slot / page_rows];
        if (blk < 0 || blk >= num_blocks) return -1;
        if (token_major) return (((long long)blk * page_rows + slot % page_rows) * Hkv + h) * chunks;
        return (((long long)blk * Hkv + h) * page_rows + slot % page_rows) * chunks;
    }
};

__global__ void __launch_bounds__(256)
kv_compact_kernel(void* const* __restrict__ cache_ptrs, int layer_begin, const int32_t* __restrict__ path,
                  const int32_t* __restrict__ accept_len, const int32_t* __restrict__ kv_len,
                  int32_t* __restrict__ kv_len_out, int N, int Hkv, int D, int S_max, int* status,
                  const int32_t* __restrict__ block_table, int table_stride, int page_rows, int num_blocks,
                  int token_major) {
    __shared__ uint4 stage[2][kCompactRows][16];   // up to 256 B per row (D = 128)
    __shared__ int32_t src_row[kCompactRows];
    const int layer = layer_begin + blockIdx.z, b = blockIdx.y, h = blockIdx.x;
    const int S = kv_len[b], L = accept_len[b];
    const bool ok = (L >= 1 && L <= N && S >= 0 && S + N <= S_max);
    if (!ok) {
        if (threadIdx.x == 0) record_status(status, VISPEC_E_RANGE);
        return;   // kv_len_out[b] keeps its previous value for a rejected sequence
    }
    const int chunks = D / 8;                        // 16-byte vectors per row
    const int tensor = threadIdx.x >> 7;             // 0: K, 1: V
    const int r = (threadIdx.x & 127) >> 3;          // row of the pass, 0..15
    const int c0 = threadIdx.x & 7;                  // this thread moves chunks c0 and c0 + 8
    uint4* const tensor_base = reinterpret_cast<uint4*>(cache_ptrs[2 * layer + tensor]);
    bool bad = false;
    const RowMap rows = {block_table, table_stride, page_rows, num_blocks, token_major};
    // a table entry outside the pool drops the move and is reported
    auto row_of = [&](int slot) -> uint4* {
        const long long o = rows.at(b, h, slot, Hkv, S_max, chunks);
        if (o < 0) { bad = true; return nullptr; }
        return tensor_base + o;
    };
    for (int k0 = 0; k0 < L; k0 += kCompactRows) {
        if (threadIdx.x < kCompactRows) {
            const int k = k0 + threadIdx.x;
            int s = (k < L) ? path[(size_t)b * N + k] : -1;
            if (k < L && (s < k || s >= N)) { s = -1; bad = true; }
            src_row[threadIdx.x] = (s == k) ? -1 : s;   // -1: nothing to move
        }
        __syncthreads();
        const int s = src_row[r];
        const uint4* src = s >= 0 ? row_of(S + s) : nullptr;
        uint4* dst = s >= 0 ? row_of(S + k0 + r) : nullptr;
        const bool move = src && dst;
        if (move) {
            if (c0 < chunks) stage[tensor][r][c0] = src[c0];
            if (c0 + 8 < chunks) stage[tensor][r][c0 + 8] = src[c0 + 8];
        }
        __syncthreads();
        if (move) {
            if (c0 < chunks) dst[c0] = stage[tensor][r][c0];
            if (c0 + 8 < chunks) dst[c0 + 8] = stage[tensor][r][c0 + 8];
        }
        __syncthreads();
    }
    if (bad) record_status(status, VISPEC_E_RANGE);
    if (kv_len_out && blockIdx.x == 0 && blockIdx.z == 0 && threadIdx.x == 0) kv_len_out[b] = S + L;
}

cudaError_t launch_kv_compact(void* const* cache_ptrs, int layer_begin, int layer_end,
                              const int32_t* path, const int32_t* accept_len, const int32_t* kv_len,
                              int32_t* kv_len_out, int B, int N, int Hkv, int D, int S_max, int* status,
                              cudaStream_t st, const int32_t* block_table, int table_stride, int page_rows,
                              int num_blocks, int token_major) {
    if (B == 0 || layer_end <= layer_begin) return cudaSuccess;
    dim3 grid(Hkv, B, layer_end - layer_begin);
    kv_compact_kernel<<<grid, 256, 0, st>>>(cache_ptrs, layer_begin, path, accept_len, kv_len, kv_len_out,
                                            N, Hkv, D, S_max, status, block_table, table_stride, page_rows, num_blocks,
                                            token_major);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Acceptance and commit in one launch (Sec. 3.1 acceptance followed by the App. A commit): every block
// (layer, sequence, kv head) repeats the cheap acceptance of its sequence in its first warp, keeps the path
// in shared memory and then moves its head's rows exactly as kv_compact_kernel does; the block of the first
// layer and head also writes path, accept_len, bonus and kv_len_out.  Saves a launch and a dependency per
// decoding cycle.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
accept_commit_kernel(void* const* __restrict__ cache_ptrs, int layer_begin, const int32_t* __restrict__ draft,
                     const int32_t* __restrict__ target, const int32_t* __restrict__ parents,
                     const int32_t* __restrict__ kv_len, int32_t* __restrict__ path, int32_t* __restrict__ accept_len,
                     int32_t* __restrict__ bonus, int32_t* __restrict__ kv_len_out, int N, int Hkv, int D, int S_max,
                     int* status, const RowMap rows) {
    __shared__ uint4 stage[2][kCompactRows][16];
    __shared__ int32_t par[VISPEC_MAX_TREE_NODES];
    __shared__ int32_t tgt[VISPEC_MAX_TREE_NODES];
    __shared__ int32_t spath[VISPEC_MAX_TREE_NODES];
    __shared__ int32_t s_len, s_bonus;
    const int layer = layer_begin + blockIdx.z, b = blockIdx.y, h = blockIdx.x;
    const size_t rb = (size_t)b * N;
    for (int i = threadIdx.x; i < N; i += 256) { par[i] = parents[rb + i]; tgt[i] = target[rb + i]; }
    __syncthreads();
    const bool writer = (blockIdx.x == 0 && blockIdx.z == 0);
    if (threadIdx.x < 32) {
        const int len = accept_warp(draft + rb, par, tgt, N, spath, &s_bonus, writer ? status : nullptr);
        if (threadIdx.x == 0) s_len = len;
    }
    __syncthreads();
    const int S = kv_len[b], L = s_len;
    if (writer) {
        for (int i = threadIdx.x; i < N; i += 256) path[rb + i] = spath[i];
        if (threadIdx.x == 0) { accept_len[b] = L; bonus[b] = s_bonus; }
    }
    const bool ok = (S >= 0 && S + N <= S_max);
    if (!ok) {
        if (threadIdx.x == 0 && writer) record_status(status, VISPEC_E_RANGE);
        return;   // kv_len_out[b] keeps its previous value for a rejected sequence
    }
    const int chunks = D / 8;
    const int tensor = threadIdx.x >> 7;             // 0: K, 1: V
    const int r = (threadIdx.x & 127) >> 3;          // row of the pass, 0..15
    const int c0 = threadIdx.x & 7;                  // this thread moves chunks c0 and c0 + 8
    uint4* const tensor_base = reinterpret_cast<uint4*>(cache_ptrs[2 * layer + tensor]);
    bool bad = false;
    for (int k0 = 0; k0 < L; k0 += kCompactRows) {
        const int k = k0 + r;
        const int s = (k < L && spath[k] != k) ? spath[k] : -1;     // -1: nothing to move
        const long long so = s >= 0 ? rows.at(b, h, S + s, Hkv, S_max, chunks) : -1;
        const long long d_off = s >= 0 ? rows.at(b, h, S + k, Hkv, S_max, chunks) : -1;
        if (s >= 0 && (so < 0 || d_off < 0)) bad = true;               // table entry outside the pool: move dropped
        const bool move = so >= 0 && d_off >= 0;
        if (move) {
            const uint4* src = tensor_base + so;
            if (c0 < chunks) stage[tensor][r][c0] = src[c0];
            if (c0 + 8 < chunks) stage[tensor][r][c0 + 8] = src[c0 + 8];
        }
        __syncthreads();
        if (move) {
            uint4* dst = tensor_base + d_off;
            if (c0 < chunks) dst[c0] = stage[tensor][r][c0];
            if (c0 + 8 < chunks) dst[c0 + 8] = stage[tensor][r][c0 + 8];
        }
        __syncthreads();
    }
    if (bad) record_status(status, VISPEC_E_RANGE);
    if (kv_len_out && writer && threadIdx.x == 0) kv_len_out[b] = S + L;
}

cudaError_t launch_accept_commit(void* const* cache_ptrs, int layer_begin, int layer_end, const int32_t* draft,
                                 const int32_t* target, const int32_t* parents, const int32_t* kv_len,
                                 int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, int B, int N,
                                 int Hkv, int D, int S_max, int* status, cudaStream_t st, const int32_t* block_table,
                                 int table_stride, int page_rows, int num_blocks, int token_major) {
    if (B == 0 || layer_end <= layer_begin) return cudaSuccess;
    dim3 grid(Hkv, B, layer_end - layer_begin);
    const RowMap rows = {block_table, table_stride, page_rows, num_blocks, token_major};
    accept_commit_kernel<<<grid, 256, 0, st>>>(cache_ptrs, layer_begin, draft, target, parents, kv_len, path,
                                               accept_len, bonus, kv_len_out, N, Hkv, D, S_max, status, rows);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Rotary embedding of the tree's q and k rows and placement of the k and v rows at slots S + i (the step
// before the attention; Sec. 3.2: the target LLM is unchanged, and LLaVA-v1.6 / Qwen2.5-VL rotate q and k by
// position with the half-split pairing, element j with element j + D/2).  Each block forms the
// D/2 angles positions[b][i] * theta^(-2j/D) of its (node, sequence) in fp64 (positions run into the thousands,
// where fp32 argument reduction would cost digits), rotates its rows' pairs in fp64 and rounds once to bf16
// (a few hundred thousand pairs: the arithmetic rate does not matter).  Latency-bound: about 1.5 MB per call.
// ------------------------------------------------------------------------------------------------
// Rows of one (node, sequence): Hq of q, Hkv of k, Hkv of v.  D/16 threads share a row, each holding 8 elements of
// the lower half and the 8 they pair with in the upper half (two 16-byte loads, issued before any arithmetic); a
// block covers 128 / (D/16) rows, blockIdx.z walks the rows, so the whole call is one wave of small blocks.
__device__ __forceinline__ void rope_rotate8(uint4& lo, uint4& hi, const double* cs, const double* sn) {
    __nv_bfloat16* a = reinterpret_cast<__nv_bfloat16*>(&lo);
    __nv_bfloat16* b = reinterpret_cast<__nv_bfloat16*>(&hi);
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const double x = (double)__bfloat162float(a[t]), y = (double)__bfloat162float(b[t]);
        a[t] = __double2bfloat16(x * cs[t] - y * sn[t]);
        b[t] = __double2bfloat16(y * cs[t] + x * sn[t]);
    }
}

__global__ void __launch_bounds__(128)
rope_rows_kernel(__nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_new,
                 const __nv_bfloat16* __restrict__ v_new, const int32_t* __restrict__ positions,
                 const int32_t* __restrict__ kv_len, __nv_bfloat16* __restrict__ k_cache,
                 __nv_bfloat16* __restrict__ v_cache, double log2_theta, int N, int Hq, int Hkv, int D, int S_max,
                 int* status, const RowMap rmap, __nv_bfloat16* __restrict__ q_out, const double2* __restrict__ table) {
    __shared__ double cs[64], sn[64];
    // First wait for the kernel before this one (q / k_new / v_new may come from it, and so may kv_len), only then let
    // the next kernel in: an attention call that follows reads kv_len and committed cache rows before its own wait,
    // and must not do so while the kernel two places back (a commit, say) is still running.  Its prologue still
    // overlaps these blocks; this kernel writes only q and slots at or above kv_len.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int i = blockIdx.x, b = blockIdx.y, half = D / 2;
    const int S = kv_len[b];
    if (S < 0 || S + N > S_max) {
        if (threadIdx.x == 0 && i == 0 && blockIdx.z == 0) record_status(status, VISPEC_E_RANGE);
        return;
    }
    const int tpr = D / 16;                                   // threads per row
    const int row = blockIdx.z * (128 / tpr) + threadIdx.x / tpr, c8 = (threadIdx.x % tpr) * 8;
    const int rows = Hq + 2 * Hkv;
    // this thread's two vectors: source and destination
    const uint4* src = nullptr;
    uint4* dst = nullptr;
    if (row < Hq) {
        const size_t o = (((size_t)b * N + i) * Hq + row) * D;
        src = reinterpret_cast<const uint4*>(q + o);
        dst = reinterpret_cast<uint4*>(q_out + o);      // q itself, or a separate rotated copy
    } else if (row < rows) {
        const bool is_k = row < Hq + Hkv;
        const int hk = row - Hq - (is_k ? 0 : Hkv);
        src = reinterpret_cast<const uint4*>((is_k ? k_new : v_new) + (((size_t)b * N + i) * Hkv + hk) * D);
        const long long o = rmap.at(b, hk, S + i, Hkv, S_max, D / 8);
        if (o >= 0) dst = reinterpret_cast<uint4*>(is_k ? k_cache : v_cache) + o;
        else { src = nullptr; if ((threadIdx.x % tpr) == 0) record_status(status, VISPEC_E_RANGE); }   // entry outside the pool: row dropped
    }
    uint4 lo = make_uint4(0, 0, 0, 0), hi = lo;
    if (src) {
        lo = src[c8 / 8];
        hi = src[(c8 + half) / 8];
    }
    if ((int)threadIdx.x < half) {
        double s_, c_;
        if (table) {                                      // the same values, formed once per cycle by rope_table_kernel
            const double2 t = table[((size_t)b * N + i) * half + threadIdx.x];
            c_ = t.x; s_ = t.y;
        } else {
            const double ang = (double)positions[(size_t)b * N + i] * exp2(-2.0 * (double)threadIdx.x / (double)D * log2_theta);
            sincos(ang, &s_, &c_);
        }
        cs[threadIdx.x] = c_;
        sn[threadIdx.x] = s_;
    }
    __syncthreads();
    if (!src) return;
    if (row < Hq + Hkv) rope_rotate8(lo, hi, cs + c8, sn + c8);
    dst[c8 / 8] = lo;
    dst[(c8 + half) / 8] = hi;
}

namespace {
// One block per (node, sequence), one thread per frequency: the angle and its sine and cosine exactly as
// rope_rows_kernel forms them, stored once as fp64 and once rounded to fp32.
__global__ void rope_table_kernel(const int32_t* __restrict__ positions, double log2_theta, int N, int D,
                                  double2* __restrict__ tab64, float2* __restrict__ tab32) {
    const int i = blockIdx.x, b = blockIdx.y, j = threadIdx.x;
    if (j >= D / 2) return;
    const double ang = (double)positions[(size_t)b * N + i] * exp2(-2.0 * (double)j / (double)D * log2_theta);
    double s_, c_;
    sincos(ang, &s_, &c_);
    const size_t o = ((size_t)b * N + i) * (D / 2) + j;
    tab64[o] = make_double2(c_, s_);
    tab32[o] = make_float2((float)c_, (float)s_);
}
}  // namespace

cudaError_t launch_rope_table(const int32_t* positions, int B, int N, int D, float theta, void* table, cudaStream_t st) {
    if (B * N == 0) return cudaSuccess;
    double2* t64 = (double2*)table;
    float2* t32 = (float2*)(t64 + (size_t)B * N * (D / 2));
    rope_table_kernel<<<dim3(N, B), D / 2, 0, st>>>(positions, log2((double)theta), N, D, t64, t32);
    return cudaGetLastError();
}

namespace {
// One thread per (sequence, node): the position a draft-tree node carries is the committed length plus its depth, and
// the depth is the number of its ancestors, i.e. the set bits of its mask row minus its own.
__global__ void check_positions_kernel(const int32_t* __restrict__ positions, const int32_t* __restrict__ kv_len,
                                       const uint64_t* __restrict__ mask, int B, int N, int* status) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * N) return;
    const int b = idx / N, W = (N + 63) >> 6;
    int bits = 0;
    for (int w = 0; w < W; ++w) bits += __popcll(mask[(size_t)idx * W + w]);
    if (positions[idx] != kv_len[b] + bits - 1) record_status(status, VISPEC_E_POSITIONS);
}
}  // namespace

cudaError_t launch_check_positions(const int32_t* positions, const int32_t* kv_len, const uint64_t* mask, int B, int N,
                                   int* status, cudaStream_t st) {
    if (B * N == 0) return cudaSuccess;
    check_positions_kernel<<<(B * N + 127) / 128, 128, 0, st>>>(positions, kv_len, mask, B, N, status);
    return cudaGetLastError();
}

cudaError_t launch_rope_rows(void* q, const void* k_new, const void* v_new, const int32_t* positions,
                             const int32_t* kv_len, void* k_cache, void* v_cache, float theta, int B, int N, int Hq,
                             int Hkv, int D, int S_max, int* status, cudaStream_t st, const int32_t* block_table,
                             int table_stride, int page_rows, int num_blocks, int token_major, void* q_out,
                             const void* angle_table) {
    if (B == 0) return cudaSuccess;
    const RowMap rmap = {block_table, table_stride, page_rows, num_blocks, token_major};
    cudaLaunchConfig_t cfg = {};
    const int rows_per_block = 128 / (D / 16);
    cfg.gridDim = dim3(N, B, (Hq + 2 * Hkv + rows_per_block - 1) / rows_per_block);
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rope_rows_kernel, (__nv_bfloat16*)q, (const __nv_bfloat16*)k_new,
                              (const __nv_bfloat16*)v_new, positions, kv_len, (__nv_bfloat16*)k_cache,
                              (__nv_bfloat16*)v_cache, angle_table ? 0.0 : log2((double)theta), N, Hq, Hkv, D, S_max, status,
                              rmap, (__nv_bfloat16*)(q_out ? q_out : q), (const double2*)angle_table);
}

// ------------------------------------------------------------------------------------------------
// Tree rerank (App. A: 30 draft tokens kept from a depth-3, width-8 expansion; the tree is EAGLE-2's, which
// keeps the candidates of highest cumulative log-probability).  One block per sequence.  Scores become
// order-preserving 32-bit keys (NaN lowest); a candidate's rank is the number of candidates ahead of it
// (higher key, or equal key and lower index), counted against the keys in shared memory: M^2 compares,
// 18 K for the paper's 136 candidates.  Kept candidates are numbered in candidate order, which keeps
// parents ahead of children.
// ------------------------------------------------------------------------------------------------
constexpr int kRerankMaxM = 2048;

__global__ void __launch_bounds__(256)
tree_rerank_kernel(const int32_t* __restrict__ cand_parent, const int32_t* __restrict__ cand_token,
                   const float* __restrict__ cand_score, int M, int K, int32_t* __restrict__ parents,
                   int32_t* __restrict__ draft_ids, int32_t* __restrict__ selected, int* status) {
    __shared__ uint32_t key[kRerankMaxM];
    __shared__ int16_t node[kRerankMaxM];        // node number of a kept candidate, 0 if dropped
    __shared__ int warp_cnt[8];
    __shared__ int sh_bad;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int32_t* cp = cand_parent + (size_t)b * M;
    if (tid == 0) sh_bad = 0;
    for (int i = tid; i < M; i += 256) {
        const float s = cand_score[(size_t)b * M + i];
        const uint32_t u = __float_as_uint(s);
        // ascending float order -> ascending unsigned order; -0 and +0 made equal; NaN below everything
        uint32_t k = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
        if (s == 0.0f) k = 0x80000000u;
        if (s != s) k = 0u;
        key[i] = k;
    }
    __syncthreads();
    // pass over the candidates in chunks of 256 (in index order) so that the node numbers can be handed out
    // by a block-wide prefix count
    int base = 0;
    for (int i0 = 0; i0 < M; i0 += 256) {
        const int i = i0 + tid;
        bool keep = false;
        if (i < M) {
            const uint32_t ki = key[i];
            int ahead = 0;
            for (int j = 0; j < M; ++j) {
                const uint32_t kj = key[j];
                ahead += (kj > ki) || (kj == ki && j < i);
            }
            keep = ahead < K;
            const int pr = cp[i];
            if (pr < -1 || pr >= i) sh_bad = 1;
        }
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_cnt[w] = __popc(m);
        __syncthreads();
        int before = base + __popc(m & ((1u << lane) - 1));
        for (int x = 0; x < w; ++x) before += warp_cnt[x];
        int total = 0;
        for (int x = 0; x < 8; ++x) total += warp_cnt[x];
        if (i < M) node[i] = keep ? (int16_t)(before + 1) : (int16_t)0;
        base += total;
        __syncthreads();
    }
    // a kept candidate whose parent was dropped breaks the tree
    for (int i = tid; i < M; i += 256) {
        const int pr = cp[i];
        if (node[i] && pr >= 0 && pr < i && !node[pr]) sh_bad = 1;
    }
    __syncthreads();
    const bool bad = sh_bad != 0;
    int32_t* po = parents + (size_t)b * (K + 1);
    int32_t* io = draft_ids + (size_t)b * (K + 1);
    if (tid == 0) {
        po[0] = -1;
        io[0] = 0;
        if (bad) record_status(status, VISPEC_E_BAD_TREE);
    }
    for (int i = tid; i < M; i += 256) {
        const int n = node[i];
        if (!n) continue;
        selected[(size_t)b * K + n - 1] = i;
        io[n] = cand_token[(size_t)b * M + i];
        const int pr = cp[i];
        po[n] = bad ? -1 : (pr == -1 ? 0 : (int)node[pr]);
    }
}

cudaError_t launch_tree_rerank(const int32_t* cand_parent, const int32_t* cand_token, const float* cand_score, int B,
                               int M, int K, int32_t* parents, int32_t* draft_ids, int32_t* selected, int* status,
                               cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    tree_rerank_kernel<<<B, 256, 0, st>>>(cand_parent, cand_token, cand_score, M, K, parents, draft_ids, selected, status);
    return cudaGetLastError();
}

}  // namespace vispec
