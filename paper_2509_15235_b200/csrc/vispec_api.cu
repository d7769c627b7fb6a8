// C ABI of libvispec: context management, argument validation, dispatch to the kernels.
#include <cstdlib>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "vispec_internal.h"

namespace vispec {

size_t workspace_bytes(const vispec_shape& s, int sm_count) {
    const int G = s.Hq / s.Hkv;
    const size_t units64 = (size_t)s.B_max * s.Hkv * ((G * s.N_max + 63) / 64);
    const size_t slot = slot_bytes(s.D);
    // generic kernel: at most 4*SMs + units partials of 64 rows (half slots);
    // persistent kernel: at most two partials of 128 rows per CTA, one CTA per SM.
    return kCounterBytes + (4 * (size_t)sm_count + units64) * (slot / 2) + 2 * (size_t)sm_count * slot + q_scratch_bytes(s);
}

// Rotated copy of q for the fused rotary call where it runs as two kernels: the last q_scratch_bytes of the workspace.
size_t q_scratch_bytes(const vispec_shape& s) {
    return ((size_t)s.B_max * s.N_max * s.Hq * s.D * 2 + 255) / 256 * 256;
}

}  // namespace vispec

using namespace vispec;

namespace {

// One NVTX range per hot entry point (a no-op costing a few nanoseconds unless a profiler is attached).
struct ApiRange {
    explicit ApiRange(const char* name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
};
#define VISPEC_RANGE() ApiRange api_range_(__func__)

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

extern "C" {

const char* vispec_strerror(int status) {
    switch (status) {
        case VISPEC_OK: return "ok";
        case VISPEC_E_NULL: return "required pointer is NULL";
        case VISPEC_E_ALIGN: return "pointer is not sufficiently aligned";
        case VISPEC_E_SHAPE: return "unsupported or inconsistent shape";
        case VISPEC_E_RANGE: return "index or length out of range";
        case VISPEC_E_UNSUPPORTED: return "request not supported by this build";
        case VISPEC_E_CUDA: return "CUDA call failed";
        case VISPEC_E_TIMEOUT: return "bounded device-side wait gave up";
        case VISPEC_E_BAD_TREE: return "parent array is not a valid tree";
        case VISPEC_E_UNREGISTERED: return "layer cache not registered (or pointers differ)";
        case VISPEC_E_WORKSPACE: return "workspace missing or too small";
        case VISPEC_E_POSITIONS: return "positions differ from kv_len + depth";
        default: return "unknown status";
    }
}

int vispec_ctx_create(vispec_ctx** out, const vispec_shape* s, int device) {
    if (!out || !s) return VISPEC_E_NULL;
    *out = nullptr;
    if (s->B_max < 1 || s->N_max < 1 || s->N_max > VISPEC_MAX_TREE_NODES || s->Hq < 1 || s->Hkv < 1 ||
        s->Hq % s->Hkv != 0 || (s->D != 64 && s->D != 128) || s->S_max < s->N_max || s->layers < 1)
        return VISPEC_E_SHAPE;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) return VISPEC_E_CUDA;
    if (device < 0 || device >= n_dev) return VISPEC_E_RANGE;
    if (cudaSetDevice(device) != cudaSuccess) return VISPEC_E_CUDA;
    vispec_ctx* c = new (std::nothrow) vispec_ctx();
    if (!c) return VISPEC_E_CUDA;
    c->shape = *s;
    c->device = device;
    bool ok = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_cache_ptrs, sizeof(void*) * 2 * s->layers) == cudaSuccess;
    ok = ok && cudaMemset(c->d_cache_ptrs, 0, sizeof(void*) * 2 * s->layers) == cudaSuccess;
    ok = ok && init_attn_generic() == cudaSuccess;
    ok = ok && init_attn_tc5() == cudaSuccess;
    ok = ok && init_stream_probe() == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) { vispec_ctx_destroy(c); return VISPEC_E_CUDA; }
    c->h_k.assign(s->layers, nullptr);
    c->h_v.assign(s->layers, nullptr);
    const char* fg = std::getenv("VISPEC_FORCE_GENERIC");
    c->force_generic = fg && fg[0] == '1';
    c->check_positions = std::getenv("VISPEC_DEBUG") != nullptr;
    c->k_map.resize(s->layers);
    c->page_rows.assign(s->layers, 0);
    c->num_blocks.assign(s->layers, 0);
    c->token_major.assign(s->layers, 0);
    c->v_map.resize(s->layers);
    *out = c;
    return VISPEC_OK;
}

int vispec_ctx_destroy(vispec_ctx* c) {
    if (!c) return VISPEC_OK;
    if (c->d_status) cudaFree(c->d_status);
    if (c->d_cache_ptrs) cudaFree(c->d_cache_ptrs);
    delete c;
    return VISPEC_OK;
}

int vispec_workspace_bytes(const vispec_ctx* c, size_t* out) {
    if (!c || !out) return VISPEC_E_NULL;
    *out = workspace_bytes(c->shape, c->sm_count);
    return VISPEC_OK;
}

int vispec_ctx_set_workspace(vispec_ctx* c, void* ws, size_t bytes) {
    if (!c || !ws) return VISPEC_E_NULL;
    if (!aligned(ws, 256)) return VISPEC_E_ALIGN;
    if (bytes < workspace_bytes(c->shape, c->sm_count)) return VISPEC_E_WORKSPACE;
    if (cudaMemset(ws, 0, kCounterBytes) != cudaSuccess) return VISPEC_E_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return VISPEC_E_CUDA;
    c->ws = ws;
    c->ws_bytes_used = workspace_bytes(c->shape, c->sm_count);
    c->ws_bytes = c->ws_bytes_used - q_scratch_bytes(c->shape);   // what the attention kernels may use for partials
    return VISPEC_OK;
}

int vispec_ctx_set_option(vispec_ctx* c, int option, int value) {
    if (!c) return VISPEC_E_NULL;
    switch (option) {
        case VISPEC_OPT_EARLY_PREFETCH: c->early_prefetch = value != 0; return VISPEC_OK;
        case VISPEC_OPT_FORCE_GENERIC: c->force_generic = value != 0; return VISPEC_OK;
        case VISPEC_OPT_SPLIT_FORM:
            if (value < 0 || value > 3) return VISPEC_E_RANGE;
            c->tc5_path = value; return VISPEC_OK;
        case VISPEC_OPT_KV_LEN_HINT:
            if (value < 0) return VISPEC_E_RANGE;
            c->kv_len_hint = value; return VISPEC_OK;
        case VISPEC_OPT_CHECK_POSITIONS: c->check_positions = value != 0; return VISPEC_OK;
        default: return VISPEC_E_UNSUPPORTED;
    }
}

int vispec_cache_register(vispec_ctx* c, int layer, void* k_cache, void* v_cache) {
    if (!c || !k_cache || !v_cache) return VISPEC_E_NULL;
    if (layer < 0 || layer >= c->shape.layers) return VISPEC_E_RANGE;
    if (!aligned(k_cache, 128) || !aligned(v_cache, 128)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (s.D == 128) {
        // 3-D view (d, slot, sequence*head) of a [B,Hkv,S_max,D] bf16 cache; one box = 64 d-columns
        // (128 bytes, the swizzle span) x 128 slots.  Slots past S_max read as zero.
        EncodeTiledFn enc = get_encode_fn();
        if (!enc) return VISPEC_E_CUDA;
        const cuuint64_t dims[3] = {(cuuint64_t)s.D, (cuuint64_t)s.S_max, (cuuint64_t)s.B_max * s.Hkv};
        const cuuint64_t strides[2] = {(cuuint64_t)s.D * 2, (cuuint64_t)s.S_max * s.D * 2};
        const cuuint32_t box[3] = {64, 128, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        void* ptrs[2] = {k_cache, v_cache};
        CUtensorMap* maps[2] = {&c->k_map[layer], &c->v_map[layer]};
        for (int t = 0; t < 2; ++t) {
            CUresult r = enc(maps[t], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptrs[t], dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return VISPEC_E_CUDA;
        }
    }
    void* pair[2] = {k_cache, v_cache};
    if (cudaMemcpy(c->d_cache_ptrs + 2 * layer, pair, sizeof(pair), cudaMemcpyHostToDevice) != cudaSuccess)
        return VISPEC_E_CUDA;
    c->h_k[layer] = k_cache;
    c->h_v[layer] = v_cache;
    c->page_rows[layer] = 0;
    c->num_blocks[layer] = 0;
    c->token_major[layer] = 0;
    return VISPEC_OK;
}

int vispec_cache_register_paged(vispec_ctx* c, int layer, void* k_pool, void* v_pool, int num_blocks, int page_rows,
                                int token_major) {
    if (!c || !k_pool || !v_pool) return VISPEC_E_NULL;
    if (layer < 0 || layer >= c->shape.layers) return VISPEC_E_RANGE;
    if (!aligned(k_pool, 128) || !aligned(v_pool, 128)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (s.D != 128) return VISPEC_E_UNSUPPORTED;
    if (num_blocks < 1 || (page_rows != 16 && page_rows != 32 && page_rows != 64 && page_rows != 128)) return VISPEC_E_SHAPE;
    if ((long long)num_blocks * s.Hkv >= (1ll << 31)) return VISPEC_E_SHAPE;
    if ((long long)num_blocks * page_rows >= (1ll << 31)) return VISPEC_E_SHAPE;
    // 3-D view of the bf16 pool, one box = 64 d-columns x one block's slots of one head: (d, slot in block, block*head)
    // for [num_blocks,Hkv,page_rows,D]; (d, head, block*page_rows + slot) for the token-major
    // [num_blocks,page_rows,Hkv,D].  A block number outside the pool reads as zero.
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return VISPEC_E_CUDA;
    const cuuint64_t row = (cuuint64_t)s.D * 2;
    const cuuint64_t dims_h[3] = {(cuuint64_t)s.D, (cuuint64_t)page_rows, (cuuint64_t)num_blocks * s.Hkv};
    const cuuint64_t dims_t[3] = {(cuuint64_t)s.D, (cuuint64_t)s.Hkv, (cuuint64_t)num_blocks * page_rows};
    const cuuint64_t strides_h[2] = {row, (cuuint64_t)page_rows * row};
    const cuuint64_t strides_t[2] = {row, (cuuint64_t)s.Hkv * row};
    const cuuint32_t box_h[3] = {64, (cuuint32_t)page_rows, 1};
    const cuuint32_t box_t[3] = {64, 1, (cuuint32_t)page_rows};
    const cuuint64_t* dims = token_major ? dims_t : dims_h;
    const cuuint64_t* strides = token_major ? strides_t : strides_h;
    const cuuint32_t* box = token_major ? box_t : box_h;
    const cuuint32_t estr[3] = {1, 1, 1};
    void* ptrs[2] = {k_pool, v_pool};
    CUtensorMap* maps[2] = {&c->k_map[layer], &c->v_map[layer]};
    for (int t = 0; t < 2; ++t) {
        CUresult r = enc(maps[t], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptrs[t], dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return VISPEC_E_CUDA;
    }
    void* pair[2] = {k_pool, v_pool};
    if (cudaMemcpy(c->d_cache_ptrs + 2 * layer, pair, sizeof(pair), cudaMemcpyHostToDevice) != cudaSuccess)
        return VISPEC_E_CUDA;
    c->h_k[layer] = k_pool;
    c->h_v[layer] = v_pool;
    c->page_rows[layer] = page_rows;
    c->num_blocks[layer] = num_blocks;
    c->token_major[layer] = token_major ? 1 : 0;
    return VISPEC_OK;
}

int vispec_tree_mask_build(vispec_ctx* c, const int32_t* parents, int B, int N, uint64_t* tree_mask,
                           int32_t* depth, void* stream) {
    VISPEC_RANGE();
    if (!c || !parents || !tree_mask) return VISPEC_E_NULL;
    if (B < 0 || B > c->shape.B_max || N < 1 || N > c->shape.N_max) return VISPEC_E_SHAPE;
    if (launch_tree_mask(parents, B, N, tree_mask, depth, c->d_status, (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_tree_verify_attn(vispec_ctx* c, int layer, const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* kv_len, const uint64_t* tree_mask, const int32_t* positions,
                            int B, int N, float scale, void* out, float* lse, void* stream) {
    VISPEC_RANGE();
    if (!c || !q || !kv_len || !tree_mask || !out) return VISPEC_E_NULL;
    if (!aligned(q, 16) || !aligned(out, 16)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    if (!c->h_k[layer]) return VISPEC_E_UNREGISTERED;
    if ((k_cache && k_cache != c->h_k[layer]) || (v_cache && v_cache != c->h_v[layer])) return VISPEC_E_UNREGISTERED;
    if (c->page_rows[layer]) return VISPEC_E_UNSUPPORTED;     // a paged layer goes through vispec_tree_verify_attn_paged
    if (!c->ws) return VISPEC_E_WORKSPACE;
    AttnArgs a = {};
    a.q = q; a.k = c->h_k[layer]; a.v = c->h_v[layer];
    a.kv_len = kv_len; a.mask = tree_mask; a.out = out; a.lse = lse;
    a.B = B; a.N = N; a.Hq = s.Hq; a.Hkv = s.Hkv; a.D = s.D; a.S_max = s.S_max;
    a.scale = scale; a.ws = c->ws; a.ws_bytes = c->ws_bytes; a.status = c->d_status;
    a.sm_count = c->sm_count;
    a.early_prefetch = c->early_prefetch;
    a.tc5_path = c->tc5_path;
    a.kv_len_hint = c->kv_len_hint;
    a.k_map = &c->k_map[layer]; a.v_map = &c->v_map[layer];
    int n = 0;
    cudaError_t err = (!c->force_generic && attn_tc5_supports(a)) ? launch_attn_tc5(a, (cudaStream_t)stream, &n)
                                                                  : launch_attn_generic(a, (cudaStream_t)stream, &n);
    c->launches += n;
    if (err == cudaSuccess && c->check_positions && positions && B > 0) {
        // after the attention, so that the attention keeps its place right behind its predecessor on the stream
        err = launch_check_positions(positions, kv_len, tree_mask, B, N, c->d_status, (cudaStream_t)stream);
        c->launches += 1;
    }
    return err == cudaSuccess ? VISPEC_OK : VISPEC_E_CUDA;
}

int vispec_rope_table_bytes(const vispec_ctx* c, int B, int N, size_t* out) {
    if (!c || !out) return VISPEC_E_NULL;
    if (B < 0 || N < 0) return VISPEC_E_SHAPE;
    *out = (size_t)B * N * (c->shape.D / 2) * (sizeof(double) * 2 + sizeof(float) * 2);
    return VISPEC_OK;
}

int vispec_rope_table_build(vispec_ctx* c, const int32_t* positions, int B, int N, float theta, void* table,
                            void* stream) {
    VISPEC_RANGE();
    if (!c || !positions || !table) return VISPEC_E_NULL;
    if (!aligned(table, 16)) return VISPEC_E_ALIGN;
    if (B < 0 || B > c->shape.B_max || N < 1 || N > c->shape.N_max || !(theta > 1.f)) return VISPEC_E_SHAPE;
    if (launch_rope_table(positions, B, N, c->shape.D, theta, table, (cudaStream_t)stream) != cudaSuccess) return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_tree_verify_attn_rope(vispec_ctx* c, int layer, const void* q, const void* k_new, const void* v_new,
                                 const void* rope_table, const int32_t* kv_len, const uint64_t* tree_mask, int B, int N,
                                 float scale, void* out, float* lse, void* stream) {
    VISPEC_RANGE();
    if (!c || !q || !k_new || !v_new || !rope_table || !kv_len || !tree_mask || !out) return VISPEC_E_NULL;
    if (!aligned(q, 16) || !aligned(out, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(rope_table, 16))
        return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    if (!c->h_k[layer]) return VISPEC_E_UNREGISTERED;
    if (c->page_rows[layer]) return VISPEC_E_UNSUPPORTED;
    if (!c->ws) return VISPEC_E_WORKSPACE;
    if (B == 0) return VISPEC_OK;
    AttnArgs a = {};
    a.q = q; a.k = c->h_k[layer]; a.v = c->h_v[layer];
    a.kv_len = kv_len; a.mask = tree_mask; a.out = out; a.lse = lse;
    a.B = B; a.N = N; a.Hq = s.Hq; a.Hkv = s.Hkv; a.D = s.D; a.S_max = s.S_max;
    a.scale = scale; a.ws = c->ws; a.ws_bytes = c->ws_bytes; a.status = c->d_status;
    a.sm_count = c->sm_count;
    a.early_prefetch = c->early_prefetch;
    a.tc5_path = c->tc5_path;
    a.kv_len_hint = c->kv_len_hint;
    a.k_map = &c->k_map[layer]; a.v_map = &c->v_map[layer];
    a.rope_table = rope_table; a.k_new = k_new; a.v_new = v_new;
    if (c->force_generic || !attn_tc5_supports(a)) return VISPEC_E_UNSUPPORTED;
    int n = 0;
    cudaError_t err = cudaSuccess;
    if (!attn_tc5_uses_clusters(a)) {
        // Where the kernel splits its work evenly over the SMs (many units, long caches) the in-kernel rotation costs
        // more than it saves: the rows go through the rotation kernel instead (the table in place of positions, q into
        // the scratch copy at the end of the workspace so that the caller's q stays as it is), then the plain attention.
        void* q_rot = (unsigned char*)c->ws + c->ws_bytes_used - q_scratch_bytes(s);
        err = launch_rope_rows(const_cast<void*>(q), k_new, v_new, nullptr, kv_len, c->h_k[layer], c->h_v[layer], 0.f, B, N,
                               s.Hq, s.Hkv, s.D, s.S_max, c->d_status, (cudaStream_t)stream, nullptr, 0, 0, 0, 0, q_rot,
                               rope_table);
        c->launches += 1;
        a.q = q_rot; a.rope_table = nullptr; a.k_new = nullptr; a.v_new = nullptr;
    }
    if (err == cudaSuccess) err = launch_attn_tc5(a, (cudaStream_t)stream, &n);
    c->launches += n;
    return err == cudaSuccess ? VISPEC_OK : VISPEC_E_CUDA;
}

int vispec_tree_verify_attn_paged(vispec_ctx* c, int layer, const void* q, const int32_t* kv_len,
                                  const int32_t* block_table, int table_stride, const uint64_t* tree_mask, int B, int N,
                                  float scale, void* out, float* lse, void* stream) {
    VISPEC_RANGE();
    if (!c || !q || !kv_len || !block_table || !tree_mask || !out) return VISPEC_E_NULL;
    if (!aligned(q, 16) || !aligned(out, 16)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max || table_stride < 1) return VISPEC_E_SHAPE;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    if (!c->h_k[layer]) return VISPEC_E_UNREGISTERED;
    if (!c->page_rows[layer]) return VISPEC_E_UNSUPPORTED;
    if ((long long)table_stride * c->page_rows[layer] > (1ll << 30)) return VISPEC_E_SHAPE;
    if (!c->ws) return VISPEC_E_WORKSPACE;
    if (B == 0) return VISPEC_OK;
    AttnArgs a = {};
    a.q = q; a.k = c->h_k[layer]; a.v = c->h_v[layer];
    a.kv_len = kv_len; a.mask = tree_mask; a.out = out; a.lse = lse;
    a.B = B; a.N = N; a.Hq = s.Hq; a.Hkv = s.Hkv; a.D = s.D;
    a.S_max = table_stride * c->page_rows[layer];
    a.scale = scale; a.ws = c->ws; a.ws_bytes = c->ws_bytes; a.status = c->d_status;
    a.sm_count = c->sm_count;
    a.early_prefetch = c->early_prefetch;
    a.tc5_path = c->tc5_path;
    a.kv_len_hint = c->kv_len_hint;
    a.k_map = &c->k_map[layer]; a.v_map = &c->v_map[layer];
    a.block_table = block_table; a.table_stride = table_stride;
    a.page_rows = c->page_rows[layer]; a.num_blocks = c->num_blocks[layer]; a.token_major = c->token_major[layer];
    if (!attn_tc5_supports(a)) return VISPEC_E_UNSUPPORTED;   // B <= 32, scale > 0, workspace large enough for the table's capacity
    int n = 0;
    cudaError_t err = launch_attn_tc5(a, (cudaStream_t)stream, &n);
    c->launches += n;
    return err == cudaSuccess ? VISPEC_OK : VISPEC_E_CUDA;
}

int vispec_kv_compact_paged(vispec_ctx* c, int layer_begin, int layer_end, const int32_t* path,
                            const int32_t* accept_len, const int32_t* kv_len, const int32_t* block_table,
                            int table_stride, int32_t* kv_len_out, int B, int N, void* stream) {
    VISPEC_RANGE();
    if (!c || !path || !accept_len || !kv_len || !block_table) return VISPEC_E_NULL;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max || table_stride < 1) return VISPEC_E_SHAPE;
    if (layer_begin < 0 || layer_end > s.layers || layer_begin > layer_end) return VISPEC_E_RANGE;
    if (kv_len_out == kv_len) return VISPEC_E_SHAPE;
    if (layer_begin == layer_end) return VISPEC_OK;
    const int pr = c->page_rows[layer_begin], nb = c->num_blocks[layer_begin];
    for (int l = layer_begin; l < layer_end; ++l) {
        if (!c->h_k[l]) return VISPEC_E_UNREGISTERED;
        if (!c->page_rows[l]) return VISPEC_E_UNSUPPORTED;
        if (c->page_rows[l] != pr || c->num_blocks[l] != nb || c->token_major[l] != c->token_major[layer_begin])
            return VISPEC_E_SHAPE;                                                   // one table serves every layer
    }
    if ((long long)table_stride * pr > (1ll << 30)) return VISPEC_E_SHAPE;
    if (launch_kv_compact(c->d_cache_ptrs, layer_begin, layer_end, path, accept_len, kv_len, kv_len_out, B, N, s.Hkv,
                          s.D, table_stride * pr, c->d_status, (cudaStream_t)stream, block_table, table_stride, pr,
                          nb, c->token_major[layer_begin]) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

// the layers [lb, le) are registered, paged, and share one pool geometry; returns VISPEC_OK or the error
static int paged_range_check(const vispec_ctx* c, int lb, int le, int table_stride) {
    if (table_stride < 1) return VISPEC_E_SHAPE;
    for (int l = lb; l < le; ++l) {
        if (!c->h_k[l]) return VISPEC_E_UNREGISTERED;
        if (!c->page_rows[l]) return VISPEC_E_UNSUPPORTED;
        if (c->page_rows[l] != c->page_rows[lb] || c->num_blocks[l] != c->num_blocks[lb] ||
            c->token_major[l] != c->token_major[lb])
            return VISPEC_E_SHAPE;
    }
    if (le > lb && (long long)table_stride * c->page_rows[lb] > (1ll << 30)) return VISPEC_E_SHAPE;
    return VISPEC_OK;
}

int vispec_accept_commit_paged(vispec_ctx* c, int layer_begin, int layer_end, const int32_t* draft_ids,
                               const int32_t* target_ids, const int32_t* parents, const int32_t* kv_len,
                               const int32_t* block_table, int table_stride, int B, int N, int32_t* path,
                               int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, void* stream) {
    VISPEC_RANGE();
    if (!c || !draft_ids || !target_ids || !parents || !kv_len || !block_table || !path || !accept_len || !bonus)
        return VISPEC_E_NULL;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (layer_begin < 0 || layer_end > s.layers || layer_begin >= layer_end) return VISPEC_E_RANGE;
    if (kv_len_out == kv_len) return VISPEC_E_SHAPE;
    const int rc = paged_range_check(c, layer_begin, layer_end, table_stride);
    if (rc != VISPEC_OK) return rc;
    const int pr = c->page_rows[layer_begin];
    if (launch_accept_commit(c->d_cache_ptrs, layer_begin, layer_end, draft_ids, target_ids, parents, kv_len, path,
                             accept_len, bonus, kv_len_out, B, N, s.Hkv, s.D, table_stride * pr, c->d_status,
                             (cudaStream_t)stream, block_table, table_stride, pr, c->num_blocks[layer_begin],
                             c->token_major[layer_begin]) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_rope_tree_rows_paged(vispec_ctx* c, int layer, void* q, const void* k_new, const void* v_new,
                                const int32_t* positions, const int32_t* kv_len, const int32_t* block_table,
                                int table_stride, int B, int N, float theta, void* stream) {
    VISPEC_RANGE();
    if (!c || !q || !k_new || !v_new || !positions || !kv_len || !block_table) return VISPEC_E_NULL;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max || !(theta > 1.f)) return VISPEC_E_SHAPE;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    const int rc = paged_range_check(c, layer, layer + 1, table_stride);
    if (rc != VISPEC_OK) return rc;
    const int pr = c->page_rows[layer];
    if (launch_rope_rows(q, k_new, v_new, positions, kv_len, c->h_k[layer], c->h_v[layer], theta, B, N, s.Hq, s.Hkv,
                         s.D, table_stride * pr, c->d_status, (cudaStream_t)stream, block_table, table_stride, pr,
                         c->num_blocks[layer], c->token_major[layer]) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_rope_tree_rows(vispec_ctx* c, int layer, void* q, const void* k_new, const void* v_new,
                          const int32_t* positions, const int32_t* kv_len, int B, int N, float theta, void* stream) {
    VISPEC_RANGE();
    if (!c || !q || !k_new || !v_new || !positions || !kv_len) return VISPEC_E_NULL;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16)) return VISPEC_E_ALIGN;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max || !(theta > 1.f)) return VISPEC_E_SHAPE;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    if (!c->h_k[layer]) return VISPEC_E_UNREGISTERED;
    if (c->page_rows[layer]) return VISPEC_E_UNSUPPORTED;
    if (launch_rope_rows(q, k_new, v_new, positions, kv_len, c->h_k[layer], c->h_v[layer], theta, B, N, s.Hq, s.Hkv,
                         s.D, s.S_max, c->d_status, (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_stream_probe(vispec_ctx* c, int layer, const int32_t* kv_len, int B, int N, void* stream) {
    VISPEC_RANGE();
    if (!c || !kv_len) return VISPEC_E_NULL;
    const vispec_shape& s = c->shape;
    if (B < 1 || B > s.B_max || B > 32 || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (s.D != 128) return VISPEC_E_UNSUPPORTED;
    if (layer < 0 || layer >= s.layers) return VISPEC_E_RANGE;
    if (!c->h_k[layer]) return VISPEC_E_UNREGISTERED;
    if (c->page_rows[layer]) return VISPEC_E_UNSUPPORTED;
    AttnArgs a = {};
    a.k = c->h_k[layer]; a.v = c->h_v[layer]; a.kv_len = kv_len;
    a.B = B; a.N = N; a.Hq = s.Hq; a.Hkv = s.Hkv; a.D = s.D; a.S_max = s.S_max;
    a.status = c->d_status; a.sm_count = c->sm_count; a.early_prefetch = c->early_prefetch;
    a.k_map = &c->k_map[layer]; a.v_map = &c->v_map[layer];
    if (launch_stream_probe(a, (cudaStream_t)stream) != cudaSuccess) return VISPEC_E_CUDA;
    c->launches += 1;
    return VISPEC_OK;
}

int vispec_accept(vispec_ctx* c, const int32_t* draft_ids, const int32_t* target_ids, const int32_t* parents,
                  int B, int N, int32_t* path, int32_t* accept_len, int32_t* bonus, void* stream) {
    VISPEC_RANGE();
    if (!c || !draft_ids || !target_ids || !parents || !path || !accept_len || !bonus) return VISPEC_E_NULL;
    if (B < 0 || B > c->shape.B_max || N < 1 || N > c->shape.N_max) return VISPEC_E_SHAPE;
    if (launch_accept(draft_ids, target_ids, parents, B, N, path, accept_len, bonus, c->d_status,
                      (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_tree_rerank(vispec_ctx* c, const int32_t* cand_parent, const int32_t* cand_token, const float* cand_score,
                       int B, int M, int K, int32_t* parents, int32_t* draft_ids, int32_t* selected, void* stream) {
    VISPEC_RANGE();
    if (!c || !cand_parent || !cand_token || !cand_score || !parents || !draft_ids || (!selected && K > 0))
        return VISPEC_E_NULL;
    if (B < 0 || B > c->shape.B_max || M < 1 || M > 2048 || K < 0 || K > M || K + 1 > c->shape.N_max)
        return VISPEC_E_SHAPE;
    if (launch_tree_rerank(cand_parent, cand_token, cand_score, B, M, K, parents, draft_ids, selected, c->d_status,
                           (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_accept_sampled(vispec_ctx* c, const int32_t* draft_ids, const int32_t* parents, const float* p_target,
                          const float* p_draft, const float* u_accept, const float* u_bonus, int B, int N, int V,
                          int32_t* path, int32_t* accept_len, int32_t* bonus, void* stream) {
    VISPEC_RANGE();
    if (!c || !draft_ids || !parents || !p_target || !p_draft || !u_accept || !u_bonus || !path || !accept_len || !bonus)
        return VISPEC_E_NULL;
    if (!aligned(p_target, 16) || !aligned(p_draft, 16)) return VISPEC_E_ALIGN;
    if (B < 0 || B > c->shape.B_max || N < 1 || N > c->shape.N_max || V < 1) return VISPEC_E_SHAPE;
    if (launch_accept_sampled(draft_ids, parents, p_target, p_draft, u_accept, u_bonus, B, N, V, path, accept_len, bonus,
                              c->d_status, (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_kv_compact(vispec_ctx* c, int layer_begin, int layer_end, const int32_t* path,
                      const int32_t* accept_len, const int32_t* kv_len, int32_t* kv_len_out, int B, int N,
                      void* stream) {
    VISPEC_RANGE();
    if (!c || !path || !accept_len || !kv_len) return VISPEC_E_NULL;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (layer_begin < 0 || layer_end > s.layers || layer_begin > layer_end) return VISPEC_E_RANGE;
    if (kv_len_out == kv_len) return VISPEC_E_SHAPE;
    for (int l = layer_begin; l < layer_end; ++l) {
        if (!c->h_k[l]) return VISPEC_E_UNREGISTERED;
        if (c->page_rows[l]) return VISPEC_E_UNSUPPORTED;
    }
    if (launch_kv_compact(c->d_cache_ptrs, layer_begin, layer_end, path, accept_len, kv_len, kv_len_out, B, N,
                          s.Hkv, s.D, s.S_max, c->d_status, (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    if (B > 0 && layer_end > layer_begin) c->launches += 1;
    return VISPEC_OK;
}

int vispec_accept_commit(vispec_ctx* c, int layer_begin, int layer_end, const int32_t* draft_ids,
                         const int32_t* target_ids, const int32_t* parents, const int32_t* kv_len, int B, int N,
                         int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, void* stream) {
    VISPEC_RANGE();
    if (!c || !draft_ids || !target_ids || !parents || !kv_len || !path || !accept_len || !bonus) return VISPEC_E_NULL;
    const vispec_shape& s = c->shape;
    if (B < 0 || B > s.B_max || N < 1 || N > s.N_max) return VISPEC_E_SHAPE;
    if (layer_begin < 0 || layer_end > s.layers || layer_begin > layer_end) return VISPEC_E_RANGE;
    if (kv_len_out == kv_len) return VISPEC_E_SHAPE;
    for (int l = layer_begin; l < layer_end; ++l) {
        if (!c->h_k[l]) return VISPEC_E_UNREGISTERED;
        if (c->page_rows[l]) return VISPEC_E_UNSUPPORTED;
    }
    if (layer_end == layer_begin) {
        // nothing to commit: plain acceptance
        if (launch_accept(draft_ids, target_ids, parents, B, N, path, accept_len, bonus, c->d_status,
                          (cudaStream_t)stream) != cudaSuccess)
            return VISPEC_E_CUDA;
    } else if (launch_accept_commit(c->d_cache_ptrs, layer_begin, layer_end, draft_ids, target_ids, parents, kv_len,
                                    path, accept_len, bonus, kv_len_out, B, N, s.Hkv, s.D, s.S_max, c->d_status,
                                    (cudaStream_t)stream) != cudaSuccess) {
        return VISPEC_E_CUDA;
    }
    if (B > 0) c->launches += 1;
    return VISPEC_OK;
}

int vispec_status_poll(vispec_ctx* c, int* code, void* stream) {
    if (!c || !code) return VISPEC_E_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    if (cudaMemcpyAsync(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return VISPEC_E_CUDA;
    if (cudaMemsetAsync(c->d_status, 0, sizeof(int), st) != cudaSuccess) return VISPEC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return VISPEC_E_CUDA;
    // a call that gave up on a wait may have left arrival counters behind: the next call finds them zero again
    if (v == VISPEC_E_TIMEOUT && c->ws && cudaMemsetAsync(c->ws, 0, kCounterBytes, st) != cudaSuccess) return VISPEC_E_CUDA;
    *code = v;
    return VISPEC_OK;
}

int vispec_selftest_bounded_wait(vispec_ctx* c, long long limit_cycles, void* stream) {
    if (!c) return VISPEC_E_NULL;
    if (limit_cycles < 1 || limit_cycles > (1ll << 31)) return VISPEC_E_RANGE;
    if (!c->ws) return VISPEC_E_WORKSPACE;
    if (launch_bounded_wait_selftest(limit_cycles, c->d_status, (int*)c->ws, (cudaStream_t)stream) != cudaSuccess)
        return VISPEC_E_CUDA;
    c->launches += 1;
    return VISPEC_OK;
}

int vispec_launch_count(const vispec_ctx* c, uint64_t* out) {
    if (!c || !out) return VISPEC_E_NULL;
    *out = c->launches;
    return VISPEC_OK;
}

}  // extern "C"
