// Internal declarations shared by the translation units of libvispec (never installed).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <vector>

#include "vispec.h"

struct vispec_ctx {
    vispec_shape shape;
    int device = 0;
    int sm_count = 0;
    int* d_status = nullptr;        // device status word (first asynchronous error wins)
    void** d_cache_ptrs = nullptr;  // device table [layers][2]: k_cache, v_cache
    std::vector<void*> h_k, h_v;    // host copy of the registered pointers
    std::vector<CUtensorMap> k_map, v_map;  // TMA descriptors per layer (D == 128 only)
    std::vector<int> page_rows, num_blocks; // per layer: slots per pool block (0 = contiguous cache), pool blocks
    std::vector<int> token_major;           // per layer: pool is [block][slot][head][D] instead of [block][head][slot][D]
    void* ws = nullptr;             // caller-owned workspace
    size_t ws_bytes = 0;            // of which the attention kernels' partials may use this much
    size_t ws_bytes_used = 0;       // vispec_workspace_bytes(): the rotated-q scratch sits at its end
    uint64_t launches = 0;
    bool force_generic = false;     // VISPEC_OPT_FORCE_GENERIC (or VISPEC_FORCE_GENERIC=1 at context creation)
    bool early_prefetch = true;     // VISPEC_OPT_EARLY_PREFETCH
    int tc5_path = 0;               // VISPEC_OPT_SPLIT_FORM: 0 automatic, 1 partials in global memory, 2 clusters, 3 merge kernel always
    int kv_len_hint = 0;            // VISPEC_OPT_KV_LEN_HINT
    bool check_positions = false;   // VISPEC_OPT_CHECK_POSITIONS (or VISPEC_DEBUG in the environment at context creation)
};

namespace vispec {

// ---- workspace layout -------------------------------------------------------------------------
// [0, kCounterBytes)            arrival counters (int32), zero between calls
// [kCounterBytes, ...)          partial-result slots, each kSlotRows rows of (D fp32 + m + l)
constexpr size_t kCounterBytes = 64 * 1024;
constexpr int kSlotRows = 128;
inline size_t slot_bytes(int D) { return (size_t)kSlotRows * ((size_t)D * 4 + 8); }
size_t workspace_bytes(const vispec_shape& s, int sm_count);
size_t q_scratch_bytes(const vispec_shape& s);

// ---- kernels' host launchers (each returns a cudaError_t from the launch) -----------------------
cudaError_t launch_tree_mask(const int32_t* parents, int B, int N, uint64_t* mask, int32_t* depth,
                             int* status, cudaStream_t st);
cudaError_t launch_accept(const int32_t* draft, const int32_t* target, const int32_t* parents, int B,
                          int N, int32_t* path, int32_t* accept_len, int32_t* bonus, int* status,
                          cudaStream_t st);
cudaError_t launch_kv_compact(void* const* cache_ptrs, int layer_begin, int layer_end,
                              const int32_t* path, const int32_t* accept_len, const int32_t* kv_len,
                              int32_t* kv_len_out, int B, int N, int Hkv, int D, int S_max, int* status,
                              cudaStream_t st, const int32_t* block_table = nullptr, int table_stride = 0,
                              int page_rows = 0, int num_blocks = 0, int token_major = 0);

cudaError_t launch_accept_commit(void* const* cache_ptrs, int layer_begin, int layer_end, const int32_t* draft,
                                 const int32_t* target, const int32_t* parents, const int32_t* kv_len,
                                 int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, int B, int N,
                                 int Hkv, int D, int S_max, int* status, cudaStream_t st,
                                 const int32_t* block_table = nullptr, int table_stride = 0, int page_rows = 0,
                                 int num_blocks = 0, int token_major = 0);

cudaError_t launch_rope_rows(void* q, const void* k_new, const void* v_new, const int32_t* positions,
                             const int32_t* kv_len, void* k_cache, void* v_cache, float theta, int B, int N, int Hq,
                             int Hkv, int D, int S_max, int* status, cudaStream_t st,
                             const int32_t* block_table = nullptr, int table_stride = 0, int page_rows = 0,
                             int num_blocks = 0, int token_major = 0, void* q_out = nullptr, const void* angle_table = nullptr);
// (q_out: where the rotated q rows go, q itself when null; angle_table: the fp64 half of a vispec_rope_table_build
// table to take cosines and sines from instead of forming them from positions and theta)

cudaError_t launch_accept_sampled(const int32_t* draft_ids, const int32_t* parents, const float* p, const float* p_hat,
                                  const float* u_accept, const float* u_bonus, int B, int N, int V, int32_t* path,
                                  int32_t* accept_len, int32_t* bonus, int* status, cudaStream_t st);

cudaError_t launch_tree_rerank(const int32_t* cand_parent, const int32_t* cand_token, const float* cand_score, int B,
                               int M, int K, int32_t* parents, int32_t* draft_ids, int32_t* selected, int* status,
                               cudaStream_t st);

struct AttnArgs {
    const void* q; const void* k; const void* v;
    const int32_t* kv_len; const uint64_t* mask;
    void* out; float* lse;
    int B, N, Hq, Hkv, D, S_max;
    float scale;
    void* ws; size_t ws_bytes;
    int* status;
    int sm_count;
    bool early_prefetch;   // committed-prefix tiles may be read before the preceding kernel has completed
    int tc5_path;          // 0 automatic, 1 partials in global memory (3: merge kernel always), 2 clusters where possible
    int kv_len_hint;       // committed length the caller expects (0: unknown, reason about S_max)
    // fused rotary embedding (TMA + tcgen05 kernel, contiguous caches): rope_table non-null turns it on
    const void* rope_table; const void* k_new; const void* v_new;
    const CUtensorMap* k_map; const CUtensorMap* v_map;
    // paged cache (page_rows != 0): pool blocks of page_rows slots, block_table [B][table_stride]; S_max is then
    // table_stride * page_rows
    const int32_t* block_table; int table_stride, page_rows, num_blocks, token_major;
};
// Generic split-KV kernel on warp-level tensor-core instructions (any supported shape).
cudaError_t init_attn_generic();   // once per device, with that device current
cudaError_t launch_attn_generic(const AttnArgs& a, cudaStream_t st, int* n_launches);

// TMA + tcgen05 kernel (D = 128), work split evenly over the SMs, followed by its merge kernel.
bool attn_tc5_supports(const AttnArgs& a);
cudaError_t init_attn_tc5();           // once per device, with that device current
cudaError_t launch_attn_tc5(const AttnArgs& a, cudaStream_t st, int* n_launches);
bool attn_tc5_uses_clusters(const AttnArgs& a);   // the call would run in the cluster form (one launch, short calls)
// The bounded wait of the attention kernels on a barrier that never completes (failure-detection self-test).
cudaError_t launch_bounded_wait_selftest(long long limit, int* status, int* counters, cudaStream_t st);
// positions[b][i] == kv_len[b] + popcount(mask row i) - 1, else status VISPEC_E_POSITIONS.
cudaError_t launch_check_positions(const int32_t* positions, const int32_t* kv_len, const uint64_t* mask, int B, int N,
                                   int* status, cudaStream_t st);
// (cos, sin) of positions[b][i] * theta^(-2j/D), j < D/2: B*N*D/2 fp64 pairs followed by the same as fp32 pairs.
cudaError_t launch_rope_table(const int32_t* positions, int B, int N, int D, float theta, void* table, cudaStream_t st);
// Streaming-read probe over the rows one attention call reads (measurement aid).
cudaError_t init_stream_probe();
cudaError_t launch_stream_probe(const AttnArgs& a, cudaStream_t st);

}  // namespace vispec
