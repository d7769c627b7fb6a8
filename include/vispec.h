/*
 * vispec.h - C ABI of the draft-tree verification step of speculative decoding for
 * vision-language models (ViSpec, arXiv 2509.15235), written for NVIDIA B200 (sm_100a).
 *
 * The paper's decoding loop (Sec. 3.1) alternates drafting and verification: the target model
 * scores a whole tree of drafted tokens in one forward, keeps the longest root path whose tokens
 * it would have produced itself, and commits that path to its pre-allocated KV cache (App. A).
 * This library is the attention-side hot path of that verification:
 *
 *   vispec_tree_mask_build   parent array of the draft tree -> per-node ancestor bitmask
 *   vispec_tree_verify_attn  tree-masked attention (Eq. 1 with scale) of all tree queries against
 *                            the long, image-token dominated bf16 KV cache of one layer
 *   vispec_accept            greedy (temperature 0) acceptance walk -> accepted path, bonus token
 *   vispec_kv_compact        gather the accepted path's K/V rows into the contiguous cache
 *
 * and the steps next to it in a decoding cycle:
 *
 *   vispec_accept_commit     acceptance and commit in one launch
 *   vispec_tree_rerank       keep the K best-scored candidates of the tree expansion (App. A) as the tree
 *   vispec_rope_tree_rows    rotary embedding of the tree's q/k rows and their placement in the cache
 *   vispec_accept_sampled    acceptance at temperature > 0 (Sec. 3.1's min(1, p/p^) rule with residual resampling)
 *   vispec_cache_register_paged and the *_paged calls: the same work on a pool of cache blocks and a block table
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  The library never takes
 *     ownership of caller memory and never frees it.
 *   - Hot calls (mask, attention, accept, compact) allocate nothing, never synchronise with the
 *     host and enqueue their work on `stream` (a cudaStream_t passed as void*; NULL = default).
 *   - Every function returns VISPEC_OK (0) or a negative vispec_status.  Errors that only the
 *     device can see (a bad parent index, kv_len + N beyond the allocation, a bounded wait that
 *     ran out) are recorded in a device status word that vispec_status_poll reads; the kernel
 *     that met the error skips the offending work instead of faulting.
 *   - Notation: B sequences, N tree nodes INCLUDING the root (node 0, the last committed token's
 *     successor; parents[b][0] = -1), W = ceil(N/64) mask words, Hq/Hkv query/KV heads,
 *     G = Hq/Hkv, D head dim, S = kv_len[b] committed slots, S_max allocated slots, L layers.
 *   - Layouts (row-major): q, out [B,N,Hq,D] bf16;  k_cache, v_cache [B,Hkv,S_max,D] bf16 per layer;
 *     tree node i's K/V rows sit at slot S+i of its sequence when attention is called;
 *     tree_mask [B,N,W] uint64 (bit t of row i: node t is visible to node i);
 *     parents, draft_ids, target_ids, path [B,N] int32; kv_len, accept_len, bonus [B] int32.
 */
#ifndef VISPEC_H_
#define VISPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum vispec_status {
    VISPEC_OK = 0,
    VISPEC_E_NULL = -1,         /* a required pointer is NULL */
    VISPEC_E_ALIGN = -2,        /* a pointer misses its alignment (16 B tensors, 128 B caches) */
    VISPEC_E_SHAPE = -3,        /* a size outside the supported set, or inconsistent with the context */
    VISPEC_E_RANGE = -4,        /* an index (layer, device, kv_len + N) out of range */
    VISPEC_E_UNSUPPORTED = -5,  /* valid request this build cannot serve */
    VISPEC_E_CUDA = -6,         /* a CUDA runtime/driver call failed */
    VISPEC_E_TIMEOUT = -7,      /* a bounded device-side wait gave up (status word only) */
    VISPEC_E_BAD_TREE = -8,     /* parents[b][i] not in [0,i) for i>0, or parents[b][0] != -1 */
    VISPEC_E_UNREGISTERED = -9, /* layer has no registered cache, or pointers differ from it */
    VISPEC_E_WORKSPACE = -10,   /* workspace missing or too small */
    VISPEC_E_POSITIONS = -11    /* positions differ from kv_len + depth (status word, VISPEC_OPT_CHECK_POSITIONS) */
} vispec_status;

#define VISPEC_MAX_TREE_NODES 128

typedef struct vispec_shape {
    int32_t B_max;   /* most sequences per call */
    int32_t N_max;   /* most tree nodes per sequence, 1..128 */
    int32_t Hq;      /* query heads */
    int32_t Hkv;     /* key/value heads, divides Hq */
    int32_t D;       /* head dimension: 64 or 128 */
    int32_t S_max;   /* allocated cache slots per (sequence, kv head) */
    int32_t layers;  /* number of cache pairs that may be registered */
} vispec_shape;

typedef struct vispec_ctx vispec_ctx;  /* opaque; owns only descriptors and a device status word */

/* Human-readable name of a status code (static storage, never NULL). */
const char* vispec_strerror(int status);

/* Create a context for one model shape on CUDA device `device`.  Not a hot call: it allocates a few
 * hundred bytes of device memory (status word, per-layer pointer table).  `*out` (host) receives the
 * context.  Errors: E_NULL, E_SHAPE (D not 64/128, Hq % Hkv != 0, N_max > 128, a non-positive size),
 * E_RANGE (no such device), E_CUDA. */
int vispec_ctx_create(vispec_ctx** out, const vispec_shape* shape /*host*/, int device);

/* Destroy a context and the small device allocations it made.  Caller memory (caches, workspace)
 * is untouched.  NULL is accepted. */
int vispec_ctx_destroy(vispec_ctx* ctx);

/* Bytes of scratch the attention needs for `shape` on the context's device: split-KV partial
 * results (fp32) plus arrival counters.  `*out` is host memory. */
int vispec_workspace_bytes(const vispec_ctx* ctx, size_t* out /*host*/);

/* Hand the context a caller-owned device buffer of at least vispec_workspace_bytes() bytes, 256-byte
 * aligned.  The library zeroes its counters once here (enqueued on the default stream and
 * synchronised: not a hot call).  The buffer must stay alive and must not be shared by calls that
 * overlap on the GPU.  Errors: E_NULL, E_ALIGN, E_WORKSPACE (too small), E_CUDA. */
int vispec_ctx_set_workspace(vispec_ctx* ctx, void* workspace, size_t bytes);

/* Options of a context (vispec_ctx_set_option). */
typedef enum vispec_option {
    /* Default 1.  vispec_tree_verify_attn is enqueued so that it may start while the kernel before it on
     * `stream` is still running (programmatic dependent launch).  Before that kernel has completed it
     * reads only kv_len and cache tiles that lie wholly inside the committed prefix [0, S) - state that
     * the previous decoding cycle committed; q, tree_mask, the tree's own K/V rows (slots S..S+N-1) are
     * read, and everything is written, only after it has completed.  Attention calls (and the stream probe) let
     * their successor start as soon as they have started themselves, so through a run of back-to-back attention
     * calls the early reads of a later call may overlap the kernel that preceded the first of them.  The rule:
     * a kernel that writes kv_len or committed cache slots (vispec_kv_compact, vispec_accept_commit) must be
     * followed by at least one kernel that does not start early - vispec_tree_mask_build, vispec_rope_tree_rows
     * (it waits for its predecessor before it lets its successor in) or any ordinary kernel - before the next
     * attention call with this option on; the decoding cycle (commit, mask build, attention x layers) satisfies
     * it.  Otherwise set 0 for the attention calls in between: then nothing is read early. */
    VISPEC_OPT_EARLY_PREFETCH = 1,
    /* Default 0 (1 if the environment has VISPEC_FORCE_GENERIC=1 at context creation).  Route attention
     * through the shape-generic warp-level kernel even where the TMA/tcgen05 kernel applies. */
    VISPEC_OPT_FORCE_GENERIC = 2,
    /* Default 0.  How the TMA/tcgen05 attention kernel combines the pieces of a (sequence, kv head) that
     * several thread blocks work on: 0 chooses per call; 1 always parks partial results in the workspace
     * (they are merged by the block that delivers a unit's last partial when a unit has at most 64 query rows,
     * by a second kernel otherwise); 2 uses thread-block clusters that merge through distributed shared memory
     * whenever the shape allows one cluster per (sequence, kv head, row block); 3 is 1 with the second kernel
     * always.  The in-kernel merge counts arrivals in the first 64 KiB of the workspace, which
     * vispec_ctx_set_workspace zeroes and every call leaves zero (a call that ended with VISPEC_E_TIMEOUT may
     * not: vispec_status_poll zeroes them again when it reports that code). */
    VISPEC_OPT_SPLIT_FORM = 3,
    /* Default 0 (none).  The committed length the caller expects its sequences to have, in slots.  The host never
     * reads kv_len, so where it must choose between ways of running the attention it reasons about the cache
     * capacity S_max; a context sized for 32 k slots that serves 2 k-token sequences is better described by this
     * hint.  It only steers that choice: any kv_len up to S_max - N stays valid. */
    VISPEC_OPT_KV_LEN_HINT = 4,
    /* Default 0 (1 if the environment has VISPEC_DEBUG set at context creation).  vispec_tree_verify_attn also
     * checks its `positions` argument on the device: positions[b][i] == kv_len[b] + (set bits of tree_mask row
     * i) - 1, the rule "position = committed length + depth" for a mask built from a parent array.  A mismatch sets
     * the status word VISPEC_E_POSITIONS; the attention itself runs unchanged (it does not use positions).  One
     * extra small launch per call, so off by default. */
    VISPEC_OPT_CHECK_POSITIONS = 5
} vispec_option;

/* Set an option of the context (host call, takes effect for later calls).  Errors: E_NULL,
 * E_UNSUPPORTED (unknown option), E_RANGE (value). */
int vispec_ctx_set_option(vispec_ctx* ctx, int option, int value);

/* Register layer `layer`'s cache pair [B_max,Hkv,S_max,D] bf16 (App. A: pre-allocated KV cache).
 * Builds the TMA tensor maps for these base pointers and records them for vispec_kv_compact; call
 * again if the allocator moves a cache.  Pointers must be 128-byte aligned.  Not a hot call (one
 * small host->device copy).  Errors: E_NULL, E_ALIGN, E_RANGE (layer), E_CUDA. */
int vispec_cache_register(vispec_ctx* ctx, int layer, void* k_cache, void* v_cache);

/* Ancestor mask of a draft tree (the tree of Sec. 3.1 / App. A, given as a parent array):
 *   tree_mask[b][i] = { i } U tree_mask[b][parents[b][i]],  depth[b][i] = |tree_mask[b][i]| - 1.
 * parents [B,N] int32 with parents[b][0] = -1 and 0 <= parents[b][i] < i.  A node whose chain
 * to the root meets an invalid link (or parents[b][0] != -1) gets a row with its own bit only and
 * depth 0, and the status word becomes VISPEC_E_BAD_TREE; nothing faults.  depth may be NULL.
 * Host errors: E_NULL, E_SHAPE (B < 0, B > B_max, N < 1, N > N_max). */
int vispec_tree_mask_build(vispec_ctx* ctx, const int32_t* parents, int B, int N,
                           uint64_t* tree_mask, int32_t* depth, void* stream);

/* Tree-masked attention of one layer (Eq. 1 of the paper, with the 1/sqrt(d) scale it omits given
 * explicitly as `scale`).  For sequence b, query head h, node i:
 *   allowed keys A = { j < S } U { S + t : bit t of tree_mask[b][i] },   S = kv_len[b]
 *   out[b][i][h] = sum_{j in A} softmax_j(scale * <q[b][i][h], k[b][h/G][j]>) * v[b][h/G][j]
 * computed with fp32 accumulation from bf16 inputs, rounded once to bf16 (nearest even).
 * lse [B,Hq,N] fp32 (optional, may be NULL) receives log sum_{j in A} exp(score_j).
 * An empty A gives out = 0 and lse = -inf.  tree_mask is an INPUT (any bit pattern is honoured,
 * it is never re-derived from parents).  Cache slots at or beyond S + N are never interpreted
 * (they may hold NaN patterns); tree rows that a node's mask hides get weight exactly 0 and must
 * hold finite values, as rows written by the K/V projection do.  `positions` [B,N] (kv_len + depth) may be
 * NULL: q and the cached k arrive already rotated (vispec_rope_tree_rows is the call that uses positions), so the
 * attention does not need it; with VISPEC_OPT_CHECK_POSITIONS on it is checked against kv_len and tree_mask.
 * k_cache / v_cache must be the pointers registered for `layer` (or NULL to use them).
 * A sequence with kv_len[b] < 0 or kv_len[b] + N > S_max gets out = 0 and the status word
 * VISPEC_E_RANGE.  Needs a workspace (vispec_ctx_set_workspace).
 * Host errors: E_NULL, E_ALIGN (q/out 16 B), E_SHAPE, E_RANGE (layer), E_UNREGISTERED, E_WORKSPACE. */
int vispec_tree_verify_attn(vispec_ctx* ctx, int layer, const void* q, const void* k_cache,
                            const void* v_cache, const int32_t* kv_len, const uint64_t* tree_mask,
                            const int32_t* positions, int B, int N, float scale, void* out,
                            float* lse, void* stream);

/* The angle table of the fused call below (Sec. 3.2: the target LLM, and with it its rotary position embedding, is
 * unchanged).  For sequence b, node i, j < D/2:  angle = positions[b][i] * theta^(-2j/D), formed in fp64;
 * `table` (DEVICE, 16-byte aligned, vispec_rope_table_bytes() bytes, caller-owned) receives B*N*D/2 (cos, sin) pairs
 * in fp64 followed by the same pairs rounded to fp32.  positions and theta mean what they mean for
 * vispec_rope_tree_rows.  One small launch; the table serves every layer of the cycle (positions do not depend on
 * the layer).  Host errors: E_NULL, E_ALIGN, E_SHAPE (B, N, theta <= 1), E_CUDA. */
int vispec_rope_table_build(vispec_ctx* ctx, const int32_t* positions, int B, int N, float theta, void* table,
                            void* stream);
/* Bytes of a table for B sequences of N nodes at the context's head size (host call). */
int vispec_rope_table_bytes(const vispec_ctx* ctx, int B, int N, size_t* out /*host*/);

/* vispec_rope_tree_rows followed by vispec_tree_verify_attn as one call (Sec. 3.2; Eq. 1), for contiguous caches at
 * D = 128, at most 32 sequences and scale > 0 (anything else: VISPEC_E_UNSUPPORTED, use the two calls).  q [B,N,Hq,D]
 * arrives UNROTATED and is not modified.  k_new, v_new [B,N,Hkv,D] are the tree's rows: k rotated in fp64 with one
 * rounding to bf16, v copied, both written to slots kv_len[b] + i of the registered caches exactly as
 * vispec_rope_tree_rows writes them.  Short calls (the form with one thread-block cluster per head) run as ONE
 * launch: every thread block rotates the q rows it needs on their way into shared memory (fp32 arithmetic from the
 * table's fp32 half; the rotated q is consumed by the score product only), and the blocks of a head's cluster each
 * write a share of the tree's rows into the cache before the block whose part of the cache contains those slots reads
 * them (a sequence with kv_len + N > S_max is left alone: nothing written, zero output, VISPEC_E_RANGE).  Long calls (work split evenly over the SMs)
 * run as two launches - the rotation kernel fed from the table, writing the rotated q into a scratch copy at the end
 * of the workspace, then the plain attention - because there the in-kernel rotation costs more than it saves.  Everything else (tree_mask, kv_len, out, lse,
 * status word, early prefix reads) as in vispec_tree_verify_attn; rope_table comes from vispec_rope_table_build
 * with the same B and N.  Host errors: those of vispec_tree_verify_attn, plus E_ALIGN for k_new / v_new / table. */
int vispec_tree_verify_attn_rope(vispec_ctx* ctx, int layer, const void* q, const void* k_new, const void* v_new,
                                 const void* rope_table, const int32_t* kv_len, const uint64_t* tree_mask, int B, int N,
                                 float scale, void* out, float* lse, void* stream);

/* Attention without any allocation (the paper has no counterpart: this entry point exists for
 * deployment, not for the method).  It is for callers that cannot obtain device memory when they
 * need to run: a serving process whose memory pool is fixed at start-up, a plugin that receives
 * tensors but no allocator, code on a latency-critical stream where cudaMalloc's implicit
 * device synchronisation is not acceptable.  It computes exactly what vispec_tree_verify_attn
 * computes, but needs no context, no registration and no workspace: the split-KV partial results go
 * to a 16 MiB array that is part of the library image (static device memory, held on every GPU that
 * loads the library until the process exits).  The function calls no cudaMalloc/cudaFree and no
 * allocating library routine.
 *   - Arguments as in vispec_tree_verify_attn, with the shape given explicitly (Hq, Hkv, D in
 *     {64,128}, S_max) and the caches passed directly ([B,Hkv,S_max,D] bf16, 16-byte aligned).
 *   - status_word: optional DEVICE int32 that receives VISPEC_E_RANGE (compare-and-swap from 0) if a
 *     sequence has kv_len < 0 or kv_len + N > S_max (that sequence's output is zero); may be NULL.
 *   - Limit: B * Hkv * ceil(G*N/64) partial-result units must fit the array with two KV splits,
 *     i.e. 64 KiB + 2 * units * 64 * (4*D + 8) bytes <= 16 MiB (at D = 128: 251 units).  Beyond
 *     that the call returns VISPEC_E_WORKSPACE and does nothing.
 *   - The first call on each device looks up the array's device address and sets one kernel
 *     attribute; make that first call outside any stream capture, with the device current.
 *   - All calls share the one array, and it keeps the previous call's contents.  Nothing in it has
 *     to start at zero (every partial is written before it is read), so no clearing is done; but two
 *     calls that overlap on the GPU (different streams, different host threads) race on it.  Run
 *     calls of this entry point one after another.
 * Errors: E_NULL, E_ALIGN, E_SHAPE, E_WORKSPACE (too large for the array), E_RANGE (device index), E_CUDA. */
int vispec_tree_verify_attn_static(const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* kv_len, const uint64_t* tree_mask, int B, int N,
                                   int Hq, int Hkv, int D, int S_max, float scale, void* out,
                                   float* lse, int* status_word, void* stream);

/* Paged cache (the paper's runtime uses one pre-allocated cache per sequence, App. A; a serving stack shares a
 * pool of fixed-size blocks between sequences instead - same arithmetic, another layout).
 *   k_pool, v_pool: bf16 [num_blocks, Hkv, page_rows, D], or [num_blocks, page_rows, Hkv, D] if token_major != 0
 *   (device, 128-byte aligned, caller-owned), page_rows in {16, 32, 64, 128}, D = 128 only (E_UNSUPPORTED
 *   otherwise).  Registering a layer replaces what was registered
 *   for it before, paged or not.  A paged layer is served by the *_paged calls only (the others answer
 *   E_UNSUPPORTED for it, and the *_paged calls answer E_UNSUPPORTED for a contiguous layer).
 * Host errors: E_NULL, E_RANGE (layer), E_ALIGN, E_UNSUPPORTED, E_SHAPE. */
int vispec_cache_register_paged(vispec_ctx* ctx, int layer, void* k_pool, void* v_pool, int num_blocks, int page_rows,
                                int token_major);

/* vispec_tree_verify_attn on a paged layer.  block_table [B, table_stride] int32 (device): entry i of row b is
 * the pool block that holds logical slots [i * page_rows, (i + 1) * page_rows) of sequence b; only the entries of
 * blocks that start below kv_len[b] + N are read.  Logical slots mean what they mean in the contiguous call
 * (prefix at [0, kv_len), tree rows at kv_len + i); capacity is table_stride * page_rows slots (a sequence with
 * kv_len + N beyond it is skipped: zero output, -inf lse, status VISPEC_E_RANGE).  A table entry outside
 * [0, num_blocks) reads as zeros and sets the status word VISPEC_E_RANGE; nothing faults.  The table, like
 * kv_len and the committed prefix, must not be written by the kernel that precedes this call on the stream.
 * Everything else (q, tree_mask, scale, out, lse, workspace, accuracy) as in vispec_tree_verify_attn.
 * Host errors: E_NULL, E_ALIGN, E_SHAPE, E_RANGE, E_UNREGISTERED, E_UNSUPPORTED (contiguous layer, B > 32,
 * scale <= 0), E_WORKSPACE. */
int vispec_tree_verify_attn_paged(vispec_ctx* ctx, int layer, const void* q, const int32_t* kv_len,
                                  const int32_t* block_table, int table_stride, const uint64_t* tree_mask, int B, int N,
                                  float scale, void* out, float* lse, void* stream);

/* vispec_kv_compact on paged layers [layer_begin, layer_end): rows move between logical slots kv_len + path[k]
 * and kv_len + k, each found through block_table (one table serves all layers of the range, which must share
 * num_blocks, page_rows and layout: E_SHAPE otherwise).  A table entry outside the pool drops that row's move and sets
 * the status word VISPEC_E_RANGE.  Other arguments and errors as in vispec_kv_compact. */
int vispec_kv_compact_paged(vispec_ctx* ctx, int layer_begin, int layer_end, const int32_t* path,
                            const int32_t* accept_len, const int32_t* kv_len, const int32_t* block_table,
                            int table_stride, int32_t* kv_len_out, int B, int N, void* stream);

/* vispec_accept_commit and vispec_rope_tree_rows on paged layers: the same work, with every logical slot found
 * through block_table (arguments as in vispec_kv_compact_paged / vispec_tree_verify_attn_paged).  A table entry
 * outside the pool drops that row's move or placement and sets the status word VISPEC_E_RANGE.  The accepted
 * range [layer_begin, layer_end) must not be empty here (E_RANGE). */
int vispec_accept_commit_paged(vispec_ctx* ctx, int layer_begin, int layer_end, const int32_t* draft_ids,
                               const int32_t* target_ids, const int32_t* parents, const int32_t* kv_len,
                               const int32_t* block_table, int table_stride, int B, int N, int32_t* path,
                               int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, void* stream);
int vispec_rope_tree_rows_paged(vispec_ctx* ctx, int layer, void* q, const void* k_new, const void* v_new,
                                const int32_t* positions, const int32_t* kv_len, const int32_t* block_table,
                                int table_stride, int B, int N, float theta, void* stream);

/* Rotary position embedding of the tree rows and their placement in the cache: the step just before
 * vispec_tree_verify_attn of the same layer (Sec. 3.2: the target LLM runs unchanged; LLaVA-v1.6 and
 * Qwen2.5-VL rotate q and k by position, pairing element j with element j + D/2).  For node i of sequence b
 * and j < D/2:   angle = positions[b][i] * theta^(-2j/D)
 *   x'[j] = x[j] cos(angle) - x[j+D/2] sin(angle),   x'[j+D/2] = x[j+D/2] cos(angle) + x[j] sin(angle)
 * q [B,N,Hq,D] bf16 is rotated IN PLACE; k_new [B,N,Hkv,D] is rotated and written, v_new [B,N,Hkv,D] copied,
 * to slots kv_len[b] + i of the caches registered for `layer`.  Angles and the rotation are formed in fp64,
 * with one rounding to bf16.  positions is what the interface names (kv_len + depth for a draft tree); theta is
 * the rotary base (> 1; 10000 for Vicuna, 1000000 for Qwen2.5).  A sequence with kv_len < 0 or kv_len + N > S_max
 * is skipped with status word VISPEC_E_RANGE.
 * Host errors: E_NULL, E_ALIGN (16 B), E_SHAPE, E_RANGE (layer), E_UNREGISTERED. */
int vispec_rope_tree_rows(vispec_ctx* ctx, int layer, void* q, const void* k_new, const void* v_new,
                          const int32_t* positions, const int32_t* kv_len, int B, int N, float theta, void* stream);

/* Measurement aid (the paper has no counterpart): reads exactly the K and V rows that
 * vispec_tree_verify_attn(layer, ..., kv_len, B, N) reads - slots [0, kv_len[b] + N) of every kv head, rounded
 * up to whole 128-slot tiles - through the same TMA rings, on every SM, and does nothing with them.  Its time
 * is the floor that streaming alone sets for an attention call on this machine.  D = 128 only (E_UNSUPPORTED
 * otherwise), B <= 32.  Sequences with kv_len out of range are skipped.
 * Host errors: E_NULL, E_SHAPE, E_RANGE (layer), E_UNREGISTERED, E_UNSUPPORTED. */
int vispec_stream_probe(vispec_ctx* ctx, int layer, const int32_t* kv_len, int B, int N, void* stream);

/* Tree rerank: the last step of building the draft tree, the one that needs scores only (App. A: 30 draft
 * tokens kept from a depth-3 expansion of 8 nodes per level; the tree is EAGLE-2's, which keeps the candidates
 * of highest cumulative log-probability).  Of M candidates per sequence
 *   cand_parent [B,M] int32: an earlier candidate, or -1 for a child of the root
 *   cand_token  [B,M] int32,  cand_score [B,M] fp32 (cumulative log-probability of the path to the candidate)
 * the K of highest score are kept (equal scores: lower index first; NaN below everything) and become nodes
 * 1..K of a tree in increasing candidate index (parents stay ahead of children); node 0 is the root:
 *   parents   [B,K+1]: parents[b][0] = -1, parents[b][j] = node number of node j's parent
 *   draft_ids [B,K+1]: draft_ids[b][0] = 0 (ignored downstream), draft_ids[b][j] = token of node j
 *   selected  [B,K]:   candidate index of node j at [j-1] (may be NULL if K == 0)
 * The outputs are the inputs of vispec_tree_mask_build / vispec_accept* with N = K + 1.  A sequence with a parent
 * index that is not an earlier candidate, or a kept candidate whose parent was not kept (impossible for
 * cumulative log-probabilities), gets parents = -1 throughout and the status word VISPEC_E_BAD_TREE; selected
 * and draft_ids are still written.  Bit-exact: only comparisons of the given floats.
 * Host errors: E_NULL, E_SHAPE (M in [1, 2048], 0 <= K <= M, K + 1 <= N_max). */
int vispec_tree_rerank(vispec_ctx* ctx, const int32_t* cand_parent, const int32_t* cand_token, const float* cand_score,
                       int B, int M, int K, int32_t* parents, int32_t* draft_ids, int32_t* selected, void* stream);

/* Greedy acceptance (Sec. 3.1 at temperature 0; Table 1 upper half).  target_ids[b][i] is the
 * target model's greedy token after node i; non-root node a is matched iff
 * draft_ids[b][a] == target_ids[b][parents[b][a]]; the accepted path ends at the deepest node whose
 * whole chain to the root is matched (smallest index among equally deep ones).
 *   path[b][0..accept_len) = that chain from the root (always node 0) downward, rest padded with -1
 *   accept_len[b] >= 1 counts its nodes; tau of Sec. 5.1 is accept_len - 1
 *   bonus[b] = target_ids[b][last path node], the next cycle's root token
 * draft_ids[b][0] is ignored.  Invalid parents: that sequence returns the root only and the status
 * word VISPEC_E_BAD_TREE.  Host errors: E_NULL, E_SHAPE. */
int vispec_accept(vispec_ctx* ctx, const int32_t* draft_ids, const int32_t* target_ids,
                  const int32_t* parents, int B, int N, int32_t* path, int32_t* accept_len,
                  int32_t* bonus, void* stream);

/* Sampled acceptance (Sec. 3.1 at temperature > 0; Table 1 lower half): a drafted token x is kept with
 * probability min(1, p(x)/p^(x)); after a rejection the target distribution is replaced by
 * norm(max(0, p - p^)).  On a tree the children of the current node are decided one after the other, in
 * increasing node index (the multi-candidate form of the works Sec. 3.1 cites); the first kept child becomes the
 * current node with its own target row; when no child is left the bonus token is drawn from what remains.
 *   p_target [B,N,V] fp32 (device): row i = the target's distribution of the token after node i
 *   p_draft  [B,N,V] fp32 (device): row i = the draft distribution node i's children were drawn from
 *   u_accept [B,N] fp32 in [0,1): the uniform deciding node i (read only if node i comes to be decided)
 *   u_bonus  [B]   fp32 in [0,1): draws the bonus token, as the smallest token whose running weight sum exceeds
 *                  u_bonus * total (the last token of positive weight if rounding leaves none)
 * The random numbers are inputs: the call is deterministic.  Decisions are taken in fp64 on the fp32 inputs.
 * If max(0, r - p^) is zero everywhere after a rejection, the walk stops and the bonus token is drawn from the
 * current node's target row; bonus = -1 if that row has no positive entry.
 * path / accept_len / bonus as in vispec_accept (the outputs feed vispec_kv_compact unchanged).
 * A sequence with invalid parents (status VISPEC_E_BAD_TREE) or a drafted token outside [0,V) (VISPEC_E_RANGE)
 * gets accept_len 0, path -1, bonus -1.  draft_ids[b][0] is ignored.
 * Host errors: E_NULL, E_ALIGN (rows 16 B), E_SHAPE. */
int vispec_accept_sampled(vispec_ctx* ctx, const int32_t* draft_ids, const int32_t* parents, const float* p_target,
                          const float* p_draft, const float* u_accept, const float* u_bonus, int B, int N, int V,
                          int32_t* path, int32_t* accept_len, int32_t* bonus, void* stream);

/* Commit (App. A): for every registered layer in [layer_begin, layer_end), sequence and kv head, the
 * rows at slots S + path[b][k], k < accept_len[b], are gathered and then written to slots S + k, for
 * K and V, in place (gather-then-scatter: correct although a destination may be another entry's
 * source).  All other slots keep their bytes.  kv_len_out[b] = S + accept_len[b] (may be NULL; must
 * NOT alias kv_len, which other thread blocks of the same launch still read: E_SHAPE).  `N` is the row
 * length of `path`; a valid path is strictly increasing with path[b][k] >= k.  A sequence whose accept_len, path entry or
 * kv_len is out of range is skipped with status word VISPEC_E_RANGE.
 * Host errors: E_NULL, E_SHAPE, E_RANGE (layers), E_UNREGISTERED. */
int vispec_kv_compact(vispec_ctx* ctx, int layer_begin, int layer_end, const int32_t* path,
                      const int32_t* accept_len, const int32_t* kv_len, int32_t* kv_len_out,
                      int B, int N, void* stream);

/* Acceptance and commit in one launch: the result of vispec_accept followed by vispec_kv_compact over the
 * registered layers [layer_begin, layer_end) (Sec. 3.1 acceptance at temperature 0, then the App. A commit of
 * the accepted path's K/V rows), without the second launch and the dependency between the two.  Arguments,
 * outputs (path, accept_len, bonus, kv_len_out = S + accept_len; kv_len_out may be NULL and must not alias
 * kv_len) and status-word behaviour are those of the two calls: an invalid tree commits the root only
 * (VISPEC_E_BAD_TREE), a sequence with kv_len < 0 or kv_len + N > S_max gets its acceptance outputs but no
 * commit (VISPEC_E_RANGE).  With layer_begin == layer_end only the acceptance runs.
 * Host errors: E_NULL, E_SHAPE, E_RANGE (layers), E_UNREGISTERED. */
int vispec_accept_commit(vispec_ctx* ctx, int layer_begin, int layer_end, const int32_t* draft_ids,
                         const int32_t* target_ids, const int32_t* parents, const int32_t* kv_len, int B, int N,
                         int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* kv_len_out, void* stream);

/* Read and clear the device status word (synchronises `stream`; not a hot call).
 * `*code` (host) receives VISPEC_OK or the first asynchronous error recorded since the last poll.  When that
 * is VISPEC_E_TIMEOUT the arrival counters at the head of the workspace are zeroed on `stream` as well.
 * out and lse of an attention call that ended in VISPEC_E_TIMEOUT are undefined (a block that gave up leaves
 * its rows unwritten or half merged); only the status word says so. */
int vispec_status_poll(vispec_ctx* ctx, int* code /*host*/, void* stream);

/* Self-test of the bounded waits (Sec. 3.1 has no counterpart: this serves failure detection).  Every device-side
 * wait of the attention kernels polls a barrier for a limited time and then gives up; this call runs that wait
 * routine on a barrier nobody ever arrives on, with `limit_cycles` SM clock cycles (1 .. 2^31) as the limit, and a
 * second waiter that must be released by the first one's give-up flag.  The kernel returns, the status word
 * becomes VISPEC_E_TIMEOUT, and - as a call that gave up half way may - it leaves a non-zero arrival counter at the
 * head of the workspace, which vispec_status_poll clears.  Nothing else is touched.  Needs a workspace.
 * Host errors: E_NULL, E_RANGE (limit), E_WORKSPACE, E_CUDA. */
int vispec_selftest_bounded_wait(vispec_ctx* ctx, long long limit_cycles, void* stream);

/* Number of kernels the library has launched through this context since creation (host counter). */
int vispec_launch_count(const vispec_ctx* ctx, uint64_t* out /*host*/);

#ifdef __cplusplus
}
#endif
#endif /* VISPEC_H_ */
