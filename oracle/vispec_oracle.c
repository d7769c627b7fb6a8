/*
 * CPU fp64 oracle for the draft-tree verification step.  TEST INFRASTRUCTURE ONLY:
 * it is called by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg, never by the product path, and it shares no source with the CUDA library.
 *
 * Everything here is the plain definition written out, with no blocking, fusion or
 * reordering, so that it can be checked against the paper by eye:
 *
 *   oracle_tree_mask    ancestor sets of a draft tree (the tree of Sec. 3.1, "context-aware
 *                       dynamic draft tree"; the mask itself is standard tree decoding
 *                       mechanics the paper inherits by citation)
 *   oracle_tree_attn    softmax attention of Eq. 1 (with the 1/sqrt(d) scale Eq. 1 drops
 *                       "for simplicity" restored as an explicit argument), restricted per
 *                       tree node to the committed prefix plus the node's ancestors
 *   oracle_accept       the acceptance rule of Sec. 3.1 at temperature 0 (Table 1, upper
 *                       half): a drafted token survives iff it equals the target's greedy
 *                       token at its parent; the result is the longest surviving root path
 *   oracle_kv_compact   commit of the accepted rows into the pre-allocated cache (App. A)
 *   oracle_accept_sampled  the acceptance rule of Sec. 3.1 at temperature > 0 (Table 1, lower half): a drafted
 *                       token x is kept with probability min(1, p(x)/p^(x)); after a rejection the target
 *                       distribution is replaced by norm(max(0, p - p^)); on a tree the rule is applied to
 *                       the children of the current node one after the other (the tree of SpecInfer, which
 *                       Sec. 3.1 cites), and the token after the last kept node is drawn from what remains
 *   oracle_tree_rerank  choice of the draft tree's nodes among the expansion's candidates (App. A: 30 draft
 *                       tokens, depth 3, 8 nodes expanded per level; the tree is EAGLE-2's, which keeps the
 *                       candidates of highest cumulative log-probability)
 *   oracle_rope_rows    rotary position embedding of the tree's q and k rows and their placement in the
 *                       cache (Sec. 3.2: the target LLM is used unchanged; LLaVA and Qwen2.5-VL rotate q and
 *                       k by position, in the half-split pairing: element j with element j + D/2)
 *
 * Layouts (row-major, C order):
 *   q, out            [B, N, Hq, D]
 *   k_cache, v_cache  [B, Hkv, S_max, D]   bf16 carried as uint16 bit patterns
 *   tree_mask         [B, N, W] uint64, W = ceil(N/64); bit t of row i <=> node t visible to node i
 *   parents, ids      [B, N] int32; parents[b][0] = -1
 *   path              [B, N] int32 padded with -1
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Ancestor mask: bit t of mask[b][i] is set iff t is i itself or is reached from i by following
 * parent links up to the root.  depth[b][i] = number of links from i to the root.
 * Returns 0, or -1 if some parent is not an earlier node (the row is still written: self bit only). */
int oracle_tree_mask(const int32_t* parents, int B, int N, uint64_t* mask, int32_t* depth) {
    int W = (N + 63) / 64, bad = 0;
    for (int b = 0; b < B; ++b) {
        const int32_t* par = parents + (size_t)b * N;
        for (int i = 0; i < N; ++i) {
            uint64_t* row = mask + ((size_t)b * N + i) * W;
            for (int w = 0; w < W; ++w) row[w] = 0;
            int ok = (par[0] == -1);
            for (int a = i; ok && a != 0; a = par[a])      /* every link must point to an earlier node */
                if (par[a] < 0 || par[a] >= a) ok = 0;
            int d = 0;
            if (!ok) {
                bad = 1;
                row[i / 64] |= (uint64_t)1 << (i % 64);
            } else {
                for (int a = i; a != -1; a = par[a]) {
                    row[a / 64] |= (uint64_t)1 << (a % 64);
                    if (par[a] != -1) ++d;
                }
            }
            if (depth) depth[(size_t)b * N + i] = d;
        }
    }
    return bad ? -1 : 0;
}

/* Tree-masked attention, Eq. 1 with scale.  For sequence b, query head h (kv head h / G) and tree
 * node i the allowed key set is A = { j : j < S } U { S + t : bit t of tree_mask[b][i] }, S = kv_len[b]:
 *     s_j = scale * <q, k_j>,  alpha_j = exp(s_j) / sum_{A} exp(s_k),  out = sum_{A} alpha_j v_j.
 * The maximum is subtracted before exponentiation (it cancels in alpha).  out is fp64;
 * lse[b][h][i] = log sum_A exp(s_j) (may be NULL).  An empty A gives out = 0, lse = -inf. */
int oracle_tree_attn(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                     const int32_t* kv_len, const uint64_t* tree_mask,
                     int B, int N, int Hq, int Hkv, int D, int S_max, double scale,
                     double* out, double* lse) {
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    int G = Hq / Hkv, W = (N + 63) / 64;
    for (int b = 0; b < B; ++b)
        if (kv_len[b] < 0 || kv_len[b] + N > S_max) return -2;
    int status = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            int S = kv_len[b], kvh = h / G;
            const uint16_t* Kh = k_cache + ((size_t)b * Hkv + kvh) * (size_t)S_max * D;
            const uint16_t* Vh = v_cache + ((size_t)b * Hkv + kvh) * (size_t)S_max * D;
            double* s = (double*)malloc(sizeof(double) * (size_t)(S + N));
            unsigned char* allowed = (unsigned char*)malloc((size_t)(S + N));
            double* qd = (double*)malloc(sizeof(double) * (size_t)D);
            if (!s || !allowed || !qd) { status = -3; free(s); free(allowed); free(qd); continue; }
            for (int i = 0; i < N; ++i) {
                const uint16_t* qi = q + (((size_t)b * N + i) * Hq + h) * D;
                const uint64_t* mrow = tree_mask + ((size_t)b * N + i) * W;
                double* o = out + (((size_t)b * N + i) * Hq + h) * D;
                for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(qi[d]);
                for (int j = 0; j < S; ++j) allowed[j] = 1;
                for (int t = 0; t < N; ++t) allowed[S + t] = (unsigned char)((mrow[t / 64] >> (t % 64)) & 1);
                double m = -INFINITY;
                for (int j = 0; j < S + N; ++j) {
                    if (!allowed[j]) continue;
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += qd[d] * bf16_to_f64(Kh[(size_t)j * D + d]);
                    s[j] = scale * acc;
                    if (s[j] > m) m = s[j];
                }
                double denom = 0.0;
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                for (int j = 0; j < S + N; ++j) {
                    if (!allowed[j]) continue;
                    double w = exp(s[j] - m);
                    denom += w;
                    for (int d = 0; d < D; ++d) o[d] += w * bf16_to_f64(Vh[(size_t)j * D + d]);
                }
                if (denom > 0.0) {
                    for (int d = 0; d < D; ++d) o[d] /= denom;
                } else {
                    for (int d = 0; d < D; ++d) o[d] = 0.0;
                }
                if (lse) lse[((size_t)b * Hq + h) * N + i] = denom > 0.0 ? m + log(denom) : -INFINITY;
            }
            free(s); free(allowed); free(qd);
        }
    }
    return status;
}

/* Greedy (temperature 0) acceptance on a tree.  A non-root node a is "matched" iff
 * draft_ids[a] == target_ids[parents[a]] (the target's greedy token after the parent is the drafted
 * token).  Node i is accepted-reachable iff every non-root node on the chain i -> root is matched.
 * The accepted path ends at the reachable node of greatest depth (smallest index among equals);
 * path lists that chain from the root down; accept_len counts its nodes (root included);
 * bonus = target_ids[last node of the path] (the token the target emits after the path). */
int oracle_accept(const int32_t* draft_ids, const int32_t* target_ids, const int32_t* parents,
                  int B, int N, int32_t* path, int32_t* accept_len, int32_t* bonus) {
    for (int b = 0; b < B; ++b) {
        const int32_t* par = parents + (size_t)b * N;
        const int32_t* dr = draft_ids + (size_t)b * N;
        const int32_t* tg = target_ids + (size_t)b * N;
        int best = 0, best_depth = 0;
        for (int i = 0; i < N; ++i) {
            int ok = 1, d = 0;
            for (int a = i; a != 0; a = par[a]) {
                if (par[a] < 0 || par[a] >= a) return -1;
                if (dr[a] != tg[par[a]]) ok = 0;
                ++d;
            }
            if (ok && d > best_depth) { best = i; best_depth = d; }
        }
        int32_t* p = path + (size_t)b * N;
        for (int k = 0; k < N; ++k) p[k] = -1;
        int k = best_depth;
        for (int a = best; ; a = par[a]) { p[k--] = a; if (a == 0) break; }
        accept_len[b] = best_depth + 1;
        bonus[b] = tg[best];
    }
    return 0;
}

/* Draw from the unnormalised weights w[0..V) with one uniform u in [0,1): the smallest v whose running sum
 * exceeds u * (sum of w); if rounding leaves none, the last v with w[v] > 0; -1 if no weight is positive. */
static int32_t draw_from_weights(const double* w, int V, double u) {
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += w[v];
    if (!(total > 0.0)) return -1;
    const double target = u * total;
    double run = 0.0;
    int32_t last = -1;
    for (int v = 0; v < V; ++v) {
        run += w[v];
        if (w[v] > 0.0) last = v;
        if (run > target) return v;
    }
    return last;
}

/* Sampled acceptance on a tree (Sec. 3.1, temperature > 0).
 *   p      [B,N,V] fp32: row i = the target's distribution of the token that follows node i
 *   p_hat  [B,N,V] fp32: row i = the draft distribution the tokens of node i's children were drawn from
 *   draft_ids [B,N]: token of node i (the root's is the last sampled token and is always kept)
 *   u_accept [B,N] in [0,1): the uniform that decides node i, if node i comes to be decided
 *   u_bonus  [B]   in [0,1): the uniform that draws the token after the last kept node
 * Walk: cur = root, r = p[cur].  The children of cur are decided in increasing index order: child c with token
 * x is kept iff u_accept[c] < min(1, r[x] / p_hat[cur][x]) (0/0 counts as 0); if kept, cur = c, r = p[c], and the
 * walk goes on with c's children; if not, r = norm(max(0, r - p_hat[cur])) and the next child is decided.  When
 * cur has no child left, the bonus token is drawn from r.  If max(0, r - p_hat[cur]) is zero everywhere the walk
 * stops and the bonus token is drawn from p[cur].
 * path / accept_len / bonus as in oracle_accept.  A sequence whose parents are not earlier nodes, or with a
 * drafted token outside [0,V), gets accept_len 0, path -1, bonus -1; the return value counts such sequences. */
int oracle_accept_sampled(const int32_t* draft_ids, const int32_t* parents, const float* p, const float* p_hat,
                          const float* u_accept, const float* u_bonus, int B, int N, int V,
                          int32_t* path, int32_t* accept_len, int32_t* bonus) {
    int bad = 0;
    double* r = (double*)malloc(sizeof(double) * (size_t)V);
    if (!r) return -1;
    for (int b = 0; b < B; ++b) {
        const int32_t* par = parents + (size_t)b * N;
        const int32_t* dr = draft_ids + (size_t)b * N;
        int32_t* pa = path + (size_t)b * N;
        for (int k = 0; k < N; ++k) pa[k] = -1;
        int ok = par[0] == -1;
        for (int i = 1; i < N; ++i)
            if (par[i] < 0 || par[i] >= i || dr[i] < 0 || dr[i] >= V) ok = 0;
        if (!ok) { accept_len[b] = 0; bonus[b] = -1; ++bad; continue; }
        int cur = 0, len = 1;
        pa[0] = 0;
        for (;;) {
            const float* pt = p + ((size_t)b * N + cur) * V;
            const float* ph = p_hat + ((size_t)b * N + cur) * V;
            for (int v = 0; v < V; ++v) r[v] = (double)pt[v];
            int kept = -1, empty = 0;
            for (int c = cur + 1; c < N && kept < 0 && !empty; ++c) {
                if (par[c] != cur) continue;
                const int x = dr[c];
                const double q = (double)ph[x];
                const double ratio = q > 0.0 ? r[x] / q : (r[x] > 0.0 ? INFINITY : 0.0);
                if ((double)u_accept[(size_t)b * N + c] < fmin(1.0, ratio)) { kept = c; break; }
                double z = 0.0;
                for (int v = 0; v < V; ++v) { r[v] = fmax(0.0, r[v] - (double)ph[v]); z += r[v]; }
                if (z > 0.0) { for (int v = 0; v < V; ++v) r[v] /= z; }
                else { empty = 1; for (int v = 0; v < V; ++v) r[v] = (double)pt[v]; }
            }
            if (kept >= 0) { cur = kept; pa[len++] = kept; continue; }
            bonus[b] = draw_from_weights(r, V, (double)u_bonus[b]);
            break;
        }
        accept_len[b] = len;
    }
    free(r);
    return bad;
}

/* a ranks before b: higher score first, NaN below everything, equal scores by lower index */
static int ranks_before(const float* score, int a, int b) {
    const float sa = score[a], sb = score[b];
    const int na = isnan(sa), nb = isnan(sb);
    if (na || nb) return na != nb ? nb : a < b;
    if (sa != sb) return sa > sb;
    return a < b;
}

/* Tree rerank: of M candidates (cand_parent[i] = an earlier candidate or -1 for a child of the root,
 * cand_score[i] = cumulative log-probability of the path to i, cand_token[i]) keep the K of highest score
 * (equal scores: lower index first; NaN last) and emit them in increasing candidate index as nodes 1..K of a
 * tree whose node 0 is the root:
 *   selected[b][j-1] = candidate index of node j;  parents[b][j] = node number of its parent (0 for -1);
 *   draft_ids[b][j] = its token;  parents[b][0] = -1, draft_ids[b][0] = 0.
 * A sequence with a parent index that is not an earlier candidate, or with a kept candidate whose parent
 * was not kept, is counted in the return value and gets parents = -1 throughout (selected and draft_ids are
 * still written). */
int oracle_tree_rerank(const int32_t* cand_parent, const int32_t* cand_token, const float* cand_score,
                       int B, int M, int K, int32_t* parents, int32_t* draft_ids, int32_t* selected) {
    if (K < 0 || K > M) return -1;
    int bad = 0;
    int* keep = (int*)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    int* node = (int*)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    if (!keep || !node) { free(keep); free(node); return -2; }
    for (int b = 0; b < B; ++b) {
        const int32_t* cp = cand_parent + (size_t)b * M;
        const int32_t* ct = cand_token + (size_t)b * M;
        const float* cs = cand_score + (size_t)b * M;
        int32_t* po = parents + (size_t)b * (K + 1);
        int32_t* io = draft_ids + (size_t)b * (K + 1);
        int32_t* so = selected + (size_t)b * K;
        int ok = 1;
        for (int i = 0; i < M; ++i) {
            if (cp[i] < -1 || cp[i] >= i) ok = 0;
            int ahead = 0;                                  /* how many candidates rank before i */
            for (int j = 0; j < M; ++j)
                if (j != i && ranks_before(cs, j, i)) ++ahead;
            keep[i] = ahead < K;
        }
        po[0] = -1; io[0] = 0;
        int n = 0;
        for (int i = 0; i < M; ++i) {
            node[i] = -1;
            if (!keep[i]) continue;
            node[i] = ++n;
            so[n - 1] = i;
            io[n] = ct[i];
            if (!ok) continue;
            if (cp[i] == -1) po[n] = 0;
            else if (keep[cp[i]]) po[n] = node[cp[i]];
            else ok = 0;
        }
        if (!ok) { ++bad; for (int j = 0; j <= K; ++j) po[j] = -1; }
    }
    free(keep); free(node);
    return bad;
}

/* KV commit for one layer's cache pair: for every sequence and kv head the rows at slots
 * S + path[k], k < accept_len, are gathered into a temporary and then written to slots S + k
 * (K and V alike).  Every other slot keeps its bytes.  kv_len_out[b] = S + accept_len (may be NULL). */
int oracle_kv_compact(uint16_t* k_cache, uint16_t* v_cache, const int32_t* path,
                      const int32_t* accept_len, const int32_t* kv_len, int32_t* kv_len_out,
                      int B, int N, int Hkv, int D, int S_max) {
    for (int b = 0; b < B; ++b) {
        int S = kv_len[b], L = accept_len[b];
        if (L < 1 || L > N || S < 0 || S + N > S_max) return -1;
        for (int k = 0; k < L; ++k) {
            int src = path[(size_t)b * N + k];
            if (src < 0 || src >= N) return -2;
        }
        uint16_t* tmp = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)L * D);
        if (!tmp) return -3;
        for (int which = 0; which < 2; ++which) {
            uint16_t* cache = which ? v_cache : k_cache;
            for (int h = 0; h < Hkv; ++h) {
                uint16_t* base = cache + ((size_t)b * Hkv + h) * (size_t)S_max * D;
                for (int k = 0; k < L; ++k)
                    memcpy(tmp + (size_t)k * D, base + (size_t)(S + path[(size_t)b * N + k]) * D,
                           sizeof(uint16_t) * D);
                for (int k = 0; k < L; ++k)
                    memcpy(base + (size_t)(S + k) * D, tmp + (size_t)k * D, sizeof(uint16_t) * D);
            }
        }
        free(tmp);
        if (kv_len_out) kv_len_out[b] = S + L;
    }
    return 0;
}

static uint16_t f64_to_bf16(double x) {
    /* one rounding to nearest even of the fp64 value: the bf16 neighbours of x are exactly
     * representable in fp64, so compare against their midpoint */
    float f = (float)x;                       /* may double-round; corrected below */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7f800000u) == 0x7f800000u) return (uint16_t)(u >> 16);   /* inf / nan */
    uint32_t lo = u & 0xffff0000u;            /* truncation toward zero */
    float flo, fhi;
    uint32_t hi = lo + 0x10000u;
    memcpy(&flo, &lo, sizeof flo);
    memcpy(&fhi, &hi, sizeof fhi);
    double dlo = (double)flo, dhi = (double)fhi;
    if (fabs(x) < fabs(dlo)) {                /* (float)x rounded away from x across a bf16 boundary */
        hi = lo; lo = lo - 0x10000u;
        memcpy(&flo, &lo, sizeof flo); memcpy(&fhi, &hi, sizeof fhi);
        dlo = (double)flo; dhi = (double)fhi;
    }
    double mid = 0.5 * (dlo + dhi);
    double ax = fabs(x), amid = fabs(mid);
    if (ax < amid) return (uint16_t)(lo >> 16);
    if (ax > amid) return (uint16_t)(hi >> 16);
    return (uint16_t)(((lo >> 16) & 1u) ? (hi >> 16) : (lo >> 16));      /* tie: even mantissa */
}

/* Rotary embedding of the tree rows, then their placement in the cache (the step before the attention):
 *   angle(b,i,j) = positions[b][i] * theta^(-2j/D),  j < D/2
 *   x'[j] = x[j] cos - x[j+D/2] sin,   x'[j+D/2] = x[j+D/2] cos + x[j] sin        (q and k rows)
 * q [B,N,Hq,D] is rotated in place; rotated k_new [B,N,Hkv,D] and v_new (unchanged) go to slots
 * kv_len[b] + i of k_cache / v_cache [B,Hkv,S_max,D].  bf16 in, fp64 arithmetic, one rounding to bf16.
 * A sequence with kv_len < 0 or kv_len + N > S_max is skipped.  Returns the number of skipped sequences. */
int oracle_rope_rows(uint16_t* q, const uint16_t* k_new, const uint16_t* v_new, const int32_t* positions,
                     const int32_t* kv_len, uint16_t* k_cache, uint16_t* v_cache, double theta,
                     int B, int N, int Hq, int Hkv, int D, int S_max) {
    int skipped = 0, half = D / 2;
    for (int b = 0; b < B; ++b) {
        int S = kv_len[b];
        if (S < 0 || S + N > S_max) { ++skipped; continue; }
        for (int i = 0; i < N; ++i) {
            double pos = (double)positions[(size_t)b * N + i];
            for (int j = 0; j < half; ++j) {
                double ang = pos * pow(theta, -2.0 * (double)j / (double)D);
                double c = cos(ang), sn = sin(ang);
                for (int h = 0; h < Hq; ++h) {
                    uint16_t* row = q + (((size_t)b * N + i) * Hq + h) * D;
                    double a = bf16_to_f64(row[j]), bb = bf16_to_f64(row[j + half]);
                    row[j] = f64_to_bf16(a * c - bb * sn);
                    row[j + half] = f64_to_bf16(bb * c + a * sn);
                }
                for (int h = 0; h < Hkv; ++h) {
                    const uint16_t* src = k_new + (((size_t)b * N + i) * Hkv + h) * D;
                    uint16_t* dst = k_cache + (((size_t)b * Hkv + h) * S_max + S + i) * D;
                    double a = bf16_to_f64(src[j]), bb = bf16_to_f64(src[j + half]);
                    dst[j] = f64_to_bf16(a * c - bb * sn);
                    dst[j + half] = f64_to_bf16(bb * c + a * sn);
                }
            }
            for (int h = 0; h < Hkv; ++h)
                memcpy(v_cache + (((size_t)b * Hkv + h) * S_max + S + i) * D,
                       v_new + (((size_t)b * N + i) * Hkv + h) * D, (size_t)D * sizeof(uint16_t));
        }
    }
    return skipped;
}
