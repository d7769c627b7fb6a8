// Sampled (temperature > 0) acceptance on a draft tree (Sec. 3.1): a drafted token x is kept with probability
// min(1, p(x)/p^(x)); after a rejection the target distribution becomes norm(max(0, p - p^)); the children of
// the current node are decided one after the other and the token after the last kept node is drawn from what
// remains.
//
// What is kept in registers instead of a residual vector: after k rejections at one node the residual is
// proportional to m_k = max(0, p - c_k p^) with c_0 = 0, c_{k+1} = c_k + S_k and S_k = sum(m_k) (S_0 taken as 1:
// the rule compares against p itself), because max(0, max(0, p - c p^)/S - p^) = max(0, p - (c + S) p^)/S.
// A decision needs two scalars of the node's rows; only a rejection needs a pass over the two rows (2 * V * 4
// bytes) to form the next S, and that pass also leaves per-warp partial sums that locate the bonus token, so the
// draw re-reads one warp's slice only.
//
// One cluster per sequence (8 CTAs for large vocabularies, 1 for small ones), 1024 threads per CTA.  Every CTA
// takes the same decisions from the same numbers: the CTA partials are exchanged through distributed shared
// memory behind a hardware cluster barrier and summed by everyone in rank order, so S is bit-identical in the
// cluster.  Sums and comparisons are fp64 (the inputs are fp32): the decisions then differ from a sequential
// fp64 evaluation only where a uniform falls within ~1e-15 of a threshold.
#include "vispec_internal.h"

namespace vispec {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxCluster = 8;

__device__ __forceinline__ void record_status_as(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}
__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cl_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ double cl_ld_f64(const double* local, uint32_t rank) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
    uint32_t ra;
    double v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(ra) : "memory");
    return v;
}

__device__ __forceinline__ double weight(float p, float ph, double c) {
    return fmax(0.0, (double)p - c * (double)ph);
}

// The slice of [0, V) that warp w of CTA `rank` sums: CTAs take consecutive ranges, warps consecutive sub-ranges,
// both rounded to 4 elements so that 16-byte loads stay aligned when V is a multiple of 4.
struct Slice { int lo, hi; };
__device__ __forceinline__ Slice warp_slice(int V, int rank, int csize, int w) {
    const int per = (((V + csize - 1) / csize) + 3) & ~3;
    const int wper = (((per + kWarps - 1) / kWarps) + 3) & ~3;
    const int clo = rank * per, chi = min(V, clo + per);
    Slice s;
    s.lo = min(chi, clo + w * wper);
    s.hi = min(chi, s.lo + wper);
    return s;
}

template <bool VEC>
__device__ __forceinline__ double slice_sum(const float* __restrict__ pt, const float* __restrict__ ph, double c,
                                            Slice s, int lane) {
    double acc = 0.0;
    if (VEC) {
#pragma unroll 8
        for (int e = s.lo + lane * 4; e < s.hi; e += 128) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(pt + e));
            const float4 b = __ldg(reinterpret_cast<const float4*>(ph + e));
            acc += (weight(a.x, b.x, c) + weight(a.y, b.y, c)) + (weight(a.z, b.z, c) + weight(a.w, b.w, c));
        }
    } else {
#pragma unroll 4
        for (int e = s.lo + lane; e < s.hi; e += 32) acc += weight(__ldg(pt + e), __ldg(ph + e), c);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

// first index i < n with (base + v[0] + ... + v[i]) > target, else the last i with v[i] > 0, else -1;
// *before = the running sum ahead of the index returned
__device__ __forceinline__ int locate(const double* v, int n, double base, double target, double* before) {
    double run = base;
    int last = -1;
    double last_before = base;
    for (int i = 0; i < n; ++i) {
        if (v[i] > 0.0) { last = i; last_before = run; }
        if (run + v[i] > target) { *before = run; return i; }
        run += v[i];
    }
    *before = last_before;
    return last;
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
accept_sampled_kernel(const int32_t* __restrict__ draft_ids, const int32_t* __restrict__ parents,
                      const float* __restrict__ p, const float* __restrict__ p_hat,
                      const float* __restrict__ u_accept, const float* __restrict__ u_bonus, int N, int V,
                      int32_t* __restrict__ path, int32_t* __restrict__ accept_len, int32_t* __restrict__ bonus,
                      int* status) {
    __shared__ int32_t par[VISPEC_MAX_TREE_NODES], ids[VISPEC_MAX_TREE_NODES], spath[VISPEC_MAX_TREE_NODES];
    __shared__ float ua[VISPEC_MAX_TREE_NODES];
    __shared__ float px_of[VISPEC_MAX_TREE_NODES], phx_of[VISPEC_MAX_TREE_NODES];   // p[parent][token], p^[parent][token] per node
    __shared__ double seg[kWarps];               // this CTA's per-warp sums of the last pass
    __shared__ double part[2];                   // this CTA's sum, by pass parity (read by the whole cluster)
    __shared__ double allpart[kMaxCluster];      // every CTA's sum of the last pass
    __shared__ double sh_c, sh_S;
    __shared__ int sh_cur, sh_action, sh_bad, sh_stop, sh_len;

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int csize = (int)cl_size(), rank = (int)cl_rank();
    const int b = blockIdx.x / csize;
    const size_t nb = (size_t)b * N;

    if (tid == 0) { sh_bad = 0; sh_stop = 0; }
    __syncthreads();
    if (tid < N) {
        const int pr = parents[nb + tid], id = draft_ids[nb + tid];
        par[tid] = pr;
        ids[tid] = id;
        ua[tid] = u_accept[nb + tid];
        const bool ok = tid == 0 ? pr == -1 : (pr >= 0 && pr < tid && id >= 0 && id < V);
        if (!ok) atomicOr(&sh_bad, tid == 0 || pr < 0 || pr >= tid ? 1 : 2);
    }
    __syncthreads();
    if (sh_bad) {                                // the same verdict in every CTA of the cluster: all leave here
        if (rank == 0) {
            if (tid < N) path[nb + tid] = -1;
            if (tid == 0) {
                accept_len[b] = 0;
                bonus[b] = -1;
                record_status_as(status, (sh_bad & 1) ? VISPEC_E_BAD_TREE : VISPEC_E_RANGE);
            }
        }
        return;
    }

    // the two scalars each decision needs, for every node at once (one round of loads instead of one per decision)
    if (tid >= 1 && tid < N) {
        const size_t row = (nb + par[tid]) * (size_t)V + ids[tid];
        px_of[tid] = __ldg(p + row);
        phx_of[tid] = __ldg(p_hat + row);
    }
    __syncthreads();

    enum { PASS = 0, DRAW = 1 };
    // walk state, meaningful in thread 0 only
    int cur = 0, len = 1, next_child = 1;
    double c = 0.0, S = 1.0;
    bool have_pass = false;
    if (tid == 0) spath[0] = 0;

    for (int iter = 0; iter < 2 * N + 4; ++iter) {
        if (tid == 0) {
            int action = -1;
            while (action < 0) {
                int ch = next_child;
                while (ch < N && par[ch] != cur) ++ch;
                if (ch >= N) {                   // no child left: draw from what remains (needs the sums of a pass)
                    action = have_pass ? DRAW : PASS;
                    break;
                }
                const double px = (double)px_of[ch], phx = (double)phx_of[ch];
                const double num = fmax(0.0, px - c * phx);
                next_child = ch + 1;
                if ((double)ua[ch] * S * phx < num) {          // kept: u < min(1, r(x)/p^(x)), r = m/S
                    cur = ch;
                    spath[len++] = ch;
                    c = 0.0; S = 1.0; have_pass = false;
                } else {                                        // rejected: next residual needs its sum
                    c += S;
                    action = PASS;
                }
            }
            sh_action = action; sh_c = c; sh_cur = cur;
        }
        __syncthreads();
        if (sh_action != PASS) break;

        // ---- one pass over the two rows of node sh_cur ----
        const float* pt = p + (nb + sh_cur) * (size_t)V;
        const float* ph = p_hat + (nb + sh_cur) * (size_t)V;
        const double sum = slice_sum<VEC>(pt, ph, sh_c, warp_slice(V, rank, csize, w), lane);
        if (lane == 0) seg[w] = sum;
        __syncthreads();
        const int parity = iter & 1;
        if (tid == 0) {
            double v[kWarps];
#pragma unroll
            for (int i = 0; i < kWarps; ++i) v[i] = seg[i];          // all loads first, then the ordered sum
            double t = 0.0;
#pragma unroll
            for (int i = 0; i < kWarps; ++i) t += v[i];
            part[parity] = t;
        }
        cl_sync();                               // every CTA's part[parity] is written and visible
        if (tid == 0) {
            double v[kMaxCluster];
#pragma unroll
            for (int r = 0; r < kMaxCluster; ++r) v[r] = r < csize ? cl_ld_f64(&part[parity], (uint32_t)r) : 0.0;
            double t = 0.0;
#pragma unroll
            for (int r = 0; r < kMaxCluster; ++r) {
                allpart[r] = v[r];
                t += v[r];
            }
            if (t > 0.0) {
                S = t; have_pass = true;
            } else if (c == 0.0) {               // the target row itself has no weight: nothing to draw
                sh_stop = 1;
            } else {                             // empty residual: stop deciding, draw from the target row
                c = 0.0; S = 1.0; have_pass = false; next_child = N;
            }
            sh_S = S;
        }
        __syncthreads();
        if (sh_stop) break;
    }

    // ---- outputs: path and length from rank 0, the bonus token from the warp whose slice holds it ----
    if (tid == 0) sh_len = len;
    __syncthreads();
    if (rank == 0) {
        if (tid == 0) accept_len[b] = sh_len;
        if (tid < N) path[nb + tid] = tid < sh_len ? spath[tid] : -1;
    }

    if (sh_stop || sh_action != DRAW) {           // no weight to draw from (or, never, the pass bound ran out)
        if (rank == 0 && tid == 0) {
            bonus[b] = -1;
            if (!sh_stop) record_status_as(status, VISPEC_E_TIMEOUT);
        }
    } else {
        const double target = (double)u_bonus[b] * sh_S;
        double base = 0.0;
        const int r_star = locate(allpart, csize, 0.0, target, &base);
        if (r_star == rank) {
            double base2 = base;
            const int w_star = locate(seg, kWarps, base, target, &base2);
            if (w_star == w) {
                const float* pt = p + (nb + sh_cur) * (size_t)V;
                const float* ph = p_hat + (nb + sh_cur) * (size_t)V;
                const Slice s = warp_slice(V, rank, csize, w);
                const double cc = sh_c;
                double run = base2;
                int found = -1, last_pos = -1;
                for (int e0 = s.lo; e0 < s.hi && found < 0; e0 += 128) {
                    double m[4];
                    const int e = e0 + lane * 4;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        m[j] = (e + j < s.hi) ? weight(__ldg(pt + e + j), __ldg(ph + e + j), cc) : 0.0;
                    const double mine = (m[0] + m[1]) + (m[2] + m[3]);
                    double incl = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double t = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += t;
                    }
                    const double chunk = __shfl_sync(0xffffffffu, incl, 31);
                    // the first lane whose running sum passes the target, then the element inside that lane
                    const unsigned hit = __ballot_sync(0xffffffffu, run + incl > target);
                    int cand = -1;
                    if (hit) {
                        const int l0 = __ffs(hit) - 1;
                        if (lane == l0) {
                            double r2 = run + (incl - mine);
                            int last_in = -1;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (m[j] > 0.0) last_in = e + j;
                                if (cand < 0 && r2 + m[j] > target) cand = e + j;
                                r2 += m[j];
                            }
                            if (cand < 0) cand = last_in;   // rounding between the two summation orders
                        }
                        cand = __shfl_sync(0xffffffffu, cand, l0);
                    }
                    int lp = -1;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (m[j] > 0.0) lp = e + j;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(0xffffffffu, lp, o));
                    if (cand >= 0) found = cand;
                    else if (lp >= 0) last_pos = lp;
                    run += chunk;
                }
                if (found < 0) found = last_pos;            // the slice's sum said "here" but the rescan fell short
                if (lane == 0) bonus[b] = found;
            }
        }
    }
    cl_sync();                                   // nobody leaves while its partial sums may still be read
}

}  // namespace

cudaError_t launch_accept_sampled(const int32_t* draft_ids, const int32_t* parents, const float* p, const float* p_hat,
                                  const float* u_accept, const float* u_bonus, int B, int N, int V, int32_t* path,
                                  int32_t* accept_len, int32_t* bonus, int* status, cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    const int cl = V >= 8192 ? kMaxCluster : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B * cl);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (V % 4 == 0)
        return cudaLaunchKernelEx(&cfg, accept_sampled_kernel<true>, draft_ids, parents, p, p_hat, u_accept, u_bonus, N,
                                  V, path, accept_len, bonus, status);
    return cudaLaunchKernelEx(&cfg, accept_sampled_kernel<false>, draft_ids, parents, p, p_hat, u_accept, u_bonus, N, V,
                              path, accept_len, bonus, status);
}

}  // namespace vispec
