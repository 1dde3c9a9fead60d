// radar_verify_accept: acceptance of the verified tree.
//   greedy     - vocabulary pass with k = 1 (row argmax, no exponentials) over the target logits of
//                the live tree rows, then one warp per sequence walks the tree with ballots.
//   stochastic - one thread-block cluster per sequence walks the tree lazily: only rows on the accepted
//                path are read, and each CTA of the cluster owns a slice of the vocabulary in every pass.
//                Probabilities are fp64.  exp((z - max) / T) of the current node's target and draft rows
//                is cached in the workspace (p, q = cached value / row sum); after j rejections the residual pair is, for every token v that has
//                not been proposed yet,  p_j(v) = max(0, p(v) - a_j q(v)) / W_j,  q_j(v) = c_j q(v),
//                and for the token proposed at trial i <= j,  p_j(x_i) = max(0, p(x_i) - a_i q(x_i)) / W_j,
//                q_j(x_i) = 0, with a_{j+1} = a_j + c_j W_j,  c_{j+1} = c_j / (1 - q_j(x_{j+1})) and
//                W_{j+1} = sum_v max(0, p(v) - a(v) q(v)).  This is the rectify / remove / renormalise
//                recursion of Eq. 2 unrolled, so each rejection costs one read-only pass.
#include <algorithm>

#include "common.cuh"

namespace radar {
namespace {

// ------------------------------------------------------------------------------------------
// greedy walk
// ------------------------------------------------------------------------------------------
struct GreedyParams {
    radar_accept_args a;
    VocabPassParams vp;
};

__global__ void __launch_bounds__(64) greedy_walk_kernel(const GreedyParams P) {
    chain_wait();
    const radar_accept_args& a = P.a;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    __shared__ int s_arg[kMaxNodes], s_tok[kMaxNodes], s_par[kMaxNodes];
    const int M = min(max(a.n_nodes[b], 1), kMaxNodes);
    const int nc = P.vp.n_chunks;
    {   // argmax of row tid: best chunk record by (value desc, token asc)
        int best_i = 0x7fffffff;
        float best_v = -CUDART_INF_F;
        if (tid < M) {
            const size_t rec0 = ((size_t)b * kMaxNodes + tid) * nc;
            for (int c = 0; c < nc; ++c) {
                const float v = P.vp.part_v[rec0 + c];
                const int i = P.vp.part_i[rec0 + c];
                if (precedes(v, i, best_v, best_i)) { best_v = v; best_i = i; }
            }
        }
        s_arg[tid] = best_i;
        s_tok[tid] = tid < M ? a.tree_tok[(size_t)b * kMaxNodes + tid] : -1;
        s_par[tid] = tid < M ? a.tree_parent[(size_t)b * kMaxNodes + tid] : -2;
    }
    __syncthreads();
    if (tid >= 32) return;
    const int W = a.t_max + 1;
    int32_t* pn = a.path_nodes + (size_t)b * W;
    int32_t* pt = a.path_tokens + (size_t)b * W;
    int cur = 0, len = 0;
    if (lane == 0) { pn[0] = 0; pt[0] = s_tok[0]; }
    while (len < a.t_max) {
        const int want = s_arg[cur];
        const unsigned lo = __ballot_sync(kFull, s_par[lane] == cur && s_tok[lane] == want && lane > 0);
        const unsigned hi = __ballot_sync(kFull, s_par[lane + 32] == cur && s_tok[lane + 32] == want);
        const int nxt = lo ? __ffs(lo) - 1 : (hi ? 32 + __ffs(hi) - 1 : -1);
        if (nxt < 0) break;
        cur = nxt;
        ++len;
        if (lane == 0) { pn[len] = cur; pt[len] = s_tok[cur]; }
    }
    for (int dd = len + 1 + lane; dd < W; dd += 32) { pn[dd] = -1; pt[dd] = -1; }
    int best = 0x7fffffff;
    const int nl = a.n_leaves[b];
    for (int r = lane; r < nl; r += 32)
        if (a.retrieve[((size_t)b * a.N + r) * W + len] == cur) best = min(best, r);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(kFull, best, o));
    if (lane == 0) {
        a.accept_len[b] = len;
        a.next_token[b] = s_arg[cur];
        a.best_retrieve_row[b] = best == 0x7fffffff ? -1 : best;
    }
}

// ------------------------------------------------------------------------------------------
// stochastic walk
// ------------------------------------------------------------------------------------------
constexpr int kSThreads = 1024;
constexpr int kMaxCluster = 8;           // portable cluster size limit

struct StochParams {
    radar_accept_args a;
    double* p_cache;     // [B][V] unnormalised exp((z_target - max) / T)
    double* q_cache;     // [B][V] same for the draft row
    int* status;
};

// The walk of one sequence is shared by the CTAs of a thread-block cluster: CTA r owns the vocabulary
// slice [V r / n, V (r + 1) / n) of every full-vocabulary pass.  Every scalar that steers the walk is
// reduced over the cluster into every CTA in a fixed order, so all CTAs take identical decisions and
// meet at the same cluster barriers.
struct ClusterRed {
    double* block_scratch;   // [32] shared
    double* slots;           // [2][kMaxCluster] shared; the same array exists in every CTA of the cluster
    unsigned rank, n;
    unsigned phase;

    __device__ double block_sum(double v) {
        v = warp_sum(v);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) block_scratch[threadIdx.x >> 5] = v;
        __syncthreads();
        double t = 0.0;
        for (int w = 0; w < kSThreads / 32; ++w) t += block_scratch[w];     // same order in every thread
        return t;
    }
    __device__ double block_max(double v) {
        v = warp_max(v);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) block_scratch[threadIdx.x >> 5] = v;
        __syncthreads();
        double t = block_scratch[0];
        for (int w = 1; w < kSThreads / 32; ++w) t = fmax(t, block_scratch[w]);
        return t;
    }
    // every CTA's value lands in out[0..n) of every CTA (rank order)
    __device__ void all_gather(double mine, double* out) {
        double* my = slots + (phase & 1) * kMaxCluster;
        if (threadIdx.x < n) {
            asm volatile(
                "{\n\t.reg .u32 ra;\n\t"
                "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
                "st.shared::cluster.f64 [ra], %2;\n\t}"
                ::"r"((uint32_t)__cvta_generic_to_shared(my + rank)), "r"(threadIdx.x), "d"(mine)
                : "memory");
        }
        cluster_sync();
        for (unsigned r = 0; r < n; ++r) out[r] = my[r];
        ++phase;                         // the other half is written next: no second barrier is needed
    }
    __device__ static void cluster_sync() {
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    __device__ double sum(double local) {
        double all[kMaxCluster];
        all_gather(block_sum(local), all);
        double t = 0.0;
        for (unsigned r = 0; r < n; ++r) t += all[r];
        return t;
    }
    __device__ double max(double local) {
        double all[kMaxCluster];
        all_gather(block_max(local), all);
        double t = all[0];
        for (unsigned r = 1; r < n; ++r) t = fmax(t, all[r]);
        return t;
    }
};

// cache[v] = exp(z[v] / T - max) over this CTA's slice; returns 1 / sum over the whole row
template <typename T>
__device__ double softmax_to_cache(const T* z, int v0, int v1, double invT, double* cache, ClusterRed& red, bool* nan_seen) {
    double m = -CUDART_INF;
    for (int v = v0 + threadIdx.x; v < v1; v += kSThreads) {
        const float zf = to_float(z[v]);
        if (zf != zf) *nan_seen = true;
        m = fmax(m, (double)zf * invT);
    }
    m = red.max(m);
    double s = 0.0;
    for (int v = v0 + threadIdx.x; v < v1; v += kSThreads) {
        const double e = exp((double)to_float(z[v]) * invT - m);
        cache[v] = e;
        s += e;
    }
    s = red.sum(s);                      // its cluster barrier also publishes every slice of the cache
    return 1.0 / s;
}

template <typename T>
__global__ void __launch_bounds__(kSThreads) stochastic_walk_kernel(const StochParams P) {
    chain_wait();
    const radar_accept_args& a = P.a;
    unsigned crank, csize;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
    const int b = blockIdx.x / csize, tid = threadIdx.x;
    const int V = a.V, W = a.t_max + 1;
    __shared__ double s_red[32];
    __shared__ double s_slots[2 * kMaxCluster];
    __shared__ int s_tok[kMaxNodes], s_par[kMaxNodes], s_drow[kMaxNodes], s_child[kMaxNodes];
    __shared__ int s_nchild;
    __shared__ int s_rx[RADAR_MAX_NODES];        // tokens proposed and rejected at the current node
    __shared__ double s_ra[RADAR_MAX_NODES];     // their frozen coefficients a_i
    __shared__ int s_pick, s_last_pos;
    ClusterRed red{s_red, s_slots, crank, csize, 0};
    const int v0 = (int)((long long)V * crank / csize), v1 = (int)((long long)V * (crank + 1) / csize);
    const bool lead = crank == 0;                 // writes the per-sequence outputs

    const int M = min(max(a.n_nodes[b], 1), kMaxNodes);
    if (tid < kMaxNodes) {
        s_tok[tid] = tid < M ? a.tree_tok[(size_t)b * kMaxNodes + tid] : -1;
        s_par[tid] = tid < M ? a.tree_parent[(size_t)b * kMaxNodes + tid] : -2;
        s_drow[tid] = tid < M ? a.tree_draft_row[(size_t)b * kMaxNodes + tid] : -1;
    }
    __syncthreads();
    ClusterRed::cluster_sync();                   // every CTA's shared memory is live before the first remote store

    const T* target = reinterpret_cast<const T*>(a.target_logits) + (size_t)b * kMaxNodes * V;
    const T* draft = reinterpret_cast<const T*>(a.draft_logits) + (size_t)b * a.R * V;
    double* pc = P.p_cache + (size_t)b * V;
    double* qc = P.q_cache + (size_t)b * V;
    const double invT = 1.0 / (double)a.temperature;
    const float* ua = a.u_accept + (size_t)b * kMaxNodes;
    bool nan_seen = false;

    int32_t* pn = a.path_nodes + (size_t)b * W;
    int32_t* pt = a.path_tokens + (size_t)b * W;
    int cur = 0, len = 0;
    if (lead && tid == 0) { pn[0] = 0; pt[0] = s_tok[0]; }

    int n_rej = 0;           // rejections at the final node (0 => weights are p itself)
    double a_coef = 0.0;     // p_j(v) = max(0, p(v) - a q(v)) / W_j for tokens not yet proposed
    double ip = 1.0, iq = 1.0;   // 1 / sum of the cached exponentials: p(v) = pc[v] * ip, q(v) = qc[v] * iq
    bool bad_tree = false;
    for (;;) {
        ip = softmax_to_cache<T>(target + (size_t)cur * V, v0, v1, invT, pc, red, &nan_seen);
        if (tid == 0) {
            int n = 0;
            for (int j = cur + 1; j < M; ++j)
                if (s_par[j] == cur) s_child[n++] = j;
            s_nchild = n;
        }
        __syncthreads();
        const int nchild = s_nchild;
        n_rej = 0;
        a_coef = 0.0;
        if (nchild == 0 || len >= a.t_max) break;
        const int drow = s_drow[cur];
        if (drow < 0 || drow >= a.R) { bad_tree = true; break; }
        iq = softmax_to_cache<T>(draft + (size_t)drow * V, v0, v1, invT, qc, red, &nan_seen);

        double Wn = 1.0, cq = 1.0;
        int accepted = -1;
        for (int ci = 0; ci < nchild; ++ci) {
            const int j = s_child[ci];
            const int x = s_tok[j];
            if (x < 0 || x >= V) { bad_tree = true; break; }
            const double px = pc[x] * ip, qx = qc[x] * iq;
            const double pj = fmax(0.0, px - a_coef * qx) / Wn;      // x has not been proposed before
            const double qj = cq * qx;
            bool acc;
            if (qj <= 0.0) acc = pj > 0.0;
            else {
                const double ratio = pj / qj;
                acc = (double)ua[j] < (ratio < 1.0 ? ratio : 1.0);
            }
            if (acc) { accepted = j; break; }
            // reject: one pass for the new residual mass
            const double a_new = a_coef + cq * Wn;
            double g = 0.0;
            for (int v = v0 + tid; v < v1; v += kSThreads) g += fmax(0.0, pc[v] * ip - a_new * (qc[v] * iq));
            g = red.sum(g);
            // tokens rejected earlier keep their own coefficient: swap their terms
            for (int r = 0; r < n_rej; ++r) {
                const int xr = s_rx[r];
                const double pr = pc[xr] * ip, qr = qc[xr] * iq;
                g += fmax(0.0, pr - s_ra[r] * qr) - fmax(0.0, pr - a_new * qr);
            }
            double frozen = a_coef;
            if (g > 0.0) { a_coef = a_new; Wn = g; frozen = a_new; }   // else: residual empty, p stays as it is
            __syncthreads();
            if (tid == 0) { s_rx[n_rej] = x; s_ra[n_rej] = frozen; }
            __syncthreads();
            ++n_rej;
            const double rest = 1.0 - qj;                               // draft mass left after removing x
            if (rest <= 0.0) break;
            cq = cq / rest;
        }
        if (bad_tree || accepted < 0) break;
        cur = accepted;
        ++len;
        if (lead && tid == 0) { pn[len] = cur; pt[len] = s_tok[cur]; }
    }

    // ---- final draw: inverse CDF over w(v) = max(0, p(v) - a(v) q(v)) (or p(v) when nothing was rejected) ----
    const int nv = v1 - v0;
    const int per = (nv + kSThreads - 1) / kSThreads;
    const int t0 = v0 + min(tid * per, nv), t1 = v0 + min(tid * per + per, nv);
    auto weight = [&](int v) -> double {
        if (n_rej == 0) return pc[v] * ip;
        double av = a_coef;
        for (int r = 0; r < n_rej; ++r)
            if (s_rx[r] == v) av = s_ra[r];
        return fmax(0.0, pc[v] * ip - av * (qc[v] * iq));
    };
    if (tid == 0) { s_pick = 0x7fffffff; s_last_pos = -1; }
    double seg = 0.0;
    int last_pos = -1;
    for (int v = t0; v < t1; ++v) {
        const double w = weight(v);
        seg += w;
        if (w > 0.0) last_pos = v;
    }
    // scan of seg over the threads of this CTA (fp64).  A thread's end and its successor's start are the
    // same expression, so at most one thread owns a point.
    double incl = seg;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
    }
    double excl = __shfl_up_sync(kFull, incl, 1);
    if (lane == 0) excl = 0.0;
    __syncthreads();
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    double woff = 0.0, slice_total = 0.0;
    for (int w = 0; w < kSThreads / 32; ++w) {
        if (w == warp) woff = slice_total;
        slice_total += s_red[w];
    }
    __syncthreads();
    // slice totals of every CTA, in rank order: the running sum gives each slice's start, and the same
    // expression is the previous slice's end
    double tots[kMaxCluster];
    red.all_gather(slice_total, tots);
    double total = 0.0, my_start = 0.0;
    for (unsigned r = 0; r < csize; ++r) {
        if (r == crank) my_start = total;
        total += tots[r];
    }
    const double tgt = (double)a.u_sample[b] * total;
    // owner: the first slice whose end exceeds the point; if rounding leaves none, the last slice with mass
    int owner = -1, last_live = 0;
    {
        double run = 0.0;
        for (unsigned r = 0; r < csize; ++r) {
            run += tots[r];
            if (tots[r] > 0.0) last_live = (int)r;
            if (owner < 0 && tgt < run) owner = (int)r;
        }
        if (owner < 0) owner = last_live;
    }
    if ((int)crank == owner) {
        const double start = my_start + (woff + excl), end = my_start + (woff + incl);
        if (last_pos >= 0) atomicMax(&s_last_pos, last_pos);
        if (start <= tgt && tgt < end) {
            double run = start;
            int pick = last_pos;                                            // rounding guard: the crossing is in here
            for (int v = t0; v < t1; ++v) {
                run += weight(v);
                if (run > tgt) { pick = v; break; }
            }
            if (pick >= 0) atomicMin(&s_pick, pick);
        }
        __syncthreads();
        if (tid == 0) a.next_token[b] = s_pick != 0x7fffffff ? s_pick : s_last_pos;
    }
    if (lead && tid == 0) {
        a.accept_len[b] = len;
        if (bad_tree) set_status(P.status, RADAR_ERR_TREE);
    }
    if (nan_seen) set_status(P.status, RADAR_ERR_NUMERIC);
    if (lead) {
        for (int dd = len + 1 + tid; dd < W; dd += kSThreads) { pn[dd] = -1; pt[dd] = -1; }
        if (tid < 32) {
            int best = 0x7fffffff;
            const int nl = a.n_leaves[b];
            for (int r = tid; r < nl; r += 32)
                if (a.retrieve[((size_t)b * a.N + r) * W + len] == cur) best = min(best, r);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(kFull, best, o));
            if (tid == 0) a.best_retrieve_row[b] = best == 0x7fffffff ? -1 : best;
        }
    }
    ClusterRed::cluster_sync();                   // no CTA leaves while another may still store into its shared memory
}

// ------------------------------------------------------------------------------------------
// acceptance-length distribution (Eq. 11-13)
// ------------------------------------------------------------------------------------------
struct AccLenParams {
    radar_acclen_args a;
    double* p_cache;     // [grid][V]
    double* q_cache;     // [grid][V]
    double* cond;        // [B][64]: P_acc(row | its parent), in the workspace
    int* status;
};

// One item = one tree row of one sequence; rows without children have nothing to do.  A persistent
// grid walks the items; each block evaluates its row's children in order with the same closed-form
// residual recursion as the stochastic walk, but follows every rejection branch: child j gets
// reach_j a_j with reach_j = prod_{i<j} (1 - a_i).
template <typename T>
__global__ void __launch_bounds__(kSThreads) accept_length_nodes_kernel(const AccLenParams P) {
    chain_wait();
    const radar_acclen_args& a = P.a;
    const int tid = threadIdx.x, V = a.V;
    __shared__ double s_red[32];
    __shared__ double s_slots[2 * kMaxCluster];
    __shared__ int s_tok[kMaxNodes], s_par[kMaxNodes];
    __shared__ int s_rx[RADAR_MAX_NODES];
    __shared__ double s_ra[RADAR_MAX_NODES];
    ClusterRed red{s_red, s_slots, 0u, 1u, 0};       // launched without clusters: every block is its own
    double* pc = P.p_cache + (size_t)blockIdx.x * V;
    double* qc = P.q_cache + (size_t)blockIdx.x * V;
    const double invT = 1.0 / (double)a.temperature;
    bool nan_seen = false, bad_tree = false;

    for (int item = blockIdx.x; item < a.B * kMaxNodes; item += gridDim.x) {
        const int b = item / kMaxNodes, c = item % kMaxNodes;
        const int M = min(max(a.n_nodes[b], 1), kMaxNodes);
        if (c >= M) {
            if (tid == 0) P.cond[item] = 0.0;
            continue;
        }
        __syncthreads();                                  // previous item's readers are done with s_tok / s_par
        if (tid < kMaxNodes) {
            s_tok[tid] = tid < M ? a.tree_tok[(size_t)b * kMaxNodes + tid] : -1;
            s_par[tid] = tid < M ? a.tree_parent[(size_t)b * kMaxNodes + tid] : -2;
        }
        __syncthreads();
        if (c == 0 && tid == 0) P.cond[item] = 1.0;       // the root is always "accepted"
        int nchild = 0;
        for (int j = c + 1; j < M; ++j) nchild += s_par[j] == c ? 1 : 0;
        if (nchild == 0) continue;
        const int drow = a.tree_draft_row[(size_t)b * kMaxNodes + c];
        if (drow < 0 || drow >= a.R) { bad_tree = true; continue; }
        const T* target = reinterpret_cast<const T*>(a.target_logits) + ((size_t)b * kMaxNodes + c) * V;
        const T* draft = reinterpret_cast<const T*>(a.draft_logits) + ((size_t)b * a.R + drow) * V;
        const double ip = softmax_to_cache<T>(target, 0, V, invT, pc, red, &nan_seen);
        const double iq = softmax_to_cache<T>(draft, 0, V, invT, qc, red, &nan_seen);

        double a_coef = 0.0, Wn = 1.0, cq = 1.0, reach = 1.0;
        int n_rej = 0;
        bool exhausted = false;
        for (int j = c + 1; j < M; ++j) {
            if (s_par[j] != c) continue;
            if (exhausted) {
                if (tid == 0) P.cond[(size_t)b * kMaxNodes + j] = 0.0;
                continue;
            }
            const int x = s_tok[j];
            if (x < 0 || x >= V) { bad_tree = true; break; }
            const double px = pc[x] * ip, qx = qc[x] * iq;
            const double pj = fmax(0.0, px - a_coef * qx) / Wn;
            const double qj = cq * qx;
            double acc;
            if (qj <= 0.0) acc = pj > 0.0 ? 1.0 : 0.0;
            else { acc = pj / qj; if (acc > 1.0) acc = 1.0; }
            if (tid == 0) P.cond[(size_t)b * kMaxNodes + j] = reach * acc;
            reach *= 1.0 - acc;
            // the rejection branch: new residual, x leaves the draft distribution
            const double a_new = a_coef + cq * Wn;
            double g = 0.0;
            for (int v = tid; v < V; v += kSThreads) g += fmax(0.0, pc[v] * ip - a_new * (qc[v] * iq));
            g = red.sum(g);
            for (int r = 0; r < n_rej; ++r) {
                const int xr = s_rx[r];
                const double pr = pc[xr] * ip, qr = qc[xr] * iq;
                g += fmax(0.0, pr - s_ra[r] * qr) - fmax(0.0, pr - a_new * qr);
            }
            double frozen = a_coef;
            if (g > 0.0) { a_coef = a_new; Wn = g; frozen = a_new; }
            __syncthreads();
            if (tid == 0) { s_rx[n_rej] = x; s_ra[n_rej] = frozen; }
            __syncthreads();
            ++n_rej;
            const double rest = 1.0 - qj;
            if (rest <= 0.0) exhausted = true;
            else cq = cq / rest;
        }
    }
    if (nan_seen) set_status(P.status, RADAR_ERR_NUMERIC);
    if (bad_tree && tid == 0) set_status(P.status, RADAR_ERR_TREE);
}

// one warp per sequence: P_acc along the paths (parents precede children), P_stop, p_i
__global__ void __launch_bounds__(32) accept_length_dist_kernel(const AccLenParams P) {
    chain_wait();
    const radar_acclen_args& a = P.a;
    const int b = blockIdx.x, lane = threadIdx.x;
    const int M = min(max(a.n_nodes[b], 1), kMaxNodes);
    __shared__ double s_pacc[kMaxNodes], s_sum[kMaxNodes], s_dist[64];
    for (int i = lane; i < kMaxNodes; i += 32) { s_pacc[i] = 0.0; s_sum[i] = 0.0; }
    for (int i = lane; i < 64; i += 32) s_dist[i] = 0.0;
    __syncwarp();
    if (lane == 0) {
        s_pacc[0] = 1.0;
        for (int j = 1; j < M; ++j) {
            const int par = a.tree_parent[(size_t)b * kMaxNodes + j];
            const double cj = (par >= 0 && par < j) ? P.cond[(size_t)b * kMaxNodes + j] : 0.0;
            s_pacc[j] = (par >= 0 && par < j ? s_pacc[par] : 0.0) * cj;
            if (par >= 0 && par < j) s_sum[par] += cj;
        }
        for (int c = 0; c < M; ++c) {
            const int dep = a.tree_depth[(size_t)b * kMaxNodes + c];
            if (dep >= 0 && dep <= a.t_max) s_dist[dep] += s_pacc[c] * (1.0 - s_sum[c]);
        }
    }
    __syncwarp();
    for (int i = lane; i < kMaxNodes; i += 32) a.p_acc_node[(size_t)b * kMaxNodes + i] = s_pacc[i];
    for (int i = lane; i <= a.t_max; i += 32) a.dist[(size_t)b * (a.t_max + 1) + i] = s_dist[i];
}

}  // namespace
}  // namespace radar

using namespace radar;

extern "C" size_t radar_accept_workspace_bytes(const radar_ctx* ctx, int B, int V, int mode) {
    if (!ctx || B <= 0 || V <= 0) return 0;
    if (mode == RADAR_GREEDY) {
        int chunk;
        const int n_chunks = vocab_pass_plan_chunks(ctx->sm_count, B * kMaxNodes, V, &chunk);
        return vocab_pass_partial_bytes(B * kMaxNodes, n_chunks, 1);
    }
    return align_up((size_t)B * V * sizeof(double), 256) * 2;
}

extern "C" int radar_verify_accept(radar_ctx* ctx, const radar_accept_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->V <= 0 || a->t_max < 1 || a->N < 1) return RADAR_ERR_INVALID_ARG;
    if (a->mode != RADAR_GREEDY && a->mode != RADAR_STOCHASTIC) return RADAR_ERR_INVALID_ARG;
    if (a->logits_dtype != RADAR_F32 && a->logits_dtype != RADAR_BF16) return RADAR_ERR_UNSUPPORTED;
    if (!a->target_logits || !a->tree_tok || !a->tree_parent || !a->n_nodes || !a->retrieve || !a->n_leaves ||
        !a->accept_len || !a->path_nodes || !a->path_tokens || !a->next_token || !a->best_retrieve_row ||
        !a->workspace)
        return RADAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->workspace) & 255) != 0) return RADAR_ERR_WORKSPACE;
    if (radar_accept_workspace_bytes(ctx, a->B, a->V, a->mode) > a->workspace_bytes) return RADAR_ERR_WORKSPACE;

    if (a->mode == RADAR_GREEDY) {
        GreedyParams gp;
        gp.a = *a;
        VocabPassParams& vp = gp.vp;
        vp.logits = a->target_logits;
        vp.dtype = a->logits_dtype;
        vp.row_stride = a->V;
        vp.seq_stride = (int64_t)kMaxNodes * a->V;
        vp.n_seq = a->B;
        vp.F = kMaxNodes;
        vp.V = a->V;
        vp.k = 1;
        vp.n_chunks = vocab_pass_plan_chunks(ctx->sm_count, a->B * kMaxNodes, a->V, &vp.chunk);
        vp.want_lse = 0;
        vp.seq_active = nullptr;
        vp.seq_rows = a->n_nodes;
        vp.status = ctx->d_status;
        vocab_pass_carve(a->workspace, a->B * kMaxNodes, vp.n_chunks, 1, &vp);
        RADAR_CUDA_CHECK(vocab_pass_launch(ctx, RADAR_K_VOCAB_ACCEPT, vp, stream));
        {
            radar_launch_scope scope(ctx, RADAR_K_GREEDY_WALK, stream);
            RADAR_CUDA_CHECK(launch_chained(greedy_walk_kernel, dim3(a->B), dim3(64), 0, stream, gp));
        }
        RADAR_CUDA_CHECK(cudaGetLastError());
        return RADAR_OK;
    }
    if (!a->tree_draft_row || !a->draft_logits || !a->u_accept || !a->u_sample || a->R < 1) return RADAR_ERR_INVALID_ARG;
    if (!(a->temperature > 0.f)) return RADAR_ERR_INVALID_ARG;
    StochParams sp;
    sp.a = *a;
    sp.p_cache = reinterpret_cast<double*>(a->workspace);
    sp.q_cache = reinterpret_cast<double*>(reinterpret_cast<char*>(a->workspace) +
                                           align_up((size_t)a->B * a->V * sizeof(double), 256));
    sp.status = ctx->d_status;
    // cluster size: as many CTAs per sequence as keep the whole batch resident at once (at most 8)
    int cs = 1;
    while (cs < kMaxCluster && (long long)a->B * cs * 2 <= ctx->sm_count) cs *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a->B * cs));
    cfg.blockDim = dim3(kSThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    {
        radar_launch_scope scope(ctx, RADAR_K_STOCH_WALK, stream);
        if (a->logits_dtype == RADAR_F32) RADAR_CUDA_CHECK(cudaLaunchKernelEx(&cfg, stochastic_walk_kernel<float>, sp));
        else RADAR_CUDA_CHECK(cudaLaunchKernelEx(&cfg, stochastic_walk_kernel<__nv_bfloat16>, sp));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}

static int acclen_grid(const radar_ctx* ctx, int B) { return std::min(B * kMaxNodes, ctx->sm_count); }

extern "C" size_t radar_acclen_workspace_bytes(const radar_ctx* ctx, int B, int V) {
    if (!ctx || B <= 0 || V <= 0) return 0;
    return 2 * align_up((size_t)acclen_grid(ctx, B) * V * sizeof(double), 256) + align_up((size_t)B * kMaxNodes * sizeof(double), 256);
}

extern "C" int radar_accept_length_distribution(radar_ctx* ctx, const radar_acclen_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->V <= 0 || a->t_max < 1 || a->R < 1 || !(a->temperature > 0.f)) return RADAR_ERR_INVALID_ARG;
    if (a->t_max >= 64) return RADAR_ERR_UNSUPPORTED;
    if (a->logits_dtype != RADAR_F32 && a->logits_dtype != RADAR_BF16) return RADAR_ERR_UNSUPPORTED;
    if (!a->target_logits || !a->draft_logits || !a->tree_tok || !a->tree_parent || !a->tree_depth || !a->tree_draft_row ||
        !a->n_nodes || !a->dist || !a->p_acc_node || !a->workspace)
        return RADAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->workspace) & 255) != 0) return RADAR_ERR_WORKSPACE;
    if (radar_acclen_workspace_bytes(ctx, a->B, a->V) > a->workspace_bytes) return RADAR_ERR_WORKSPACE;
    const int grid = acclen_grid(ctx, a->B);
    AccLenParams P;
    P.a = *a;
    char* w = reinterpret_cast<char*>(a->workspace);
    const size_t cache = align_up((size_t)grid * a->V * sizeof(double), 256);
    P.p_cache = reinterpret_cast<double*>(w);
    P.q_cache = reinterpret_cast<double*>(w + cache);
    P.cond = reinterpret_cast<double*>(w + 2 * cache);
    P.status = ctx->d_status;
    {
        radar_launch_scope scope(ctx, RADAR_K_ACCLEN_NODES, stream);
        if (a->logits_dtype == RADAR_F32) RADAR_CUDA_CHECK(launch_chained(accept_length_nodes_kernel<float>, dim3(grid), dim3(kSThreads), 0, stream, P));
        else RADAR_CUDA_CHECK(launch_chained(accept_length_nodes_kernel<__nv_bfloat16>, dim3(grid), dim3(kSThreads), 0, stream, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    {
        radar_launch_scope scope(ctx, RADAR_K_ACCLEN_DIST, stream);
        RADAR_CUDA_CHECK(launch_chained(accept_length_dist_kernel, dim3(a->B), dim3(32), 0, stream, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}

// ------------------------------------------------------------------------------------------
// Greedy acceptance for callers that cannot hand over a workspace.
//
// Who needs this: code that runs after its host application has frozen device memory.  A serving
// engine typically gives every free byte of the GPU to its own KV-cache pool at start-up; from
// then on a cudaMalloc either fails or has to be carved out of that pool by hand, and cudaMalloc /
// cudaFree also synchronise the whole device, which a decode loop cannot afford per step.  Such a
// caller has inputs and outputs (they are part of its own pre-planned buffers) but no spare
// scratch to lend.  For it the scratch lives in this library's image: one fixed array per GPU.
// The driver loads a library's device image lazily and allocates the array (and the kernels'
// code) when it does, so radar_create makes that happen for its device - it resolves the array's
// address and loads the two kernels of this path - and the array then stays until the process
// exits.  Create the context BEFORE the host freezes device memory; the calls themselves then
// allocate nothing.
//
// Consequences of that choice, all of which the caller must know:
//   * the array has a fixed size (RADAR_NOALLOC_SCRATCH_BYTES = 1 MiB); a batch / vocabulary whose
//     chunk records do not fit is refused with RADAR_ERR_UNSUPPORTED before anything is launched;
//   * all calls on a device share it.  Two calls whose kernels may overlap on the GPU (different
//     streams, or graphs replayed concurrently) race on it and give undefined results; calls on
//     one stream are safe;
//   * it keeps whatever the previous call left.  Nothing in this path needs zeroed scratch: every
//     record that is read has been written earlier in the same call, so no clearing is done;
//   * in host code the array's name is only a handle.  radar_create looks up the real device
//     address with cudaGetSymbolAddress (with its device current) and caches it per device; a call
//     that finds no cached address (a context made by other means) does the look-up itself, so
//     make the first call outside any stream capture.
// ------------------------------------------------------------------------------------------
#include <mutex>

namespace {
constexpr size_t kNoAllocScratchBytes = 1u << 20;
constexpr int kNoAllocMaxDevices = 64;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];
std::mutex g_noalloc_mutex;
void* g_noalloc_addr[kNoAllocMaxDevices] = {nullptr};      // per device: device address of g_noalloc_scratch
}  // namespace

namespace radar {
int noalloc_prepare_device(int device) {
    if (device < 0 || device >= kNoAllocMaxDevices) return RADAR_OK;       // beyond the table: resolved per call
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_addr[device] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return RADAR_ERR_CUDA;
        g_noalloc_addr[device] = p;
    }
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, greedy_walk_kernel) != cudaSuccess || vocab_pass_preload_argbest() != cudaSuccess)
        return RADAR_ERR_CUDA;
    return RADAR_OK;
}
}  // namespace radar

extern "C" size_t radar_noalloc_scratch_bytes(void) { return kNoAllocScratchBytes; }

extern "C" int radar_verify_accept_greedy_noalloc(radar_ctx* ctx, const radar_accept_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->V <= 0 || a->t_max < 1 || a->N < 1) return RADAR_ERR_INVALID_ARG;
    if (a->mode != RADAR_GREEDY) return RADAR_ERR_UNSUPPORTED;        // the stochastic walk needs 16 * B * V bytes
    if (a->logits_dtype != RADAR_F32 && a->logits_dtype != RADAR_BF16) return RADAR_ERR_UNSUPPORTED;
    // size first: a request that cannot fit is refused whatever else it carries
    int chunk = 0;
    const int n_chunks = vocab_pass_plan_chunks(ctx->sm_count, a->B * kMaxNodes, a->V, &chunk);
    if ((long long)a->B * kMaxNodes > 0x7fffffff / (n_chunks > 0 ? n_chunks : 1)) return RADAR_ERR_UNSUPPORTED;
    if (vocab_pass_partial_bytes(a->B * kMaxNodes, n_chunks, 1) > kNoAllocScratchBytes) return RADAR_ERR_UNSUPPORTED;
    if (!a->target_logits || !a->tree_tok || !a->tree_parent || !a->n_nodes || !a->retrieve || !a->n_leaves ||
        !a->accept_len || !a->path_nodes || !a->path_tokens || !a->next_token || !a->best_retrieve_row)
        return RADAR_ERR_INVALID_ARG;

    int cur = -1;
    RADAR_CUDA_CHECK(cudaGetDevice(&cur));
    if (cur != ctx->device || cur < 0 || cur >= kNoAllocMaxDevices) return RADAR_ERR_INVALID_ARG;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (g_noalloc_addr[cur] == nullptr) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return RADAR_ERR_CUDA;
            g_noalloc_addr[cur] = p;
        }
        scratch = g_noalloc_addr[cur];
    }

    GreedyParams gp;
    gp.a = *a;
    gp.a.workspace = scratch;
    gp.a.workspace_bytes = kNoAllocScratchBytes;
    VocabPassParams& vp = gp.vp;
    vp.logits = a->target_logits;
    vp.dtype = a->logits_dtype;
    vp.row_stride = a->V;
    vp.seq_stride = (int64_t)kMaxNodes * a->V;
    vp.n_seq = a->B;
    vp.F = kMaxNodes;
    vp.V = a->V;
    vp.k = 1;
    vp.n_chunks = n_chunks;
    vp.chunk = chunk;
    vp.want_lse = 0;
    vp.seq_active = nullptr;
    vp.seq_rows = a->n_nodes;
    vp.status = ctx->d_status;
    vocab_pass_carve(scratch, a->B * kMaxNodes, n_chunks, 1, &vp);
    RADAR_CUDA_CHECK(vocab_pass_launch(ctx, RADAR_K_VOCAB_ACCEPT, vp, stream));
    {
        radar_launch_scope scope(ctx, RADAR_K_GREEDY_WALK, stream);
        RADAR_CUDA_CHECK(launch_chained(greedy_walk_kernel, dim3(a->B), dim3(64), 0, stream, gp));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}
