// radar_verify_accept: acceptance of the verified tree.
//   greedy     - vocabulary pass with k = 1 (row argmax, no exponentials) over the target logits of
//                the live tree rows, then one warp per sequence walks the tree with ballots.
//   stochastic - one block per sequence walks the tree lazily: only rows on the accepted path are
//                read.  Probabilities are fp64.  p and q of the current node are cached (normalised)
//                in the workspace; after j rejections the residual pair is, for every token v that has
//                not been proposed yet,  p_j(v) = max(0, p(v) - a_j q(v)) / W_j,  q_j(v) = c_j q(v),
//                and for the token proposed at trial i <= j,  p_j(x_i) = max(0, p(x_i) - a_i q(x_i)) / W_j,
//                q_j(x_i) = 0, with a_{j+1} = a_j + c_j W_j,  c_{j+1} = c_j / (1 - q_j(x_{j+1})) and
//                W_{j+1} = sum_v max(0, p(v) - a(v) q(v)).  This is the rectify / remove / renormalise
//                recursion of Eq. 2 unrolled, so each rejection costs one read-only pass.
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

struct StochParams {
    radar_accept_args a;
    double* p_cache;     // [B][V]
    double* q_cache;     // [B][V]
    int* status;
};

struct BlockRed {
    double* scratch;     // [32] shared
    __device__ double sum(double v) {
        v = warp_sum(v);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
        __syncthreads();
        double t = 0.0;
        for (int w = 0; w < kSThreads / 32; ++w) t += scratch[w];     // same order in every thread
        return t;
    }
    __device__ double max(double v) {
        v = warp_max(v);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
        __syncthreads();
        double t = scratch[0];
        for (int w = 1; w < kSThreads / 32; ++w) t = fmax(t, scratch[w]);
        return t;
    }
};

// cache[v] = softmax(z / T)[v] in fp64; every thread returns after the cache is complete
template <typename T>
__device__ void softmax_to_cache(const T* z, int V, double invT, double* cache, BlockRed& red, bool* nan_seen) {
    double m = -CUDART_INF;
    for (int v = threadIdx.x; v < V; v += kSThreads) {
        const float zf = to_float(z[v]);
        if (zf != zf) *nan_seen = true;
        m = fmax(m, (double)zf * invT);
    }
    m = red.max(m);
    double s = 0.0;
    for (int v = threadIdx.x; v < V; v += kSThreads) {
        const double e = exp((double)to_float(z[v]) * invT - m);
        cache[v] = e;
        s += e;
    }
    s = red.sum(s);
    const double inv = 1.0 / s;
    for (int v = threadIdx.x; v < V; v += kSThreads) cache[v] *= inv;
    __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kSThreads) stochastic_walk_kernel(const StochParams P) {
    const radar_accept_args& a = P.a;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int V = a.V, W = a.t_max + 1;
    __shared__ double s_red[32];
    __shared__ int s_tok[kMaxNodes], s_par[kMaxNodes], s_drow[kMaxNodes], s_child[kMaxNodes];
    __shared__ int s_nchild;
    __shared__ int s_rx[RADAR_MAX_NODES];        // tokens proposed and rejected at the current node
    __shared__ double s_ra[RADAR_MAX_NODES];     // their frozen coefficients a_i
    __shared__ int s_pick, s_last_pos;
    BlockRed red{s_red};

    const int M = min(max(a.n_nodes[b], 1), kMaxNodes);
    if (tid < kMaxNodes) {
        s_tok[tid] = tid < M ? a.tree_tok[(size_t)b * kMaxNodes + tid] : -1;
        s_par[tid] = tid < M ? a.tree_parent[(size_t)b * kMaxNodes + tid] : -2;
        s_drow[tid] = tid < M ? a.tree_draft_row[(size_t)b * kMaxNodes + tid] : -1;
    }
    __syncthreads();

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
    if (tid == 0) { pn[0] = 0; pt[0] = s_tok[0]; }

    int n_rej = 0;           // rejections at the final node (0 => weights are p itself)
    double a_coef = 0.0;
    bool bad_tree = false;
    for (;;) {
        softmax_to_cache<T>(target + (size_t)cur * V, V, invT, pc, red, &nan_seen);
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
        softmax_to_cache<T>(draft + (size_t)drow * V, V, invT, qc, red, &nan_seen);

        double Wn = 1.0, cq = 1.0;
        int accepted = -1;
        for (int ci = 0; ci < nchild; ++ci) {
            const int j = s_child[ci];
            const int x = s_tok[j];
            if (x < 0 || x >= V) { bad_tree = true; break; }
            const double px = pc[x], qx = qc[x];
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
            for (int v = tid; v < V; v += kSThreads) g += fmax(0.0, pc[v] - a_new * qc[v]);
            g = red.sum(g);
            // tokens rejected earlier keep their own coefficient: swap their terms
            for (int r = 0; r < n_rej; ++r) {
                const int xr = s_rx[r];
                g += fmax(0.0, pc[xr] - s_ra[r] * qc[xr]) - fmax(0.0, pc[xr] - a_new * qc[xr]);
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
        if (tid == 0) { pn[len] = cur; pt[len] = s_tok[cur]; }
    }

    // ---- final draw: inverse CDF over w(v) = max(0, p(v) - a(v) q(v)) (or p(v) when nothing was rejected) ----
    const int per = (V + kSThreads - 1) / kSThreads;
    const int v0 = min(tid * per, V), v1 = min(v0 + per, V);
    auto weight = [&](int v) -> double {
        if (n_rej == 0) return pc[v];
        double av = a_coef;
        for (int r = 0; r < n_rej; ++r)
            if (s_rx[r] == v) av = s_ra[r];
        return fmax(0.0, pc[v] - av * qc[v]);
    };
    if (tid == 0) { s_pick = 0x7fffffff; s_last_pos = -1; }
    double seg = 0.0;
    int last_pos = -1;
    for (int v = v0; v < v1; ++v) {
        const double w = weight(v);
        seg += w;
        if (w > 0.0) last_pos = v;
    }
    // scan of seg over threads (fp64).  A thread's end and its successor's start are the same
    // expression, so exactly one thread owns the point u * total.
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
    double woff = 0.0, total = 0.0;
    for (int w = 0; w < kSThreads / 32; ++w) {
        if (w == warp) woff = total;
        total += s_red[w];
    }
    const double start = woff + excl, end = woff + incl;
    const double tgt = (double)a.u_sample[b] * total;
    if (last_pos >= 0) atomicMax(&s_last_pos, last_pos);
    if (start <= tgt && tgt < end) {
        double run = start;
        int pick = last_pos;                                            // rounding guard: the crossing is in here
        for (int v = v0; v < v1; ++v) {
            run += weight(v);
            if (run > tgt) { pick = v; break; }
        }
        atomicMin(&s_pick, pick);
    }
    __syncthreads();
    if (tid == 0) {
        int nt = s_pick != 0x7fffffff ? s_pick : s_last_pos;
        a.next_token[b] = nt;
        a.accept_len[b] = len;
        if (bad_tree) set_status(P.status, RADAR_ERR_TREE);
    }
    if (nan_seen) set_status(P.status, RADAR_ERR_NUMERIC);
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
            greedy_walk_kernel<<<a->B, 64, 0, stream>>>(gp);
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
    {
        radar_launch_scope scope(ctx, RADAR_K_STOCH_WALK, stream);
        if (a->logits_dtype == RADAR_F32) stochastic_walk_kernel<float><<<a->B, kSThreads, 0, stream>>>(sp);
        else stochastic_walk_kernel<__nv_bfloat16><<<a->B, kSThreads, 0, stream>>>(sp);
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
// scratch to lend.  For it the scratch lives in this library's image: one fixed array in device
// memory that exists on every GPU from the moment the library is loaded there until the process
// exits.
//
// Consequences of that choice, all of which the caller must know:
//   * the array has a fixed size (RADAR_NOALLOC_SCRATCH_BYTES = 1 MiB); a batch / vocabulary whose
//     chunk records do not fit is refused with RADAR_ERR_UNSUPPORTED before anything is launched;
//   * all calls on a device share it.  Two calls whose kernels may overlap on the GPU (different
//     streams, or graphs replayed concurrently) race on it and give undefined results; calls on
//     one stream are safe;
//   * it keeps whatever the previous call left.  Nothing in this path needs zeroed scratch: every
//     record that is read has been written earlier in the same call, so no clearing is done;
//   * in host code the array's name is only a handle.  The first call on each device looks up the
//     real device address with cudaGetSymbolAddress (that device must be current) and caches it;
//     make that first call outside any stream capture.
// ------------------------------------------------------------------------------------------
#include <mutex>

namespace {
constexpr size_t kNoAllocScratchBytes = 1u << 20;
constexpr int kNoAllocMaxDevices = 64;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];
std::mutex g_noalloc_mutex;
void* g_noalloc_addr[kNoAllocMaxDevices] = {nullptr};      // per device: device address of g_noalloc_scratch
}  // namespace

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
        greedy_walk_kernel<<<a->B, 64, 0, stream>>>(gp);
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}
