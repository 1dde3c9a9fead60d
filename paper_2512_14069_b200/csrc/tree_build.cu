// radar_rerank_build_tree: one block per sequence finds the n best (score desc, pool index asc) keys of the
// pool (threshold filter + rank count for pools of up to 1024 entries, a shared-memory bitonic network
// beyond), keeps them, compacts them in pool order with a block
// scan and derives parent rows, depths, position ids, ancestor masks, leaves and retrieve rows.
#include "common.cuh"

namespace radar {
namespace {

constexpr int kThreads = 1024;

struct TreeParams {
    radar_tree_args a;
    int* status;
    int n2;              // pool capacity rounded up to a power of two
};

// ascending order of this key == (score descending, pool index ascending); -0 and +0 compare equal
__device__ __forceinline__ unsigned long long sort_key(float score, int idx) {
    unsigned u = __float_as_uint(score == 0.f ? 0.f : score);
    u ^= (u >> 31) ? 0xffffffffu : 0x80000000u;          // monotone map of the float order onto unsigned
    return ((unsigned long long)(~u) << 32) | (unsigned)idx;
}

__global__ void __launch_bounds__(kThreads) rerank_build_tree_kernel(const TreeParams P) {
    chain_wait();
    const radar_tree_args& a = P.a;
    extern __shared__ unsigned char smem_raw[];
    unsigned long long* s_key = reinterpret_cast<unsigned long long*>(smem_raw);        // [n2] sort keys
    float* s_score = reinterpret_cast<float*>(smem_raw + (size_t)(P.n2 + 32) * 8);              // [C]
    short* s_node = reinterpret_cast<short*>(smem_raw + (size_t)(P.n2 + 32) * 8 + (size_t)a.pool_capacity * 4);   // [C] tree row or 0
    __shared__ int s_warp_cnt[kThreads / 32];
    __shared__ int s_parent[kMaxNodes], s_depth[kMaxNodes], s_haschild[kMaxNodes], s_leaf_rank[kMaxNodes];
    __shared__ int s_nleaves;

    const int b = blockIdx.x;
    const int n2_cap = P.n2 + 32;                                          // key array: n2 sort slots + 32 per-warp thresholds
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = a.pool_capacity;
    const size_t pb = (size_t)b * C;
    int L = a.pool_len[b];
    L = max(0, min(L, C));
    int want = a.n_keep != nullptr ? a.n_keep[b] : a.N;
    want = max(0, min(want, a.N));
    const int n_eff = min(min(want, L), kMaxNodes - 1);
    const int M = n_eff + 1;

    for (int i = tid; i < L; i += kThreads) s_score[i] = a.pool_score[pb + i];
    if (tid < kMaxNodes) { s_parent[tid] = -1; s_depth[tid] = 0; s_haschild[tid] = 0; }
    __syncthreads();
    for (int i = tid; i < L; i += kThreads) s_node[i] = 0;
    if (L <= kThreads) {
        // One key per thread, dealt out like cards (lane l of warp w holds pool entry 32 l + w) so that every warp
        // sees all depths of the pool.  With j = ceil(n_eff / 32), the j-th best key of every warp, taken at its
        // worst over the warps, has at least n_eff keys at or before it: those few are ranked by counting.
        // If some warp holds fewer than j entries, every entry is a candidate.
        const int mine = lane * 32 + warp;
        const unsigned long long key = mine < L ? sort_key(s_score[mine], mine) : ~0ull;
        const int jth = (n_eff + 31) / 32;
        unsigned long long cur = key, best = ~0ull;
        if (L / 32 >= jth) {
            for (int r = 0; r < jth; ++r) {
                best = cur;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(kFull, best, o));
                if (cur == best) cur = ~0ull;                              // keys are distinct: one lane leaves
            }
        }
        if (tid == 0) s_nleaves = 0;                                       // reused as the candidate counter
        if (lane == 0) s_key[n2_cap - 32 + warp] = best;                   // tail of the key array: per-warp thresholds
        __syncthreads();
        unsigned long long thr = 0ull;
        for (int w = 0; w < kThreads / 32; ++w) thr = max(thr, s_key[n2_cap - 32 + w]);
        __syncthreads();
        {   // one shared-memory atomic per warp, not per candidate
            const bool cand = mine < L && key <= thr;
            const unsigned m = __ballot_sync(kFull, cand);
            int base = 0;
            if (lane == 0 && m) base = atomicAdd(&s_nleaves, __popc(m));
            base = __shfl_sync(kFull, base, 0);
            if (cand) s_key[base + __popc(m & ((1u << lane) - 1u))] = key;
        }
        __syncthreads();
        const int C = s_nleaves;                                           // <= L <= 1024 - 32 entries are free below the tail
        for (int c = tid; c < C; c += kThreads) {
            const unsigned long long kc = s_key[c];
            int rank = 0;
            for (int j = 0; j < C; ++j) rank += s_key[j] < kc ? 1 : 0;
            if (rank < n_eff) s_node[(int)(kc & 0xffffffffu)] = 1;
        }
        __syncthreads();
    } else {
        // larger pools: bitonic network over the smallest power of two that holds the live entries
        int n2 = 2;
        while (n2 < L) n2 <<= 1;
        for (int i = tid; i < n2; i += kThreads) s_key[i] = i < L ? sort_key(s_score[i], i) : ~0ull;
        __syncthreads();
        for (int size = 2; size <= n2; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int t = tid; t < (n2 >> 1); t += kThreads) {
                    const int lo = ((t & ~(stride - 1)) << 1) | (t & (stride - 1));
                    const int hi = lo | stride;
                    const bool up = (lo & size) == 0;
                    const unsigned long long x = s_key[lo], y = s_key[hi];
                    if ((x > y) == up) { s_key[lo] = y; s_key[hi] = x; }
                }
                __syncthreads();
            }
        }
        for (int p = tid; p < n_eff; p += kThreads) s_node[(int)(s_key[p] & 0xffffffffu)] = 1;
        __syncthreads();
    }

    // each thread owns a contiguous run of pool entries so that the scan keeps pool order
    const int per = (L + kThreads - 1) / kThreads;
    const int i0 = min(tid * per, L), i1 = min(i0 + per, L);
    int kept_cnt = 0;
    for (int i = i0; i < i1; ++i) kept_cnt += s_node[i];
    // exclusive scan of kept_cnt over threads
    int incl = kept_cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp_cnt[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = s_warp_cnt[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(kFull, w, o);
            if (lane >= o) w += v;
        }
        s_warp_cnt[lane] = w;
    }
    __syncthreads();
    int run = incl - kept_cnt + (warp > 0 ? s_warp_cnt[warp - 1] : 0);
    for (int i = i0; i < i1; ++i) {
        if (s_node[i]) { ++run; s_node[i] = (short)run; }       // tree row = 1 + rank in pool order
    }
    __syncthreads();

    // ---- per kept entry: write its row ----
    const size_t tb = (size_t)b * kMaxNodes;
    const int P_b = a.prefix_len[b];
    for (int i = i0; i < i1; ++i) {
        const int row = s_node[i];
        if (row == 0) continue;
        const int pp = a.pool_parent[pb + i];
        int prow = 0;
        if (pp >= 0) {
            prow = (pp < L) ? s_node[pp] : 0;
            if (prow == 0) set_status(P.status, RADAR_ERR_TREE);    // parent pruned: not ancestor-closed
        }
        const int dep = a.pool_depth[pb + i];
        a.tree_tok[tb + row] = a.pool_tok[pb + i];
        a.tree_parent[tb + row] = prow;
        a.tree_depth[tb + row] = dep;
        a.tree_pos[tb + row] = P_b + dep;
        a.tree_pool_idx[tb + row] = i;
        a.tree_score[tb + row] = s_score[i];
        s_parent[row] = prow;
        s_depth[row] = dep;
        s_haschild[prow] = 1;                                      // benign race: same value
        s_leaf_rank[row] = a.pool_draft_row[pb + i];               // parked here until leaves are known
    }
    if (tid == 0) {
        a.tree_tok[tb] = a.root_tok[b];
        a.tree_parent[tb] = -1;
        a.tree_depth[tb] = 0;
        a.tree_pos[tb] = P_b;
        a.tree_pool_idx[tb] = -1;
        a.tree_score[tb] = 0.f;
        s_leaf_rank[0] = 0;                                         // the root's children come from draft row 0
        a.n_nodes[b] = M;
    }
    // padding rows
    for (int r = M + tid; r < kMaxNodes; r += kThreads) {
        a.tree_tok[tb + r] = -1; a.tree_parent[tb + r] = -1; a.tree_depth[tb + r] = 0; a.tree_pos[tb + r] = 0;
        a.tree_pool_idx[tb + r] = -1; a.tree_score[tb + r] = 0.f; a.tree_draft_row[tb + r] = -1;
        a.tree_mask[tb + r] = 0ull;
    }
    __syncthreads();

    // ---- masks, draft rows, leaves ----
    const int W = a.t_max + 1;
    int my_leaf = 0;
    if (tid < kMaxNodes) {
        const int r = tid;
        if (r < M) {
            unsigned long long m = 0ull;
            int j = r, guard = 0;
            while (j >= 0 && guard++ < kMaxNodes) { m |= 1ull << j; j = s_parent[j]; }
            a.tree_mask[tb + r] = m;
            a.tree_draft_row[tb + r] = s_haschild[r] ? s_leaf_rank[r] : -1;
            my_leaf = (!s_haschild[r] && M > 1) ? 1 : 0;
        }
    }
    __syncthreads();                                               // s_leaf_rank is re-used below
    if (tid < kMaxNodes) {
        const unsigned bal = __ballot_sync(kFull, my_leaf != 0);
        if (lane == 0) s_warp_cnt[warp] = __popc(bal);
        const int before = __popc(bal & ((1u << lane) - 1));
        s_leaf_rank[tid] = before;
    }
    __syncthreads();
    if (tid < kMaxNodes && my_leaf) {
        const int l = s_leaf_rank[tid] + (warp == 1 ? s_warp_cnt[0] : 0);
        int32_t* rowp = a.retrieve + ((size_t)b * a.N + l) * W;
        const int dep = s_depth[tid];
        for (int dd = dep + 1; dd < W; ++dd) rowp[dd] = -1;
        int j = tid;
        for (int dd = min(dep, W - 1); dd >= 0 && j >= 0; --dd) { rowp[dd] = j; j = s_parent[j]; }
    }
    if (tid == 0) {
        s_nleaves = s_warp_cnt[0] + s_warp_cnt[1];
        a.n_leaves[b] = s_nleaves;
    }
    __syncthreads();
    const int nl = s_nleaves;
    for (int e = nl * W + tid; e < a.N * W; e += kThreads) a.retrieve[(size_t)b * a.N * W + e] = -1;
}

}  // namespace
}  // namespace radar

using namespace radar;

extern "C" int radar_rerank_build_tree(radar_ctx* ctx, const radar_tree_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->N < 1 || a->t_max < 1 || a->pool_capacity < 1) return RADAR_ERR_INVALID_ARG;
    if (a->N >= RADAR_MAX_NODES || a->pool_capacity > RADAR_MAX_POOL || a->t_max >= 64) return RADAR_ERR_UNSUPPORTED;
    if (!a->pool_tok || !a->pool_parent || !a->pool_depth || !a->pool_draft_row || !a->pool_score || !a->pool_len ||
        !a->root_tok || !a->prefix_len || !a->tree_tok || !a->tree_parent || !a->tree_depth || !a->tree_pos ||
        !a->tree_pool_idx || !a->tree_draft_row || !a->tree_score || !a->tree_mask || !a->n_nodes || !a->retrieve ||
        !a->n_leaves)
        return RADAR_ERR_INVALID_ARG;
    TreeParams p;
    p.a = *a;
    p.status = ctx->d_status;
    p.n2 = 2;
    while (p.n2 < a->pool_capacity) p.n2 <<= 1;
    const size_t smem = (size_t)(p.n2 + 32) * 8 + (size_t)a->pool_capacity * 6;
    RADAR_CUDA_CHECK(radar_opt_in_smem(ctx, RADAR_SMEM_TREE_BUILD, rerank_build_tree_kernel, smem));
    {
        radar_launch_scope scope(ctx, RADAR_K_TREE_BUILD, stream);
        RADAR_CUDA_CHECK(launch_chained(rerank_build_tree_kernel, dim3(a->B), dim3(kThreads), smem, stream, p));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}
