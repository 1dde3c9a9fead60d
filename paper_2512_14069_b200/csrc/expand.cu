// radar_expand_step: vocabulary pass (vocab_pass.cu) followed by one block per sequence that
// merges the chunk partials into each row's top-k and log-normaliser, forms the candidate
// scores, appends them to the pool, selects the k best over all parents and runs the
// prediction model (LSTM cell + MLP head) on their confidence scores.  The block is built for
// latency: everything it reads from global memory is fetched in a few wide, independent batches.
#include "common.cuh"

namespace radar {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kMergeWarps = 16;                      // warps 0..15 merge chunk records, warps 16..31 prepare the gate
constexpr int kMaxF = 32;
constexpr size_t kStageLimit = 96 * 1024;            // chunk records are staged in shared memory up to this size
constexpr int kSurvCap = 256;                        // per-row survivor list of the parallel merge
constexpr int kSelCluster = 4;                       // blocks per sequence when the recurrent product is shared out
constexpr long long kShortPassLogits = 4 << 20;      // ... which is done while a vocabulary pass reads at most this many logits

struct SelectParams {
    radar_expand_args a;
    VocabPassParams vp;
    int* status;
    int staged;                                      // 1: the block's chunk records fit the staging area
    int split;                                       // 1: launched on its own (RADAR_EXPAND_SELECT): the stream predecessor
                                                     //    is not this call's vocabulary pass, so nothing is read before the wait
    const float* feat_pre;                           // hidden-state policy: [B][4H] W_ih f and [B][H] W_1[:, H:] f,
    const float* feat_hid;                           // written by gate_features_kernel
    int cluster;                                     // blocks per sequence: block 0 of a cluster does the work below,
                                                     // the others hold W_hh in shared memory and multiply it by h
};

// Hidden-state policy (Table 3): the input-side products of the prediction model, W_ih f_b (4H rows) and the
// head's columns for the input, W_1[:, H:] f_b (H rows), for every sequence.  One block per output row, one
// warp per 512-element segment of it: every weight is requested at once (the matrix is read at memory speed,
// once), the feature rows come from L1/L2, the segments meet in shared memory.  It needs nothing from the
// vocabulary pass and is launched ahead of it.
constexpr int kFeatSeg = 512;                        // elements of a row per warp: 4 x float4 per lane
__global__ void __launch_bounds__(1024) gate_features_kernel(const radar_expand_args a, float* pre, float* hid) {
    chain_wait();
    const int H = kHidden, lane = threadIdx.x & 31, seg = threadIdx.x >> 5, nseg = blockDim.x >> 5;
    const int r = blockIdx.x;                        // 0 .. 5H-1
    const int d = a.feat_dim;
    __shared__ float s_part[32][8];
    const float* w = r < 4 * H ? a.w_ih + (size_t)r * d : a.w1 + (size_t)(r - 4 * H) * (H + d) + H;
    float4 wv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = seg * kFeatSeg + i * 128 + lane * 4;
        wv[i] = c < d ? __ldg(reinterpret_cast<const float4*>(w + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int b0 = 0; b0 < a.B; b0 += 8) {
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = seg * kFeatSeg + i * 128 + lane * 4;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (c < d && b0 + j < a.B) {
                    const float4 f = __ldg(reinterpret_cast<const float4*>(a.features + (size_t)(b0 + j) * d + c));
                    acc[j] = fmaf(wv[i].x, f.x, fmaf(wv[i].y, f.y, fmaf(wv[i].z, f.z, fmaf(wv[i].w, f.w, acc[j]))));
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float v = warp_sum(acc[j]);
            if (lane == 0) s_part[seg][j] = v;
        }
        __syncthreads();
        if (threadIdx.x < 8 && b0 + (int)threadIdx.x < a.B) {
            float v = 0.f;
            for (int q = 0; q < nseg; ++q) v += s_part[q][threadIdx.x];
            const int b = b0 + threadIdx.x;
            if (r < 4 * H) pre[(size_t)b * 4 * H + r] = v;
            else hid[(size_t)b * H + (r - 4 * H)] = v;
        }
        __syncthreads();
    }
}

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + expf(-x)); }

__device__ __forceinline__ void group_barrier(int id) { asm volatile("bar.sync %0, 512;" ::"r"(id) : "memory"); }
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__host__ __device__ inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

// Thread-block cluster pieces of the select + gate block: stores and barrier arrivals into block 0's shared memory.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f32(const float* local, uint32_t rank, float v) {
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\tst.shared::cluster.f32 [ra], %2;\n\t}" ::"r"(
                     smem_addr(local)), "r"(rank), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(const uint64_t* local, uint32_t rank) {
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\t"
                 "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}" ::"r"(smem_addr(local)), "r"(rank) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(const uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
constexpr int kHelperRows(int n_help) { return (4 * kHidden + n_help - 1) / n_help; }

// (value, index) as one 64-bit word whose unsigned order is the merge's order: a precedes b (larger value, then
// smaller index) exactly if key(a) > key(b).  -0 is folded into +0 first, as the comparison of values does.
__device__ __forceinline__ unsigned long long order_key(float v, int i) {
    uint32_t u = __float_as_uint(v + 0.f);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (uint32_t)(0x7fffffff - i);
}
__device__ __forceinline__ float key_value(unsigned long long key) {
    const uint32_t u = (uint32_t)(key >> 32);
    return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}
__device__ __forceinline__ int key_index(unsigned long long key) { return 0x7fffffff - (int)(uint32_t)key; }

// One block per sequence.  Phase 1 runs two things side by side: warps 0-15 merge the vocabulary pass's
// chunk records into each row's top-k and log-normaliser, warps 16-31 do everything of the prediction
// model that does not depend on this call's candidates (W_hh h + biases, weights into shared memory).
// Phase 2 appends the candidates to the pool and selects the frontier; phase 3 finishes the LSTM cell
// and the MLP head from shared memory only.
template <bool kHelpers>
__global__ void __launch_bounds__(kSelThreads, 1) expand_select_gate_kernel(const SelectParams P) {
    // Launched behind its vocabulary pass in one call, the predecessor is that pass, whose blocks wait for
    // everything before them: the previous call's state (active, h, c, pool_len) is complete when this block
    // starts.  Only the chunk records need the pass itself, so the gate warps never wait for it.
    // Launched on its own (split), the predecessor on the stream is the previous call's select + gate block, or,
    // at call 1, anything at all.  The only thing read before the wait for it are the gate's weights, and only
    // from call 2 on: they may not change during an expansion, and whoever wrote them before call 1 is complete
    // when the block of call 2 starts, because the block of call 1 lets its successor start only after its own
    // wait (the trigger below sits behind the wait in this form).
    if (!P.split) chain_trigger();
    const radar_expand_args& a = P.a;
    const bool early = !P.split || a.t >= 2;           // weights may be fetched before the wait
    const int n_help = kHelpers ? P.cluster - 1 : 0;   // blocks of the cluster that only multiply W_hh by h
    const int b = kHelpers ? blockIdx.x / P.cluster : blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    extern __shared__ __align__(16) unsigned char sel_smem[];
    __shared__ float s_pre[4 * kHidden];
    __shared__ __align__(8) uint64_t s_pre_bar;        // block 0's: counts the helper warps that have delivered
    uint32_t crank = 0;
    if (kHelpers) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));

    if (crank != 0) {
        // ---- helper block: rows [hr0, hr1) of W_hh h + biases, into block 0's s_pre ----
        // The weights are constants: they are in shared memory before the predecessor is done, so that the
        // product costs block 0 no global-memory traffic at all once the state is there.
        const int H = kHidden;
        const int hr0 = ((int)crank - 1) * kHelperRows(n_help), hr1 = min(4 * H, hr0 + kHelperRows(n_help));
        float* s_w = reinterpret_cast<float*>(sel_smem);
        if (early)
            for (int e = tid; e < (hr1 - hr0) * H / 4; e += kSelThreads) cp_async16(s_w + 4 * e, a.w_hh + (size_t)hr0 * H + 4 * e);
        cluster_barrier();                             // block 0 has started and its barrier word is initialised
        if (P.split) { chain_sync(); chain_trigger(); }
        if (!early)
            for (int e = tid; e < (hr1 - hr0) * H / 4; e += kSelThreads) cp_async16(s_w + 4 * e, a.w_hh + (size_t)hr0 * H + 4 * e);
        if (!(a.t > 1 && a.active[b] == 0)) {          // (block 0 takes the same decision and waits for nobody)
            cp_async_wait_all();
            __syncthreads();
            const bool state = a.t > 1;
            const float* hb = a.h + (size_t)b * H + lane * 4;
            const float4 h4 = state ? make_float4(hb[0], hb[1], hb[2], hb[3]) : make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = hr0 + warp; r < hr1; r += kSelWarps) {
                const float4 w = *reinterpret_cast<const float4*>(s_w + (size_t)(r - hr0) * H + lane * 4);
                float acc = w.x * h4.x;                // the same arithmetic, in the same order, as block 0's own loop
                acc = fmaf(w.y, h4.y, acc);
                acc = fmaf(w.z, h4.z, acc);
                acc = fmaf(w.w, h4.w, acc);
                acc = warp_sum(acc);
                if (lane == 0) st_cluster_f32(&s_pre[r], 0, acc + a.b_ih[r] + a.b_hh[r]);
            }
            if (lane == 0) mbar_arrive_cluster(&s_pre_bar, 0);       // release: after this lane's stores
        }
        cp_async_wait_all();
        chain_sync();
        return;
    }
    const int F = a.F, k = a.k, H = kHidden;
    const int n_chunks = P.vp.n_chunks;
    const int per_row = n_chunks * k;
    const bool run_gate = a.t < a.t_max;
    const int policy = a.policy;
    const int kx = policy == RADAR_POLICY_LSTM_HIDDEN ? 0 : k;      // input columns the block itself multiplies

    const size_t stage_elems = P.staged ? (size_t)F * per_row : 0;
    float* st_v = reinterpret_cast<float*>(sel_smem);                              // [F][n_chunks][k] if staged
    int* st_i = reinterpret_cast<int*>(sel_smem + up16(stage_elems * 4));
    float* sv_v = reinterpret_cast<float*>(sel_smem + 2 * up16(stage_elems * 4));   // [kMergeWarps][kSurvCap]
    int* sv_i = reinterpret_cast<int*>(sv_v + kMergeWarps * kSurvCap);
    float* s_wih = reinterpret_cast<float*>(sv_i + kMergeWarps * kSurvCap);         // [4H][k]
    float* s_w1 = s_wih + 4 * H * k;                                                // [H][H + k]

    // The gate's weights are constants: their copies into shared memory are issued before the wait where that is
    // allowed, so that they cross the SM's load path while the predecessor still runs and not beside the merge.
    auto stage_weights = [&]() {
        if (warp < kMergeWarps || !run_gate) return;
        const int gt = tid - kMergeWarps * 32;          // 0..511
        if (policy == RADAR_POLICY_MLP_SCORES) {
            for (int e = gt; e < H * k / 4; e += 512) cp_async16(s_w1 + 4 * e, a.w1 + 4 * e);     // [H][k]
        } else if (policy == RADAR_POLICY_LSTM_HIDDEN) {
            // only the head's columns for the LSTM output; the input columns were applied by gate_features_kernel
            for (int e = gt; e < H * H / 4; e += 512) {
                const int r = e / (H / 4), c4 = e % (H / 4);
                cp_async16(s_w1 + r * H + c4 * 4, a.w1 + (size_t)r * (H + a.feat_dim) + c4 * 4);
            }
        } else {
            for (int e = gt; e < H * k; e += 512) cp_async16(s_wih + 4 * e, a.w_ih + 4 * e);          // 4H*k floats
            for (int e = gt; e < H * (H + k) / 4; e += 512) cp_async16(s_w1 + 4 * e, a.w1 + 4 * e);
        }
    };
    if (early) stage_weights();
    if (n_help > 0) {
        if (tid == 0) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(&s_pre_bar)), "r"(n_help * kSelWarps) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        cluster_barrier();
    }
    if (P.split) { chain_sync(); chain_trigger(); }
    if (!early) stage_weights();
    if (a.t > 1 && a.active[b] == 0) {                 // call 1 always runs: it (re)starts every sequence
        cp_async_wait_all();                           // nothing of this block is in flight when it leaves
        chain_sync();
        if (tid == 0) a.cont[b] = 0;
        return;
    }
    __shared__ double s_cand[kMaxF * RADAR_MAX_K];     // candidate scores, flat (f, j)
    __shared__ int s_ctok[kMaxF * RADAR_MAX_K];
    __shared__ float s_x[RADAR_MAX_K];                 // gate input
    __shared__ __align__(16) float s_h[kHidden];
    __shared__ float s_hn[kHidden], s_hid[kHidden], s_c[kHidden];
    __shared__ float s_b1[kHidden], s_w2[2 * kHidden], s_b2[2];
    __shared__ float s_y[2];
    __shared__ int s_base;
    __shared__ float s_tv[kMergeWarps], s_rv[kMergeWarps][32];
    __shared__ int s_ti[kMergeWarps], s_ri[kMergeWarps][32];

    if (tid == 0) s_base = a.t > 1 ? a.pool_len[b] : 0;
    // previous call's state, needed late: requested now so that nothing waits for it (F * k <= the block's threads)
    const int my_parent = tid < F * k ? a.parent_pool_idx[(size_t)b * F + tid / k] : 0;
    const int forced = a.force_calls != nullptr ? a.force_calls[b] : -1;     // read now, needed at the very end

    if (warp < kMergeWarps) {
        // ---- 1a. chunk records -> shared memory (coalesced), then per row: top-k, log-normaliser, scores ----
        const size_t row0 = (size_t)b * F;
        const float* gv = P.vp.part_v + row0 * per_row;
        const int* gi = P.vp.part_i + row0 * per_row;
        chain_sync();
        if (P.staged) {
            if ((per_row & 3) == 0) {       // rows of records are 16-byte aligned (the partial arrays are 256-byte aligned)
                for (int e = tid; e < F * per_row / 4; e += kMergeWarps * 32) { cp_async16(st_v + 4 * e, gv + 4 * e); cp_async16(st_i + 4 * e, gi + 4 * e); }
            } else {
                for (int e = tid; e < F * per_row; e += kMergeWarps * 32) { cp_async4(st_v + e, gv + e); cp_async4(st_i + e, gi + e); }
            }
            cp_async_wait_all();
            group_barrier(2);
        }
        for (int f = warp; f < F; f += kMergeWarps) {
            const size_t row = row0 + f;
            // log-sum-exp over the chunks in fp64: the first loads are issued here and consumed after the merge
            // (always from a valid address, and not looked at before the merge is done: nothing below waits for them)
            const float pm0_raw = P.vp.part_m[row * n_chunks + min(lane, n_chunks - 1)];
            const float ps0_raw = P.vp.part_s[row * n_chunks + min(lane, n_chunks - 1)];
            const float parent_sc = a.parent_score[(size_t)b * F + f];
            WarpTopList<float> top;
            top.reset();
            bool merged = false;
            if (P.staged) {
                // Parallel merge of the sorted chunk lists.  The k-th best chunk head bounds the row's k-th
                // best from below; what is not after it survives, and survivors are ranked by counting.
                const float* pv = st_v + (size_t)f * per_row;
                const int* pi = st_i + (size_t)f * per_row;
                // survivors as order keys, in the space of this warp's value and index lists
                unsigned long long* lk = reinterpret_cast<unsigned long long*>(sv_v) + warp * kSurvCap;
                if (lane == 0) { s_tv[warp] = -CUDART_INF_F; s_ti[warp] = 0x7fffffff; }
                s_rv[warp][lane] = -CUDART_INF_F;
                s_ri[warp][lane] = 0x7fffffff;
                __syncwarp();
                if (n_chunks <= 32) {
                    // lane c holds the head of chunk c; its rank among the heads by shuffling the heads' order keys
                    // (one 64-bit comparison per pair: the warp's instruction count is what this phase costs)
                    const float hv = lane < n_chunks ? pv[lane * k] : -CUDART_INF_F;
                    const int hi = lane < n_chunks ? pi[lane * k] : 0x7fffffff;
                    const unsigned long long hk = order_key(hv, hi);
                    int rank = 0;
#pragma unroll 4
                    for (int o = 0; o < n_chunks; ++o) rank += __shfl_sync(kFull, hk, o) > hk ? 1 : 0;
                    if (lane < n_chunks && rank == k - 1) { s_tv[warp] = hv; s_ti[warp] = hi; }
                } else {
                    for (int c = lane; c < n_chunks; c += 32) {
                        const float hv = pv[c * k];
                        const int hi = pi[c * k];
                        int rank = 0;
                        for (int o = 0; o < n_chunks; ++o) rank += precedes(pv[o * k], pi[o * k], hv, hi) ? 1 : 0;
                        if (rank == k - 1) { s_tv[warp] = hv; s_ti[warp] = hi; }
                    }
                }
                __syncwarp();
                const float tv = s_tv[warp];
                const int ti = s_ti[warp];
                int total = 0;
                for (int c0 = 0; c0 < n_chunks; c0 += 32) {
                    const int c = c0 + lane;
                    int cnt = 0;
                    if (c < n_chunks)
                        while (cnt < k && !precedes(tv, ti, pv[c * k + cnt], pi[c * k + cnt])) ++cnt;
                    int incl = cnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int v = __shfl_up_sync(kFull, incl, o);
                        if (lane >= o) incl += v;
                    }
                    const int off = total + incl - cnt;
                    for (int e = 0; e < cnt; ++e)
                        if (off + e < kSurvCap) lk[off + e] = order_key(pv[c * k + e], pi[c * k + e]);
                    total += __shfl_sync(kFull, incl, 31);
                }
                __syncwarp();
                if (total <= kSurvCap) {
                    for (int e = lane; e < total; e += 32) {
                        const unsigned long long ck = lk[e];
                        int rank = 0;
#pragma unroll 4
                        for (int j = 0; j < total; ++j) rank += lk[j] > ck ? 1 : 0;
                        if (rank < k) { s_rv[warp][rank] = key_value(ck); s_ri[warp][rank] = key_index(ck); }
                    }
                    __syncwarp();
                    top.v = s_rv[warp][lane];
                    top.i = s_ri[warp][lane];
                    merged = true;
                }
                __syncwarp();
            }
            if (!merged) {
                // serial merge (records too large to stage, or a survivor list that overflowed)
                const float* pv = (P.staged ? st_v : gv) + (size_t)f * per_row;
                const int* pi = (P.staged ? st_i : gi) + (size_t)f * per_row;
                float thr = -CUDART_INF_F;
                int thr_i = 0x7fffffff;
                for (int c = 0; c < n_chunks; ++c) {
                    for (int e = 0; e < k; ++e) {
                        const float cv = pv[c * k + e];
                        const int ci = pi[c * k + e];
                        if (!precedes(cv, ci, thr, thr_i)) break;          // each chunk's list is sorted
                        top.insert(cv, ci);
                        thr = top.value_at(k - 1);
                        thr_i = top.index_at(k - 1);
                    }
                }
            }
            const float pm0 = lane < n_chunks ? pm0_raw : -CUDART_INF_F;
            const float ps0 = lane < n_chunks ? ps0_raw : 0.f;
            float mloc = pm0;
            for (int c = lane + 32; c < n_chunks; c += 32) mloc = fmaxf(mloc, P.vp.part_m[row * n_chunks + c]);
            const float M = warp_max(mloc);
            double sloc = pm0 > -CUDART_INF_F ? (double)ps0 * exp((double)pm0 - (double)M) : 0.0;
            for (int c = lane + 32; c < n_chunks; c += 32) {
                const float mc = P.vp.part_m[row * n_chunks + c];
                if (mc > -CUDART_INF_F) sloc += (double)P.vp.part_s[row * n_chunks + c] * exp((double)mc - (double)M);
            }
            const double S = warp_sum(sloc);
            const double lse = (double)M + log(S);
            if (lane < k) {
                const double logp = (double)top.v - lse;
                const double sc = (double)parent_sc + logp;
                a.topk_tok[row * k + lane] = top.i;
                a.topk_logp[row * k + lane] = (float)logp;
                s_cand[f * k + lane] = sc;
                s_ctok[f * k + lane] = top.i;
            }
        }
    } else if (run_gate) {
        // ---- 1b. the part of the prediction model that only needs the previous state ----
        const int gt = tid - kMergeWarps * 32;          // 0..511
        const int gw = warp - kMergeWarps;              // 0..15
        if (gt < H) {
            const bool state = a.t > 1 && policy != RADAR_POLICY_MLP_SCORES;
            s_h[gt] = state ? a.h[(size_t)b * H + gt] : 0.f;
            s_c[gt] = state ? a.c[(size_t)b * H + gt] : 0.f;
        }
        group_barrier(3);
        const float4 h4 = *reinterpret_cast<const float4*>(&s_h[lane * 4]);
        constexpr int kBatch = 8;
        for (int r0 = gw * 32; n_help == 0 && policy != RADAR_POLICY_MLP_SCORES && r0 < gw * 32 + 32; r0 += kBatch) {
            float4 w[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                w[i] = __ldg(reinterpret_cast<const float4*>(a.w_hh + (size_t)(r0 + i) * H) + lane);
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                float acc = w[i].x * h4.x;
                acc = fmaf(w[i].y, h4.y, acc);
                acc = fmaf(w[i].z, h4.z, acc);
                acc = fmaf(w[i].w, h4.w, acc);
                acc = warp_sum(acc);
                if (lane == 0) s_pre[r0 + i] = acc + a.b_ih[r0 + i] + a.b_hh[r0 + i];
            }
        }
        if (gt < H) s_b1[gt] = a.b1[gt];
        if (gt < 2 * H) s_w2[gt] = a.w2[gt];
        if (gt < 2) s_b2[gt] = a.b2[gt];
        cp_async_wait_all();
        if (n_help > 0 && gt == 0) {                   // the helpers' rows of s_pre; the barrier below publishes them
            bool ok = false;
            for (uint32_t it = 0; it < (1u << 22) && !(ok = mbar_try_wait_cluster(&s_pre_bar, 0)); ++it) {}
            if (!ok) set_status(P.status, RADAR_ERR_TIMEOUT);
        }
    }
    __syncthreads();
    const int base = s_base;
    const int n_cand = F * k;
    if (base + n_cand > a.pool_capacity) {             // never write past the pool
        if (tid == 0) { set_status(P.status, RADAR_ERR_INVALID_ARG); a.cont[b] = 0; a.active[b] = 0; }
        return;
    }

    // ---- 2. append every candidate to the pool ----
    const size_t pb = (size_t)b * a.pool_capacity + base;
    static_assert(kMaxF * RADAR_MAX_K <= kSelThreads, "one candidate per thread");
    if (tid < n_cand) {
        const int e = tid;
        a.pool_tok[pb + e] = s_ctok[e];
        a.pool_parent[pb + e] = my_parent;
        a.pool_score[pb + e] = (float)s_cand[e];
        a.pool_depth[pb + e] = a.t;
    }                     // (its draft row is written below, by the thread that knows whether it survives)

    // ---- 3. the k best candidates over all parents (score desc, flat index asc) ----
    // eight threads share a candidate's rank count (n_cand <= 1024: at most 8 rounds)
    for (int e0 = 0; e0 < n_cand; e0 += kSelThreads / 8) {
        const int e = e0 + (tid >> 3), part = tid & 7;
        const bool have = e < n_cand;
        const double v = have ? s_cand[e] : 0.0;
        int rank = 0;
        if (have)
            for (int j = part; j < n_cand; j += 8) rank += precedes(s_cand[j], j, v, e) ? 1 : 0;
        rank += __shfl_xor_sync(kFull, rank, 1);
        rank += __shfl_xor_sync(kFull, rank, 2);
        rank += __shfl_xor_sync(kFull, rank, 4);
        if (have && part == 0) a.pool_draft_row[pb + e] = rank < k ? 1 + (a.t - 1) * k + rank : -1;
        if (have && part == 0 && rank < k) {
            const float sc = (float)v;
            const size_t o = (size_t)b * k + rank;
            a.frontier_tok[o] = s_ctok[e];
            a.frontier_score[o] = sc;
            a.frontier_pool_idx[o] = base + e;
            a.frontier_src_row[o] = e / k;
            s_x[rank] = expf(sc);                                // confidence score in [0,1]
        }
    }
    if (tid == 0) a.pool_len[b] = base + n_cand;
    __syncthreads();

    // ---- 4. prediction model, from shared memory ----
    bool cont = false;
    if (run_gate && policy == RADAR_POLICY_MLP_SCORES) {
        if (tid < H) {
            float acc = s_b1[tid];
            const float* w = s_w1 + tid * k;
            for (int j = 0; j < k; ++j) acc = fmaf(w[j], s_x[j], acc);
            s_hid[tid] = fmaxf(acc, 0.f);
        }
        __syncthreads();
        if (warp < 2) {
            float acc = 0.f;
            for (int c = lane; c < H; c += 32) acc = fmaf(s_w2[warp * H + c], s_hid[c], acc);
            acc = warp_sum(acc);
            if (lane == 0) s_y[warp] = acc + s_b2[warp];
        }
        __syncthreads();
        cont = s_y[1] > s_y[0];
        if (tid < 2) a.gate_logits[(size_t)b * 2 + tid] = s_y[tid];
        if (forced >= 0) cont = a.t < forced;
    } else if (run_gate) {
        if (tid < 4 * H) {
            float acc = s_pre[tid];
            if (policy == RADAR_POLICY_LSTM_HIDDEN) {
                acc += P.feat_pre[(size_t)b * 4 * H + tid];
            } else {
                const float* w = s_wih + tid * k;
#pragma unroll 4                                       // the loads of four terms at once, the sum in the order of before
                for (int j = 0; j < k; ++j) acc = fmaf(w[j], s_x[j], acc);
            }
            s_pre[tid] = acc;
        }
        __syncthreads();
        if (tid < H) {
            const float ig = sigmoidf_(s_pre[tid]);
            const float fg = sigmoidf_(s_pre[H + tid]);
            const float gg = tanhf(s_pre[2 * H + tid]);
            const float og = sigmoidf_(s_pre[3 * H + tid]);
            const float cn = fg * s_c[tid] + ig * gg;
            const float hn = og * tanhf(cn);
            a.c[(size_t)b * H + tid] = cn;
            a.h[(size_t)b * H + tid] = hn;
            s_hn[tid] = hn;
        }
        __syncthreads();
        {
            // a warp's four rows side by side: the inputs are read once and the four reductions run interleaved
            static_assert(kHidden == 4 * kSelWarps, "four rows of the hidden layer per warp");
            const float hv[4] = {s_hn[lane], s_hn[lane + 32], s_hn[lane + 64], s_hn[lane + 96]};
            const float xv = lane < kx ? s_x[lane] : 0.f;
            float acc[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float* w = s_w1 + (warp + i * kSelWarps) * (H + kx);
                float t = w[lane] * hv[0];
                t = fmaf(w[lane + 32], hv[1], t);
                t = fmaf(w[lane + 64], hv[2], t);
                t = fmaf(w[lane + 96], hv[3], t);
                if (lane < kx) t = fmaf(w[H + lane], xv, t);
                acc[i] = t;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i] += __shfl_xor_sync(kFull, acc[i], o);
            }
            if (lane < 4) {
                const int r = warp + lane * kSelWarps;
                const float v = lane == 0 ? acc[0] : lane == 1 ? acc[1] : lane == 2 ? acc[2] : acc[3];
                s_hid[r] = fmaxf(v + s_b1[r] + (policy == RADAR_POLICY_LSTM_HIDDEN ? P.feat_hid[(size_t)b * H + r] : 0.f), 0.f);
            }
        }
        __syncthreads();
        if (warp == 0) {                               // both logits in one warp: nothing else has to wait for them
            float y0 = 0.f, y1 = 0.f;
            for (int c = lane; c < H; c += 32) {
                y0 = fmaf(s_w2[c], s_hid[c], y0);
                y1 = fmaf(s_w2[H + c], s_hid[c], y1);
            }
            y0 = warp_sum(y0) + s_b2[0];
            y1 = warp_sum(y1) + s_b2[1];
            cont = y1 > y0;
            if (lane < 2) a.gate_logits[(size_t)b * 2 + lane] = lane == 0 ? y0 : y1;
        }
        if (forced >= 0) cont = a.t < forced;
    } else {
        if (tid < 2) a.gate_logits[(size_t)b * 2 + tid] = 0.f;
    }
    if (tid == 0) {
        a.cont[b] = cont ? 1 : 0;
        a.active[b] = cont ? 1 : 0;
    }
}

}  // namespace
}  // namespace radar

using namespace radar;

extern "C" size_t radar_expand_workspace_bytes(const radar_ctx* ctx, int B, int F, int V, int k) {
    if (!ctx || B <= 0 || F <= 0 || V <= 0 || k <= 0) return 0;
    int chunk;
    const int n_chunks = vocab_pass_plan_chunks(ctx->sm_count, B * F, V, &chunk);
    return align_up(vocab_pass_partial_bytes(B * F, n_chunks, k), 256) + (size_t)B * 5 * kHidden * sizeof(float);
}

extern "C" int radar_expand_step(radar_ctx* ctx, const radar_expand_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->F <= 0 || a->V <= 0 || a->k <= 0 || a->t < 1 || a->t > a->t_max) return RADAR_ERR_INVALID_ARG;
    if (a->k > RADAR_MAX_K || a->F > kMaxF || a->V < a->k) return RADAR_ERR_UNSUPPORTED;
    if (a->logits_dtype != RADAR_F32 && a->logits_dtype != RADAR_BF16) return RADAR_ERR_UNSUPPORTED;
    if (a->logits_row_stride < a->V) return RADAR_ERR_INVALID_ARG;
    if (a->phase != RADAR_EXPAND_ALL && a->phase != RADAR_EXPAND_VOCAB && a->phase != RADAR_EXPAND_SELECT) return RADAR_ERR_INVALID_ARG;
    if (!a->logits || !a->parent_score || !a->parent_pool_idx || (!a->active && a->phase != RADAR_EXPAND_VOCAB) || !a->h || !a->c || !a->pool_tok ||
        !a->pool_parent || !a->pool_depth || !a->pool_draft_row || !a->pool_score || !a->pool_len ||
        !a->frontier_tok || !a->frontier_score || !a->frontier_pool_idx || !a->frontier_src_row || !a->topk_tok ||
        !a->topk_logp || !a->gate_logits || !a->cont || !a->workspace)
        return RADAR_ERR_INVALID_ARG;
    if (a->policy != RADAR_POLICY_LSTM_SCORES && a->policy != RADAR_POLICY_MLP_SCORES && a->policy != RADAR_POLICY_LSTM_HIDDEN)
        return RADAR_ERR_INVALID_ARG;
    const bool gate_runs = a->t < a->t_max;
    if (gate_runs && (!a->w1 || !a->b1 || !a->w2 || !a->b2 || (reinterpret_cast<uintptr_t>(a->w1) & 15) != 0))
        return RADAR_ERR_INVALID_ARG;
    if (gate_runs && a->policy != RADAR_POLICY_MLP_SCORES &&
        (!a->w_ih || !a->w_hh || !a->b_ih || !a->b_hh ||
         ((reinterpret_cast<uintptr_t>(a->w_hh) | reinterpret_cast<uintptr_t>(a->w_ih)) & 15) != 0))
        return RADAR_ERR_INVALID_ARG;
    if (gate_runs && a->policy == RADAR_POLICY_LSTM_HIDDEN &&
        (!a->features || a->feat_dim < 4 || a->feat_dim > 16384 || (a->feat_dim & 3) != 0 ||
         (reinterpret_cast<uintptr_t>(a->features) & 15) != 0))
        return RADAR_ERR_INVALID_ARG;
    if (a->pool_capacity < a->F * a->k) return RADAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->workspace) & 255) != 0) return RADAR_ERR_WORKSPACE;

    SelectParams sp;
    sp.a = *a;
    sp.status = ctx->d_status;
    VocabPassParams& vp = sp.vp;
    vp.logits = a->logits;
    vp.dtype = a->logits_dtype;
    vp.row_stride = a->logits_row_stride;
    vp.seq_stride = a->logits_seq_stride;
    vp.n_seq = a->B;
    vp.F = a->F;
    vp.V = a->V;
    vp.k = a->k;
    vp.n_chunks = vocab_pass_plan_chunks(ctx->sm_count, a->B * a->F, a->V, &vp.chunk);
    vp.want_lse = 1;
    vp.seq_active = a->t > 1 ? a->active : nullptr;          // RADAR_EXPAND_VOCAB: the caller's (possibly older) mask, or NULL
    vp.seq_rows = nullptr;
    vp.status = ctx->d_status;
    const size_t part_bytes = align_up(vocab_pass_partial_bytes(a->B * a->F, vp.n_chunks, a->k), 256);
    if (part_bytes + (size_t)a->B * 5 * kHidden * sizeof(float) > a->workspace_bytes) return RADAR_ERR_WORKSPACE;
    vocab_pass_carve(a->workspace, a->B * a->F, vp.n_chunks, a->k, &vp);
    float* feat_pre = reinterpret_cast<float*>(reinterpret_cast<char*>(a->workspace) + part_bytes);
    sp.feat_pre = feat_pre;
    sp.feat_hid = feat_pre + (size_t)a->B * 4 * kHidden;
    if (gate_runs && a->policy == RADAR_POLICY_LSTM_HIDDEN && a->phase != RADAR_EXPAND_SELECT) {
        radar_launch_scope scope(ctx, RADAR_K_GATE_FEATURES, stream);
        const int nseg = (a->feat_dim + kFeatSeg - 1) / kFeatSeg;
        RADAR_CUDA_CHECK(launch_chained(gate_features_kernel, dim3(5 * kHidden), dim3(nseg * 32), 0, stream, *a, feat_pre,
                                        feat_pre + (size_t)a->B * 4 * kHidden));
    }

    if (a->phase != RADAR_EXPAND_SELECT) RADAR_CUDA_CHECK(vocab_pass_launch(ctx, RADAR_K_VOCAB_EXPAND, vp, stream));
    if (a->phase == RADAR_EXPAND_VOCAB) return RADAR_OK;
    sp.split = a->phase == RADAR_EXPAND_SELECT ? 1 : 0;
    // The chunk records are staged in shared memory only if they fit next to the survivor lists and the gate
    // weights inside the 227 KB a block may have; otherwise the merge reads them from global memory.
    const size_t stage_bytes = (size_t)a->F * vp.n_chunks * a->k * 8;
    const size_t fixed_smem = (size_t)kMergeWarps * kSurvCap * 8 +
                              sizeof(float) * ((size_t)4 * kHidden * a->k + (size_t)kHidden * (kHidden + a->k));
    sp.staged = stage_bytes <= kStageLimit && 2 * up16(stage_bytes / 2) + fixed_smem <= 227 * 1024 ? 1 : 0;
    const size_t smem = 2 * up16(sp.staged ? stage_bytes / 2 : 0) + fixed_smem;
    // Blocks per sequence.  With a recurrent policy, three more blocks per sequence hold W_hh (256 KB, more than
    // one block has room for) in their shared memory, loaded while the predecessor still runs, and deliver
    // W_hh h + biases into block 0: the block then streams none of it after the wait (measured: 1.3 us less per
    // draft call at B = 1 and B = 4).  That pays while the draft calls are a chain of short, latency-bound
    // kernels.  Once the next call's vocabulary pass, which shares the device with this kernel, is long enough
    // to be the slower of the two, the waiting helper blocks only take SMs from it (B = 8, V = 128256: 0.8 us
    // MORE per call), so larger passes keep one block per sequence.
    const bool recurrent = gate_runs && a->policy != RADAR_POLICY_MLP_SCORES;
    const size_t helper_bytes = (size_t)kHelperRows(kSelCluster - 1) * kHidden * sizeof(float);
    const bool short_pass = (long long)a->B * a->k * a->V <= kShortPassLogits;
    sp.cluster = recurrent && short_pass && a->B * kSelCluster * 2 <= ctx->sm_count && smem >= helper_bytes ? kSelCluster : 1;
    {
        radar_launch_scope scope(ctx, RADAR_K_SELECT_GATE, stream);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(a->B * sp.cluster));
        cfg.blockDim = dim3(kSelThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)sp.cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = sp.cluster > 1 ? 2 : 1;
        if (sp.cluster > 1) {
            RADAR_CUDA_CHECK(radar_opt_in_smem(ctx, RADAR_SMEM_SELECT_GATE_CLUSTER, expand_select_gate_kernel<true>, smem));
            RADAR_CUDA_CHECK(cudaLaunchKernelEx(&cfg, expand_select_gate_kernel<true>, sp));
        } else {
            RADAR_CUDA_CHECK(radar_opt_in_smem(ctx, RADAR_SMEM_SELECT_GATE, expand_select_gate_kernel<false>, smem));
            RADAR_CUDA_CHECK(cudaLaunchKernelEx(&cfg, expand_select_gate_kernel<false>, sp));
        }
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}
