// Vocabulary pass: one coalesced, vectorised read of every logits row produces, per
// (row, chunk), the chunk's k best (logit, token) pairs and its (max, sum exp) pair.
//
// The pass is HBM-bound, so each logit is read exactly once, with 16-byte streaming loads, and a
// block keeps its whole chunk (16 or 32 values per thread) in registers: every load of the chunk is
// in flight at once, and nothing is re-read from memory for the selection.  Selection is a filter,
// not a running list: with j = ceil(k / 8), the j-th largest of each warp's 32 per-thread maxima, taken
// at its lowest over the 8 warps, is a lower bound of the chunk's k-th best value; the few
// values that reach it go to a shared-memory candidate list, and their exact ranks by
// (logit desc, token asc) are counted there.  If an adversarial chunk overflows the list, k rounds
// of a block-wide arg-best over the registers give the same result.
#include "common.cuh"

namespace radar {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCandCap = 1024;
constexpr int kEmptyIdx = 0x40000000;          // empty slots sort after every real token id

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float (&out)[4]) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(p));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&out)[8]) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            out[2 * j] = __uint_as_float(w[j] << 16);
            out[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float max_nan(float a, float b) {
    float y;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
    return y;
}

// best (value desc, index asc) pair over the warp, in every lane
__device__ __forceinline__ void warp_best(float& v, int& i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(kFull, v, o);
        const int oi = __shfl_xor_sync(kFull, i, o);
        if (precedes(ov, oi, v, i)) { v = ov; i = oi; }
    }
}

// EPT = values per thread kept in registers (a multiple of the vector width), chunk = kThreads * EPT
template <typename T, int EPT, bool WANT_LSE>
__global__ void __launch_bounds__(kThreads, WANT_LSE ? (EPT == 32 ? 5 : 6) : 5) vocab_pass_kernel(const VocabPassParams p) {
    chain_wait();
    using VT = Vec<T>;
    constexpr int N = VT::N;
    constexpr int NV = EPT / N;
    // grid = (chunks, rows of a sequence, sequences): no division on the way to the block's data
    const int chunk_id = blockIdx.x, f = blockIdx.y, seq = blockIdx.z;
    const int row = seq * p.F + f;
    if (p.seq_active != nullptr && p.seq_active[seq] == 0) return;
    if (p.seq_rows != nullptr && f >= p.seq_rows[seq]) return;

    const T* base = reinterpret_cast<const T*>(p.logits) + (int64_t)seq * p.seq_stride + (int64_t)f * p.row_stride;
    const int e0 = min(chunk_id * p.chunk, p.V);
    const int e1 = min(e0 + p.chunk, p.V);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k = p.k;

    // scalar head up to the first 16-byte boundary, vector body, scalar tail
    const uintptr_t addr = reinterpret_cast<uintptr_t>(base + e0);
    int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
    head = min(head, e1 - e0);
    const int body0 = e0 + head;
    const int nvec = (e1 - body0) / N;             // <= kThreads * NV because chunk == kThreads * EPT
    const int tail0 = body0 + nvec * N;
    const int ntail = e1 - tail0;

    // ---- every load of the chunk in flight ----
    float x[NV][N];
    const T* vbase = base + body0;
    if (head == 0 && nvec == kThreads * NV) {        // a whole, aligned chunk (all but a row's last one): nothing to check
        const T* vp = vbase + (int64_t)tid * N;
#pragma unroll
        for (int u = 0; u < NV; ++u) VT::load(vp + (int64_t)u * (kThreads * N), x[u]);
    } else {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int j = tid + u * kThreads;
            if (j < nvec) {
                VT::load(vbase + (int64_t)j * N, x[u]);
            } else {
#pragma unroll
                for (int e = 0; e < N; ++e) x[u][e] = -CUDART_INF_F;
            }
        }
    }
    // head and tail (each shorter than one vector): one value for threads 0..N-1 and N..2N-1
    float xs = -CUDART_INF_F;
    int xs_idx = -1;
    if (tid < head) xs_idx = e0 + tid;
    else if (tid >= N && tid - N < ntail) xs_idx = tail0 + tid - N;
    if (xs_idx >= 0) xs = to_float(base[xs_idx]);

    // ---- per-thread max (NaN-propagating) ----
    float mxa[4] = {xs, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int u = 0; u < NV; ++u)
#pragma unroll
        for (int e = 0; e < N; ++e) mxa[e & 3] = max_nan(mxa[e & 3], x[u][e]);
    const float bv = max_nan(max_nan(mxa[0], mxa[1]), max_nan(mxa[2], mxa[3]));
    const bool nan = bv != bv;
    float ssum = 0.f;
    if (WANT_LSE) {
        if (bv > -CUDART_INF_F) {
            const float mb = bv * 1.4426950408889634f;
#pragma unroll
            for (int u = 0; u < NV; ++u)
#pragma unroll
                for (int e = 0; e < N; ++e) ssum += fast_exp2(fmaf(x[u][e], 1.4426950408889634f, -mb));
            if (xs_idx >= 0) ssum += fast_exp2(fmaf(xs, 1.4426950408889634f, -mb));
        }
    }

    __shared__ float sh_m[kWarps], sh_s[kWarps];
    __shared__ float sh_tv[kWarps];
    __shared__ int sh_ti[kWarps];
    __shared__ int sh_nan, sh_cnt;
    __shared__ float sh_cv[kCandCap];
    __shared__ int sh_ci[kCandCap];
    if (tid == 0) { sh_nan = 0; sh_cnt = 0; }

    const size_t rec = (size_t)row * p.n_chunks + chunk_id;
    if (WANT_LSE) {
        const float wm = warp_max(bv);
        const float ws = warp_sum(wm > -CUDART_INF_F ? ssum * __expf(bv - wm) : 0.f);
        if (lane == 0) { sh_m[warp] = wm; sh_s[warp] = ws; }
    }

    if (!WANT_LSE || k == 1) {
        // ---- arg-best only (the pass without the normaliser is always run with k = 1) ----
        // lowest index that holds the thread's max (index order: head scalar < vector elements < tail scalar)
        int bi = kEmptyIdx + tid;
        if (xs_idx >= 0 && tid >= N && xs == bv) bi = xs_idx;
#pragma unroll
        for (int u = NV - 1; u >= 0; --u) {
            const int idx0 = body0 + (tid + u * kThreads) * N;
            if (tid + u * kThreads < nvec) {
#pragma unroll
                for (int e = N - 1; e >= 0; --e)
                    if (x[u][e] == bv) bi = idx0 + e;
            }
        }
        if (xs_idx >= 0 && tid < N && xs == bv) bi = xs_idx;
        float wv = bv;
        int wi = bi;
        warp_best(wv, wi);
        if (lane == 0) { sh_tv[warp] = wv; sh_ti[warp] = wi; }
        __syncthreads();
        if (nan) atomicOr(&sh_nan, 1);
        __syncthreads();
        if (warp == 0) {
            float v = lane < kWarps ? sh_tv[lane] : -CUDART_INF_F;
            int i = lane < kWarps ? sh_ti[lane] : 0x7fffffff;
            warp_best(v, i);
            if (lane == 0) {
                p.part_v[rec] = v;
                p.part_i[rec] = i >= kEmptyIdx ? 0x7fffffff : i;
            }
        }
    } else {
        // ---- threshold: the j-th largest per-thread max of every warp (with multiplicity), j = ceil(k / warps);
        //      the smallest of these over the warps has at least k elements of the chunk at or above it ----
        {
            const int jth = (k + kWarps - 1) / kWarps;
            float cv = bv, wv = bv;
            for (int r = 0; r < jth; ++r) {
                wv = warp_max(cv);
                const unsigned who = __ballot_sync(kFull, cv == wv);
                if (lane == __ffs(who) - 1) cv = -CUDART_INF_F;                // one holder of the max leaves
            }
            if (lane == 0) sh_tv[warp] = wv;
        }
        __syncthreads();
        if (nan) atomicOr(&sh_nan, 1);
        float tv = sh_tv[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) tv = fminf(tv, sh_tv[w]);
        // ---- candidates: every element at or above the threshold value.  One bit per register value; the few
        //      that qualify are re-read from memory by position, so no register is indexed dynamically ----
        unsigned mask = 0;
#pragma unroll
        for (int u = 0; u < NV; ++u)
#pragma unroll
            for (int e = 0; e < N; ++e) mask |= (x[u][e] >= tv ? 1u : 0u) << (u * N + e);
        if (xs_idx >= 0 && xs >= tv) {
            const int slot = atomicAdd(&sh_cnt, 1);
            if (slot < kCandCap) { sh_cv[slot] = xs; sh_ci[slot] = xs_idx; }
        }
        while (mask) {
            const int bit = __ffs(mask) - 1;
            mask &= mask - 1;
            const int j = tid + (bit / N) * kThreads;
            if (j < nvec) {                                                     // padding of a short chunk is not an element
                const int idx = body0 + j * N + bit % N;
                const int slot = atomicAdd(&sh_cnt, 1);
                if (slot < kCandCap) { sh_cv[slot] = to_float(base[idx]); sh_ci[slot] = idx; }
            }
        }
        __syncthreads();
        const int C = sh_cnt;
        float* out_v = p.part_v + rec * k;
        int32_t* out_i = p.part_i + rec * k;
        if (C <= kCandCap) {
            for (int c = tid; c < C; c += kThreads) {
                const float cv = sh_cv[c];
                const int ci = sh_ci[c];
                int rank = 0;
                for (int j = 0; j < C; ++j) rank += precedes(sh_cv[j], sh_ci[j], cv, ci) ? 1 : 0;
                if (rank < k) { out_v[rank] = cv; out_i[rank] = ci; }
            }
            for (int r = C + tid; r < k; r += kThreads) { out_v[r] = -CUDART_INF_F; out_i[r] = 0x7fffffff; }
        } else {
            // ---- exact fallback: k rounds of a block-wide arg-best over the registers ----
            float pv = CUDART_INF_F;                   // previous winner: everything real comes after it
            int pi = -1;
            for (int r = 0; r < k; ++r) {
                float cv = -CUDART_INF_F;
                int ci = 0x7fffffff;
                auto offer = [&](float v, int idx) {
                    if (precedes(pv, pi, v, idx) && precedes(v, idx, cv, ci)) { cv = v; ci = idx; }
                };
#pragma unroll
                for (int u = 0; u < NV; ++u) {
                    const int idx0 = body0 + (tid + u * kThreads) * N;
                    if (tid + u * kThreads < nvec) {
#pragma unroll
                        for (int e = 0; e < N; ++e) offer(x[u][e], idx0 + e);
                    }
                }
                if (xs_idx >= 0) offer(xs, xs_idx);
                warp_best(cv, ci);
                __syncthreads();                        // previous round's readers are done
                if (lane == 0) { sh_tv[warp] = cv; sh_ti[warp] = ci; }
                __syncthreads();
                cv = sh_tv[0];
                ci = sh_ti[0];
#pragma unroll
                for (int w = 1; w < kWarps; ++w)
                    if (precedes(sh_tv[w], sh_ti[w], cv, ci)) { cv = sh_tv[w]; ci = sh_ti[w]; }
                if (tid == 0) { out_v[r] = cv; out_i[r] = ci; }
                pv = cv;
                pi = ci;
            }
        }
    }

    if (WANT_LSE && tid == 0) {
        float M = sh_m[0];
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, sh_m[w]);
        float S = 0.f;
        if (M > -CUDART_INF_F)
            for (int w = 0; w < kWarps; ++w) S += sh_s[w] * __expf(sh_m[w] - M);
        p.part_m[rec] = M;
        p.part_s[rec] = S;
    }
    if (tid == 0 && sh_nan) set_status(p.status, RADAR_ERR_NUMERIC);
}

template <typename T, bool WANT_LSE>
cudaError_t launch_ept(const VocabPassParams& p, dim3 grid, cudaStream_t stream) {
    if (p.chunk / kThreads == 16) return launch_chained(vocab_pass_kernel<T, 16, WANT_LSE>, grid, dim3(kThreads), 0, stream, p);
    return launch_chained(vocab_pass_kernel<T, 32, WANT_LSE>, grid, dim3(kThreads), 0, stream, p);
}

}  // namespace

// chunk is 8192 values (32 per thread, five blocks per SM), or 4096 (16 per thread, six blocks) when
// the larger one would leave SMs without work
int vocab_pass_plan_chunks(int sm_count, int rows, int V, int* chunk_out) {
    int chunk = 8192;
    if ((long long)rows * ((V + chunk - 1) / chunk) < 5LL * sm_count) chunk = 4096;
    *chunk_out = chunk;
    return (V + chunk - 1) / chunk;
}

size_t vocab_pass_partial_bytes(int rows, int n_chunks, int k) {
    const size_t rec = (size_t)rows * n_chunks;
    return align_up(rec * k * 4, 256) * 2 + align_up(rec * 4, 256) * 2;
}

void vocab_pass_carve(void* ws, int rows, int n_chunks, int k, VocabPassParams* p) {
    const size_t rec = (size_t)rows * n_chunks;
    char* c = reinterpret_cast<char*>(ws);
    p->part_v = reinterpret_cast<float*>(c); c += align_up(rec * k * 4, 256);
    p->part_i = reinterpret_cast<int32_t*>(c); c += align_up(rec * k * 4, 256);
    p->part_m = reinterpret_cast<float*>(c); c += align_up(rec * 4, 256);
    p->part_s = reinterpret_cast<float*>(c);
}

// Makes the driver load the arg-best instantiations on the current device (kernel images are loaded lazily, at
// first use, and loading allocates): a caller that must not allocate later can have it done at set-up.
cudaError_t vocab_pass_preload_argbest() {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, vocab_pass_kernel<float, 16, false>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, vocab_pass_kernel<float, 32, false>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, vocab_pass_kernel<__nv_bfloat16, 16, false>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, vocab_pass_kernel<__nv_bfloat16, 32, false>);
    return e;
}

cudaError_t vocab_pass_launch(radar_ctx* ctx, int kernel_id, const VocabPassParams& p, cudaStream_t stream) {
    if (p.n_seq <= 0 || p.F <= 0 || p.n_chunks <= 0) return cudaSuccess;
    if (p.n_seq > 65535 || p.F > 65535) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)p.n_chunks, (unsigned)p.F, (unsigned)p.n_seq);
    if (!p.want_lse && p.k != 1) return cudaErrorInvalidValue;
    radar_launch_scope scope(ctx, kernel_id, stream);
    if (p.dtype == RADAR_F32) return p.want_lse ? launch_ept<float, true>(p, grid, stream) : launch_ept<float, false>(p, grid, stream);
    return p.want_lse ? launch_ept<__nv_bfloat16, true>(p, grid, stream) : launch_ept<__nv_bfloat16, false>(p, grid, stream);
}

}  // namespace radar
