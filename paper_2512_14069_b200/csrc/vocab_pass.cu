// Vocabulary pass: one coalesced, vectorised read of every logits row produces, per
// (row, chunk), the chunk's k best (logit, token) pairs and its (max, sum exp) pair.
// The pass is HBM-bound: each logit is read exactly once with 16-byte loads; selection keeps
// a sorted 32-entry list per warp (one entry per lane) that is touched only when an element
// beats the current k-th best, which after the first few vectors is rare.
#include "common.cuh"

namespace radar {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

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

struct Scan {
    WarpTopList<float> top;
    float thr;      // k-th best value so far (warp-uniform)
    int thr_i;
    float m, s;     // per-thread running max and sum of exp(x - m)
    bool nan;
    int k;

    __device__ __forceinline__ void init(int k_) {
        top.reset();
        thr = -CUDART_INF_F;
        thr_i = 0x7fffffff;
        m = -CUDART_INF_F;
        s = 0.f;
        nan = false;
        k = k_;
    }
    // warp-collective: offer one element per lane
    __device__ __forceinline__ void offer(float v, int idx, bool valid) {
        const bool cand = valid && precedes(v, idx, thr, thr_i);
        unsigned mk = __ballot_sync(kFull, cand);
        if (mk == 0) return;
        while (mk) {
            const int src = __ffs(mk) - 1;
            mk &= mk - 1;
            top.insert(__shfl_sync(kFull, v, src), __shfl_sync(kFull, idx, src));
        }
        thr = top.value_at(k - 1);
        thr_i = top.index_at(k - 1);
    }
};

template <typename T, bool WANT_LSE>
__global__ void __launch_bounds__(kThreads) vocab_pass_kernel(const VocabPassParams p) {
    using VT = Vec<T>;
    constexpr int N = VT::N;
    const int row = blockIdx.x / p.n_chunks;
    const int chunk_id = blockIdx.x - row * p.n_chunks;
    const int seq = row / p.F;
    const int f = row - seq * p.F;
    if (p.seq_active != nullptr && p.seq_active[seq] == 0) return;
    if (p.seq_rows != nullptr && f >= p.seq_rows[seq]) return;

    const T* base = reinterpret_cast<const T*>(p.logits) + (int64_t)seq * p.seq_stride + (int64_t)f * p.row_stride;
    const int e0 = min(chunk_id * p.chunk, p.V);
    const int e1 = min(e0 + p.chunk, p.V);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    Scan sc;
    sc.init(p.k);

    // scalar head up to the first 16-byte boundary, vector body, scalar tail
    const uintptr_t addr = reinterpret_cast<uintptr_t>(base + e0);
    int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
    head = min(head, e1 - e0);
    const int body0 = e0 + head;
    const int nvec = (e1 - body0) / N;
    const int tail0 = body0 + nvec * N;

    auto scalar = [&](int idx, bool valid) {
        float v = valid ? to_float(base[idx]) : -CUDART_INF_F;
        if (valid) {
            if (v != v) sc.nan = true;
            if (WANT_LSE) {
                if (v > sc.m) { sc.s *= __expf(sc.m - v); sc.m = v; }
                if (sc.m > -CUDART_INF_F) sc.s += __expf(v - sc.m);
            }
        }
        sc.offer(v, idx, valid);
    };
    if (warp == 0) {                        // head and tail are shorter than one vector
        scalar(e0 + lane, lane < head);
        scalar(tail0 + lane, tail0 + lane < e1);
    }

    const T* vbase = base + body0;
    constexpr int U = 4;                    // independent 16-byte loads in flight per thread
    for (int j0 = 0; j0 < nvec; j0 += kThreads * U) {
        float x[U][N];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = j0 + u * kThreads + tid;
            ok[u] = j < nvec;
            if (ok[u]) VT::load(vbase + (int64_t)j * N, x[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = j0 + u * kThreads + tid;
            bool any = false;
            if (ok[u]) {
                float vmax = x[u][0];
#pragma unroll
                for (int e = 1; e < N; ++e) vmax = fmaxf(vmax, x[u][e]);
                bool bad = false;
#pragma unroll
                for (int e = 0; e < N; ++e) bad |= (x[u][e] != x[u][e]);
                sc.nan |= bad;
                if (WANT_LSE) {
                    if (vmax > sc.m) { sc.s *= __expf(sc.m - vmax); sc.m = vmax; }
                    if (sc.m > -CUDART_INF_F) {
#pragma unroll
                        for (int e = 0; e < N; ++e) sc.s += __expf(x[u][e] - sc.m);
                    }
                }
                any = vmax >= sc.thr;
            }
            if (__any_sync(kFull, any)) {
                const int idx0 = body0 + j * N;
#pragma unroll
                for (int e = 0; e < N; ++e) sc.offer(ok[u] ? x[u][e] : -CUDART_INF_F, idx0 + e, ok[u]);
            }
        }
    }

    // ---- combine the warps of the block ----
    __shared__ float sh_v[kWarps][32];
    __shared__ int sh_i[kWarps][32];
    __shared__ float sh_m[kWarps], sh_s[kWarps];
    __shared__ int sh_nan;
    if (tid == 0) sh_nan = 0;
    sh_v[warp][lane] = sc.top.v;
    sh_i[warp][lane] = sc.top.i;
    if (WANT_LSE) {
        const float wm = warp_max(sc.m);
        const float ws = warp_sum(wm > -CUDART_INF_F ? sc.s * __expf(sc.m - wm) : 0.f);
        if (lane == 0) { sh_m[warp] = wm; sh_s[warp] = ws; }
    }
    __syncthreads();
    if (sc.nan) atomicOr(&sh_nan, 1);
    __syncthreads();
    if (warp == 0) {
        for (int w = 1; w < kWarps; ++w) {
            for (int e = 0; e < p.k; ++e) {
                const float cv = sh_v[w][e];
                const int ci = sh_i[w][e];
                if (!precedes(cv, ci, sc.thr, sc.thr_i)) break;      // that warp's list is sorted
                sc.top.insert(cv, ci);
                sc.thr = sc.top.value_at(p.k - 1);
                sc.thr_i = sc.top.index_at(p.k - 1);
            }
        }
        const size_t rec = (size_t)row * p.n_chunks + chunk_id;
        if (lane < p.k) {
            p.part_v[rec * p.k + lane] = sc.top.v;
            p.part_i[rec * p.k + lane] = sc.top.i;
        }
        if (WANT_LSE && lane == 0) {
            float M = sh_m[0];
            for (int w = 1; w < kWarps; ++w) M = fmaxf(M, sh_m[w]);
            float S = 0.f;
            if (M > -CUDART_INF_F)
                for (int w = 0; w < kWarps; ++w) S += sh_s[w] * __expf(sh_m[w] - M);
            p.part_m[rec] = M;
            p.part_s[rec] = S;
        }
        if (lane == 0 && sh_nan) set_status(p.status, RADAR_ERR_NUMERIC);
    }
}

}  // namespace

int vocab_pass_plan_chunks(int sm_count, int rows, int V, int* chunk_out) {
    const int min_chunk = 2048, max_chunk = 16384;
    int want = (2 * sm_count + rows - 1) / rows;                 // about two blocks per SM for small inputs
    if (want < 1) want = 1;
    int chunk = (V + want - 1) / want;
    if (chunk < min_chunk) chunk = min_chunk;
    if (chunk > max_chunk) chunk = max_chunk;
    chunk = (chunk + 255) / 256 * 256;
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

cudaError_t vocab_pass_launch(radar_ctx* ctx, int kernel_id, const VocabPassParams& p, cudaStream_t stream) {
    const int rows = p.n_seq * p.F;
    const unsigned grid = (unsigned)rows * (unsigned)p.n_chunks;
    if (grid == 0) return cudaSuccess;
    radar_launch_scope scope(ctx, kernel_id, stream);
    if (p.dtype == RADAR_F32) {
        if (p.want_lse) vocab_pass_kernel<float, true><<<grid, kThreads, 0, stream>>>(p);
        else vocab_pass_kernel<float, false><<<grid, kThreads, 0, stream>>>(p);
    } else {
        if (p.want_lse) vocab_pass_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, stream>>>(p);
        else vocab_pass_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace radar
