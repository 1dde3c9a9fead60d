// radar_tree_attention: tree-masked GQA attention of the draft tree's queries against the
// prefix KV cache plus the tree's own KV.
//
// This file holds the fp32-arithmetic kernel (exact enough for the 1e-5 fp32 contract, also
// serving bf16 storage) and the split-KV combine.  Work is split over (sequence, KV head,
// block of 32 query rows, KV split); all G query heads that share a KV head are rows of the
// same block so that a K/V tile staged in shared memory is reused G * rows times.
#include <algorithm>

#include "common.cuh"

namespace radar {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerWarp = 4;
constexpr int kRowsPerBlock = kWarps * kRowsPerWarp;     // 32
constexpr int kTile = 32;                                // keys per shared-memory tile

struct AttnParams {
    radar_attn_args a;
    int G;
    int split_len, n_splits;
    float scale;
    float2* part_ml;     // [B][Hq][64][S] (running max, normaliser)
    float* part_o;       // [B][Hq][64][S][d]
    int* status;
};

template <typename T> __device__ __forceinline__ void load16(const T* src, float* dst);
template <> __device__ __forceinline__ void load16<float>(const float* src, float* dst) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(src + 4 * q);
        dst[4 * q] = v.x; dst[4 * q + 1] = v.y; dst[4 * q + 2] = v.z; dst[4 * q + 3] = v.w;
    }
}
template <> __device__ __forceinline__ void load16<__nv_bfloat16>(const __nv_bfloat16* src, float* dst) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint4 v = *reinterpret_cast<const uint4*>(src + 8 * q);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            dst[8 * q + 2 * j] = __uint_as_float(w[j] << 16);
            dst[8 * q + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) tree_attn_fp32_kernel(const AttnParams P) {
    chain_wait();
    const radar_attn_args& a = P.a;
    constexpr int KS = D + 4;                       // padded K row: conflict-free 16-byte reads by 32 lanes
    extern __shared__ float smem[];
    float* Qs = smem;                               // [32][D]
    float* Ks = Qs + kRowsPerBlock * D;             // [32][KS]
    float* Vs = Ks + kTile * KS;                    // [32][D]

    const int split = blockIdx.x % P.n_splits;
    const int rblock = blockIdx.x / P.n_splits;
    const int g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = P.G, Hq = a.Hq, Hkv = a.Hkv;

    const int M = min(max(a.n_nodes[b], 0), kMaxNodes);
    const int Pb = a.prefix_len[b];
    const bool paged = a.block_table != nullptr;
    const int64_t kv0 = paged ? 0 : a.kv_start[b];
    // the same bounds as the tensor-core kernel: a sequence whose prefix does not lie inside the cache is
    // reported and skipped before anything of the cache is read
    if (Pb < 0 || Pb > a.max_prefix_len || kv0 < 0 || kv0 + Pb > a.cache_rows) {
        if (tid == 0) set_status(P.status, RADAR_ERR_INVALID_ARG);
        return;
    }
    const int R = M * G;
    const int row0 = rblock * kRowsPerBlock;
    if (row0 >= R) return;
    const int Ltot = Pb + M;
    const int k_begin = split * P.split_len;
    const int k_end = min(k_begin + P.split_len, Ltot);
    if (k_begin >= k_end) return;

    const T* Q = reinterpret_cast<const T*>(a.Q);
    const T* Kc = reinterpret_cast<const T*>(a.Kc);
    const T* Vc = reinterpret_cast<const T*>(a.Vc);
    const T* Kt = reinterpret_cast<const T*>(a.Kt);
    const T* Vt = reinterpret_cast<const T*>(a.Vt);
    const int64_t n_cache_pages = paged ? P.a.cache_rows / a.page_size : 0;

    // ---- stage the block's query rows (pre-scaled) ----
    for (int e = tid; e < kRowsPerBlock * (D / 16); e += kThreads) {
        const int rl = e / (D / 16), seg = e % (D / 16);
        const int r = row0 + rl;
        float tmp[16];
        if (r < R) {
            const int node = r / G, hq = g * G + r % G;
            load16<T>(Q + (((int64_t)b * kMaxNodes + node) * Hq + hq) * D + seg * 16, tmp);
        } else {
#pragma unroll
            for (int q = 0; q < 16; ++q) tmp[q] = 0.f;
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) Qs[rl * D + seg * 16 + q] = tmp[q] * P.scale;
    }

    unsigned long long rmask[kRowsPerWarp];
    bool rvalid[kRowsPerWarp];
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) {
        const int r = row0 + warp * kRowsPerWarp + i;
        rvalid[i] = r < R;
        rmask[i] = rvalid[i] ? a.mask[(int64_t)b * kMaxNodes + r / G] : 0ull;
    }
    float m_run[kRowsPerWarp], l_run[kRowsPerWarp], acc[kRowsPerWarp][D / 32];
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) {
        m_run[i] = -CUDART_INF_F;
        l_run[i] = 0.f;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) acc[i][c] = 0.f;
    }

    for (int k0 = k_begin; k0 < k_end; k0 += kTile) {
        __syncthreads();                            // previous tile fully consumed (and Qs visible)
        for (int e = tid; e < kTile * (D / 16); e += kThreads) {
            const int j = e / (D / 16), seg = e % (D / 16);
            const int kidx = k0 + j;
            float tk[16], tv[16];
            if (kidx < k_end) {
                const T *ksrc, *vsrc;
                if (kidx < Pb) {
                    int64_t row = kv0 + kidx;
                    if (paged) {
                        int64_t page = a.block_table[(int64_t)b * a.max_pages + kidx / a.page_size];
                        if (page < 0 || page >= n_cache_pages) { set_status(P.status, RADAR_ERR_INVALID_ARG); page = 0; }
                        row = page * a.page_size + kidx % a.page_size;
                    }
                    const int64_t off = (row * Hkv + g) * D + seg * 16;
                    ksrc = Kc + off; vsrc = Vc + off;
                } else {
                    const int64_t off = (((int64_t)b * kMaxNodes + (kidx - Pb)) * Hkv + g) * D + seg * 16;
                    ksrc = Kt + off; vsrc = Vt + off;
                }
                load16<T>(ksrc, tk);
                load16<T>(vsrc, tv);
            } else {
#pragma unroll
                for (int q = 0; q < 16; ++q) { tk[q] = 0.f; tv[q] = 0.f; }
            }
#pragma unroll
            for (int q = 0; q < 16; q += 4) {
                *reinterpret_cast<float4*>(&Ks[j * KS + seg * 16 + q]) = make_float4(tk[q], tk[q + 1], tk[q + 2], tk[q + 3]);
                *reinterpret_cast<float4*>(&Vs[j * D + seg * 16 + q]) = make_float4(tv[q], tv[q + 1], tv[q + 2], tv[q + 3]);
            }
        }
        __syncthreads();

        // scores: lane = key
        float s[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) s[i] = 0.f;
        const float* krow = Ks + lane * KS;
        const float* qrow = Qs + (warp * kRowsPerWarp) * D;
#pragma unroll 4
        for (int c = 0; c < D; c += 4) {
            const float4 kv = *reinterpret_cast<const float4*>(krow + c);
#pragma unroll
            for (int i = 0; i < kRowsPerWarp; ++i) {
                const float4 qv = *reinterpret_cast<const float4*>(qrow + i * D + c);
                s[i] = fmaf(qv.x, kv.x, s[i]);
                s[i] = fmaf(qv.y, kv.y, s[i]);
                s[i] = fmaf(qv.z, kv.z, s[i]);
                s[i] = fmaf(qv.w, kv.w, s[i]);
            }
        }
        const int kidx = k0 + lane;
        float pr[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            bool ok = rvalid[i] && kidx < k_end;
            if (ok && kidx >= Pb) ok = (rmask[i] >> (kidx - Pb)) & 1ull;
            const float sv = ok ? s[i] : -CUDART_INF_F;
            const float tmax = warp_max(sv);
            const float m_new = fmaxf(m_run[i], tmax);
            float p = 0.f, corr = 1.f;
            if (m_new > -CUDART_INF_F) {
                p = ok ? __expf(sv - m_new) : 0.f;
                corr = __expf(m_run[i] - m_new);       // exp(-inf) = 0 on the first live tile
            }
            const float psum = warp_sum(p);
            l_run[i] = l_run[i] * corr + psum;
            m_run[i] = m_new;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) acc[i][c] *= corr;
            pr[i] = p;
        }
        // O += P V : lane owns output dims [lane * D/32, +D/32)
        for (int j = 0; j < kTile; ++j) {
            float vv[D / 32];
            if (D == 128) {
                const float4 t = *reinterpret_cast<const float4*>(Vs + j * D + lane * 4);
                vv[0] = t.x; vv[1] = t.y; vv[2] = t.z; vv[3] = t.w;
            } else {
                const float2 t = *reinterpret_cast<const float2*>(Vs + j * D + lane * 2);
                vv[0] = t.x; vv[1] = t.y;
            }
#pragma unroll
            for (int i = 0; i < kRowsPerWarp; ++i) {
                const float pj = __shfl_sync(kFull, pr[i], j);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) acc[i][c] = fmaf(pj, vv[c], acc[i][c]);
            }
        }
    }

    // ---- partial results ----
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) {
        const int r = row0 + warp * kRowsPerWarp + i;
        if (r >= R) continue;
        const int node = r / G, hq = g * G + r % G;
        const int64_t rec = (((int64_t)b * Hq + hq) * kMaxNodes + node) * P.n_splits + split;
        if (lane == 0) P.part_ml[rec] = make_float2(m_run[i], l_run[i]);
        float* dst = P.part_o + rec * D + lane * (D / 32);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) dst[c] = acc[i][c];
    }
}

// one warp per (sequence, query head, tree row): merge the KV splits
template <typename T, int D>
__global__ void __launch_bounds__(128) tree_attn_combine_kernel(const AttnParams P) {
    chain_wait();
    const radar_attn_args& a = P.a;
    const int lane = threadIdx.x & 31;
    const int64_t item = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int node = (int)(item % kMaxNodes);
    const int hq = (int)((item / kMaxNodes) % a.Hq);
    const int b = (int)(item / ((int64_t)kMaxNodes * a.Hq));
    if (b >= a.B) return;
    const int M = min(max(a.n_nodes[b], 0), kMaxNodes);
    const int Pb = a.prefix_len[b];
    const int64_t kv0 = a.block_table != nullptr ? 0 : a.kv_start[b];
    if (node >= M || Pb < 0 || Pb > a.max_prefix_len || kv0 < 0 || kv0 + Pb > a.cache_rows) return;   // skipped by the main kernel
    const int n_valid = (Pb + M + P.split_len - 1) / P.split_len;
    const int64_t rec0 = (((int64_t)b * a.Hq + hq) * kMaxNodes + node) * P.n_splits;
    float mx = -CUDART_INF_F;
    for (int s = 0; s < n_valid; ++s) mx = fmaxf(mx, P.part_ml[rec0 + s].x);
    float den = 0.f, o[D / 32];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) o[c] = 0.f;
    for (int s = 0; s < n_valid; ++s) {
        const float2 ml = P.part_ml[rec0 + s];
        if (ml.x == -CUDART_INF_F) continue;
        const float w = __expf(ml.x - mx);
        den += ml.y * w;
        const float* src = P.part_o + (rec0 + s) * D + lane * (D / 32);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) o[c] = fmaf(src[c], w, o[c]);
    }
    const float inv = 1.f / den;
    T* dst = reinterpret_cast<T*>(a.O) + (((int64_t)b * kMaxNodes + node) * a.Hq + hq) * D + lane * (D / 32);
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        if constexpr (sizeof(T) == 4) dst[c] = o[c] * inv;
        else dst[c] = __float2bfloat16(o[c] * inv);
    }
    if (a.lse != nullptr && lane == 0) a.lse[((int64_t)b * a.Hq + hq) * kMaxNodes + node] = mx + logf(den);
}

void plan(const radar_ctx* ctx, int B, int Hq, int Hkv, int max_prefix_len, int* split_len, int* n_splits) {
    const int G = Hq / Hkv;
    const int rblocks = (kMaxNodes * G + kRowsPerBlock - 1) / kRowsPerBlock;
    const int Lmax = max_prefix_len + kMaxNodes;
    long long base = (long long)B * Hkv * rblocks;
    int want = (int)((4LL * ctx->sm_count + base - 1) / base);
    if (want < 1) want = 1;
    int len = (Lmax + want - 1) / want;
    if (len < 256) len = 256;
    len = (len + kTile - 1) / kTile * kTile;
    *split_len = len;
    *n_splits = (Lmax + len - 1) / len;
}

template <typename T, int D>
int launch(radar_ctx* ctx, const AttnParams& P, cudaStream_t stream) {
    const radar_attn_args& a = P.a;
    const int rblocks = (kMaxNodes * P.G + kRowsPerBlock - 1) / kRowsPerBlock;
    const size_t smem = sizeof(float) * (kRowsPerBlock * D + kTile * (D + 4) + kTile * D);
    RADAR_CUDA_CHECK(radar_opt_in_smem(ctx, RADAR_SMEM_ATTN_FMA + 2 * (sizeof(T) == 2) + (D == 128), tree_attn_fp32_kernel<T, D>, smem));
    dim3 grid((unsigned)(rblocks * P.n_splits), (unsigned)a.Hkv, (unsigned)a.B);
    {
        radar_launch_scope scope(ctx, RADAR_K_ATTN, stream);
        RADAR_CUDA_CHECK(launch_chained(tree_attn_fp32_kernel<T, D>, grid, dim3(kThreads), smem, stream, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    const int64_t items = (int64_t)a.B * a.Hq * kMaxNodes;
    {
        radar_launch_scope scope(ctx, RADAR_K_ATTN_COMBINE, stream);
        RADAR_CUDA_CHECK(launch_chained(tree_attn_combine_kernel<T, D>, dim3((unsigned)((items + 3) / 4)), dim3(128), 0, stream, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}

}  // namespace
}  // namespace radar

using namespace radar;

extern "C" size_t radar_attn_workspace_bytes(const radar_ctx* ctx, int B, int Hq, int Hkv, int d, int dtype,
                                             int max_prefix_len) {
    if (!ctx || B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || max_prefix_len < 0) return 0;
    int split_len, n_splits;
    plan(ctx, B, Hq, Hkv, max_prefix_len, &split_len, &n_splits);
    const size_t rec = (size_t)B * Hq * kMaxNodes * n_splits;
    size_t need = align_up(rec * sizeof(float2), 256) + align_up(rec * d * sizeof(float), 256);
    // the same buffer serves whichever kernel the call dispatches to
    if (dtype == RADAR_BF16) need = std::max(need, tree_attn_tc_workspace_bytes(ctx, B, Hq, Hkv, d, max_prefix_len));
    return need;
}

extern "C" int radar_tree_attention_path(const radar_attn_args* a) {
    if (!a) return RADAR_ERR_INVALID_ARG;
    return tree_attn_tc_supported(a) ? RADAR_ATTN_PATH_TENSOR_CORE : RADAR_ATTN_PATH_FMA;
}

extern "C" int radar_tree_attention(radar_ctx* ctx, const radar_attn_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (a->B <= 0 || a->Hq <= 0 || a->Hkv <= 0 || a->max_prefix_len < 0) return RADAR_ERR_INVALID_ARG;
    if (a->Hq % a->Hkv != 0) return RADAR_ERR_INVALID_ARG;
    if (a->d != 64 && a->d != 128) return RADAR_ERR_UNSUPPORTED;
    if (a->dtype != RADAR_F32 && a->dtype != RADAR_BF16) return RADAR_ERR_UNSUPPORTED;
    const bool paged = a->block_table != nullptr;
    if (paged && (a->max_pages <= 0 || !(a->page_size == 16 || a->page_size == 32 || a->page_size == 64 ||
                                         (a->page_size > 0 && a->page_size % 128 == 0)) ||
                  (long long)a->max_pages * a->page_size < a->max_prefix_len || a->cache_rows < a->page_size))
        return RADAR_ERR_INVALID_ARG;
    if (!a->Q || (!paged && !a->kv_start) || !a->prefix_len || !a->Kt || !a->Vt || !a->mask || !a->n_nodes || !a->O ||
        !a->workspace)
        return RADAR_ERR_INVALID_ARG;
    if (a->max_prefix_len > 0 && (!a->Kc || !a->Vc)) return RADAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->workspace) & 255) != 0) return RADAR_ERR_WORKSPACE;
    // both kernels move Q, K, V and O in 16-byte pieces
    if (((reinterpret_cast<uintptr_t>(a->Q) | reinterpret_cast<uintptr_t>(a->Kc) | reinterpret_cast<uintptr_t>(a->Vc) |
          reinterpret_cast<uintptr_t>(a->Kt) | reinterpret_cast<uintptr_t>(a->Vt) | reinterpret_cast<uintptr_t>(a->O)) & 15) != 0)
        return RADAR_ERR_INVALID_ARG;
    if (a->max_prefix_len > 0 && a->cache_rows <= 0) return RADAR_ERR_INVALID_ARG;
    const int n_layers = a->n_layers > 1 ? a->n_layers : 1;
    if (n_layers > 1 && (((a->q_layer_stride | a->cache_layer_stride | a->tree_kv_layer_stride | a->o_layer_stride) & 7) != 0 ||
                         a->q_layer_stride <= 0 || a->tree_kv_layer_stride <= 0 || a->o_layer_stride <= 0 ||
                         (a->max_prefix_len > 0 && a->cache_layer_stride <= 0) || (a->lse != nullptr && a->lse_layer_stride <= 0)))
        return RADAR_ERR_INVALID_ARG;
    if (tree_attn_tc_supported(a)) return tree_attn_tc_launch(ctx, a, stream);
    if (n_layers > 1) {
        // the FMA kernel takes one layer per launch
        const size_t es = a->dtype == RADAR_F32 ? 4 : 2;
        for (int l = 0; l < n_layers; ++l) {
            radar_attn_args one = *a;
            one.n_layers = 1;
            one.Q = reinterpret_cast<const char*>(a->Q) + (size_t)l * a->q_layer_stride * es;
            one.Kt = reinterpret_cast<const char*>(a->Kt) + (size_t)l * a->tree_kv_layer_stride * es;
            one.Vt = reinterpret_cast<const char*>(a->Vt) + (size_t)l * a->tree_kv_layer_stride * es;
            if (a->Kc) one.Kc = reinterpret_cast<const char*>(a->Kc) + (size_t)l * a->cache_layer_stride * es;
            if (a->Vc) one.Vc = reinterpret_cast<const char*>(a->Vc) + (size_t)l * a->cache_layer_stride * es;
            one.O = reinterpret_cast<char*>(a->O) + (size_t)l * a->o_layer_stride * es;
            if (a->lse) one.lse = a->lse + (size_t)l * a->lse_layer_stride;
            const int rc = radar_tree_attention(ctx, &one, stream_);
            if (rc != RADAR_OK) return rc;
        }
        return RADAR_OK;
    }

    AttnParams P;
    P.a = *a;
    P.G = a->Hq / a->Hkv;
    P.scale = a->scale > 0.f ? a->scale : 1.f / sqrtf((float)a->d);
    P.status = ctx->d_status;
    plan(ctx, a->B, a->Hq, a->Hkv, a->max_prefix_len, &P.split_len, &P.n_splits);
    const size_t rec = (size_t)a->B * a->Hq * kMaxNodes * P.n_splits;
    const size_t need = align_up(rec * sizeof(float2), 256) + align_up(rec * a->d * sizeof(float), 256);
    if (need > a->workspace_bytes) return RADAR_ERR_WORKSPACE;
    P.part_ml = reinterpret_cast<float2*>(a->workspace);
    P.part_o = reinterpret_cast<float*>(reinterpret_cast<char*>(a->workspace) + align_up(rec * sizeof(float2), 256));

    if (a->dtype == RADAR_F32) {
        return a->d == 128 ? launch<float, 128>(ctx, P, stream) : launch<float, 64>(ctx, P, stream);
    }
    return a->d == 128 ? launch<__nv_bfloat16, 128>(ctx, P, stream) : launch<__nv_bfloat16, 64>(ctx, P, stream);
}
