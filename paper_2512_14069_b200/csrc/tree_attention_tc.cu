// Tree-masked GQA attention for bf16 on the 5th-generation tensor cores (tcgen05 + tensor memory),
// with K/V tiles staged by TMA.
//
// Work decomposition.  All G query heads of one KV head, for all tree rows, form R = n_nodes * G
// query rows (row r = node * G + head-in-group).  They are cut into row blocks of 128 (the MMA M
// dimension); one CTA owns (sequence, KV head, row block, KV split) and streams its range of the
// prefix in tiles of 128 keys, plus - in the last split - one tile holding the tree's own 64 keys.
//
// Inside the CTA (10 warps):
//   warp 8     TMA producer: Q once, then K and V tiles into two 3-slot rings (128-byte swizzle).
//   warp 9     MMA issuer (one lane): S = Q K^T into one of two tensor-memory score buffers, and
//              O (+)= P V with P read back from tensor memory (bf16, overlaying S) and V consumed
//              N-major straight from the row-major tile.
//   warps 0-3  softmax group 0: tiles 0, 2, 4, ... of the CTA's range;  warps 4-7: group 1, odd tiles.
//              One thread per query row: S row from tensor memory, prefix-boundary / ancestor-bit
//              masking in registers, running max with lazy rescaling of the O accumulator, exp2,
//              P back to tensor memory.  The two groups keep separate (m, l, O) and are merged
//              through shared memory at the end, so tile t+1's QK^T and softmax overlap tile t's PV.
// A sequence that fits one split is normalised and written to O directly; otherwise the CTA writes
// an fp32 partial (m, l, O) that tree_attn_tc_combine_kernel merges.
//
// Every mbarrier wait is bounded; a wait that runs out sets RADAR_ERR_TIMEOUT on the device status
// word, the CTA drains, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc05.cuh"

namespace radar {
namespace {

using namespace tc05;

constexpr int kTcThreads = 320;
constexpr int kTileKeys = 128;       // keys per prefix tile
constexpr int kTreeKeys = 64;        // keys of the tree tile (RADAR_MAX_NODES)
constexpr int kRing = 3;
constexpr float kRescaleThreshold = 8.f;   // in log2 units: P stays below 2^8

struct TcParams {
    radar_attn_args a;
    int G, nodes_per_rb, nrb_max;
    int tiles_per_split, n_splits_max;
    float scale_log2;
    long long cache_rows;
    float2* part_ml;     // [B][Hq][64][n_splits_max]  (m natural-log units, l)
    float* part_o;       // [B][Hq][64][n_splits_max][D]
    int* status;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D>
struct Smem {
    static constexpr int kHalves = D / 64;
    static constexpr int kQBytes = 128 * D * 2;
    static constexpr int kTileBytes = kTileKeys * D * 2;
    static constexpr int kRingBytes = kRing * kTileBytes;
    static constexpr int kTotal = kQBytes + 2 * kRingBytes;
    static constexpr int kDynamic = kTotal + 1024;          // slack for the 1024-byte alignment
};

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKc,
                    const __grid_constant__ CUtensorMap tmVc, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, const TcParams P) {
    using SM = Smem<D>;
    constexpr int H = SM::kHalves;
    const radar_attn_args& a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rb = blockIdx.x % P.nrb_max;
    const int split = blockIdx.x / P.nrb_max;
    const int g = blockIdx.y, b = blockIdx.z;
    const int G = P.G;

    // ---- which part of the problem is ours (uniform over the CTA) ----
    const int M = min(max(a.n_nodes[b], 0), kMaxNodes);
    const int Pb = a.prefix_len[b];
    const long long kv0 = a.kv_start[b];
    if (Pb < 0 || Pb > a.max_prefix_len || kv0 < 0 || kv0 + Pb > P.cache_rows) {
        if (tid == 0) set_status(P.status, RADAR_ERR_INVALID_ARG);
        return;
    }
    const int R = M * G;
    if (rb * 128 >= R) return;
    const int ntp_all = (Pb + kTileKeys - 1) / kTileKeys;                       // prefix tiles of the sequence
    const int n_splits = max(1, (ntp_all + P.tiles_per_split - 1) / P.tiles_per_split);
    if (split >= n_splits) return;
    const int tile0 = split * P.tiles_per_split;
    const int ntp = min(P.tiles_per_split, ntp_all - tile0);                     // prefix tiles of this CTA (may be 0)
    const bool has_tree = split == n_splits - 1;
    const int nt = max(ntp, 0) + (has_tree ? 1 : 0);                              // >= 1

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* sQ = smem;
    unsigned char* sK = smem + SM::kQBytes;
    unsigned char* sV = sK + SM::kRingBytes;
    __shared__ uint64_t bar_q, bar_kfull[kRing], bar_kempty[kRing], bar_vfull[kRing], bar_vempty[kRing];
    __shared__ uint64_t bar_sfull[2], bar_pready[2], bar_odone[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ float s_xm[128], s_xl[128];

    if (tid == 0) {
        s_abort = 0;
        mbar_init(&bar_q, 1);
        for (int i = 0; i < kRing; ++i) {
            mbar_init(&bar_kfull[i], 1); mbar_init(&bar_kempty[i], 1);
            mbar_init(&bar_vfull[i], 1); mbar_init(&bar_vempty[i], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&bar_sfull[i], 1); mbar_init(&bar_pready[i], 4); mbar_init(&bar_odone[i], 1); }
        fence_barrier_init();
    }
    if (warp == 8) {
        tmem_alloc(&s_tmem_base, 512);
        tmem_relinquish();
        if (lane == 0) {
            tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmKc); tma_prefetch_desc(&tmVc);
            tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s_tmem_base;
    // tensor-memory columns: S/P buffers at 0 and 128, O accumulators at 256 and 384
    volatile int* ab = &s_abort;

    // tile t of this CTA: prefix tile (128 keys) or, last, the tree tile (64 keys)
    auto tile_is_tree = [&](int t) { return has_tree && t == nt - 1; };

    if (warp == 8) {
        // =================================== TMA producer ===================================
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar_q, SM::kQBytes);
            for (int h = 0; h < H; ++h)
                tma_load_3d(sQ + h * (128 * 128), &tmQ, &bar_q, h * 64, g * G, b * kMaxNodes + rb * P.nodes_per_rb);
            auto load_tile = [&](int t, bool is_k) {
                const int slot = t % kRing;
                uint64_t* full = is_k ? &bar_kfull[slot] : &bar_vfull[slot];
                uint64_t* empty = is_k ? &bar_kempty[slot] : &bar_vempty[slot];
                unsigned char* dst = (is_k ? sK : sV) + slot * SM::kTileBytes;
                if (!mbar_wait(empty, ((t / kRing) & 1) ^ 1, ab)) return false;
                if (tile_is_tree(t)) {
                    mbar_arrive_expect_tx(full, kTreeKeys * D * 2);
                    for (int h = 0; h < H; ++h)
                        tma_load_3d(dst + h * (kTreeKeys * 128), is_k ? &tmKt : &tmVt, full, h * 64, g, b * kMaxNodes);
                } else {
                    mbar_arrive_expect_tx(full, kTileKeys * D * 2);
                    const int row = (int)(kv0 + (long long)(tile0 + t) * kTileKeys);
                    for (int h = 0; h < H; ++h)
                        tma_load_3d(dst + h * (kTileKeys * 128), is_k ? &tmKc : &tmVc, full, h * 64, g, row);
                }
                return true;
            };
            // same order as the MMA warp consumes: K0, K1, then V(t), K(t+2)
            bool ok = load_tile(0, true);
            if (ok && nt > 1) ok = load_tile(1, true);
            for (int t = 0; ok && t < nt; ++t) {
                ok = load_tile(t, false);
                if (ok && t + 2 < nt) ok = load_tile(t + 2, true);
            }
        }
        __syncwarp();
    } else if (warp == 9) {
        // =================================== MMA issuer ===================================
        constexpr uint32_t idesc_s128 = idesc_bf16_f32(128, kTileKeys, false, false);
        constexpr uint32_t idesc_s64 = idesc_bf16_f32(128, kTreeKeys, false, false);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
        bool ok = mbar_wait(&bar_q, 0, ab);
        auto issue_s = [&](int t) {
            const int slot = t % kRing, grp = t & 1;
            if (!mbar_wait(&bar_kfull[slot], (t / kRing) & 1, ab)) return false;
            tc_fence_after_sync();
            if (lane == 0) {
                const bool tree = tile_is_tree(t);
                const int nk = tree ? kTreeKeys : kTileKeys;
                const uint32_t kbase = smem_u32(sK + slot * SM::kTileBytes);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const int h = kk >> 2, ko = (kk & 3) * 32;
                    const uint64_t ad = smem_desc_sw128(smem_u32(sQ) + h * (128 * 128) + ko, 16, 1024);
                    const uint64_t bd = smem_desc_sw128(kbase + h * (nk * 128) + ko, 16, 1024);
                    mma_ss(tmem + grp * 128, ad, bd, tree ? idesc_s64 : idesc_s128, kk > 0);
                }
                mma_commit(&bar_kempty[slot]);
                mma_commit(&bar_sfull[grp]);
            }
            __syncwarp();
            return true;
        };
        if (ok) ok = issue_s(0);
        if (ok && nt > 1) ok = issue_s(1);
        for (int t = 0; ok && t < nt; ++t) {
            const int slot = t % kRing, grp = t & 1, j = t >> 1;
            if (!mbar_wait(&bar_pready[grp], j & 1, ab)) { ok = false; break; }
            if (!mbar_wait(&bar_vfull[slot], (t / kRing) & 1, ab)) { ok = false; break; }
            tc_fence_after_sync();
            const bool tree = tile_is_tree(t);
            const int nk = tree ? kTreeKeys : kTileKeys;
            const int valid = tree ? M : min(kTileKeys, Pb - (tile0 + t) * kTileKeys);
            const int ksteps = (valid + 15) >> 4;
            unsigned char* vtile = sV + slot * SM::kTileBytes;
            if (valid < ksteps * 16) {
                // rows past the last live key are multiplied by P = 0; they must not hold NaN/Inf bit patterns
                const int nrows = ksteps * 16 - valid;
                for (int e = lane; e < nrows * 8 * H; e += 32) {
                    const int h = e / (nrows * 8), rem = e % (nrows * 8);
                    const int r = valid + rem / 8, c = rem % 8;
                    *reinterpret_cast<uint4*>(vtile + h * (nk * 128) + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            if (lane == 0) {
                const uint32_t vbase = smem_u32(vtile);
                for (int kk = 0; kk < ksteps; ++kk) {
                    const uint64_t bd = smem_desc_sw128(vbase + kk * 2048, nk * 128, 1024);
                    mma_ts(tmem + 256 + grp * 128, tmem + grp * 128 + kk * 8, bd, idesc_pv, (j > 0) || (kk > 0));
                }
                mma_commit(&bar_vempty[slot]);
                if (t + 2 >= nt) mma_commit(&bar_odone[grp]);       // this group's last tile
            }
            __syncwarp();
            if (t + 2 < nt) ok = issue_s(t + 2);
        }
    } else {
        // =================================== softmax groups ===================================
        const int grp = warp >> 2;
        const int row = (warp & 3) * 32 + lane;                 // row of the block == tensor-memory lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + grp * 128 + lane_addr;
        const uint32_t tO = tmem + 256 + grp * 128 + lane_addr;
        const int r_glob = rb * 128 + row;
        const int node = r_glob / G;
        const int hq = g * G + r_glob % G;
        const bool row_live = r_glob < R;
        const unsigned long long live_bits = M >= 64 ? ~0ull : ((1ull << M) - 1ull);
        const unsigned long long mask_bits = row_live ? (a.mask[(int64_t)b * kMaxNodes + node] & live_bits) : 0ull;
        const int n_my = (nt - grp + 1) >> 1;
        float m_run = -CUDART_INF_F, l_run = 0.f;
        bool ok = true;

        for (int j = 0; j < n_my && ok; ++j) {
            const int t = 2 * j + grp;
            if (!mbar_wait(&bar_sfull[grp], j & 1, ab)) { ok = false; break; }
            tc_fence_after_sync();
            const bool tree = tile_is_tree(t);
            const int nchunks = tree ? kTreeKeys / 32 : kTileKeys / 32;
            uint32_t sv[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nchunks) tmem_ld32(tS + c * 32, sv[c]);
            tmem_wait_ld();
            // ---- masking ----
            if (tree) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (!((mask_bits >> (c * 32 + i)) & 1ull)) sv[c][i] = 0xff800000u;     // -inf
            } else {
                const int valid = min(kTileKeys, Pb - (tile0 + t) * kTileKeys);
                if (valid < kTileKeys) {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (c * 32 + i >= valid) sv[c][i] = 0xff800000u;
                }
            }
            // ---- running max (log2 units), lazy rescale decision ----
            float mx = -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nchunks)
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(sv[c][i]));
            const float m_tile = mx * P.scale_log2;
            float factor = 1.f;
            if (j == 0) {
                m_run = m_tile;
            } else if (m_tile > m_run + kRescaleThreshold) {
                factor = ex2(m_run - m_tile);               // m_run may be -inf: factor 0 clears O and l
                m_run = m_tile;
            }
            const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;
            // ---- P = exp2(s * scale - m), row sum, bf16 pairs back to tensor memory (over S) ----
            float lsum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (c < nchunks) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float p0 = ex2(fmaf(__uint_as_float(sv[c][2 * i]), P.scale_log2, -m_use));
                        const float p1 = ex2(fmaf(__uint_as_float(sv[c][2 * i + 1]), P.scale_log2, -m_use));
                        lsum += p0 + p1;
                        const __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
                        pk[i] = *reinterpret_cast<const uint32_t*>(&v);
                    }
                    tmem_st16(tS + c * 16, pk);
                }
            }
            l_run = l_run * factor + lsum;
            // ---- rescale the accumulator when some row of this warp moved its reference max ----
            if (j > 0 && __any_sync(kFull, factor != 1.f)) {
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                    tmem_st32(tO + c * 32, o);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_pready[grp]);
        }

        // ---- epilogue: merge the two groups, then write the final rows or the split's partial ----
        if (ok && n_my > 0) ok = mbar_wait(&bar_odone[grp], 0, ab);
        tc_fence_after_sync();
        float* xo = reinterpret_cast<float*>(sK);            // [D][128] exchange buffer (rings are idle by now)
        if (grp == 1) {
            if (ok && n_my > 0) {
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) xo[(c * 32 + i) * 128 + row] = __uint_as_float(o[i]);
                }
                s_xm[row] = m_run;
                s_xl[row] = l_run;
            } else {
                s_xm[row] = -CUDART_INF_F;
                s_xl[row] = 0.f;
            }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (grp == 0 && ok) {
            const float m1 = s_xm[row], l1 = s_xl[row];
            const float m = fmaxf(m_run, m1);
            const float m_safe = m == -CUDART_INF_F ? 0.f : m;
            const float w0 = ex2(m_run - m_safe), w1 = ex2(m1 - m_safe);      // exp2(-inf) = 0
            const float l = l_run * w0 + l1 * w1;
            const bool merge = m1 != -CUDART_INF_F;
            const bool final_rows = n_splits == 1;
            const float inv = final_rows ? 1.f / l : 1.f;
            const int64_t out_row = ((int64_t)b * kMaxNodes + node) * a.Hq + hq;
            const int64_t rec = (((int64_t)b * a.Hq + hq) * kMaxNodes + node) * P.n_splits_max + split;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                tmem_wait_ld();
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    v[i] = __uint_as_float(o[i]) * w0;
                    if (merge) v[i] = fmaf(xo[(c * 32 + i) * 128 + row], w1, v[i]);
                    v[i] *= inv;
                }
                if (row_live) {
                    if (final_rows) {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.O) + out_row * D + c * 32;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t w[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const __nv_bfloat162 t2 = __floats2bfloat162_rn(v[q * 8 + 2 * i], v[q * 8 + 2 * i + 1]);
                                w[i] = *reinterpret_cast<const uint32_t*>(&t2);
                            }
                            *reinterpret_cast<uint4*>(dst + q * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    } else {
                        float* dst = P.part_o + rec * D + c * 32;
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            *reinterpret_cast<float4*>(dst + q * 4) = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
                    }
                }
            }
            if (row_live) {
                const float m_nat = m_safe * 0.6931471805599453f;
                if (final_rows) {
                    if (a.lse != nullptr) a.lse[((int64_t)b * a.Hq + hq) * kMaxNodes + node] = m_nat + logf(l);
                } else {
                    P.part_ml[rec] = make_float2(m == -CUDART_INF_F ? -CUDART_INF_F : m_nat, l);
                }
            }
        }
    }

    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) {
        if (s_abort) {
            // let loads that are still in flight land before the CTA's shared memory is released
            if (lane == 0) {
                int dummy = 0;
                for (int i = 0; i < kRing; ++i) {
                    mbar_wait(&bar_kfull[i], 0, &dummy, 1u << 12);
                    mbar_wait(&bar_vfull[i], 0, &dummy, 1u << 12);
                }
                set_status(P.status, RADAR_ERR_TIMEOUT);
            }
            __syncwarp();
        }
        tmem_dealloc(tmem, 512);
    }
}

// one warp per (sequence, query head, tree row) of a sequence that was split: merge the partials
template <int D>
__global__ void __launch_bounds__(128) tree_attn_tc_combine_kernel(const TcParams P) {
    const radar_attn_args& a = P.a;
    const int lane = threadIdx.x & 31;
    const int64_t item = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int node = (int)(item % kMaxNodes);
    const int hq = (int)((item / kMaxNodes) % a.Hq);
    const int b = (int)(item / ((int64_t)kMaxNodes * a.Hq));
    if (b >= a.B) return;
    const int M = min(max(a.n_nodes[b], 0), kMaxNodes);
    const int Pb = a.prefix_len[b];
    if (node >= M || Pb < 0 || Pb > a.max_prefix_len) return;
    const int ntp_all = (Pb + kTileKeys - 1) / kTileKeys;
    const int n_splits = max(1, (ntp_all + P.tiles_per_split - 1) / P.tiles_per_split);
    if (n_splits == 1) return;                              // written directly by the attention kernel
    const int64_t rec0 = (((int64_t)b * a.Hq + hq) * kMaxNodes + node) * P.n_splits_max;
    float mx = -CUDART_INF_F;
    for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, P.part_ml[rec0 + s].x);
    float den = 0.f, o[D / 32];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) o[c] = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float2 ml = P.part_ml[rec0 + s];
        if (ml.x == -CUDART_INF_F) continue;
        const float w = __expf(ml.x - mx);
        den += ml.y * w;
        const float* src = P.part_o + (rec0 + s) * D + lane * (D / 32);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) o[c] = fmaf(src[c], w, o[c]);
    }
    const float inv = 1.f / den;
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.O) + (((int64_t)b * kMaxNodes + node) * a.Hq + hq) * D + lane * (D / 32);
#pragma unroll
    for (int c = 0; c < D / 32; ++c) dst[c] = __float2bfloat16(o[c] * inv);
    if (a.lse != nullptr && lane == 0) a.lse[((int64_t)b * a.Hq + hq) * kMaxNodes + node] = mx + logf(den);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
        return q == cudaDriverEntryPointSuccess ? reinterpret_cast<EncodeTiledFn>(p) : nullptr;
    }();
    return fn;
}

// [rows][heads][d] bf16 tensor, box = (64 elements, box_heads, box_rows), 128-byte swizzle, zero fill
bool make_map(CUtensorMap* tm, const void* base, int d, int heads, long long rows, int box_heads, int box_rows) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * heads};
    cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
    cuuint32_t es[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tree_attn_tc_supported(const radar_attn_args* a) {
    if (a->dtype != RADAR_BF16 || (a->d != 64 && a->d != 128)) return false;
    const int G = a->Hq / a->Hkv;
    if (G < 1 || G > 128 || (128 % G) != 0) return false;
    if (a->cache_rows < 0 || a->cache_rows >= (1ll << 31) || (long long)a->B * kMaxNodes >= (1ll << 31)) return false;
    const uintptr_t al = reinterpret_cast<uintptr_t>(a->Q) | reinterpret_cast<uintptr_t>(a->Kc) |
                         reinterpret_cast<uintptr_t>(a->Vc) | reinterpret_cast<uintptr_t>(a->Kt) |
                         reinterpret_cast<uintptr_t>(a->Vt) | reinterpret_cast<uintptr_t>(a->O);
    return (al & 15) == 0 && encode_fn() != nullptr;
}

void tree_attn_tc_plan(const radar_ctx* ctx, int B, int Hq, int Hkv, int max_prefix_len, int* tiles_per_split,
                       int* n_splits_max) {
    const int G = Hq / Hkv;
    const int nrb = (kMaxNodes * G + 127) / 128;
    const int nt = (max_prefix_len + kTileKeys - 1) / kTileKeys;
    const long long units = (long long)B * Hkv * nrb;
    // enough CTAs to cover the machine about twice, but at least 4 tiles (512 keys) per CTA
    int want = (int)((2LL * ctx->sm_count + units - 1) / units);
    if (want < 1) want = 1;
    int tps = (nt + want - 1) / want;
    if (tps < 4) tps = 4;
    if (tps > nt && nt > 0) tps = nt;
    *tiles_per_split = tps;
    *n_splits_max = nt > 0 ? (nt + tps - 1) / tps : 1;
}

size_t tree_attn_tc_workspace_bytes(const radar_ctx* ctx, int B, int Hq, int Hkv, int d, int max_prefix_len) {
    int tps, ns;
    tree_attn_tc_plan(ctx, B, Hq, Hkv, max_prefix_len, &tps, &ns);
    if (ns == 1) return 256;
    const size_t rec = (size_t)B * Hq * kMaxNodes * ns;
    return align_up(rec * sizeof(float2), 256) + align_up(rec * d * sizeof(float), 256);
}

template <int D>
static int launch_tc(radar_ctx* ctx, TcParams& P, cudaStream_t stream) {
    const radar_attn_args& a = P.a;
    CUtensorMap tmQ, tmKc, tmVc, tmKt, tmVt;
    const long long tree_rows = (long long)a.B * kMaxNodes;
    const bool have_prefix = a.Kc != nullptr && a.Vc != nullptr && a.cache_rows > 0;
    if (!make_map(&tmQ, a.Q, D, a.Hq, tree_rows, P.G, P.nodes_per_rb) ||
        !make_map(&tmKt, a.Kt, D, a.Hkv, tree_rows, 1, kTreeKeys) ||
        !make_map(&tmVt, a.Vt, D, a.Hkv, tree_rows, 1, kTreeKeys) ||
        !make_map(&tmKc, have_prefix ? a.Kc : a.Kt, D, a.Hkv, have_prefix ? a.cache_rows : tree_rows, 1, kTileKeys) ||
        !make_map(&tmVc, have_prefix ? a.Vc : a.Vt, D, a.Hkv, have_prefix ? a.cache_rows : tree_rows, 1, kTileKeys))
        return RADAR_ERR_CUDA;
    static bool attr_done = false;                  // once per process: not a stream operation
    if (!attr_done) {
        RADAR_CUDA_CHECK(cudaFuncSetAttribute(tree_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              Smem<D>::kDynamic));
        attr_done = true;
    }
    dim3 grid((unsigned)(P.nrb_max * P.n_splits_max), (unsigned)a.Hkv, (unsigned)a.B);
    {
        radar_launch_scope scope(ctx, RADAR_K_ATTN, stream);
        tree_attn_tc_kernel<D><<<grid, kTcThreads, Smem<D>::kDynamic, stream>>>(tmQ, tmKc, tmVc, tmKt, tmVt, P);
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    if (P.n_splits_max > 1) {
        const int64_t items = (int64_t)a.B * a.Hq * kMaxNodes;
        radar_launch_scope scope(ctx, RADAR_K_ATTN_COMBINE, stream);
        tree_attn_tc_combine_kernel<D><<<(unsigned)((items + 3) / 4), 128, 0, stream>>>(P);
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}

int tree_attn_tc_launch(radar_ctx* ctx, const radar_attn_args* a, cudaStream_t stream) {
    TcParams P;
    P.a = *a;
    P.G = a->Hq / a->Hkv;
    P.nodes_per_rb = 128 / P.G;
    P.nrb_max = (kMaxNodes * P.G + 127) / 128;
    const float scale = a->scale > 0.f ? a->scale : 1.f / sqrtf((float)a->d);
    P.scale_log2 = scale * 1.4426950408889634f;
    P.cache_rows = a->cache_rows;
    P.status = ctx->d_status;
    tree_attn_tc_plan(ctx, a->B, a->Hq, a->Hkv, a->max_prefix_len, &P.tiles_per_split, &P.n_splits_max);
    if (tree_attn_tc_workspace_bytes(ctx, a->B, a->Hq, a->Hkv, a->d, a->max_prefix_len) > a->workspace_bytes)
        return RADAR_ERR_WORKSPACE;
    const size_t rec = (size_t)a->B * a->Hq * kMaxNodes * P.n_splits_max;
    P.part_ml = reinterpret_cast<float2*>(a->workspace);
    P.part_o = reinterpret_cast<float*>(reinterpret_cast<char*>(a->workspace) + align_up(rec * sizeof(float2), 256));
    return a->d == 128 ? launch_tc<128>(ctx, P, stream) : launch_tc<64>(ctx, P, stream);
}

}  // namespace radar
