// Tree-masked GQA attention for bf16 on the 5th-generation tensor cores (tcgen05 + tensor memory),
// with K/V tiles staged by TMA.
//
// Work decomposition.  All G query heads of one KV head, for all tree rows, form R = n_nodes * G
// query rows (row r = node * G + head-in-group), cut into row blocks of 128 (the MMA M dimension)
// and these into pairs.  A unit is (sequence, KV head, row-block pair); it has to visit the
// sequence's prefix in tiles of 128 keys plus one tile holding the tree's own 64 keys.  The tiles of
// all units, weighted by their cost, are laid end to end and cut into equal ranges, one per CTA, so
// every CTA gets about the same amount of time whatever the mix of prefix lengths and tree sizes;
// the grid is one CTA per SM.  A CTA therefore works through a few segments (unit, tile range).  A
// unit that falls into one CTA is normalised and written to O directly; the pieces of a unit that
// was cut are written as fp32 partials (m, l, O) and merged by tree_attn_tc_combine_kernel.  When
// there are several pairs per KV head, CTAs alternate between them so that they stream the same K/V
// at the same time and all but the first read hit L2.
//
// Inside the CTA (10 warps):
//   warp 8     TMA producer: per segment the Q rows, then K and V tiles into two rings (128-byte
//              swizzle), in the order the MMA warp consumes them.
//   warp 9     MMA issuer (one lane): S = Q K^T into one of two tensor-memory score buffers, and
//              O (+)= P V with P read back from tensor memory (bf16, overlaying S) and V consumed
//              N-major straight from the row-major tile.
//   warps 0-3 / 4-7  softmax groups 0 / 1, one thread per query row: S row from tensor memory,
//              prefix-boundary / ancestor-bit masking in registers, running max with lazy rescaling
//              of the O accumulator, exp2, P back to tensor memory.
//              Unit with two live row blocks: group s owns row block s and sees every tile, so each
//              K/V tile is loaded once for 256 query rows.  Unit with one live row block: the
//              groups take alternate tiles with separate (m, l, O) and are merged at the end.
//              Either way one group's softmax overlaps the other's MMAs.
// Every mbarrier wait is bounded; a wait that runs out sets RADAR_ERR_TIMEOUT on the device status
// word, the CTA drains without skipping any hardware barrier, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "tc05.cuh"

namespace radar {
namespace {

using namespace tc05;

constexpr int kTcThreads = 576;      // 16 softmax warps, TMA producer, MMA issuer
constexpr int kProducerWarp = 16, kMmaWarp = 17;
constexpr int kStaticSmem = 3072;    // barriers and exchange arrays: with the tiles exactly the 227 KB a block may have
constexpr int kTileKeys = 128;       // keys per prefix tile
constexpr int kTreeKeys = 64;        // keys of the tree tile (RADAR_MAX_NODES)
constexpr int kPairRows = 256;       // query rows of a row-block pair (and the stride of partial records)
constexpr float kRescaleThreshold = 8.f;   // in log2 units: P stays below 2^8

// Written by every CTA of the attention kernel, read by the combine kernel.
struct CutUnit {
    int valid;           // 1: this CTA's last segment starts a unit that continues in the following CTAs
    int b, g, nt;        // the unit and its number of tiles
    int layer;           // the layer it belongs to
    int slot;            // partial slot of that first piece in this CTA (0 or 1)
    int rows;            // live query rows of the unit
    int w;               // cost of one of its tiles
    long long u0;        // position of the unit's first tile in the class's space
    long long tot;       // size of that space
};

struct TcParams {
    radar_attn_args a;
    int G, g_log2, nodes_per_rb;   // G divides 128 on this path, so it is a power of two
    int pair_rows;       // query rows of a class's units: 256 (two row blocks share each K/V tile) or 128
    int n_layers;        // layers run by this launch (the same tree, masks and prefix lengths for all)
    long long o_ls, lse_ls;   // elements between consecutive layers of O and of lse
    int n_cls;           // classes = units per KV head
    int ncc;             // CTAs per class; grid = n_cls * ncc
    int cost_one, cost_two, unit_cost;   // tile_costs(n_cls)
    float scale_log2;
    long long cache_rows;
    float2* part_ml;     // [grid][2][256]     (m in natural-log units, l)
    float* part_o;       // [grid][2][256][D]
    CutUnit* cut;        // [grid]
    int* status;
};

__device__ __forceinline__ float max3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}
// one 32-byte store: a whole sector per lane (the epilogue's lanes write to different rows, so every store
// instruction is split into one transaction per lane; with 16-byte stores each of them filled half a sector)
__device__ __forceinline__ void st_global_32b(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
                 "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- the tile space of one class (unit index pp within a KV head) ---------------------------------
// Positions are in cost units: a tile of a unit with two live row blocks (four MMAs) weighs cost_two, a tile of
// a unit with one live row block cost_one, and every unit books cost_unit in front of its first tile for what it
// costs beside its tiles (pipeline fill, epilogue), so that a CTA whose range holds several unit starts gets fewer
// tiles; equal position ranges are then about equal amounts of time.  A tile belongs to the CTA whose range
// contains the tile's start position.  The weights are measured, not derived (attention kernel inside whole steps,
// A/B on one GPU, against 3 : 5 without the unit term): with one class per KV head 2 : 4 + 12 (ragged batch of 32:
// 605 -> 554 us; batch 1 is not of this kind), with several classes 3 : 5 + 15 (batch 1: 27.3 -> 23.3 us; batch 8 with
// ragged trees: 167 -> 165 us, where 2 : 4 + 12 gave 175 us).
struct TileCosts { int one, two, unit; };
inline TileCosts tile_costs(int n_cls) { return n_cls == 1 ? TileCosts{2, 4, 12} : TileCosts{3, 5, 15}; }

struct SeqInfo {
    int M, Pb, nt;       // tree rows, prefix length, tiles of a unit (prefix tiles + the tree tile)
    int rows;            // live query rows of this class's unit (0: it does not exist for this sequence)
    int w;               // cost of one tile
    long long kv0;
};

template <bool PAGED>
__device__ __forceinline__ SeqInfo seq_info(const TcParams& P, int b, int pp) {
    const radar_attn_args& a = P.a;
    SeqInfo s;
    s.M = min(max(a.n_nodes[b], 0), kMaxNodes);
    s.Pb = a.prefix_len[b];
    s.kv0 = PAGED ? 0 : a.kv_start[b];          // paged: the host has checked max_pages * page_size >= max_prefix_len
    const bool ok = s.Pb >= 0 && s.Pb <= a.max_prefix_len && s.kv0 >= 0 && s.kv0 + s.Pb <= P.cache_rows;
    s.rows = ok ? min(max(s.M * P.G - pp * P.pair_rows, 0), P.pair_rows) : 0;
    s.nt = (max(s.Pb, 0) + kTileKeys - 1) / kTileKeys + 1;
    s.w = s.rows > 128 ? P.cost_two : P.cost_one;
    return s;
}
template <bool PAGED>
__device__ __forceinline__ long long seq_cost(const TcParams& P, int b, int pp) {
    const SeqInfo s = seq_info<PAGED>(P, b, pp);
    return s.rows > 0 ? (long long)P.a.Hkv * (s.nt * s.w + P.unit_cost) : 0;
}
// number of tiles of a unit (start position U, nt tiles of cost w) that start before position x
__device__ __forceinline__ int tiles_before(long long x, long long U, int nt, int w, int unit_cost) {
    const long long d = x - U - unit_cost;           // clamped first, so that the division is a 32-bit one
    if (d <= 0) return 0;
    if (d >= (long long)nt * w) return nt;
    return ((int)d + w - 1) / w;
}

// One CTA's walk over its range [.., hi) of the class's space: segments (sequence b, KV head g, tiles [t0, t1)).
template <bool PAGED>
struct Cursor {
    int b, g, t0, t1;
    int layer;           // layers follow one another in the space, each with the same sequence of units
    long long U, hi;     // start position of the current unit, end of the CTA's range
    int unit_cost;
    SeqInfo s;
    __device__ __forceinline__ bool valid() const { return t1 > t0; }
    __device__ __forceinline__ void clip() { t1 = tiles_before(hi, U, s.nt, s.w, unit_cost); }
    __device__ __forceinline__ void next_unit(const TcParams& P, int pp) {
        U += (long long)s.nt * s.w + unit_cost;
        t0 = 0;
        if (++g == P.a.Hkv) {
            g = 0;
            do {
                if (++b >= P.a.B) {                               // the next layer starts over at the first sequence
                    if (++layer >= P.n_layers) { t1 = 0; return; }
                    b = 0;
                }
                s = seq_info<PAGED>(P, b, pp);
            } while (s.rows == 0);
        }
        clip();
    }
    __device__ __forceinline__ void next(const TcParams& P, int pp) {
        if (t1 < s.nt) { t0 = t1; return; }                  // the range ended inside this unit
        next_unit(P, pp);
    }
    __device__ __forceinline__ bool complete() const { return t0 == 0 && t1 == s.nt; }
    __device__ __forceinline__ bool two_rb() const { return s.rows > 128; }
};

template <int D, bool TWO>
struct Smem {
    static constexpr int kHalves = D / 64;
    static constexpr int kQBlock = 128 * D * 2;
    static constexpr int kQBytes = (TWO ? 2 : 1) * kQBlock;
    static constexpr int kTileBytes = kTileKeys * D * 2;
    static constexpr int kRingK = 3;
    static constexpr int kRingV = TWO ? 2 : 3;
    static constexpr int kTotal = kQBytes + (kRingK + kRingV) * kTileBytes;
    static constexpr int kDynamic = kTotal;                 // starts on a 1024-byte boundary behind the static block
};

// TWO: the launch may contain units with two live row blocks; decides the shared-memory layout
// PAGED: the prefix cache is read through a block table (a separate instantiation, so that the contiguous
// layout's code is not touched by it)
template <int D, bool TWO, bool PAGED>
__global__ void __launch_bounds__(kTcThreads, 1)      // 18 warps are allocated as 20: 96 registers per thread
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKc,
                    const __grid_constant__ CUtensorMap tmVc, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, const TcParams P) {
    chain_trigger();                     // warp 0 waits for the predecessor below; the barrier, tensor-memory and
                                         // descriptor set-up of the other warps needs nothing from global memory
    using SM = Smem<D, TWO>;
    constexpr int H = SM::kHalves;
    constexpr int RK = SM::kRingK, RV = SM::kRingV;
    const radar_attn_args& a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pp = blockIdx.x % P.n_cls;                    // class
    const int ci = blockIdx.x / P.n_cls;
    const int G = P.G;

    // Static block first (padded to a multiple of 1024 bytes and aligned to it), the tiles behind it: the
    // swizzled tiles need a 1024-byte boundary and there is no room left for alignment slack.
    struct __align__(1024) Static {
        uint64_t bar_qfull, bar_qempty, bar_kfull[3], bar_kempty[3], bar_vfull[3], bar_vempty[3];
        uint64_t bar_sfull[2], bar_pready[2], bar_odone[2], bar_ofree[2];
        long long range[4];      // this CTA's range [lo, hi), size of the class's space (all layers), start of its first unit
        int start[3];            // sequence, KV head and layer of the unit that contains lo
        int start_pad;
        uint32_t tmem_base;
        int abort;
        float xm[128];           // group 1's running max at the end of a segment (one live row block)
        float mx[2][2][128];     // per group and column half: row maxima of a tile; row sums at the end of a segment
        unsigned char pad[kStaticSmem - (22 * 8 + 4 * 8 + 4 * 4 + 4 + 4 + 128 * 4 + 2 * 2 * 128 * 4)];
    };
    static_assert(sizeof(Static) == kStaticSmem, "static shared-memory block");
    __shared__ Static st;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = smem_raw;
    unsigned char* sQ = smem;
    unsigned char* sK = smem + SM::kQBytes;
    unsigned char* sV = sK + RK * SM::kTileBytes;
    uint64_t& bar_qfull = st.bar_qfull;
    uint64_t& bar_qempty = st.bar_qempty;
    uint64_t (&bar_kfull)[3] = st.bar_kfull;
    uint64_t (&bar_kempty)[3] = st.bar_kempty;
    uint64_t (&bar_vfull)[3] = st.bar_vfull;
    uint64_t (&bar_vempty)[3] = st.bar_vempty;
    uint64_t (&bar_sfull)[2] = st.bar_sfull;
    uint64_t (&bar_pready)[2] = st.bar_pready;
    uint64_t (&bar_odone)[2] = st.bar_odone;
    uint64_t (&bar_ofree)[2] = st.bar_ofree;
    uint32_t& s_tmem_base = st.tmem_base;
    int& s_abort = st.abort;
    float (&s_xm)[128] = st.xm;
    float (&s_mx)[2][2][128] = st.mx;
    float (&s_xl)[2][2][128] = st.mx;        // same storage: the two uses never overlap in time
    long long (&s_range)[4] = st.range;
    int (&s_start)[3] = st.start;
    const bool smem_aligned = (smem_u32(smem_raw) & 1023u) == 0;

    // ---- set-up: warp 0 finds this CTA's range while the barriers and tensor memory are prepared ----
    if (warp == 0) {
        chain_sync();                    // every global access of the CTA comes after the block barrier below
        long long tot = 0;
        for (int b0 = 0; b0 < a.B; b0 += 32) {
            const int b = b0 + lane;
            long long sz = b < a.B ? seq_cost<PAGED>(P, b, pp) : 0;
            if (pp == 0 && ci == 0 && b < a.B) {
                const int Pb = a.prefix_len[b];
                const long long kv0 = PAGED ? 0 : a.kv_start[b];
                if (Pb < 0 || Pb > a.max_prefix_len || kv0 < 0 || kv0 + Pb > P.cache_rows) set_status(P.status, RADAR_ERR_INVALID_ARG);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sz += __shfl_xor_sync(kFull, sz, o);
            tot += sz;
        }
        // the space of all layers: layer l occupies [l * tot, (l + 1) * tot)
        const long long tot_all = tot * P.n_layers;
        const long long lo_all = tot_all * ci / P.ncc, hi = tot_all * (ci + 1) / P.ncc;
        const int layer0 = tot > 0 ? (int)(lo_all / tot) : 0;
        const long long lo = lo_all - (long long)layer0 * tot;
        long long cum = 0, fU = 0;
        int fb = -1, fg = 0;
        for (int b0 = 0; b0 < a.B && fb < 0; b0 += 32) {
            const int b = b0 + lane;
            const long long sz = b < a.B ? seq_cost<PAGED>(P, b, pp) : 0;
            long long incl = sz;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long v = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += v;
            }
            const unsigned hit = __ballot_sync(kFull, cum + incl > lo);
            if (hit) {
                const int src = __ffs(hit) - 1;
                const long long before = cum + __shfl_sync(kFull, incl - sz, src);
                fb = b0 + src;
                const SeqInfo si = seq_info<PAGED>(P, fb, pp);
                const long long unit = (long long)si.nt * si.w + P.unit_cost;
                fg = (int)((lo - before) / unit);
                fU = before + fg * unit;
            }
            cum += __shfl_sync(kFull, incl, 31);
        }
        if (lane == 0) {
            s_range[0] = lo_all; s_range[1] = hi; s_range[2] = tot_all; s_range[3] = fU + (long long)layer0 * tot;
            s_start[0] = layer0 < P.n_layers ? fb : -1; s_start[1] = fg; s_start[2] = layer0;
        }
    } else if (warp == 1) {
        if (lane == 0) {
            s_abort = 0;
            mbar_init(&bar_qfull, 1);
            mbar_init(&bar_qempty, 1);
            for (int i = 0; i < 3; ++i) {
                mbar_init(&bar_kfull[i], 1); mbar_init(&bar_kempty[i], 1);
                mbar_init(&bar_vfull[i], 1); mbar_init(&bar_vempty[i], 1);
            }
            for (int i = 0; i < 2; ++i) {
                mbar_init(&bar_sfull[i], 1); mbar_init(&bar_pready[i], 8);
                mbar_init(&bar_odone[i], 1); mbar_init(&bar_ofree[i], 8);
            }
            fence_barrier_init();
        }
    } else if (warp == kProducerWarp) {
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
    const uint32_t tmem = s_tmem_base;      // columns: S/P buffers at 0 and 128, O accumulators at 256 and 384
    volatile int* ab = &s_abort;

    // first segment: the unit that contains the range's start, from its first tile starting at or after it
    Cursor<PAGED> cur;
    cur.b = s_start[0]; cur.g = s_start[1]; cur.layer = s_start[2];
    cur.hi = s_range[1];
    cur.unit_cost = P.unit_cost;
    cur.U = s_range[3];
    cur.t0 = cur.t1 = 0;
    if (cur.b >= 0) {
        cur.s = seq_info<PAGED>(P, cur.b, pp);
        cur.t0 = tiles_before(s_range[0], cur.U, cur.s.nt, cur.s.w, P.unit_cost);
        if (cur.t0 >= cur.s.nt) cur.next_unit(P, pp);       // every tile of that unit starts before the range
        else cur.clip();
    }
    if (!cur.valid() || !smem_aligned) {                    // nothing for this CTA (uniform)
        if (tid == 0) {
            P.cut[blockIdx.x].valid = 0;
            if (!smem_aligned) set_status(P.status, RADAR_ERR_CUDA);   // the tiles would not sit on their swizzle boundary
        }
        tc_fence_before_sync();
        __syncthreads();
        if (warp == kProducerWarp) tmem_dealloc(tmem, 512);
        return;
    }

    if (warp == kProducerWarp) {
        // =================================== TMA producer ===================================
        // One lane does everything for the contiguous cache.  With a paged cache the whole warp walks the same
        // loop and lane p looks up and fetches page p of a tile (up to eight boxes per tile), the leading lane
        // still doing the waits, the byte counts, Q and the tree tile.
        if (PAGED || lane == 0) {
            const bool lead = lane == 0;
            uint32_t kc = 0, vc = 0;
            bool ok = true;
            CutUnit cu;
            cu.valid = 0;
            for (uint32_t seg = 0; cur.valid(); cur.next(P, pp), ++seg) {
                const int b = cur.b, g = cur.g, n = cur.t1 - cur.t0;
                const bool two = TWO && cur.two_rb();
                if (cur.t0 == 0 && cur.t1 < cur.s.nt) {          // necessarily the last segment of this CTA
                    cu.valid = 1; cu.b = b; cu.g = g; cu.nt = cur.s.nt; cu.slot = seg == 0 ? 0 : 1; cu.layer = cur.layer;
                    cu.rows = cur.s.rows; cu.w = cur.s.w; cu.u0 = cur.U; cu.tot = s_range[2];
                }
                if (lead) ok = ok && mbar_wait(&bar_qempty, (seg & 1) ^ 1, ab);
                if (lead && ok) {
                    mbar_arrive_expect_tx(&bar_qfull, two ? 2 * SM::kQBlock : SM::kQBlock);
                    for (int q = 0; q < (two ? 2 : 1); ++q)
                        for (int h = 0; h < H; ++h)
                            tma_load_4d(sQ + q * SM::kQBlock + h * (128 * 128), &tmQ, &bar_qfull, h * 64, g * G,
                                        b * kMaxNodes + (pp * (P.pair_rows / 128) + q) * P.nodes_per_rb, cur.layer);
                }
                auto load_tile = [&](int t, bool is_k) {
                    uint32_t& cnt = is_k ? kc : vc;
                    const int ring = is_k ? RK : RV;
                    const int slot = cnt % ring;
                    const uint32_t use = cnt / ring;
                    ++cnt;
                    uint64_t* full = is_k ? &bar_kfull[slot] : &bar_vfull[slot];
                    uint64_t* empty = is_k ? &bar_kempty[slot] : &bar_vempty[slot];
                    unsigned char* dst = (is_k ? sK : sV) + slot * SM::kTileBytes;
                    if (lead && (!ok || !mbar_wait(empty, (use & 1) ^ 1, ab))) ok = false;
                    if (PAGED) ok = __shfl_sync(kFull, ok, 0);
                    if (!ok) return;
                    if (t == cur.s.nt - 1) {
                        if (lead) {
                            mbar_arrive_expect_tx(full, kTreeKeys * D * 2);
                            for (int h = 0; h < H; ++h)
                                tma_load_4d(dst + h * (kTreeKeys * 128), is_k ? &tmKt : &tmVt, full, h * 64, g, b * kMaxNodes, cur.layer);
                        }
                    } else if (!PAGED) {
                        mbar_arrive_expect_tx(full, kTileKeys * D * 2);
                        const int row = (int)(cur.s.kv0 + (long long)t * kTileKeys);
                        for (int h = 0; h < H; ++h)
                            tma_load_4d(dst + h * (kTileKeys * 128), is_k ? &tmKc : &tmVc, full, h * 64, g, row, cur.layer);
                    } else {
                        // paged cache: one box per page (or per tile when a page holds whole tiles); only pages
                        // that hold live keys are fetched, what stays stale in the slot is masked / never read
                        const int ps = a.page_size, per = min(ps, kTileKeys);
                        const int key0 = t * kTileKeys;
                        const int n_ld = (min(kTileKeys, cur.s.Pb - key0) + per - 1) / per;
                        const long long n_cache_pages = P.cache_rows / ps;
                        if (lead) mbar_arrive_expect_tx(full, n_ld * per * D * 2);
                        __syncwarp();
                        if (const int p = lane; p < n_ld) {
                            const int key = key0 + p * per;
                            long long page = __ldg(a.block_table + (long long)b * a.max_pages + key / ps);
                            if (page < 0 || page >= n_cache_pages) { set_status(P.status, RADAR_ERR_INVALID_ARG); page = 0; }
                            const int row = (int)(page * ps + key % ps);
                            for (int h = 0; h < H; ++h)
                                tma_load_4d(dst + h * (kTileKeys * 128) + p * per * 128, is_k ? &tmKc : &tmVc, full, h * 64, g, row, cur.layer);
                        }
                    }
                };
                // same order as the MMA warp consumes: the first K tile(s), then V(i), K(i + lookahead)
                const int la = two ? 1 : 2;
                for (int i = 0; i < la && i < n; ++i) load_tile(cur.t0 + i, true);
                for (int i = 0; i < n; ++i) {
                    load_tile(cur.t0 + i, false);
                    if (i + la < n) load_tile(cur.t0 + i + la, true);
                }
            }
            if (lead) P.cut[blockIdx.x] = cu;
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // =================================== MMA issuer ===================================
        // The warp runs converged: every lane waits on the barriers and executes the same straight-line issue
        // sequences with warp-uniform descriptor words, and the elected lane issues the instructions and the
        // commits (predicated, no branch around them).  Whatever this warp executes between two MMAs costs
        // tensor-pipe time, so no control flow depends on a wait's outcome: after a wait that ran out the
        // predicate is off and the loops run dry.
        constexpr uint32_t idesc_s128 = idesc_bf16_f32(128, kTileKeys, false, false);
        constexpr uint32_t idesc_s64 = idesc_bf16_f32(128, kTreeKeys, false, false);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
        // high word of every shared-memory descriptor (stride between 8-row groups 1024 B, version, swizzle)
        constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
        const uint32_t q_lo = ((smem_u32(sQ) & 0x3ffff) >> 4) | (1u << 16);
        const uint32_t k_lo = ((smem_u32(sK) & 0x3ffff) >> 4) | (1u << 16);
        const uint32_t v_lo = (smem_u32(sV) & 0x3ffff) >> 4;
        const uint32_t elected = elect_one();
        uint32_t k_next = 0, k_par = 0, v_next = 0, v_par = 0;   // ring slot to take next and its phase parity
        uint32_t p_par[2] = {0, 0};              // phase parity of the next P tile per group
        bool ok = true;
        // The segment's shape comes from global memory; passing it through a broadcast from lane 0 tells the
        // compiler that it is the same in every lane, so that the loops below and the descriptor arithmetic in
        // them stay on the uniform datapath (this warp's own instruction stream is what bounds the issue rate).
        auto uni = [](int v) { return __shfl_sync(kFull, v, 0); };
        for (uint32_t seg = 0; uni(cur.valid()); cur.next(P, pp), ++seg) {
            const int seg_t0 = uni(cur.t0);
            const int n = uni(cur.t1) - seg_t0;
            const bool two = TWO && uni(cur.two_rb());
            const int M = uni(cur.s.M), Pb = uni(cur.s.Pb), nt_unit = uni(cur.s.nt);
            ok = ok && mbar_wait(&bar_qfull, seg & 1, ab);
            uint32_t k_slot = 0, v_slot = 0;      // ring slots of the K and V tiles in use
            bool acc[2] = {false, false};         // accumulator holds a product of this segment

            // ---- O[q] (+)= P[q] V for tile i (q is a literal at every call site) ----
            auto pv = [&](const int q, const int i, const bool fresh_v, const bool release_v) {
                const bool tree = seg_t0 + i == nt_unit - 1;
                const int nk = tree ? kTreeKeys : kTileKeys;
                const int valid = tree ? M : min(kTileKeys, Pb - (seg_t0 + i) * kTileKeys);
                const int ksteps = (valid + 15) >> 4;
                ok = ok && mbar_wait(&bar_pready[q], p_par[q], ab);
                p_par[q] ^= 1;
                if (fresh_v) {
                    v_slot = v_next;
                    ok = ok && mbar_wait(&bar_vfull[v_slot], v_par, ab);
                    if (++v_next == RV) { v_next = 0; v_par ^= 1; }
                    if (valid < ksteps * 16) {
                        // rows past the last live key meet P = 0; they must not hold NaN/Inf bit patterns
                        unsigned char* vtile = sV + v_slot * SM::kTileBytes;
                        const int nrows = ksteps * 16 - valid;
                        for (int e = lane; e < nrows * 8 * H; e += 32) {
                            const int h = e / (nrows * 8), rem = e % (nrows * 8);
                            const int r = valid + rem / 8, c = rem % 8;
                            *reinterpret_cast<uint4*>(vtile + h * (nk * 128) + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                    }
                    if (i == 0) {                 // the previous segment's epilogue has read both accumulators
                        ok = ok && mbar_wait(&bar_ofree[0], (seg & 1) ^ 1, ab);
                        ok = ok && mbar_wait(&bar_ofree[1], (seg & 1) ^ 1, ab);
                    }
                }
                tc_fence_after_sync();
                const uint32_t go = ok ? elected : 0u;
                // V is consumed N-major: 16 keys are 2048 B; 64-column blocks are nk * 128 B apart
                const uint32_t b_lo = (v_lo + v_slot * (SM::kTileBytes >> 4)) | ((uint32_t)(nk * 128 >> 4) << 16);
                // P of the first half of the tile's keys sits at column 0 of the group's buffer, of the second half
                // at column 64 (each softmax thread writes inside its own column range)
                const int hs = tree ? 2 : 4;
                const uint32_t n1 = (uint32_t)min(ksteps, hs), n2 = (uint32_t)ksteps - n1;
                mma_ts_x4(go, n1, tmem + 256 + q * 128, tmem + q * 128, b_lo, kDescHi, idesc_pv, acc[q]);
                mma_ts_x4(go, n2, tmem + 256 + q * 128, tmem + q * 128 + 64, b_lo + hs * 128, kDescHi, idesc_pv, true);
                acc[q] = true;
                if (release_v) mma_commit_if(go, &bar_vempty[v_slot]);
                if (two ? i == n - 1 : i + 2 >= n) mma_commit_if(go, &bar_odone[q]);
            };
            // ---- S[q] = Q K^T for tile si.  Nothing in tensor memory changes hands here: K arrives through the
            // async proxy, and the buffer was last read by this thread's own P V, which runs first. ----
            auto qk = [&](const int q, const int si, const bool fresh_k, const bool release_k) {
                if (fresh_k) {
                    k_slot = k_next;
                    ok = ok && mbar_wait(&bar_kfull[k_slot], k_par, ab);
                    if (++k_next == RK) { k_next = 0; k_par ^= 1; }
                }
                const uint32_t go = ok ? elected : 0u;
                const bool tree = seg_t0 + si == nt_unit - 1;
                const uint32_t a0 = q_lo + (two ? q : 0) * (SM::kQBlock >> 4);
                const uint32_t b0 = k_lo + k_slot * (SM::kTileBytes >> 4);
                const uint32_t idesc = tree ? idesc_s64 : idesc_s128;
                mma_ss_x4(go, tmem + q * 128, a0, b0, kDescHi, idesc, false);
                if (D == 128)                     // second 64-column block of Q and K
                    mma_ss_x4(go, tmem + q * 128, a0 + (128 * 128 >> 4), b0 + ((uint32_t)((tree ? kTreeKeys : kTileKeys) * 128) >> 4),
                              kDescHi, idesc, true);
                if (release_k) mma_commit_if(go, &bar_kempty[k_slot]);
                mma_commit_if(go, &bar_sfull[q]);
                // the last S of the segment: Q may be overwritten once it has run
                if (si == n - 1 && release_k) mma_commit_if(go, &bar_qempty);
            };
            // Schedule.  Two live row blocks: group s owns row block s; per tile PV0(i) S0(i+1) PV1(i) S1(i+1),
            // both groups sharing K(i+1) and V(i).  One live row block: the groups take alternate tiles,
            // PV(i) S(i+2) for group i & 1.  S of the first tile(s) comes from the iterations with i < 0.
            // Steady state (both tiles involved are full prefix tiles): the same steps with nothing to decide,
            // so that the issuing warp executes as few instructions per MMA as possible.
            const uint32_t a_q0 = q_lo, a_q1 = q_lo + (SM::kQBlock >> 4);
            auto wait_all = [&](uint64_t* bar, uint32_t parity) { ok = mbar_wait(bar, parity, ab) && ok; };
            auto pv_full = [&](const int q, const bool fresh_v, const bool release_v) {
                wait_all(&bar_pready[q], p_par[q]);
                p_par[q] ^= 1;
                if (fresh_v) {
                    v_slot = v_next;
                    wait_all(&bar_vfull[v_slot], v_par);
                    if (++v_next == RV) { v_next = 0; v_par ^= 1; }
                }
                tc_fence_after_sync();
                const uint32_t go = ok ? elected : 0u;
                const uint32_t b_lo = (v_lo + v_slot * (SM::kTileBytes >> 4)) | ((uint32_t)(kTileKeys * 128 >> 4) << 16);
                mma_ts_x4_full(go, tmem + 256 + q * 128, tmem + q * 128, b_lo, kDescHi, idesc_pv, acc[q]);
                mma_ts_x4_full(go, tmem + 256 + q * 128, tmem + q * 128 + 64, b_lo + 4 * 128, kDescHi, idesc_pv, true);
                acc[q] = true;
                if (release_v) mma_commit_if(go, &bar_vempty[v_slot]);
            };
            auto qk_full = [&](const int q, const uint32_t a0, const bool fresh_k, const bool release_k) {
                if (fresh_k) {
                    k_slot = k_next;
                    wait_all(&bar_kfull[k_slot], k_par);
                    if (++k_next == RK) { k_next = 0; k_par ^= 1; }
                }
                const uint32_t go = ok ? elected : 0u;
                const uint32_t b0 = k_lo + k_slot * (SM::kTileBytes >> 4);
                mma_ss_x4(go, tmem + q * 128, a0, b0, kDescHi, idesc_s128, false);
                if (D == 128) mma_ss_x4(go, tmem + q * 128, a0 + (128 * 128 >> 4), b0 + (kTileKeys * 128 >> 4), kDescHi, idesc_s128, true);
                if (release_k) mma_commit_if(go, &bar_kempty[k_slot]);
                mma_commit_if(go, &bar_sfull[q]);
            };
            const int n_full = min(n, Pb / kTileKeys - seg_t0);   // tiles [0, n_full) of the segment are full prefix tiles
            if (two) {
                for (int i = -1; i < n; ++i) {
                    if (i >= 0 && i + 2 < n_full) {           // tiles i and i+1 full, and S(i+1) is not the segment's last
                        pv_full(0, true, false);
                        qk_full(0, a_q0, true, false);
                        pv_full(1, false, true);
                        qk_full(1, a_q1, false, true);
                    } else {
                        if (i >= 0) pv(0, i, true, false);
                        if (i + 1 < n) qk(0, i + 1, true, false);
                        if (i >= 0) pv(1, i, false, true);
                        if (i + 1 < n) qk(1, i + 1, false, true);
                    }
                }
            } else {
                for (int i = -2; i < n; ++i) {
                    const bool fast = i >= 0 && i + 3 < n_full;   // tiles i and i+2 full, S(i+2) not the last
                    if (i & 1) {
                        if (fast) { pv_full(1, true, true); qk_full(1, a_q0, true, true); }
                        else {
                            if (i >= 0) pv(1, i, true, true);
                            if (i + 2 < n) qk(1, i + 2, true, true);
                        }
                    } else {
                        if (fast) { pv_full(0, true, true); qk_full(0, a_q0, true, true); }
                        else {
                            if (i >= 0) pv(0, i, true, true);
                            if (i + 2 < n) qk(0, i + 2, true, true);
                        }
                    }
                }
            }
        }
        __syncwarp();
    } else {
        // =================================== softmax groups ===================================
        // Two threads per query row: warp w of a group's eight serves tensor-memory lanes 32 (w & 3) .. + 31
        // and the column half (w >> 2) & 1, so a row's 128 scores are exponentiated by two threads at once
        // and the chain S -> softmax -> P V of a group is about half as long.
        const int grp = warp >> 3;
        const int half = (warp >> 2) & 1;
        const int row = (warp & 3) * 32 + lane;                 // row of the block == tensor-memory lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + grp * 128 + lane_addr;
        const uint32_t tO = tmem + 256 + grp * 128 + lane_addr;
        const uint32_t tO_other = tmem + 256 + (grp ^ 1) * 128 + lane_addr;
        constexpr int DH = D / 2;                               // accumulator columns per thread
        uint32_t sc = 0, oc = 0;                 // S tiles and accumulators this group has waited for
        bool ok = true;
        for (uint32_t seg = 0; cur.valid(); cur.next(P, pp), ++seg) {
            const int b = cur.b, g = cur.g, n = cur.t1 - cur.t0;
            const bool two = TWO && cur.two_rb();
            const int M = cur.s.M, Pb = cur.s.Pb, nt_unit = cur.s.nt;
            const int prow = (two ? grp * 128 : 0) + row;        // row within the unit
            const int r_glob = pp * P.pair_rows + prow;
            const int node = r_glob >> P.g_log2;
            const int hq = g * G + (r_glob & (G - 1));
            const bool row_live = prow < cur.s.rows;
            // A warp none of whose 32 rows is live does no arithmetic (the products of its rows are never read):
            // it only keeps the barriers going.
            const bool warp_live = prow - lane < cur.s.rows;
            const unsigned long long live_bits = M >= 64 ? ~0ull : ((1ull << M) - 1ull);
            // the row's ancestor word is needed by the tree tile only (the unit's last): it is loaded here and first
            // touched there, so that the segment does not start with a wait for global memory
            const unsigned long long mask_word = a.mask[(int64_t)b * kMaxNodes + min(node, kMaxNodes - 1)];
            const int n_my = two ? n : (n - grp + 1) >> 1;
            float m_run = -CUDART_INF_F, l_run = 0.f;            // l_run: this thread's columns only

            for (int j = 0; j < n_my; ++j) {
                const int i = two ? j : 2 * j + grp;             // local tile index
                const int t = cur.t0 + i;
                ok = __all_sync(kFull, ok && mbar_wait(&bar_sfull[grp], sc & 1, ab));    // warp-uniform: guards .aligned ops
                ++sc;
                tc_fence_after_sync();
                // This thread's chunks of 32 score columns: a prefix tile has four (two per thread), the tree tile
                // two (one per thread).  Half h of a row works in columns 64 h .. 64 h + 63 of the buffer only: its
                // scores sit there (the tree tile's second chunk is read from columns 32 .. 63 but belongs to
                // half 1 alone) and its P goes to columns 64 h + 16 cc, so the halves never touch each other's
                // columns and a thread overwrites only scores it has already taken into registers.
                const bool tree = t == nt_unit - 1;
                const int nch = tree ? 1 : 2;
                const int c0 = tree ? half : 2 * half;
                const int valid = tree ? kTreeKeys : min(kTileKeys, Pb - t * kTileKeys);
                const bool partial = tree || valid < kTileKeys;
                auto allowed_bits = [&](int c) -> uint32_t {        // keys of chunk c this row may attend to
                    if (tree) return row_live ? (uint32_t)((mask_word & live_bits) >> (c * 32)) : 0u;
                    const int lim = valid - c * 32;
                    return lim >= 32 ? 0xffffffffu : (lim <= 0 ? 0u : ((1u << lim) - 1u));
                };
                float mx = -CUDART_INF_F;
                if (ok && warp_live) {
#pragma unroll 1
                    for (int cc = 0; cc < nch; ++cc) {
                        uint32_t sv[32];
                        tmem_ld32(tS + (c0 + cc) * 32, sv);
                        tmem_wait_ld();
                        if (partial) {
                            const uint32_t al = allowed_bits(c0 + cc);
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (!((al >> e) & 1u)) sv[e] = 0xff800000u;     // -inf
                        }
                        float mxa[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                        for (int e = 0; e < 32; e += 2)                     // three-input maxima: half the instructions
                            mxa[(e >> 1) & 3] = max3(mxa[(e >> 1) & 3], __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
                        mx = fmaxf(mx, fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3])));
                    }
                }
                // the two halves of a row exchange their maxima
                s_mx[grp][half][row] = mx;
                if (grp == 0) asm volatile("bar.sync 1, 256;" ::: "memory"); else asm volatile("bar.sync 2, 256;" ::: "memory");
                if (ok && warp_live) {
                    mx = fmaxf(mx, s_mx[grp][half ^ 1][row]);
                    // ---- running max (log2 units), lazy rescale decision: the same in both halves of a row ----
                    const float m_tile = mx * P.scale_log2;
                    float factor = 1.f;
                    if (j == 0) {
                        m_run = m_tile;
                    } else if (m_tile > m_run + kRescaleThreshold) {
                        factor = ex2(m_run - m_tile);           // m_run may be -inf: factor 0 clears O and l
                        m_run = m_tile;
                    }
                    const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;
                    // ---- P = exp2(s * scale - m), row sum, bf16 pairs back to tensor memory ----
                    // (the scaling and the row sum work on pairs: one packed fp32x2 instruction per two values)
                    float2 ls[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                    const float2 sc2 = make_float2(P.scale_log2, P.scale_log2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll 1
                    for (int cc = 0; cc < nch; ++cc) {
                        uint32_t sv[32];
                        tmem_ld32(tS + (c0 + cc) * 32, sv);
                        tmem_wait_ld();
                        if (partial) {
                            const uint32_t al = allowed_bits(c0 + cc);
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (!((al >> e) & 1u)) sv[e] = 0xff800000u;
                        }
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float2 t = __ffma2_rn(make_float2(__uint_as_float(sv[2 * e]), __uint_as_float(sv[2 * e + 1])), sc2, nm2);
                            const float p0 = ex2(t.x), p1 = ex2(t.y);
                            ls[e & 1] = __fadd2_rn(ls[e & 1], make_float2(p0, p1));
                            const __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
                            pk[e] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                        tmem_st16(tS + half * 64 + cc * 16, pk);
                    }
                    l_run = l_run * factor + ((ls[0].x + ls[0].y) + (ls[1].x + ls[1].y));
                    // ---- rescale this thread's half of the accumulator when some row of the warp moved its max ----
                    if (j > 0 && __any_sync(kFull, factor != 1.f)) {
#pragma unroll 1
                        for (int c = 0; c < DH / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tO + half * DH + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
                            tmem_st32(tO + half * DH + c * 32, o);
                        }
                    }
                    tmem_wait_st();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_pready[grp]);
            }

            // ---- epilogue of the segment ----
            if (n_my > 0) {
                ok = __all_sync(kFull, ok && mbar_wait(&bar_odone[grp], oc & 1, ab));
                ++oc;
            }
            tc_fence_after_sync();
            const bool final_rows = cur.complete();
            const int slot = seg == 0 ? 0 : 1;                   // a CTA has at most a cut first and a cut last segment
            const int64_t rec = ((int64_t)blockIdx.x * 2 + slot) * kPairRows + prow;
            // the row sum is the two halves' sums; with one live row block group 1 also hands its (m, l) to group 0
            s_xl[grp][half][row] = l_run;
            if (grp == 1 && half == 0) s_xm[row] = n_my > 0 ? m_run : -CUDART_INF_F;
            asm volatile("bar.sync 3, 512;" ::: "memory");
            float l_out = s_xl[grp][0][row] + s_xl[grp][1][row];
            float m_out = m_run, w0 = 1.f, w1 = 0.f;
            bool writer = true, merge_any = false;
            if (!two) {
                // group 0 merges group 1's accumulator, which sits in the same tensor-memory lanes
                writer = grp == 0;
                if (writer) {
                    const float m1 = s_xm[row], l1 = s_xl[1][0][row] + s_xl[1][1][row];
                    const bool merge = m1 != -CUDART_INF_F;
                    m_out = fmaxf(m_run, m1);
                    const float ms = m_out == -CUDART_INF_F ? 0.f : m_out;
                    w0 = ex2(m_run - ms);                        // exp2(-inf) = 0
                    w1 = ex2(m1 - ms);
                    l_out = l_out * w0 + l1 * w1;
                    merge_any = __any_sync(kFull, merge);        // rows that do not merge carry w1 = 0
                }
            }
            if (writer && ok && warp_live) {
                const float m_safe = m_out == -CUDART_INF_F ? 0.f : m_out;
                const float inv = final_rows ? 1.f / l_out : 1.f;
                const int64_t out_row = ((int64_t)b * kMaxNodes + node) * a.Hq + hq;
#pragma unroll 1
                for (int c = 0; c < DH / 32; ++c) {
                    const int col = half * DH + c * 32;          // first accumulator column of this chunk
                    uint32_t o[32];
                    tmem_ld32(tO + col, o);
                    tmem_wait_ld();
                    float v[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(o[e]) * w0;
                    if (merge_any) {
                        tmem_ld32(tO_other + col, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = fmaf(__uint_as_float(o[e]), w1, v[e]);
                    }
                    if (row_live) {
                        if (final_rows) {
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.O) + cur.layer * P.o_ls + out_row * D + col;
                            const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31) == 0;
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                uint32_t w[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const __nv_bfloat162 t2 = __floats2bfloat162_rn(v[q * 16 + 2 * e] * inv, v[q * 16 + 2 * e + 1] * inv);
                                    w[e] = *reinterpret_cast<const uint32_t*>(&t2);
                                }
                                if (wide) {
                                    st_global_32b(dst + q * 16, w);
                                } else {
                                    *reinterpret_cast<uint4*>(dst + q * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                                    *reinterpret_cast<uint4*>(dst + q * 16 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
                                }
                            }
                        } else {
                            float* dst = P.part_o + rec * D + col;          // 128-byte aligned (workspace carve)
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                uint32_t w[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(v[q * 8 + e]);
                                st_global_32b(dst + q * 8, w);
                            }
                        }
                    }
                }
                if (row_live && half == 0) {
                    const float m_nat = m_safe * 0.6931471805599453f;
                    if (final_rows) {
                        if (a.lse != nullptr) a.lse[cur.layer * P.lse_ls + ((int64_t)b * a.Hq + hq) * kMaxNodes + node] = m_nat + logf(l_out);
                    } else {
                        P.part_ml[rec] = make_float2(m_out == -CUDART_INF_F ? -CUDART_INF_F : m_nat, l_out);
                    }
                }
            }
            asm volatile("bar.sync 4, 512;" ::: "memory");       // the exchanged (m, l) and group 1's accumulator have been read
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_ofree[grp]);
        }
    }

    // ---- teardown ----
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kProducerWarp) {
        if (s_abort) {
            // let loads that are still in flight land before the CTA's shared memory is released
            if (lane == 0) {
                int dummy = 0;
                for (int i = 0; i < 3; ++i) {
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

// Merges the pieces of the units that were cut across CTAs.  Block (c, y): CTA c of the attention
// kernel holds the first piece of a cut unit (or the block exits); the following CTAs of the same
// class hold the rest, each as its first segment.  A warp owns up to eight query rows
// (y * 8 + warp + 32 r); it works out the unit's pieces once and fetches four rows at a time, every
// piece of them in flight together.
constexpr int kCombineY = 4;                 // blocks per cut unit: 4 * 8 warps * 8 rows = 256 rows
template <int D>
__global__ void __launch_bounds__(256) tree_attn_tc_combine_kernel(const TcParams P) {
    chain_wait();
    const radar_attn_args& a = P.a;
    const CutUnit cu = P.cut[blockIdx.x];
    if (!cu.valid) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pp = blockIdx.x % P.n_cls, c0 = blockIdx.x / P.n_cls;
    const long long u1 = cu.u0 + (long long)cu.nt * cu.w + P.unit_cost;
    const int row0 = blockIdx.y * 8 + warp;
    if (row0 >= cu.rows) return;                             // rows of a unit are live from 0 up
    // pieces: class-local CTAs c0, c0 + 1, ... while their range starts before the unit's end
    int n_pieces = 1;
    while (c0 + n_pieces < P.ncc && cu.tot * (c0 + n_pieces) / P.ncc < u1) ++n_pieces;
    const int G = P.G;
    constexpr int E = D / 32;                                // output elements per lane
    auto rec_of = [&](int j) {                               // record of row 0 of piece j
        const int slot = j == 0 ? cu.slot : 0;
        return ((int64_t)((c0 + j) * P.n_cls + pp) * 2 + slot) * kPairRows;
    };
    auto live = [&](int j) {                                 // a CTA whose range holds no tile start has no piece
        return tiles_before(cu.tot * (c0 + j + 1) / P.ncc, cu.u0, cu.nt, cu.w, P.unit_cost) >
               tiles_before(cu.tot * (c0 + j) / P.ncc, cu.u0, cu.nt, cu.w, P.unit_cost);
    };
    auto store_row = [&](int prow, const float (&o)[E], float mx, float den) {
        const float inv = 1.f / den;
        const int r_glob = pp * P.pair_rows + prow;
        const int node = r_glob / G, hq = cu.g * G + r_glob % G;
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.O) + cu.layer * P.o_ls + (((int64_t)cu.b * kMaxNodes + node) * a.Hq + hq) * D + lane * E;
#pragma unroll
        for (int q = 0; q < E; q += 2) *reinterpret_cast<__nv_bfloat162*>(dst + q) = __floats2bfloat162_rn(o[q] * inv, o[q + 1] * inv);
        if (a.lse != nullptr && lane == 0) a.lse[cu.layer * P.lse_ls + ((int64_t)cu.b * a.Hq + hq) * kMaxNodes + node] = mx + logf(den);
    };

    if (n_pieces <= 4) {
        // ---- the usual case: a unit spread over a few CTAs ----
        int64_t rec[4];
        bool on[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { on[j] = j < n_pieces && live(j); rec[j] = rec_of(min(j, n_pieces - 1)); }
        for (int rb = 0; rb < 8; rb += 4) {
            if (row0 + 32 * rb >= cu.rows) break;
            float2 ml[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int prow = row0 + 32 * (rb + r);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    ml[r][j] = on[j] && prow < cu.rows ? P.part_ml[rec[j] + prow] : make_float2(-CUDART_INF_F, 0.f);
            }
            float v[4][4][E];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int prow = row0 + 32 * (rb + r);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool take = on[j] && prow < cu.rows;
                    const float* src = P.part_o + (rec[j] + (take ? prow : 0)) * D + lane * E;
                    if (E == 4) {
                        const float4 t = take ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
                        v[r][j][0] = t.x; v[r][j][1] = t.y; v[r][j][E - 2] = t.z; v[r][j][E - 1] = t.w;
                    } else {
                        const float2 t = take ? *reinterpret_cast<const float2*>(src) : make_float2(0.f, 0.f);
                        v[r][j][0] = t.x; v[r][j][1] = t.y;
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int prow = row0 + 32 * (rb + r);
                if (prow >= cu.rows) break;
                const float mx = fmaxf(fmaxf(ml[r][0].x, ml[r][1].x), fmaxf(ml[r][2].x, ml[r][3].x));
                float den = 0.f, o[E];
#pragma unroll
                for (int q = 0; q < E; ++q) o[q] = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float w = ml[r][j].x == -CUDART_INF_F ? 0.f : __expf(ml[r][j].x - mx);
                    den = fmaf(ml[r][j].y, w, den);
#pragma unroll
                    for (int q = 0; q < E; ++q) o[q] = fmaf(v[r][j][q], w, o[q]);
                }
                store_row(prow, o, mx, den);
            }
        }
        return;
    }

    // ---- a unit spread over many CTAs (very long prefixes): one row at a time, lane j holds piece j's (m, l) ----
    for (int prow = row0; prow < cu.rows; prow += 32) {
        float den = 0.f, mx = -CUDART_INF_F, o[E];
#pragma unroll
        for (int q = 0; q < E; ++q) o[q] = 0.f;
        for (int j0 = 0; j0 < n_pieces; j0 += 32) {
            const int jl = j0 + lane;
            float2 ml = make_float2(-CUDART_INF_F, 0.f);
            if (jl < n_pieces && live(jl)) ml = P.part_ml[rec_of(jl) + prow];
            const float mnew = fmaxf(mx, warp_max(ml.x));
            if (mnew == -CUDART_INF_F) continue;
            const float rescale = __expf(mx - mnew);             // 0 on the first live batch
            den *= rescale;
#pragma unroll
            for (int q = 0; q < E; ++q) o[q] *= rescale;
            mx = mnew;
            const float wl = ml.x == -CUDART_INF_F ? 0.f : __expf(ml.x - mx);
            den += warp_sum(ml.y * wl);
            const int nb = min(32, n_pieces - j0);
            for (int u0 = 0; u0 < nb; u0 += 4) {
                float v[4][E], w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    w[u] = u0 + u < nb ? __shfl_sync(kFull, wl, u0 + u) : 0.f;
                    const float* src = P.part_o + (rec_of(j0 + min(u0 + u, nb - 1)) + prow) * D + lane * E;
#pragma unroll
                    for (int q = 0; q < E; ++q) v[u][q] = w[u] != 0.f ? src[q] : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int q = 0; q < E; ++q) o[q] = fmaf(v[u][q], w[u], o[q]);
            }
        }
        store_row(prow, o, mx, den);
    }
}

// The same merge for launches with few cut units, where latency counts: block (c, y): CTA c of the attention
// kernel holds the first piece of a cut unit (or the block exits); the following CTAs of the same
// class hold the rest, each as its first segment.  One warp per query row, 8 rows per block.
template <int D>
__global__ void __launch_bounds__(256) tree_attn_tc_combine_wide_kernel(const TcParams P) {
    chain_wait();
    const radar_attn_args& a = P.a;
    const CutUnit cu = P.cut[blockIdx.x];
    if (!cu.valid) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pp = blockIdx.x % P.n_cls, c0 = blockIdx.x / P.n_cls;
    const long long u1 = cu.u0 + (long long)cu.nt * cu.w + P.unit_cost;
    // pieces: class-local CTAs c0, c0 + 1, ... while their range starts before the unit's end
    int n_pieces = 1;
    while (c0 + n_pieces < P.ncc && cu.tot * (c0 + n_pieces) / P.ncc < u1) ++n_pieces;
    const int G = P.G;
    const int prow = blockIdx.y * 8 + warp;
    if (prow >= cu.rows) return;                             // rows of a unit are live from 0 up
    auto rec_of = [&](int j) {
        const int slot = j == 0 ? cu.slot : 0;
        return ((int64_t)((c0 + j) * P.n_cls + pp) * 2 + slot) * kPairRows + prow;
    };
    auto live = [&](int j) {                                 // a CTA whose range holds no tile start has no piece
        return tiles_before(cu.tot * (c0 + j + 1) / P.ncc, cu.u0, cu.nt, cu.w, P.unit_cost) >
               tiles_before(cu.tot * (c0 + j) / P.ncc, cu.u0, cu.nt, cu.w, P.unit_cost);
    };
    float den = 0.f, mx = -CUDART_INF_F, o[D / 32];
#pragma unroll
    for (int q = 0; q < D / 32; ++q) o[q] = 0.f;
    // lane j holds piece j's (m, l); the accumulator rows of up to four pieces are fetched together
    for (int j0 = 0; j0 < n_pieces; j0 += 32) {
        const int jl = j0 + lane;
        float2 ml = make_float2(-CUDART_INF_F, 0.f);
        if (jl < n_pieces && live(jl)) ml = P.part_ml[rec_of(jl)];
        const float mnew = fmaxf(mx, warp_max(ml.x));
        if (mnew == -CUDART_INF_F) continue;
        const float rescale = __expf(mx - mnew);             // 0 on the first live batch
        den *= rescale;
#pragma unroll
        for (int q = 0; q < D / 32; ++q) o[q] *= rescale;
        mx = mnew;
        const float wl = ml.x == -CUDART_INF_F ? 0.f : __expf(ml.x - mx);
        den += warp_sum(ml.y * wl);
        const int nb = min(32, n_pieces - j0);
        for (int u0 = 0; u0 < nb; u0 += 4) {
            float v[4][D / 32], w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                w[u] = u0 + u < nb ? __shfl_sync(kFull, wl, u0 + u) : 0.f;
                const float* src = P.part_o + rec_of(j0 + min(u0 + u, nb - 1)) * D + lane * (D / 32);
#pragma unroll
                for (int q = 0; q < D / 32; ++q) v[u][q] = w[u] != 0.f ? src[q] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int q = 0; q < D / 32; ++q) o[q] = fmaf(v[u][q], w[u], o[q]);
        }
    }
    const float inv = 1.f / den;
    const int r_glob = pp * P.pair_rows + prow;
    const int node = r_glob / G, hq = cu.g * G + r_glob % G;
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.O) + cu.layer * P.o_ls + (((int64_t)cu.b * kMaxNodes + node) * a.Hq + hq) * D + lane * (D / 32);
#pragma unroll
    for (int q = 0; q < D / 32; ++q) dst[q] = __float2bfloat16(o[q] * inv);
    if (a.lse != nullptr && lane == 0) a.lse[cu.layer * P.lse_ls + ((int64_t)cu.b * a.Hq + hq) * kMaxNodes + node] = mx + logf(den);
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

// [layers][rows][heads][d] bf16 tensor (layer_stride elements between layers), box = (64 elements, box_heads,
// box_rows, one layer), 128-byte swizzle, zero fill
bool make_map(CUtensorMap* tm, const void* base, int d, int heads, long long rows, int box_heads, int box_rows, int layers,
              long long layer_stride) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    if (layers <= 1) { layers = 1; layer_stride = rows * heads * d; }
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)rows, (cuuint64_t)layers};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * heads, (cuuint64_t)layer_stride * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Grid shape.  A class is one row-block pair (256 query rows: both row blocks share every K/V tile in
// shared memory) or, when such fused units would leave most SMs without work, one row block (128 rows).
// CTAs per class: the grid is one CTA per SM, but at least four tiles per CTA when every sequence
// has the longest prefix.
void plan_grid(const radar_ctx* ctx, int B, int Hq, int Hkv, int max_prefix_len, int* pair_rows, int* n_cls, int* ncc) {
    const int G = Hq / Hkv;
    const int rows_max = kMaxNodes * G;
    const long long unit_tiles = (long long)B * Hkv * ((max_prefix_len + kTileKeys - 1) / kTileKeys + 1);
    int pr = kPairRows;
    if (rows_max > 128 && unit_tiles * ((rows_max + 255) / 256) < 4LL * ctx->sm_count) pr = 128;
    const int cls = (rows_max + pr - 1) / pr;
    long long per = ctx->sm_count / cls;
    if (per < 1) per = 1;
    const long long cap = (unit_tiles + 3) / 4;
    if (per > cap) per = cap;
    if (per < 1) per = 1;
    *pair_rows = pr;
    *n_cls = cls;
    *ncc = (int)per;
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

size_t tree_attn_tc_workspace_bytes(const radar_ctx* ctx, int B, int Hq, int Hkv, int d, int max_prefix_len) {
    int pair_rows, n_cls, ncc;
    plan_grid(ctx, B, Hq, Hkv, max_prefix_len, &pair_rows, &n_cls, &ncc);
    const size_t rec = (size_t)n_cls * ncc * 2 * kPairRows;
    return align_up(rec * sizeof(float2), 256) + align_up(rec * d * sizeof(float), 256) +
           align_up((size_t)n_cls * ncc * sizeof(CutUnit), 256);
}

template <int D, bool TWO, bool PAGED>
static int launch_tc(radar_ctx* ctx, TcParams& P, cudaStream_t stream) {
    const radar_attn_args& a = P.a;
    CUtensorMap tmQ, tmKc, tmVc, tmKt, tmVt;
    const long long tree_rows = (long long)a.B * kMaxNodes;
    const bool have_prefix = a.Kc != nullptr && a.Vc != nullptr && a.cache_rows > 0;
    const int cache_box = a.block_table != nullptr && a.page_size < kTileKeys ? a.page_size : kTileKeys;   // rows per TMA box
    const int L = P.n_layers;
    if (!make_map(&tmQ, a.Q, D, a.Hq, tree_rows, P.G, P.nodes_per_rb, L, a.q_layer_stride) ||
        !make_map(&tmKt, a.Kt, D, a.Hkv, tree_rows, 1, kTreeKeys, L, a.tree_kv_layer_stride) ||
        !make_map(&tmVt, a.Vt, D, a.Hkv, tree_rows, 1, kTreeKeys, L, a.tree_kv_layer_stride) ||
        !make_map(&tmKc, have_prefix ? a.Kc : a.Kt, D, a.Hkv, have_prefix ? a.cache_rows : tree_rows, 1, cache_box, L,
                  have_prefix ? a.cache_layer_stride : a.tree_kv_layer_stride) ||
        !make_map(&tmVc, have_prefix ? a.Vc : a.Vt, D, a.Hkv, have_prefix ? a.cache_rows : tree_rows, 1, cache_box, L,
                  have_prefix ? a.cache_layer_stride : a.tree_kv_layer_stride))
        return RADAR_ERR_CUDA;
    RADAR_CUDA_CHECK(radar_opt_in_smem(ctx, RADAR_SMEM_ATTN_TC + 4 * (D == 128) + 2 * TWO + PAGED, tree_attn_tc_kernel<D, TWO, PAGED>,
                                       (size_t)Smem<D, TWO>::kDynamic));
    {
        radar_launch_scope scope(ctx, RADAR_K_ATTN, stream);
        RADAR_CUDA_CHECK(launch_chained(tree_attn_tc_kernel<D, TWO, PAGED>, dim3((unsigned)(P.n_cls * P.ncc)), dim3(kTcThreads),
                                        (size_t)Smem<D, TWO>::kDynamic, stream, tmQ, tmKc, tmVc, tmKt, tmVt, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    {
        radar_launch_scope scope(ctx, RADAR_K_ATTN_COMBINE, stream);
        // few cut units: one row per warp and many small blocks; many: eight rows per warp, fewer waves of blocks
        if ((long long)P.n_cls * P.ncc * (kPairRows / 8) <= 16ll * ctx->sm_count)
            RADAR_CUDA_CHECK(launch_chained(tree_attn_tc_combine_wide_kernel<D>, dim3((unsigned)(P.n_cls * P.ncc), kPairRows / 8), dim3(256), 0, stream, P));
        else
            RADAR_CUDA_CHECK(launch_chained(tree_attn_tc_combine_kernel<D>, dim3((unsigned)(P.n_cls * P.ncc), kCombineY), dim3(256), 0, stream, P));
    }
    RADAR_CUDA_CHECK(cudaGetLastError());
    return RADAR_OK;
}

int tree_attn_tc_launch(radar_ctx* ctx, const radar_attn_args* a, cudaStream_t stream) {
    TcParams P;
    P.a = *a;
    P.G = a->Hq / a->Hkv;
    P.g_log2 = 0;
    while ((1 << P.g_log2) < P.G) ++P.g_log2;
    P.nodes_per_rb = 128 / P.G;
    const float scale = a->scale > 0.f ? a->scale : 1.f / sqrtf((float)a->d);
    P.scale_log2 = scale * 1.4426950408889634f;
    P.cache_rows = a->cache_rows;
    P.status = ctx->d_status;
    P.n_layers = a->n_layers > 1 ? a->n_layers : 1;
    P.o_ls = P.n_layers > 1 ? a->o_layer_stride : 0;
    P.lse_ls = P.n_layers > 1 ? a->lse_layer_stride : 0;
    plan_grid(ctx, a->B, a->Hq, a->Hkv, a->max_prefix_len, &P.pair_rows, &P.n_cls, &P.ncc);
    const TileCosts tc = tile_costs(P.n_cls);
    P.cost_one = tc.one; P.cost_two = tc.two; P.unit_cost = tc.unit;
    if (tree_attn_tc_workspace_bytes(ctx, a->B, a->Hq, a->Hkv, a->d, a->max_prefix_len) > a->workspace_bytes)
        return RADAR_ERR_WORKSPACE;
    const size_t rec = (size_t)P.n_cls * P.ncc * 2 * kPairRows;
    P.part_ml = reinterpret_cast<float2*>(a->workspace);
    P.part_o = reinterpret_cast<float*>(reinterpret_cast<char*>(a->workspace) + align_up(rec * sizeof(float2), 256));
    P.cut = reinterpret_cast<CutUnit*>(reinterpret_cast<char*>(P.part_o) + align_up(rec * a->d * sizeof(float), 256));
    const bool two = P.pair_rows > 128 && P.G * kMaxNodes > 128;      // some unit can have two live row blocks
    if (a->block_table != nullptr) {
        if (a->d == 128) return two ? launch_tc<128, true, true>(ctx, P, stream) : launch_tc<128, false, true>(ctx, P, stream);
        return two ? launch_tc<64, true, true>(ctx, P, stream) : launch_tc<64, false, true>(ctx, P, stream);
    }
    if (a->d == 128) return two ? launch_tc<128, true, false>(ctx, P, stream) : launch_tc<128, false, false>(ctx, P, stream);
    return two ? launch_tc<64, true, false>(ctx, P, stream) : launch_tc<64, false, false>(ctx, P, stream);
}

}  // namespace radar
