// Shared device/host helpers of the RADAR hot-path library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "../../include/radar.h"

// kernels the library launches (index into the profiling tables)
enum radar_kernel_id {
    RADAR_K_VOCAB_EXPAND = 0,   // vocabulary pass of radar_expand_step
    RADAR_K_SELECT_GATE,        // partial merge + frontier selection + prediction model
    RADAR_K_TREE_BUILD,
    RADAR_K_ATTN,               // tree attention main kernel
    RADAR_K_ATTN_COMBINE,
    RADAR_K_VOCAB_ACCEPT,       // row-argmax pass of greedy acceptance
    RADAR_K_GREEDY_WALK,
    RADAR_K_STOCH_WALK,
    RADAR_K_ACCLEN_NODES,       // per-row conditional acceptance probabilities (Eq. 13)
    RADAR_K_ACCLEN_DIST,        // path products and the length distribution (Eq. 11-12)
    RADAR_K_GATE_FEATURES,      // input-side products of the hidden-state policy (Table 3)
    RADAR_K_TRAIN_ROLLOUT,      // REINFORCE step: rollout + backpropagation through time per data point
    RADAR_K_TRAIN_OUTER,        // REINFORCE step: parameter gradients
    RADAR_K_TRAIN_ADAM,         // REINFORCE step: batch loss + Adam update
    RADAR_K_COUNT
};

// kernels that opt in to more than 48 KB of dynamic shared memory: one slot per instantiation
enum radar_smem_slot {
    RADAR_SMEM_SELECT_GATE = 0,
    RADAR_SMEM_SELECT_GATE_CLUSTER,   // the instantiation with helper blocks
    RADAR_SMEM_TREE_BUILD,
    RADAR_SMEM_ATTN_FMA,        // + 2 * (bf16) + (d == 128)
    RADAR_SMEM_ATTN_TC = RADAR_SMEM_ATTN_FMA + 4,   // + 4 * (d == 128) + 2 * two + paged
    RADAR_SMEM_COUNT = RADAR_SMEM_ATTN_TC + 8
};

struct radar_ctx {
    int device;
    int sm_count;
    // largest dynamic shared-memory size opted in to so far, per kernel, ON THIS CONTEXT'S DEVICE (the attribute
    // is per device: a second device in the same process needs its own opt-in)
    size_t smem_opt_in[RADAR_SMEM_COUNT];
    int* d_status;          // sticky device status word
    // launch accounting (host side)
    long long launches[RADAR_K_COUNT];
    // optional per-kernel CUDA-event timing
    bool profiling;
    cudaEvent_t* ev;        // 2 * ev_cap events
    int* ev_kernel;         // kernel id of record i
    int ev_cap, ev_used;
    double prof_ms[RADAR_K_COUNT];
    long long prof_n[RADAR_K_COUNT];
};

// Brackets one kernel launch: counts it and, while profiling, records an event pair on its stream.
struct radar_launch_scope {
    radar_ctx* c;
    cudaStream_t s;
    int slot;
    radar_launch_scope(radar_ctx* ctx, int kernel, cudaStream_t stream) : c(ctx), s(stream), slot(-1) {
        c->launches[kernel]++;
        if (c->profiling && c->ev_used < c->ev_cap) {
            slot = c->ev_used++;
            c->ev_kernel[slot] = kernel;
            cudaEventRecord(c->ev[2 * slot], s);
        }
    }
    ~radar_launch_scope() {
        if (slot >= 0) cudaEventRecord(c->ev[2 * slot + 1], s);
    }
};

// Every kernel of the library is launched with programmatic stream serialization and begins with
// chain_wait(): the next kernel's launch and block scheduling overlap the tail of the previous one, and
// nothing of a kernel touches memory before its predecessor (and, transitively, every earlier kernel of
// the stream) has completed and flushed.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void chain_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// The two halves, for kernels that do work that cannot depend on the predecessor before they wait for
// it.  Rules that keep the chain sound: (1) every block runs chain_sync() in at least one thread
// before it exits, so "kernel N complete" always implies "kernel N-1 complete"; (2) nothing written by
// the immediate predecessor is read, and nothing it reads is written, before chain_sync() (or a block
// barrier behind a thread that ran it).  Whatever kernels before the predecessor wrote is complete
// when the block starts, because the predecessor's blocks trigger only after their own wait.
__device__ __forceinline__ void chain_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_sync() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// A failing runtime call becomes RADAR_ERR_CUDA; with RADAR_DEBUG set in the environment the call and the
// runtime's message are also written to stderr.
// Raises a kernel's dynamic shared-memory limit on the context's device when `bytes` exceeds what has been
// set there before (48 KB need no opt-in).  Not a stream operation.
template <typename K>
inline cudaError_t radar_opt_in_smem(radar_ctx* ctx, int slot, K kernel, size_t bytes) {
    const size_t have = ctx->smem_opt_in[slot] > 48 * 1024 ? ctx->smem_opt_in[slot] : 48 * 1024;
    if (bytes <= have) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) ctx->smem_opt_in[slot] = bytes;
    return e;
}

#define RADAR_CUDA_CHECK(expr)                                                                     \
    do {                                                                                           \
        cudaError_t _e = (expr);                                                                   \
        if (_e != cudaSuccess) {                                                                   \
            if (getenv("RADAR_DEBUG")) fprintf(stderr, "radar: %s -> %s\n", #expr, cudaGetErrorString(_e)); \
            return RADAR_ERR_CUDA;                                                                 \
        }                                                                                          \
    } while (0)

namespace radar {

constexpr int kMaxNodes = RADAR_MAX_NODES;
constexpr int kHidden = RADAR_GATE_HIDDEN;
constexpr unsigned kFull = 0xffffffffu;

// first error wins
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// (value desc, index asc) ordering: true if a precedes b
__device__ __forceinline__ bool precedes(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}
__device__ __forceinline__ bool precedes(double va, int ia, double vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

template <typename T>
__device__ __forceinline__ T warp_max(T v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
template <typename T>
__device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// Sorted list of the 32 best (value, index) pairs seen by a warp, one per lane (lane 0 = best).
// V is float or double.  Empty slots hold (-inf, INT_MAX).
template <typename V>
struct WarpTopList {
    V v;
    int i;
    __device__ __forceinline__ void reset() {
        v = -CUDART_INF_F;
        i = 0x7fffffff;
    }
    // all lanes call with the same candidate
    __device__ __forceinline__ void insert(V cv, int ci) {
        const bool worse = precedes(cv, ci, v, i);               // this lane's entry comes after the candidate
        const unsigned w = __ballot_sync(kFull, worse);
        if (w == 0) return;
        const int pos = __ffs(w) - 1;                             // entries are sorted: worse lanes are a suffix
        const V uv = __shfl_up_sync(kFull, v, 1);
        const int ui = __shfl_up_sync(kFull, i, 1);
        const int lane = threadIdx.x & 31;
        if (lane == pos) { v = cv; i = ci; }
        else if (lane > pos) { v = uv; i = ui; }
    }
    __device__ __forceinline__ V value_at(int lane) const { return __shfl_sync(kFull, v, lane); }
    __device__ __forceinline__ int index_at(int lane) const { return __shfl_sync(kFull, i, lane); }
};

// --- vocabulary pass (vocab_pass.cu) ------------------------------------------------------
// One launch reduces every (row, chunk) of a [rows][V] logits matrix to a partial record:
//   topv/topi [k] best (logit, token) of the chunk, sorted; m = max logit; s = sum exp(logit - m).
// rows are addressed as base + seq * seq_stride + f * row_stride with row = seq * F + f; rows whose
// sequence has skip[seq] == 0 (if skip != NULL) or whose index within the sequence is >= nrows[seq]
// (if nrows != NULL) are not read.
struct VocabPassParams {
    const void* logits;
    int dtype;
    int64_t row_stride, seq_stride;
    int n_seq, F, V, k;
    int n_chunks, chunk;             // chunk = elements per chunk (multiple of 8)
    int want_lse;                    // 0: top-k only (argmax pass), 1: also (m, s)
    const uint8_t* seq_active;       // or NULL
    const int32_t* seq_rows;         // or NULL: rows to process per sequence
    float* part_v;                   // [rows][n_chunks][k]
    int32_t* part_i;                 // [rows][n_chunks][k]
    float* part_m;                   // [rows][n_chunks]
    float* part_s;                   // [rows][n_chunks]
    int* status;
};
int vocab_pass_plan_chunks(int sm_count, int rows, int V, int* chunk_out);   // returns n_chunks
size_t vocab_pass_partial_bytes(int rows, int n_chunks, int k);
void vocab_pass_carve(void* ws, int rows, int n_chunks, int k, VocabPassParams* p);
cudaError_t vocab_pass_launch(radar_ctx* ctx, int kernel_id, const VocabPassParams& p, cudaStream_t stream);
cudaError_t vocab_pass_preload_argbest();

// --- workspace-free greedy acceptance (verify_accept.cu) --------------------------------------
// Resolves the device address of the library's scratch array on the current device and loads the two kernels of
// that path, so that nothing is left for the driver to allocate at the first call.  Called by radar_create.
int noalloc_prepare_device(int device);

// --- tensor-core tree attention (tree_attention_tc.cu) --------------------------------------
bool tree_attn_tc_supported(const radar_attn_args* a);
size_t tree_attn_tc_workspace_bytes(const radar_ctx* ctx, int B, int Hq, int Hkv, int d, int max_prefix_len);
int tree_attn_tc_launch(radar_ctx* ctx, const radar_attn_args* a, cudaStream_t stream);

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace radar
