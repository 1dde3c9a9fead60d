// Context, status word and status strings of the RADAR hot-path library.
#include <new>

#include "common.cuh"

namespace {
__global__ void read_and_clear_status_kernel(int* status, int* out) {
    *out = atomicExch(status, 0);
}
}  // namespace

extern "C" int radar_create(radar_ctx** out, int device) {
    if (!out) return RADAR_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return RADAR_ERR_CUDA;
    RADAR_CUDA_CHECK(cudaSetDevice(device));
    radar_ctx* c = new (std::nothrow) radar_ctx;
    if (!c) return RADAR_ERR_CUDA;
    c->device = device;
    c->d_status = nullptr;
    c->profiling = false;
    c->ev = nullptr;
    c->ev_kernel = nullptr;
    c->ev_cap = c->ev_used = 0;
    for (int i = 0; i < RADAR_K_COUNT; ++i) { c->launches[i] = 0; c->prof_ms[i] = 0.0; c->prof_n[i] = 0; }
    for (int i = 0; i < RADAR_SMEM_COUNT; ++i) c->smem_opt_in[i] = 0;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaMalloc(&c->d_status, 2 * sizeof(int)) != cudaSuccess ||
        cudaMemset(c->d_status, 0, 2 * sizeof(int)) != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        delete c;
        return RADAR_ERR_CUDA;
    }
    // the workspace-free acceptance path must find everything in place later, when its host may not allocate
    if (radar::noalloc_prepare_device(device) != RADAR_OK) {
        cudaFree(c->d_status);
        delete c;
        return RADAR_ERR_CUDA;
    }
    *out = c;
    return RADAR_OK;
}

static void free_events(radar_ctx* c) {
    for (int i = 0; i < 2 * c->ev_cap; ++i) cudaEventDestroy(c->ev[i]);
    delete[] c->ev;
    delete[] c->ev_kernel;
    c->ev = nullptr;
    c->ev_kernel = nullptr;
    c->ev_cap = c->ev_used = 0;
    c->profiling = false;
}

extern "C" int radar_profile_begin(radar_ctx* ctx, int max_records) {
    if (!ctx || max_records <= 0) return RADAR_ERR_INVALID_ARG;
    if (ctx->ev) free_events(ctx);
    ctx->ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_records];
    ctx->ev_kernel = new (std::nothrow) int[max_records];
    if (!ctx->ev || !ctx->ev_kernel) return RADAR_ERR_CUDA;
    for (int i = 0; i < 2 * max_records; ++i) RADAR_CUDA_CHECK(cudaEventCreate(&ctx->ev[i]));
    ctx->ev_cap = max_records;
    ctx->ev_used = 0;
    for (int i = 0; i < RADAR_K_COUNT; ++i) { ctx->prof_ms[i] = 0.0; ctx->prof_n[i] = 0; }
    ctx->profiling = true;
    return RADAR_OK;
}

extern "C" int radar_profile_end(radar_ctx* ctx) {
    if (!ctx || !ctx->ev) return RADAR_ERR_INVALID_ARG;
    ctx->profiling = false;
    RADAR_CUDA_CHECK(cudaDeviceSynchronize());
    for (int r = 0; r < ctx->ev_used; ++r) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ctx->ev[2 * r], ctx->ev[2 * r + 1]) == cudaSuccess) {
            ctx->prof_ms[ctx->ev_kernel[r]] += ms;
            ctx->prof_n[ctx->ev_kernel[r]] += 1;
        }
    }
    free_events(ctx);
    return RADAR_OK;
}

extern "C" int radar_kernel_count(void) { return RADAR_K_COUNT; }

extern "C" const char* radar_kernel_name(int id) {
    switch (id) {
        case RADAR_K_VOCAB_EXPAND: return "vocab_pass(expand)";
        case RADAR_K_SELECT_GATE: return "expand_select_gate";
        case RADAR_K_TREE_BUILD: return "rerank_build_tree";
        case RADAR_K_ATTN: return "tree_attention";
        case RADAR_K_ATTN_COMBINE: return "tree_attention_combine";
        case RADAR_K_VOCAB_ACCEPT: return "vocab_pass(accept)";
        case RADAR_K_GREEDY_WALK: return "greedy_walk";
        case RADAR_K_STOCH_WALK: return "stochastic_walk";
        case RADAR_K_ACCLEN_NODES: return "accept_length_nodes";
        case RADAR_K_ACCLEN_DIST: return "accept_length_dist";
        case RADAR_K_GATE_FEATURES: return "gate_features";
        case RADAR_K_TRAIN_ROLLOUT: return "train_rollout";
        case RADAR_K_TRAIN_OUTER: return "train_outer";
        case RADAR_K_TRAIN_ADAM: return "train_adam";
        default: return "?";
    }
}

extern "C" int radar_kernel_stats(const radar_ctx* ctx, int id, long long* launches, double* timed_ms,
                                  long long* timed_launches) {
    if (!ctx || id < 0 || id >= RADAR_K_COUNT) return RADAR_ERR_INVALID_ARG;
    if (launches) *launches = ctx->launches[id];
    if (timed_ms) *timed_ms = ctx->prof_ms[id];
    if (timed_launches) *timed_launches = ctx->prof_n[id];
    return RADAR_OK;
}

extern "C" int radar_reset_launch_counts(radar_ctx* ctx) {
    if (!ctx) return RADAR_ERR_INVALID_ARG;
    for (int i = 0; i < RADAR_K_COUNT; ++i) ctx->launches[i] = 0;
    return RADAR_OK;
}

extern "C" int radar_destroy(radar_ctx* ctx) {
    if (!ctx) return RADAR_ERR_INVALID_ARG;
    if (ctx->ev) free_events(ctx);
    cudaFree(ctx->d_status);
    delete ctx;
    return RADAR_OK;
}

extern "C" int radar_read_device_status(radar_ctx* ctx, void* stream_) {
    if (!ctx) return RADAR_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int host = 0;
    read_and_clear_status_kernel<<<1, 1, 0, stream>>>(ctx->d_status, ctx->d_status + 1);
    RADAR_CUDA_CHECK(cudaGetLastError());
    RADAR_CUDA_CHECK(cudaMemcpyAsync(&host, ctx->d_status + 1, sizeof(int), cudaMemcpyDeviceToHost, stream));
    RADAR_CUDA_CHECK(cudaStreamSynchronize(stream));
    return host;
}

extern "C" const char* radar_status_string(int status) {
    switch (status) {
        case RADAR_OK: return "ok";
        case RADAR_ERR_INVALID_ARG: return "invalid argument";
        case RADAR_ERR_UNSUPPORTED: return "unsupported size or type";
        case RADAR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case RADAR_ERR_CUDA: return "CUDA runtime error";
        case RADAR_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case RADAR_ERR_NUMERIC: return "NaN in the logits";
        case RADAR_ERR_TREE: return "inconsistent tree (pruned parent, bad draft row or token)";
        default: return "unknown status";
    }
}
