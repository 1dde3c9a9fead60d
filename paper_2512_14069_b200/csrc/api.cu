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
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaMalloc(&c->d_status, 2 * sizeof(int)) != cudaSuccess ||
        cudaMemset(c->d_status, 0, 2 * sizeof(int)) != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        delete c;
        return RADAR_ERR_CUDA;
    }
    *out = c;
    return RADAR_OK;
}

extern "C" int radar_destroy(radar_ctx* ctx) {
    if (!ctx) return RADAR_ERR_INVALID_ARG;
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
