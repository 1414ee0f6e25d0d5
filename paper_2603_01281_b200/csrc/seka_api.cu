// Host-side entry points that launch nothing heavy: validation, workspace sizing, status.
#include <math.h>

#include "seka_kernels.h"

namespace seka {

std::atomic<unsigned long long> g_launches{0};

seka_status validate_shape(const seka_shape* s) {
    if (s == nullptr) return SEKA_ERR_INVALID_ARG;
    if (s->batch < 0 || s->max_seqlen < 0 || s->total_tokens < 0) return SEKA_ERR_INVALID_ARG;
    if (s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->n_q_heads % s->n_kv_heads != 0) return SEKA_ERR_INVALID_ARG;
    if (s->dtype != SEKA_F32 && s->dtype != SEKA_BF16) return SEKA_ERR_INVALID_ARG;
    if (s->rank <= 0 || s->n_experts <= 0) return SEKA_ERR_INVALID_ARG;
    if (s->cu_seqlens != nullptr && s->total_tokens == 0 && s->batch > 0 && s->max_seqlen > 0)
        return SEKA_ERR_INVALID_ARG;                 // packed layout needs the token count
    if (s->cu_seqlens == nullptr && s->total_tokens != 0 &&
        (long long)s->total_tokens != (long long)s->batch * s->max_seqlen) return SEKA_ERR_INVALID_ARG;
    if (!(s->softmax_scale >= 0.f) || isinf(s->softmax_scale)) return SEKA_ERR_INVALID_ARG;
    if ((long long)s->batch * s->max_seqlen > 0x7fffffffLL) return SEKA_ERR_UNSUPPORTED;
    if (s->head_dim != 64 && s->head_dim != 128) return SEKA_ERR_UNSUPPORTED;
    if (s->rank > s->head_dim) return SEKA_ERR_INVALID_ARG;
    if ((long long)s->rank * s->n_experts > 4096) return SEKA_ERR_UNSUPPORTED;
    return SEKA_OK;
}

}  // namespace seka

extern "C" size_t seka_workspace_bytes(const seka_shape* shape) {
    if (seka::validate_shape(shape) != SEKA_OK) return 0;
    return seka::workspace_layout(shape).total;
}

extern "C" seka_status seka_reset_status(void* workspace, void* cuda_stream) {
    if (workspace == nullptr) return SEKA_ERR_WORKSPACE;
    return cudaMemsetAsync(workspace, 0, seka::kStatusBytes, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? SEKA_OK : SEKA_ERR_CUDA;
}

extern "C" seka_status seka_poll_status(const void* workspace, void* cuda_stream) {
    if (workspace == nullptr) return SEKA_ERR_WORKSPACE;
    int word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SEKA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SEKA_ERR_CUDA;
    return (word >= SEKA_OK && word <= SEKA_ERR_TIMEOUT) ? static_cast<seka_status>(word) : SEKA_ERR_CUDA;
}

extern "C" const char* seka_status_string(seka_status status) {
    switch (status) {
        case SEKA_OK: return "ok";
        case SEKA_ERR_INVALID_ARG: return "invalid argument";
        case SEKA_ERR_UNSUPPORTED: return "unsupported shape";
        case SEKA_ERR_WORKSPACE: return "workspace missing or too small";
        case SEKA_ERR_CUDA: return "CUDA call failed";
        case SEKA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown status";
}

extern "C" uint64_t seka_launch_count(void) { return seka::g_launches.load(); }
