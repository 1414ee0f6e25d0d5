// AdaSEKA routing coefficients (Eq. 6, Section 3.3): one CTA per (sequence, KV head).
#include "seka_kernels.h"
#include "seka_route.cuh"

namespace seka {

__global__ void route_kernel(const void* __restrict__ Q, int q_is_f32, const float* __restrict__ U,
                             const float* __restrict__ sigma, const int* __restrict__ cu_seqlens, int L, int Hq, int Hkv,
                             int D, int r, int M, int k_route, float* __restrict__ alpha_out) {
    extern __shared__ double sm[];
    const int b = blockIdx.x / Hkv, h = blockIdx.x % Hkv;
    const double* a = route_group(Q, q_is_f32, U, sigma, cu_seqlens, L, Hq, Hkv, D, r, M, k_route, b, h, sm);
    for (int m = threadIdx.x; m < M; m += blockDim.x) alpha_out[((size_t)b * Hkv + h) * M + m] = (float)a[m];
}

seka_status launch_route(const seka_shape* shape, const void* Q, const float* U, const float* sigma, int k_route,
                         float* alpha_out, cudaStream_t stream) {
    const size_t smem = route_smem_bytes(shape->head_dim, shape->n_experts, k_route);
    if (smem > 48 * 1024 &&      // very wide banks of rank-1 experts: up to 66 KB
        cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SEKA_ERR_CUDA;
    route_kernel<<<shape->batch * shape->n_kv_heads, 1024, smem, stream>>>(
        Q, shape->dtype == SEKA_F32 ? 1 : 0, U, sigma, shape->cu_seqlens, shape->max_seqlen, shape->n_q_heads,
        shape->n_kv_heads, shape->head_dim, shape->rank, shape->n_experts, k_route, alpha_out);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

}  // namespace seka

extern "C" seka_status adaseka_route(const seka_shape* shape, const void* Q, const float* U, const float* sigma,
                                     int32_t k_route, float* alpha_out, void* cuda_stream) {
    using namespace seka;
    seka_status st = validate_shape(shape);
    if (st != SEKA_OK) return st;
    if (!U || !sigma || !alpha_out) return SEKA_ERR_INVALID_ARG;
    if (k_route < 0 || k_route > shape->rank) return SEKA_ERR_INVALID_ARG;
    if (k_route == 0) k_route = shape->rank;
    if (shape->batch == 0) return SEKA_OK;
    if (!Q) return SEKA_ERR_INVALID_ARG;
    return launch_route(shape, Q, U, sigma, k_route, alpha_out, static_cast<cudaStream_t>(cuda_stream));
}
