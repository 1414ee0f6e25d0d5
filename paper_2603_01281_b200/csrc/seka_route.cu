// AdaSEKA routing coefficients (Eq. 6, Section 3.3): one CTA per (sequence, KV head).
#include "seka_kernels.h"

namespace seka {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// s_m = sum_{k < k_route} (qbar . U_m[:, k]) sigma_m[k];  alpha_m = s_m / max_m' |s_m'|  (0 if all s are 0).
// qbar = sum of the last token's query over the G query heads of the group.  Sums run in fp64:
// the whole call is about a megaflop and the result steers every highlighted key of the prompt.
template <typename T>
__global__ void route_kernel(const T* __restrict__ Q, const float* __restrict__ U, const float* __restrict__ sigma,
                             const int* __restrict__ cu_seqlens, int L, int Hq, int Hkv, int D, int r, int M,
                             int k_route, float* __restrict__ alpha_out) {
    extern __shared__ double sm[];
    double* qbar = sm;            // [D]
    double* part = sm + D;        // [blockDim.x]
    double* s = part + blockDim.x;   // [M]
    const int b = blockIdx.x / Hkv, h = blockIdx.x % Hkv, G = Hq / Hkv;
    const int last = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - 1;
    const int first = cu_seqlens ? cu_seqlens[b] : b * L;
    const bool empty = last < first;
    for (int i = threadIdx.x; i < D; i += blockDim.x) {
        double a = 0.0;
        if (!empty)
            for (int g = 0; g < G; ++g) a += (double)to_f32(Q[((size_t)last * Hq + h * G + g) * D + i]);
        qbar[i] = a;
    }
    __syncthreads();
    for (int m = 0; m < M; ++m) {
        const float* Um = U + ((size_t)m * Hkv + h) * D * r;
        const float* sg = sigma + ((size_t)m * Hkv + h) * r;
        double acc = 0.0;
        for (int k = threadIdx.x; k < k_route; k += blockDim.x) {
            double dot = 0.0;
            for (int i = 0; i < D; ++i) dot += qbar[i] * (double)Um[(size_t)i * r + k];
            acc += dot * (double)sg[k];
        }
        part[threadIdx.x] = acc;
        __syncthreads();
        if (threadIdx.x == 0) {
            double tot = 0.0;
            for (int i = 0; i < blockDim.x; ++i) tot += part[i];
            s[m] = tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double mx = 0.0;
        for (int m = 0; m < M; ++m) mx = fmax(mx, fabs(s[m]));
        for (int m = 0; m < M; ++m)
            alpha_out[((size_t)b * Hkv + h) * M + m] = mx > 0.0 ? (float)(s[m] / mx) : 0.f;
    }
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
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int threads = 64;
    const size_t smem = sizeof(double) * (shape->head_dim + threads + shape->n_experts);
    const dim3 grid(shape->batch * shape->n_kv_heads);
    if (shape->dtype == SEKA_F32)
        route_kernel<float><<<grid, threads, smem, stream>>>(
            static_cast<const float*>(Q), U, sigma, shape->cu_seqlens, shape->max_seqlen, shape->n_q_heads,
            shape->n_kv_heads, shape->head_dim, shape->rank, shape->n_experts, k_route, alpha_out);
    else
        route_kernel<__nv_bfloat16><<<grid, threads, smem, stream>>>(
            static_cast<const __nv_bfloat16*>(Q), U, sigma, shape->cu_seqlens, shape->max_seqlen, shape->n_q_heads,
            shape->n_kv_heads, shape->head_dim, shape->rank, shape->n_experts, k_route, alpha_out);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}
