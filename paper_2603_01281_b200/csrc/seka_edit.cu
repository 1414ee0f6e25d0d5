// Standalone key-editing kernel (the hook of Algorithm 1 / Algorithm 2 applied to a key tensor in HBM).
#include <mutex>

#include "seka_kernels.h"

namespace seka {

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

__device__ __forceinline__ int find_sequence(const int* __restrict__ cu, int B, int L, int t) {
    if (cu == nullptr) return t / L;
    int lo = 0, hi = B - 1;            // largest b with cu[b] <= t
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (cu[mid] <= t) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// One warp per (highlighted token, KV head) row, fp32 arithmetic:
//   c = U_m^T k (lanes over the rank),  k' = k + g * sum_m alpha_m U_m c (lanes over head_dim).
template <typename T, int D>
__global__ void edit_rows_kernel(const T* K_in, T* K_out, const int* __restrict__ list,
                                 const int* __restrict__ count, const float* __restrict__ U,
                                 const float* __restrict__ alpha, const float* __restrict__ gain,
                                 const uint8_t* __restrict__ head_enable, const int* __restrict__ cu, int B, int L,
                                 int Hkv, int r, int M) {
    constexpr int Q = D / 32;
    const int lane = threadIdx.x & 31;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long items = (long long)(*count) * Hkv;
    for (long long it = warp0; it < items; it += nwarps) {
        const int h = (int)(it % Hkv);
        if (head_enable != nullptr && head_enable[h] == 0) continue;
        const int t = list[it / Hkv];
        const int b = find_sequence(cu, B, L, t);
        const float g = gain[b];
        const size_t row = ((size_t)t * Hkv + h) * D;
        float k[Q], dk[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) { k[q] = Elem<T>::load(K_in + row + q * 32 + lane); dk[q] = 0.f; }
        for (int m = 0; m < M; ++m) {
            const float a = g * (alpha != nullptr ? alpha[((size_t)b * Hkv + h) * M + m] : 1.f);
            const float* Um = U + ((size_t)m * Hkv + h) * D * r;
            for (int j0 = 0; j0 < r; j0 += 32) {
                const int j = j0 + lane;
                float c = 0.f;
#pragma unroll
                for (int q = 0; q < Q; ++q)
#pragma unroll 8
                    for (int ii = 0; ii < 32; ++ii) {
                        const float kv = __shfl_sync(0xffffffffu, k[q], ii);
                        if (j < r) c = fmaf(__ldg(Um + (size_t)(q * 32 + ii) * r + j), kv, c);
                    }
                c *= a;
                const int jn = min(32, r - j0);
                for (int jj = 0; jj < jn; ++jj) {
                    const float cj = __shfl_sync(0xffffffffu, c, jj);
#pragma unroll
                    for (int q = 0; q < Q; ++q) dk[q] = fmaf(__ldg(Um + (size_t)(q * 32 + lane) * r + j0 + jj), cj, dk[q]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < Q; ++q) Elem<T>::store(K_out + row + q * 32 + lane, k[q] + dk[q]);
    }
}

template <typename T>
static void launch_edit_rows(const seka_shape* s, const void* K_in, void* K_out, const int* list, const int* count,
                             const float* U, const float* alpha, const float* gain, const uint8_t* he,
                             cudaStream_t st) {
    const int blocks = 148 * 8, threads = 256;
    if (s->head_dim == 128)
        edit_rows_kernel<T, 128><<<blocks, threads, 0, st>>>(
            static_cast<const T*>(K_in), static_cast<T*>(K_out), list, count, U, alpha, gain, he, s->cu_seqlens,
            s->batch, s->max_seqlen, s->n_kv_heads, s->rank, s->n_experts);
    else
        edit_rows_kernel<T, 64><<<blocks, threads, 0, st>>>(
            static_cast<const T*>(K_in), static_cast<T*>(K_out), list, count, U, alpha, gain, he, s->cu_seqlens,
            s->batch, s->max_seqlen, s->n_kv_heads, s->rank, s->n_experts);
    ++g_launches;
}

}  // namespace seka

extern "C" seka_status seka_edit_keys(const seka_shape* shape, const void* K_in, void* K_out, const uint8_t* mask,
                                      const float* U, const float* alpha, const float* gain,
                                      const uint8_t* head_enable, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_shape(shape);
    if (stc != SEKA_OK) return stc;
    const int T = shape_total_tokens(shape);
    if (T == 0) return SEKA_OK;
    if (!K_in || !K_out || !mask || !U || !gain) return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)K_in | (uintptr_t)K_out) & 15) return SEKA_ERR_INVALID_ARG;
    const WorkspaceLayout w = workspace_layout(shape);
    if (!workspace || workspace_bytes < w.total) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    int* list = reinterpret_cast<int*>(ws + w.list_off);
    const size_t esz = shape->dtype == SEKA_F32 ? 4 : 2;
    if (K_out != K_in) {
        const size_t bytes = (size_t)T * shape->n_kv_heads * shape->head_dim * esz;
        if (cudaMemcpyAsync(K_out, K_in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SEKA_ERR_CUDA;
    }
    launch_compact_mask(mask, T, list, status + 2, st);
    if (shape->dtype == SEKA_F32)
        launch_edit_rows<float>(shape, K_in, K_out, list, status + 2, U, alpha, gain, head_enable, st);
    else
        launch_edit_rows<__nv_bfloat16>(shape, K_in, K_out, list, status + 2, U, alpha, gain, head_enable, st);
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

// ---------------------------------------------------------------- allocation-free variant
namespace seka {

// Scratch of seka_edit_keys_static, resident in the device image of every GPU that loads the
// library: a 256-byte header whose first word is the list counter, then one int32 per token.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_static_scratch[256 + (size_t)SEKA_STATIC_MAX_TOKENS * 4];

// Device address of the array on the current device, looked up once per device.
static seka_status static_scratch_of_current_device(char** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static char* table[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SEKA_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SEKA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (table[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return SEKA_ERR_CUDA;
        table[dev] = static_cast<char*>(p);
    }
    *out = table[dev];
    return SEKA_OK;
}

}  // namespace seka

extern "C" seka_status seka_edit_keys_static(const seka_shape* shape, const void* K_in, void* K_out,
                                             const uint8_t* mask, const float* U, const float* alpha,
                                             const float* gain, const uint8_t* head_enable, void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_shape(shape);
    if (stc != SEKA_OK) return stc;
    const int T = shape_total_tokens(shape);
    if (T > SEKA_STATIC_MAX_TOKENS) return SEKA_ERR_UNSUPPORTED;   // beyond the built-in scratch
    if (T == 0) return SEKA_OK;
    if (!K_in || !K_out || !mask || !U || !gain) return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)K_in | (uintptr_t)K_out) & 15) return SEKA_ERR_INVALID_ARG;
    char* scratch = nullptr;
    stc = static_scratch_of_current_device(&scratch);
    if (stc != SEKA_OK) return stc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int* count = reinterpret_cast<int*>(scratch);
    int* list = reinterpret_cast<int*>(scratch + 256);
    const size_t esz = shape->dtype == SEKA_F32 ? 4 : 2;
    if (K_out != K_in) {
        const size_t bytes = (size_t)T * shape->n_kv_heads * shape->head_dim * esz;
        if (cudaMemcpyAsync(K_out, K_in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SEKA_ERR_CUDA;
    }
    launch_compact_mask(mask, T, list, count, st);     // zeroes the counter on the stream first
    if (shape->dtype == SEKA_F32)
        launch_edit_rows<float>(shape, K_in, K_out, list, count, U, alpha, gain, head_enable, st);
    else
        launch_edit_rows<__nv_bfloat16>(shape, K_in, K_out, list, count, U, alpha, gain, head_enable, st);
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}
