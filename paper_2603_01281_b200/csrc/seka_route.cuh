// AdaSEKA routing coefficients (Eq. 6, Section 3.3) of one (sequence, KV head), as a device routine shared by the
// stand-alone routing kernel and the operand preparation of the fused forward (so that both give the same bits).
#pragma once

#include "seka_common.cuh"

namespace seka {

// Each dot product qbar . U_m[:, k] is cut into route_chunks() pieces of consecutive rows that different threads
// take (the loads of a piece are independent, so one memory latency covers them); the pieces are added in order.
#ifdef __CUDACC__
__host__ __device__
#endif
static inline int route_chunks(int M, int k_route) {
    const long long pairs = (long long)M * k_route;
    return pairs <= 512 ? 8 : (pairs <= 2048 ? 2 : 1);
}
// shared memory of route_group: the summed query, one term per (expert, piece, singular direction), the coefficients
#ifdef __CUDACC__
__host__ __device__
#endif
static inline size_t route_smem_bytes(int D, int M, int k_route) {
    return sizeof(double) * ((size_t)D + (size_t)M * k_route * route_chunks(M, k_route) + M + 1);
}

#ifdef __CUDACC__
__device__ __forceinline__ float route_load_q(const void* Q, int q_is_f32, size_t idx) {
    return q_is_f32 ? static_cast<const float*>(Q)[idx]
                    : __bfloat162float(static_cast<const __nv_bfloat16*>(Q)[idx]);
}

// s_m = sum_{k < k_route} (qbar . U_m[:, k]) sigma_m[k]  (each piece of a dot product is scaled by sigma_m[k]);  alpha_m = s_m / max_m' |s_m'|  (0 if all s are 0).
// qbar = sum of the last token's query over the G query heads of the group.  Sums run in fp64: the whole call is
// about a megaflop and the result steers every highlighted key of the prompt.
// Every thread of the CTA calls this (it synchronises the CTA); `sm` holds route_smem_bytes() bytes.  The order of
// every sum is fixed (it does not depend on the number of threads), so any kernel that calls this gets the same bits.
// Returns the M coefficients (as doubles, in shared memory), valid for every thread on return.
__device__ __forceinline__ const double* route_group(const void* Q, int q_is_f32, const float* __restrict__ U,
                                                     const float* __restrict__ sigma, const int* __restrict__ cu_seqlens,
                                                     int L, int Hq, int Hkv, int D, int r, int M, int k_route,
                                                     int b, int h, double* sm) {
    const int C = route_chunks(M, k_route);
    double* qbar = sm;                          // [D]
    double* term = sm + D;                      // [M][C][k_route]: partial dot products
    double* s = term + (size_t)M * C * k_route; // [M] (+ 1: the largest magnitude)
    const int G = Hq / Hkv, tid = threadIdx.x;
    const int last = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - 1;
    const int first = cu_seqlens ? cu_seqlens[b] : b * L;
    const bool empty = last < first;
    for (int i = tid; i < D; i += blockDim.x) {
        double a = 0.0;
        if (!empty) {
#pragma unroll 4
            for (int g = 0; g < G; ++g) a += (double)route_load_q(Q, q_is_f32, ((size_t)last * Hq + h * G + g) * D + i);
        }
        qbar[i] = a;
    }
    __syncthreads();
    const int rows = D / C;                     // D is 64 or 128, C divides it
    for (int u = tid; u < M * C * k_route; u += blockDim.x) {
        const int k = u % k_route, mc = u / k_route, c = mc % C, m = mc / C;
        const float* Um = U + (((size_t)m * Hkv + h) * D + (size_t)c * rows) * r + k;   // neighbouring threads: neighbouring columns
        const double sg = (double)sigma[((size_t)m * Hkv + h) * r + k];
        const double* qc = qbar + c * rows;
        double dot = 0.0;
#pragma unroll 16
        for (int i = 0; i < rows; ++i) dot += qc[i] * (double)Um[(size_t)i * r];
        term[u] = dot * sg;
    }
    __syncthreads();
    // pieces of a (expert, direction) pair in order, into the slot of piece 0; then the directions of an expert in order
    for (int p = tid; p < M * k_route; p += blockDim.x) {
        const int m = p / k_route, k = p - m * k_route;
        double t = 0.0;
        for (int c = 0; c < C; ++c) t += term[((size_t)m * C + c) * k_route + k];
        term[(size_t)m * C * k_route + k] = t;
    }
    __syncthreads();
    for (int m = tid; m < M; m += blockDim.x) {
        double tot = 0.0;
        for (int k = 0; k < k_route; ++k) tot += term[(size_t)m * C * k_route + k];
        s[m] = tot;
    }
    __syncthreads();
    if (tid == 0) {
        double mx = 0.0;
        for (int m = 0; m < M; ++m) mx = fmax(mx, fabs(s[m]));
        s[M] = mx;
    }
    __syncthreads();
    const double mx = s[M];
    __syncthreads();
    for (int m = tid; m < M; m += blockDim.x) s[m] = mx > 0.0 ? s[m] / mx : 0.0;
    __syncthreads();
    return s;
}
#endif

}  // namespace seka
