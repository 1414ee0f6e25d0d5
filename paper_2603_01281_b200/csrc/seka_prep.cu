// Small preparation kernels: dense edit operators and per-tile highlight flags for the fused kernel,
// highlight-mask compaction, fp32 -> bf16 input conversion.
#include "seka_kernels.h"
#include "seka_route.cuh"

namespace seka {

// Operand preparation of the fused kernel, one launch:
//   blocks [0, n_w):   a 32 x 32 tile of W[b][h] = gain_b * sum_m alpha_{b,h,m} U_m[h] U_m[h]^T  (bf16 [D x D]; the
//                      dynamic projector of Section 3.3 times the gain, or g U U^T for plain SEKA), so that the
//                      edit of a key tile is one product  K' = K + K W  (W is symmetric).  Pairs (b, h) that are
//                      not steered (zero gain, head switched off) are skipped: the fused kernel never reads them.
//   blocks [n_w, ...): one warp per (sequence, 128-key tile): does the tile hold a highlighted token?
// With `route.sigma` set the routing coefficients of Eq. 6 are computed here as well (each block of a (b, h) pair
// repeats the few thousand multiply-adds, from the last token's query), so that AdaSEKA needs no launch of its own
// before the forward; the coefficients are also written to `route.alpha_out` if that is set.
struct RouteArgs {
    const void* Q; int q_is_f32; const float* sigma; int k_route; int Hq; float* alpha_out;
};

__global__ void prep_steering_kernel(const float* __restrict__ U, const float* __restrict__ alpha,
                                     const float* __restrict__ gain, const uint8_t* __restrict__ head_enable,
                                     const uint8_t* __restrict__ mask, const int* __restrict__ cu_seqlens,
                                     __nv_bfloat16* __restrict__ W, uint8_t* __restrict__ tile_hot,
                                     int B, int L, int Hkv, int D, int r, int M, int n_tiles, int n_w,
                                     const RouteArgs route) {
    const int tid = threadIdx.x;
    extern __shared__ double route_sm[];
    if ((int)blockIdx.x < n_w) {
        const int tiles = D / 32;
        const int bh = blockIdx.x / (tiles * tiles), t = blockIdx.x % (tiles * tiles);
        const int b = bh / Hkv, h = bh % Hkv;
        const float g = gain[b];
        const double* routed = nullptr;
        if (route.sigma != nullptr) {
            routed = route_group(route.Q, route.q_is_f32, U, route.sigma, cu_seqlens, L, route.Hq, Hkv, D, r, M,
                                 route.k_route, b, h, route_sm);
            if (t == 0 && route.alpha_out != nullptr)
                for (int m = tid; m < M; m += blockDim.x) route.alpha_out[(size_t)bh * M + m] = (float)routed[m];
        }
        if (g == 0.f || (head_enable != nullptr && head_enable[h] == 0)) return;
        const int i0 = (t / tiles) * 32, j0 = (t % tiles) * 32;
        __shared__ float ui[32][33], uj[32][33];
        const int tx = tid & 31, ty = tid >> 5;          // 256 threads: 8 rows of 32
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int m = 0; m < M; ++m) {
            const float a = g * (routed != nullptr ? (float)routed[m]
                                                   : (alpha != nullptr ? alpha[((size_t)b * Hkv + h) * M + m] : 1.f));
            const float* Um = U + ((size_t)m * Hkv + h) * D * r;
            for (int k0 = 0; k0 < r; k0 += 32) {
                __syncthreads();
                for (int q = ty; q < 32; q += 8) {
                    const bool in = k0 + tx < r;
                    ui[q][tx] = in ? a * Um[(size_t)(i0 + q) * r + k0 + tx] : 0.f;
                    uj[q][tx] = in ? Um[(size_t)(j0 + q) * r + k0 + tx] : 0.f;
                }
                __syncthreads();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int i = ty + 8 * q;
#pragma unroll 8
                    for (int k = 0; k < 32; ++k) acc[q] = fmaf(ui[i][k], uj[tx][k], acc[q]);
                }
            }
        }
        __nv_bfloat16* Wbh = W + (size_t)bh * D * D;
#pragma unroll
        for (int q = 0; q < 4; ++q) Wbh[(size_t)(i0 + ty + 8 * q) * D + j0 + tx] = __float2bfloat16_rn(acc[q]);
    } else {
        const int item = ((int)blockIdx.x - n_w) * 8 + (tid >> 5), lane = tid & 31;
        if (item >= B * n_tiles) return;
        const int b = item / n_tiles, t = item % n_tiles;
        const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
        const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
        bool any = false;
        for (int q = 0; q < 4; ++q) {
            const int pos = t * 128 + q * 32 + lane;
            any = any || (pos < Lb && mask[seq0 + pos] != 0);
        }
        any = __any_sync(0xffffffffu, any);
        if (lane == 0) tile_hot[item] = any ? 1 : 0;
    }
}

// Operand preparation of the stand-alone edit, one launch:
//   blocks [0, n_p):   a 32 x 32 tile of the projector P[m][h] = U_m[h] U_m[h]^T (bf16 [D x D], as a high and a low
//                      part: [M, Hkv] matrices of high parts, then as many of low parts); gain and routing
//                      coefficients are applied per row when dK is added, so this does not depend on the batch;
//   blocks [n_p, ...): one warp per (sequence, 128-key tile): flag, and the tiles that hold a highlighted token
//                      appended to `hot_list` (any order).
__global__ void prep_edit_kernel(const float* __restrict__ U, const uint8_t* __restrict__ mask,
                                 const int* __restrict__ cu_seqlens, __nv_bfloat16* __restrict__ P,
                                 uint8_t* __restrict__ tile_hot, int* __restrict__ hot_list, int* __restrict__ hot_count,
                                 int B, int L, int Hkv, int D, int r, int M, int n_tiles, int n_p) {
    const int tid = threadIdx.x;
    if ((int)blockIdx.x < n_p) {
        const int tiles = D / 32;
        const int mh = blockIdx.x / (tiles * tiles), t = blockIdx.x % (tiles * tiles);
        const int i0 = (t / tiles) * 32, j0 = (t % tiles) * 32;
        __shared__ float ui[32][33], uj[32][33];
        const int tx = tid & 31, ty = tid >> 5;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const float* Um = U + (size_t)mh * D * r;          // U is [M, Hkv, D, r]: (m, h) pairs are consecutive
        for (int k0 = 0; k0 < r; k0 += 32) {
            __syncthreads();
            for (int q = ty; q < 32; q += 8) {
                const bool in = k0 + tx < r;
                ui[q][tx] = in ? Um[(size_t)(i0 + q) * r + k0 + tx] : 0.f;
                uj[q][tx] = in ? Um[(size_t)(j0 + q) * r + k0 + tx] : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int i = ty + 8 * q;
#pragma unroll 8
                for (int k = 0; k < 32; ++k) acc[q] = fmaf(ui[i][k], uj[tx][k], acc[q]);
            }
        }
        // two bf16 parts, P = hi + lo to about 2^-17: the edit keeps fp32-like accuracy on bf16 tensor cores
        __nv_bfloat16* Phi = P + (size_t)mh * D * D;
        __nv_bfloat16* Plo = P + ((size_t)M * Hkv + mh) * D * D;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(acc[q]);
            Phi[(size_t)(i0 + ty + 8 * q) * D + j0 + tx] = hi;
            Plo[(size_t)(i0 + ty + 8 * q) * D + j0 + tx] = __float2bfloat16_rn(acc[q] - __bfloat162float(hi));
        }
    } else {
        const int item = ((int)blockIdx.x - n_p) * 8 + (tid >> 5), lane = tid & 31;
        if (item >= B * n_tiles) return;
        const int b = item / n_tiles, t = item % n_tiles;
        const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
        const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
        bool any = false;
        for (int q = 0; q < 4; ++q) {
            const int pos = t * 128 + q * 32 + lane;
            any = any || (pos < Lb && mask[seq0 + pos] != 0);
        }
        any = __any_sync(0xffffffffu, any);
        if (lane == 0) {
            tile_hot[item] = any ? 1 : 0;
            if (any) hot_list[atomicAdd(hot_count, 1)] = item;
        }
    }
}

// Item table of the fused kernel: slot idx (heaviest row tiles first; the items of one (sequence, KV head)
// next to each other) decoded into an ItemRecord.  Returns false for a slot whose tiles lie beyond the
// sequence.
__device__ __forceinline__ bool decode_item(long long idx, int B, int L, int Hq, int Hkv, int n_qt, int pair_heads,
                                            const int* __restrict__ cu, int steer_call, const float* __restrict__ gain,
                                            const uint8_t* __restrict__ head_enable, ItemRecord& r) {
    int hqA, hqB, qtA, qtB;
    if (pair_heads) {
        const int per_qt = B * (Hq >> 1);
        const int qt = n_qt - 1 - (int)(idx / per_qt);
        const int rem = (int)(idx % per_qt);
        r.b = rem / (Hq >> 1);
        const int hp = rem % (Hq >> 1);
        hqA = 2 * hp; hqB = 2 * hp + 1; qtA = qtB = qt;
    } else {
        const int per_qt = B * Hq;
        const int qt2 = ((n_qt + 1) >> 1) - 1 - (int)(idx / per_qt);
        const int rem = (int)(idx % per_qt);
        r.b = rem / Hq;
        hqA = hqB = rem % Hq; qtA = 2 * qt2; qtB = 2 * qt2 + 1;
    }
    r.hkv = hqA / (Hq / Hkv);
    r.seq0 = cu ? cu[r.b] : r.b * L;
    r.Lb = (cu ? cu[r.b + 1] : (r.b + 1) * L) - r.seq0;
    const int nA = qtA * 128 < r.Lb ? qtA + 1 : 0, nB = qtB * 128 < r.Lb ? qtB + 1 : 0;
    r.hq = hqA | (hqB << 16); r.qt = qtA | (qtB << 16); r.n = nA | (nB << 16);
    r.steer = (steer_call && gain[r.b] != 0.f && (head_enable == nullptr || head_enable[r.hkv] != 0)) ? 1 : 0;
    return nA > 0;
}

// Fixed-length batches have no empty slots: one thread per item.
__global__ void build_items_kernel(long long n, int B, int L, int Hq, int Hkv, int n_qt, int pair_heads, int steer_call,
                                   const float* __restrict__ gain, const uint8_t* __restrict__ head_enable,
                                   ItemRecord* __restrict__ items, int* __restrict__ count) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx == 0) *count = (int)n;
    if (idx >= n) return;
    ItemRecord r;
    decode_item(idx, B, L, Hq, Hkv, n_qt, pair_heads, nullptr, steer_call, gain, head_enable, r);
    items[idx] = r;
}

// Packed variable-length batches: slots beyond a short sequence are dropped, order kept (one CTA scans).
__global__ void build_items_varlen_kernel(long long n, int B, int L, int Hq, int Hkv, int n_qt, int pair_heads,
                                          const int* __restrict__ cu, int steer_call, const float* __restrict__ gain,
                                          const uint8_t* __restrict__ head_enable, ItemRecord* __restrict__ items,
                                          int* __restrict__ count) {
    __shared__ int warp_tot[32];
    __shared__ int base_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
    if (tid == 0) base_s = 0;
    __syncthreads();
    for (long long start = 0; start < n; start += blockDim.x) {
        const long long idx = start + tid;
        ItemRecord r;
        const bool keep = idx < n && decode_item(idx, B, L, Hq, Hkv, n_qt, pair_heads, cu, steer_call, gain, head_enable, r);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_tot[wid] = __popc(bal);
        __syncthreads();
        int off = base_s;
        for (int q = 0; q < wid; ++q) off += warp_tot[q];
        if (keep) items[off + __popc(bal & ((1u << lane) - 1))] = r;
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int q = 0; q < nw; ++q) tot += warp_tot[q];
            base_s += tot;
        }
        __syncthreads();
    }
    if (tid == 0) *count = base_s;
}

// Appends the indices of highlighted tokens to `list` (order within a warp preserved).
__global__ void compact_mask_kernel(const uint8_t* __restrict__ mask, int T, int* __restrict__ list,
                                    int* __restrict__ count) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const bool hl = t < T && mask[t] != 0;
    const unsigned b = __ballot_sync(0xffffffffu, hl);
    if (b == 0) return;
    const int lane = threadIdx.x & 31;
    int base = 0;
    if (lane == 0) base = atomicAdd(count, __popc(b));
    base = __shfl_sync(0xffffffffu, base, 0);
    if (hl) list[base + __popc(b & ((1u << lane) - 1))] = t;
}

__global__ void convert_f32_bf16_kernel(const float4* __restrict__ in, uint2* __restrict__ out, size_t n4) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 v = in[i];
    out[i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
}

void launch_prep_steering(const seka_shape* sh, const float* U, const float* alpha, const float* gain,
                          const uint8_t* head_enable, const uint8_t* mask, void* W, uint8_t* tile_hot, int n_tiles,
                          cudaStream_t st, const void* Q_route, const float* sigma, int k_route, float* alpha_out) {
    const int D = sh->head_dim, tiles = D / 32;
    const int n_w = sh->batch * sh->n_kv_heads * tiles * tiles;
    const int n_flag = (sh->batch * n_tiles + 7) / 8;
    RouteArgs route{Q_route, sh->dtype == SEKA_F32 ? 1 : 0, sigma, k_route, sh->n_q_heads, alpha_out};
    const size_t smem = sigma != nullptr ? route_smem_bytes(D, sh->n_experts, k_route) : 0;
    if (smem > 48 * 1024) cudaFuncSetAttribute(prep_steering_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    prep_steering_kernel<<<n_w + n_flag, 256, smem, st>>>(U, alpha, gain, head_enable, mask, sh->cu_seqlens,
                                                         static_cast<__nv_bfloat16*>(W), tile_hot, sh->batch,
                                                         sh->max_seqlen, sh->n_kv_heads, D, sh->rank, sh->n_experts,
                                                         n_tiles, n_w, route);
    ++g_launches;
}

void launch_prep_edit(const seka_shape* sh, const float* U, const uint8_t* mask, void* P, uint8_t* tile_hot, int n_tiles,
                      int* hot_list, int* hot_count, cudaStream_t st) {
    const int D = sh->head_dim, tiles = D / 32;
    const int n_p = sh->n_experts * sh->n_kv_heads * tiles * tiles;
    const int n_flag = (sh->batch * n_tiles + 7) / 8;
    cudaMemsetAsync(hot_count, 0, sizeof(int), st);
    prep_edit_kernel<<<n_p + n_flag, 256, 0, st>>>(U, mask, sh->cu_seqlens, static_cast<__nv_bfloat16*>(P), tile_hot, hot_list,
                                                  hot_count, sh->batch, sh->max_seqlen, sh->n_kv_heads, D, sh->rank,
                                                  sh->n_experts, n_tiles, n_p);
    ++g_launches;
}

void launch_build_items(const seka_shape* sh, const WorkspaceLayout& w, bool steer, const float* gain,
                        const uint8_t* head_enable, ItemRecord* items, int* count, cudaStream_t st) {
    const long long n = w.n_items_max;
    if (sh->cu_seqlens == nullptr)
        build_items_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(n, sh->batch, sh->max_seqlen, sh->n_q_heads,
                                                                       sh->n_kv_heads, w.n_tiles, w.pair_heads, steer ? 1 : 0,
                                                                       gain, head_enable, items, count);
    else
        build_items_varlen_kernel<<<1, 1024, 0, st>>>(n, sh->batch, sh->max_seqlen, sh->n_q_heads, sh->n_kv_heads, w.n_tiles,
                                                      w.pair_heads, sh->cu_seqlens, steer ? 1 : 0, gain, head_enable, items, count);
    ++g_launches;
}

void launch_compact_mask(const uint8_t* mask, int T, int* list, int* count, cudaStream_t st) {
    cudaMemsetAsync(count, 0, sizeof(int), st);
    if (T == 0) return;
    compact_mask_kernel<<<(T + 255) / 256, 256, 0, st>>>(mask, T, list, count);
    ++g_launches;
}

void launch_convert_bf16(const float* in, void* out, size_t n, cudaStream_t st) {
    const size_t n4 = n / 4;   // head_dim is a multiple of 4, so n is too
    if (n4 == 0) return;
    convert_f32_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const float4*>(in), reinterpret_cast<uint2*>(out), n4);
    ++g_launches;
}

}  // namespace seka
