// Small preparation kernels: U -> MMA operand fragments, highlight-mask compaction,
// fp32 -> bf16 input conversion.
#include "seka_edit_tile.cuh"
#include "seka_kernels.h"

namespace seka {

// Ustack[i][j] = U[m = j / r][h][i][j % r] for j < M*r, 0 on the padding columns.
__device__ __forceinline__ float ustack(const float* __restrict__ U, int Hkv, int D, int r, int M, int h, int i, int j) {
    if (j >= M * r) return 0.f;
    const int m = j / r, jj = j - m * r;
    return U[(((size_t)m * Hkv + h) * D + i) * r + jj];
}

// One thread per uint4 of the fragment store (layout documented in seka_edit_tile.cuh).
__global__ void prep_fragments_kernel(const float* __restrict__ U, uint4* __restrict__ frags,
                                      int Hkv, int D, int r, int M, int r_pad) {
    const int KB = D / 16, NR = r_pad / 16;
    const size_t per_half = (size_t)KB * NR * 32;
    const size_t total = (size_t)Hkv * 2 * per_half;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int h = (int)(idx / (2 * per_half));
    size_t rem = idx - (size_t)h * 2 * per_half;
    const bool second = rem >= per_half;
    if (second) rem -= per_half;
    const int lane = (int)(rem & 31);
    const int g = lane >> 2, t = lane & 3;
    uint32_t w[4];
    if (!second) {
        // operand of T = K * Ustack: B[k = head-dim index][n = stacked column]
        const int np = (int)((rem >> 5) % NR), kb = (int)((rem >> 5) / NR);
        for (int q = 0; q < 2; ++q) {
            const int n = (2 * np + q) * 8 + g, k = kb * 16 + 2 * t;
            w[2 * q + 0] = pack_bf16(ustack(U, Hkv, D, r, M, h, k, n), ustack(U, Hkv, D, r, M, h, k + 1, n));
            w[2 * q + 1] = pack_bf16(ustack(U, Hkv, D, r, M, h, k + 8, n), ustack(U, Hkv, D, r, M, h, k + 9, n));
        }
    } else {
        // operand of dK = T * Ustack^T: B[k = stacked column][n = head-dim index]
        const int np2 = (int)((rem >> 5) % KB), kb2 = (int)((rem >> 5) / KB);
        for (int q = 0; q < 2; ++q) {
            const int i = (2 * np2 + q) * 8 + g, k = kb2 * 16 + 2 * t;
            w[2 * q + 0] = pack_bf16(ustack(U, Hkv, D, r, M, h, i, k), ustack(U, Hkv, D, r, M, h, i, k + 1));
            w[2 * q + 1] = pack_bf16(ustack(U, Hkv, D, r, M, h, i, k + 8), ustack(U, Hkv, D, r, M, h, i, k + 9));
        }
    }
    frags[idx] = make_uint4(w[0], w[1], w[2], w[3]);
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

void launch_prep_fragments(const float* U, uint4* frags, int Hkv, int D, int r, int M, int r_pad, cudaStream_t st) {
    const size_t total = (size_t)Hkv * frag_uint4_per_head(D, r_pad);
    prep_fragments_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(U, frags, Hkv, D, r, M, r_pad);
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
