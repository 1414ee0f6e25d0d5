// Rank-R key edit of a tile of keys held in shared memory, on warp-level tensor-core MMAs.
//
// For the rows of a [rows x D] bf16 key tile whose flag is set:
//     k' = k + sum_j colscale[j] * Ustack[:, j] * (Ustack[:, j] . k)
// where Ustack = [U_1 | ... | U_M | 0-pad] (D x R, R = M*r rounded up to 16) and
// colscale[j] = gain * alpha_{j / r} (0 on the padding).  That is k' = k + g * sum_m alpha_m
// U_m U_m^T k, the edit of Section 2 / Section 3.3, evaluated as two skinny products
// T = K * Ustack (16 x R per row block) and dK = (T * colscale) * Ustack^T, with fp32
// accumulation; rows whose flag is clear are not touched.
//
// The tile uses the 128-byte-swizzled block layout that TMA writes and the UMMA descriptors
// read ([rows x 64] blocks, `blk_stride` bytes apart), so the same routine serves the fused
// attention kernel (edit in place between the TMA load and the score MMA) and the standalone
// cache-editing kernel.  Ustack comes pre-arranged in MMA fragment order (built once per call
// by prep_fragments_kernel) so every operand load is one coalesced 16-byte read per lane.
#pragma once

#include "seka_common.cuh"

namespace seka {

#ifdef __CUDACC__

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}

// Fragment store of one KV head (uint4 units):
//   fragB [D/16][R/16][32]: operand of T = K * Ustack        (contraction over head_dim)
//   fragA [R/16][D/16][32]: operand of dK = T * Ustack^T     (contraction over the stacked rank)
__host__ __device__ inline size_t frag_uint4_per_head(int D, int r_pad) { return (size_t)2 * (D / 16) * (r_pad / 16) * 32; }

// Edits one block of 16 rows (rows r0 .. r0+15 of the tile); called by a whole warp.
// NR16 = stacked rank / 16 (1, 2, 4 or 8: the stacked rank is padded to a power of two with zero columns).
template <int D, int NR16>
__device__ __forceinline__ void edit_rows16(uint8_t* tile, uint32_t blk_stride, int r0, const uint8_t* rowflag,
                                            const uint4* __restrict__ fragB, const uint4* __restrict__ fragA,
                                            const float* colscale, int lane) {
    constexpr int KB = D / 16;
    constexpr int nR16 = NR16;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t tile_s = smem_u32(tile);

    // T = K_block * Ustack, 32 stacked columns at a time (keeps the accumulators small: this routine runs in
    // warps that gave most of their registers away); the columns are scaled by gain * alpha and the
    // accumulators repacked as the A operand of the next product
    uint32_t ta[NR16][4];
    const int lrow = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int np0 = 0; np0 < NR16; np0 += 2) {
        {
            float acc[2][2][4];
#pragma unroll
            for (int n2 = 0; n2 < 2; ++n2)
#pragma unroll
                for (int q = 0; q < 2; ++q)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[n2][q][e] = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const int col = kb * 16 + (lane >> 4) * 8;
                uint32_t a[4];
                ldmatrix_x4(a, tile_s + (uint32_t)(col >> 6) * blk_stride + sw128_offset(lrow, col & 63));
#pragma unroll
                for (int n2 = 0; n2 < 2; ++n2) {
                    const int np = np0 + n2;
                    if (np < nR16) {
                        const uint4 f = __ldg(fragB + ((size_t)kb * nR16 + np) * 32 + lane);
                        mma_bf16_16816(acc[n2][0], a, f.x, f.y);
                        mma_bf16_16816(acc[n2][1], a, f.z, f.w);
                    }
                }
            }
#pragma unroll
            for (int n2 = 0; n2 < 2; ++n2) {
                const int np = np0 + n2;
                if (np < nR16) {
                    const float2 s0 = *reinterpret_cast<const float2*>(colscale + np * 16 + 2 * t);
                    const float2 s1 = *reinterpret_cast<const float2*>(colscale + np * 16 + 8 + 2 * t);
                    ta[np][0] = pack_bf16(acc[n2][0][0] * s0.x, acc[n2][0][1] * s0.y);
                    ta[np][1] = pack_bf16(acc[n2][0][2] * s0.x, acc[n2][0][3] * s0.y);
                    ta[np][2] = pack_bf16(acc[n2][1][0] * s1.x, acc[n2][1][1] * s1.y);
                    ta[np][3] = pack_bf16(acc[n2][1][2] * s1.x, acc[n2][1][3] * s1.y);
                }
            }
        }
    }

    const bool hi0 = rowflag[r0 + g] != 0, hi1 = rowflag[r0 + g + 8] != 0;

    // dK = T * Ustack^T, added to the flagged rows in place
#pragma unroll
    for (int np2 = 0; np2 < KB; ++np2) {
        float c[2][4];
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e) c[q][e] = 0.f;
#pragma unroll
        for (int kb2 = 0; kb2 < NR16; ++kb2) {
            const uint4 f = __ldg(fragA + ((size_t)kb2 * KB + np2) * 32 + lane);
            mma_bf16_16816(c[0], ta[kb2], f.x, f.y);
            mma_bf16_16816(c[1], ta[kb2], f.z, f.w);
        }
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int col = (2 * np2 + q) * 8 + 2 * t;
            uint8_t* base = tile + (size_t)(col >> 6) * blk_stride;
            if (hi0) {
                __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(base + sw128_offset(r0 + g, col & 63));
                const float2 k = __bfloat1622float2(*p);
                *p = __floats2bfloat162_rn(k.x + c[q][0], k.y + c[q][1]);
            }
            if (hi1) {
                __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(base + sw128_offset(r0 + g + 8, col & 63));
                const float2 k = __bfloat1622float2(*p);
                *p = __floats2bfloat162_rn(k.x + c[q][2], k.y + c[q][3]);
            }
        }
    }
}

// Run-time dispatch on the padded stacked rank.
template <int D>
__device__ __forceinline__ void edit_rows16_any(uint8_t* tile, uint32_t blk_stride, int r0, const uint8_t* rowflag,
                                                const uint4* __restrict__ fragB, const uint4* __restrict__ fragA,
                                                const float* colscale, int nR16, int lane) {
    switch (nR16) {
        case 1: edit_rows16<D, 1>(tile, blk_stride, r0, rowflag, fragB, fragA, colscale, lane); break;
        case 2: edit_rows16<D, 2>(tile, blk_stride, r0, rowflag, fragB, fragA, colscale, lane); break;
        case 4: edit_rows16<D, 4>(tile, blk_stride, r0, rowflag, fragB, fragA, colscale, lane); break;
        default: edit_rows16<D, 8>(tile, blk_stride, r0, rowflag, fragB, fragA, colscale, lane); break;
    }
}

#endif  // __CUDACC__

}  // namespace seka
