// Fused SEKA / AdaSEKA steered causal GQA attention forward for sm_100a.
//
// One CTA owns a tile of 128 queries of one query head and walks the key tiles 0 .. diagonal:
//   TMA (128-byte swizzle) stages K and V tiles in shared memory, double buffered;
//   key tiles that contain highlighted tokens are edited in place, k' = k + g * sum_m alpha_m U_m U_m^T k
//     (Section 2 / Section 3.3; hook of Algorithm 1/2), by warp-level tensor-core MMAs (seka_edit_tile.cuh);
//   S = Q K'^T runs on tcgen05 with the accumulator in tensor memory (score of Section 2);
//   each thread owns one query row: causal mask on the diagonal tile, online softmax in base 2,
//     P written to shared memory as bf16 in UMMA operand layout;
//   P V runs on tcgen05 into tensor memory and is folded into the running output in registers.
// Neither K' nor the score matrix ever reaches global memory; K and V are read only.
#include <math.h>

#include "seka_edit_tile.cuh"
#include "seka_kernels.h"

namespace seka {

struct AttnParams {
    void* O;
    float* lse;
    const uint8_t* mask;
    const float* alpha;
    const float* gain;
    const uint8_t* head_enable;
    const int* cu_seqlens;
    const uint4* frags;
    int* status;
    int B, L, Hq, Hkv, rank, M, r_pad, n_qt;
    int steer;
    float scale_log2;
};

constexpr int BM = 128, BN = 128;
constexpr uint32_t BLK_BYTES = 128 * 128;   // one [128 x 64] bf16 block

template <int D>
struct SmemLayout {
    static constexpr uint32_t TILE = (D / 64) * BLK_BYTES;
    static constexpr uint32_t Q = 0;
    static constexpr uint32_t K = Q + TILE;          // 2 stages
    static constexpr uint32_t V = K + 2 * TILE;      // 2 stages
    static constexpr uint32_t P = V + 2 * TILE;      // [128 x 128] bf16
    static constexpr uint32_t ROWFLAG = P + 2 * BLK_BYTES;   // 128 bytes
    static constexpr uint32_t COLSCALE = ROWFLAG + 128;      // 128 floats
    static constexpr uint32_t BARS = COLSCALE + 512;         // 8 mbarriers
    static constexpr uint32_t MISC = BARS + 64;              // tmem holder, abort flag
    static constexpr uint32_t TOTAL = MISC + 16;
    static constexpr uint32_t DYN_BYTES = TOTAL + 1024;      // slack for the 1024-byte alignment
};

template <typename OutT> __device__ __forceinline__ void store_row(OutT* dst, const float* o, int n, float inv);
template <> __device__ __forceinline__ void store_row<__nv_bfloat16>(__nv_bfloat16* dst, const float* o, int n, float inv) {
    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int c = 0; c < n / 8; ++c)
        d4[c] = make_uint4(pack_bf16(o[8 * c] * inv, o[8 * c + 1] * inv), pack_bf16(o[8 * c + 2] * inv, o[8 * c + 3] * inv),
                           pack_bf16(o[8 * c + 4] * inv, o[8 * c + 5] * inv), pack_bf16(o[8 * c + 6] * inv, o[8 * c + 7] * inv));
}
template <> __device__ __forceinline__ void store_row<float>(float* dst, const float* o, int n, float inv) {
    float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int c = 0; c < n / 4; ++c)
        d4[c] = make_float4(o[4 * c] * inv, o[4 * c + 1] * inv, o[4 * c + 2] * inv, o[4 * c + 3] * inv);
}

template <int D, typename OutT>
__global__ void __launch_bounds__(128, 1)
seka_attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    using SL = SmemLayout<D>;
    constexpr int NBLK = D / 64;
    constexpr uint32_t TMEM_COLS = 256;   // S: columns [0,128), P*V: columns [128, 128 + D)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + SL::Q;
    uint8_t* sP = smem + SL::P;
    uint8_t* rowflag = smem + SL::ROWFLAG;
    float* colscale = reinterpret_cast<float*>(smem + SL::COLSCALE);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::BARS);
    uint64_t* bar_q = bars + 0;
    uint64_t* bar_kv = bars + 1;   // [2]
    uint64_t* bar_s = bars + 3;
    uint64_t* bar_pv = bars + 4;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + SL::MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // heaviest query tiles first; CTAs of one (sequence, KV head) are neighbours
    const int per_qt = p.B * p.Hq;
    const int qt = p.n_qt - 1 - (int)(blockIdx.x / per_qt);
    const int rem = (int)(blockIdx.x % per_qt);
    const int b = rem / p.Hq, hq = rem % p.Hq;
    const int hkv = hq / (p.Hq / p.Hkv);
    const int seq0 = p.cu_seqlens ? p.cu_seqlens[b] : b * p.L;
    const int Lb = p.cu_seqlens ? (p.cu_seqlens[b + 1] - seq0) : p.L;
    if (qt * BM >= Lb) return;                      // nothing allocated yet
    if (*reinterpret_cast<volatile int*>(p.status) != 0) return;   // an earlier CTA gave up: do not pile on

    if (tid == 0) {
        mbar_init(bar_q, 1); mbar_init(bar_kv + 0, 1); mbar_init(bar_kv + 1, 1);
        mbar_init(bar_s, 1); mbar_init(bar_pv, 1);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, TMEM_COLS); tmem_relinquish(); }

    // steering parameters of this (sequence, KV head)
    const float g = p.steer ? p.gain[b] : 0.f;
    const bool steer = p.steer && g != 0.f && (p.head_enable == nullptr || p.head_enable[hkv] != 0);
    if (steer) {
        const int j = tid;   // 128 threads cover the 128 possible stacked columns
        float cs = 0.f;
        if (j < p.M * p.rank) cs = g * (p.alpha ? p.alpha[((size_t)b * p.Hkv + hkv) * p.M + j / p.rank] : 1.f);
        colscale[j] = cs;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t tS = t_lane, tPV = t_lane + 128;

    const int n_kv = qt + 1;
    constexpr uint32_t KV_BYTES = 2 * SL::TILE;
    if (tid == 0) {
        mbar_expect_tx(bar_q, SL::TILE);
#pragma unroll
        for (int c = 0; c < NBLK; ++c) tma_load_3d(sQ + c * BLK_BYTES, &tmQ, bar_q, c * 64, hq, seq0 + qt * BM);
        mbar_expect_tx(bar_kv + 0, KV_BYTES);
#pragma unroll
        for (int c = 0; c < NBLK; ++c) {
            tma_load_3d(smem + SL::K + c * BLK_BYTES, &tmK, bar_kv + 0, c * 64, hkv, seq0);
            tma_load_3d(smem + SL::V + c * BLK_BYTES, &tmV, bar_kv + 0, c * 64, hkv, seq0);
        }
    }
    int loads_issued = 1, loads_waited = 0;   // meaningful on thread 0 only

    const size_t fr_head = frag_uint4_per_head(D, p.r_pad);
    const uint4* fragB = p.frags + (size_t)hkv * fr_head;
    const uint4* fragA = fragB + fr_head / 2;
    const int nR16 = p.r_pad / 16;

    constexpr uint32_t IDESC_S = umma_idesc_bf16(BN, false);
    constexpr uint32_t IDESC_PV = umma_idesc_bf16(D, true);

    float o[D];
#pragma unroll
    for (int c = 0; c < D; ++c) o[c] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    const int row = tid;
    bool ok = true;

    for (int j = 0; j < n_kv; ++j) {
        const int s = j & 1;
        uint8_t* sK = smem + SL::K + s * SL::TILE;
        uint8_t* sV = smem + SL::V + s * SL::TILE;
        if (tid == 0 && j + 1 < n_kv) {
            const int s2 = s ^ 1;
            mbar_expect_tx(bar_kv + s2, KV_BYTES);
#pragma unroll
            for (int c = 0; c < NBLK; ++c) {
                tma_load_3d(smem + SL::K + s2 * SL::TILE + c * BLK_BYTES, &tmK, bar_kv + s2, c * 64, hkv, seq0 + (j + 1) * BN);
                tma_load_3d(smem + SL::V + s2 * SL::TILE + c * BLK_BYTES, &tmV, bar_kv + s2, c * 64, hkv, seq0 + (j + 1) * BN);
            }
            ++loads_issued;
        }
        // which keys of this tile are highlighted
        int hl = 0;
        if (steer) {
            const int kpos = j * BN + tid;
            hl = (kpos < Lb && p.mask[seq0 + kpos] != 0) ? 1 : 0;
            rowflag[tid] = (uint8_t)hl;
        }
        const int any_hl = __syncthreads_or(hl);

        ok = mbar_wait(bar_kv + s, (uint32_t)((j >> 1) & 1), abort_flag, p.status, 1);
        if (tid == 0) ++loads_waited;
        __syncwarp();
        if (__all_sync(0xffffffffu, ok) && any_hl) {
#pragma unroll 1
            for (int blk = 0; blk < 2; ++blk) {
                const int r0 = warp * 32 + blk * 16;
                const uint32_t f4 = *reinterpret_cast<const uint32_t*>(rowflag + r0) | *reinterpret_cast<const uint32_t*>(rowflag + r0 + 4) |
                                    *reinterpret_cast<const uint32_t*>(rowflag + r0 + 8) | *reinterpret_cast<const uint32_t*>(rowflag + r0 + 12);
                if (f4 != 0) edit_rows16<D>(sK, BLK_BYTES, r0, rowflag, fragB, fragA, colscale, nR16, lane);
            }
            fence_proxy_async();
        }
        if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }

        // S = Q K'^T
        if (tid == 0) {
            if (j == 0) ok = mbar_wait(bar_q, 0, abort_flag, p.status, 2);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32;
                    umma_ss(tmem_base, umma_desc_sw128(smem_u32(sQ) + off, 16, 1024),
                            umma_desc_sw128(smem_u32(sK) + off, 16, 1024), IDESC_S, ks > 0 ? 1u : 0u);
                }
                umma_commit(bar_s);
            }
        }
        ok = mbar_wait(bar_s, (uint32_t)(j & 1), abort_flag, p.status, 3) && ok;
        __syncwarp();
        tc_fence_after();

        float corr = 1.f;
        if (ok) {
            const bool diag = (j == qt);
            uint32_t v[32];
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                tmem_ld32(tS + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    float x = __uint_as_float(v[e]);
                    if (diag && (c * 32 + e) > row) x = -INFINITY;
                    mx = fmaxf(mx, x);
                }
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            corr = fast_exp2(m_run - m_new);
            float psum = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                tmem_ld32(tS + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int e8 = 0; e8 < 4; ++e8) {
                    float pv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int col = c * 32 + e8 * 8 + e;
                        float x = fast_exp2(fmaf(__uint_as_float(v[e8 * 8 + e]), p.scale_log2, -m_new));
                        if (diag && col > row) x = 0.f;
                        pv[e] = x;
                        psum += x;
                    }
                    const int col0 = c * 32 + e8 * 8;
                    uint4 pk = make_uint4(pack_bf16(pv[0], pv[1]), pack_bf16(pv[2], pv[3]), pack_bf16(pv[4], pv[5]), pack_bf16(pv[6], pv[7]));
                    *reinterpret_cast<uint4*>(sP + (uint32_t)(col0 >> 6) * BLK_BYTES + sw128_offset(row, col0 & 63)) = pk;
                }
            }
            l_run = l_run * corr + psum;
            m_run = m_new;
            fence_proxy_async();
        }
        tc_fence_before();
        if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }

        // PV = P V
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < BN / 16; ++ks) {
                const uint32_t offP = (uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32;
                umma_ss(tmem_base + 128, umma_desc_sw128(smem_u32(sP) + offP, 16, 1024),
                        umma_desc_sw128(smem_u32(sV) + (uint32_t)ks * 2048, BLK_BYTES, 1024), IDESC_PV, ks > 0 ? 1u : 0u);
            }
            umma_commit(bar_pv);
        }
        ok = mbar_wait(bar_pv, (uint32_t)(j & 1), abort_flag, p.status, 4);
        __syncwarp();
        tc_fence_after();
        if (ok) {
            uint32_t v[32];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(tPV + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) o[c * 32 + e] = fmaf(o[c * 32 + e], corr, __uint_as_float(v[e]));
            }
        }
        tc_fence_before();
        if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }
    }

    if (ok) {
        const int qpos = qt * BM + row;
        if (qpos < Lb) {
            const size_t orow = (size_t)(seq0 + qpos) * p.Hq + hq;
            store_row<OutT>(static_cast<OutT*>(p.O) + orow * D, o, D, 1.f / l_run);
            if (p.lse != nullptr) p.lse[orow] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
    } else if (tid == 0) {
        // let any tile load still in flight land before the CTA's shared memory is released
        int dummy = 0;
        while (loads_waited < loads_issued) {
            mbar_wait(bar_kv + (loads_waited & 1), (uint32_t)((loads_waited >> 1) & 1), &dummy, nullptr, 0);
            ++loads_waited;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// bf16 tensor [T, H, d] viewed as (d, H, T); tiles of 64 x 1 x 128 with the 128-byte swizzle.
static bool make_tile_map(CUtensorMap* m, const void* base, int d, int H, int T) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)H * d * 2};
    cuuint32_t box[3] = {64, 1, 128};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, typename OutT>
static seka_status launch_attn(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const AttnParams& p, cudaStream_t st) {
    using SL = SmemLayout<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(seka_attn_fwd_kernel<D, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)SL::DYN_BYTES) != cudaSuccess) return SEKA_ERR_CUDA;
        configured = true;
    }
    const unsigned grid = (unsigned)p.n_qt * p.B * p.Hq;
    seka_attn_fwd_kernel<D, OutT><<<grid, 128, SL::DYN_BYTES, st>>>(tq, tk, tv, p);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

}  // namespace seka

extern "C" seka_status seka_attention_fwd(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                          void* O, float* lse, const uint8_t* mask, const float* U,
                                          const float* alpha, const float* gain, const uint8_t* head_enable,
                                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_shape(shape);
    if (stc != SEKA_OK) return stc;
    const int T = shape_total_tokens(shape);
    if (T == 0 || shape->batch == 0 || shape->max_seqlen == 0) return SEKA_OK;
    if (!Q || !K || !V || !O) return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15) return SEKA_ERR_INVALID_ARG;
    const bool steer = mask != nullptr && U != nullptr;
    if (steer && !gain) return SEKA_ERR_INVALID_ARG;
    const WorkspaceLayout w = workspace_layout(shape);
    if (!workspace || workspace_bytes < w.total || ((uintptr_t)workspace & 255)) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    const int D = shape->head_dim, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads;

    const void *q16 = Q, *k16 = K, *v16 = V;
    if (shape->dtype == SEKA_F32) {
        const size_t nq = (size_t)T * Hq * D, nk = (size_t)T * Hkv * D;
        char* cq = ws + w.cvt_off;
        char* ck = cq + align_up(nq * 2, 256);
        char* cv = ck + align_up(nk * 2, 256);
        launch_convert_bf16(static_cast<const float*>(Q), cq, nq, st);
        launch_convert_bf16(static_cast<const float*>(K), ck, nk, st);
        launch_convert_bf16(static_cast<const float*>(V), cv, nk, st);
        q16 = cq; k16 = ck; v16 = cv;
    }
    uint4* frags = reinterpret_cast<uint4*>(ws + w.frag_off);
    if (steer) launch_prep_fragments(U, frags, Hkv, D, shape->rank, shape->n_experts, w.r_pad, st);

    CUtensorMap tq, tk, tv;
    if (!make_tile_map(&tq, q16, D, Hq, T) || !make_tile_map(&tk, k16, D, Hkv, T) || !make_tile_map(&tv, v16, D, Hkv, T))
        return SEKA_ERR_CUDA;

    AttnParams p;
    p.O = O; p.lse = lse; p.mask = mask; p.alpha = alpha; p.gain = gain; p.head_enable = head_enable;
    p.cu_seqlens = shape->cu_seqlens; p.frags = frags; p.status = reinterpret_cast<int*>(ws);
    p.B = shape->batch; p.L = shape->max_seqlen; p.Hq = Hq; p.Hkv = Hkv; p.rank = shape->rank; p.M = shape->n_experts;
    p.r_pad = w.r_pad; p.n_qt = (shape->max_seqlen + BM - 1) / BM; p.steer = steer ? 1 : 0;
    const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;

    if (D == 128) {
        return shape->dtype == SEKA_F32 ? launch_attn<128, float>(tq, tk, tv, p, st)
                                        : launch_attn<128, __nv_bfloat16>(tq, tk, tv, p, st);
    }
    return shape->dtype == SEKA_F32 ? launch_attn<64, float>(tq, tk, tv, p, st)
                                    : launch_attn<64, __nv_bfloat16>(tq, tk, tv, p, st);
}

extern "C" size_t seka_host_staging_bytes(const seka_shape* shape) {
    using namespace seka;
    if (validate_shape(shape) != SEKA_OK) return 0;
    const size_t T = (size_t)shape_total_tokens(shape), esz = shape->dtype == SEKA_F32 ? 4 : 2;
    const size_t nq = align_up(T * shape->n_q_heads * shape->head_dim * esz, 256);
    const size_t nk = align_up(T * shape->n_kv_heads * shape->head_dim * esz, 256);
    return 2 * nq + 2 * nk + align_up(T, 256) + align_up(T * shape->n_q_heads * 4, 256);
}

extern "C" seka_status seka_attention_fwd_host(const seka_shape* shape, const void* h_Q, const void* h_K,
                                               const void* h_V, void* h_O, float* h_lse, const uint8_t* h_mask,
                                               const float* U, const float* alpha, const float* gain,
                                               const uint8_t* head_enable, void* staging, size_t staging_bytes,
                                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_shape(shape);
    if (stc != SEKA_OK) return stc;
    const size_t T = (size_t)shape_total_tokens(shape);
    if (T == 0) return SEKA_OK;
    if (!h_Q || !h_K || !h_V || !h_O) return SEKA_ERR_INVALID_ARG;
    if (!staging || staging_bytes < seka_host_staging_bytes(shape) || ((uintptr_t)staging & 255)) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t esz = shape->dtype == SEKA_F32 ? 4 : 2;
    const size_t bq = T * shape->n_q_heads * shape->head_dim * esz, bk = T * shape->n_kv_heads * shape->head_dim * esz;
    char* dq = static_cast<char*>(staging);
    char* dk = dq + align_up(bq, 256);
    char* dv = dk + align_up(bk, 256);
    char* dO = dv + align_up(bk, 256);
    char* dm = dO + align_up(bq, 256);
    char* dl = dm + align_up(T, 256);
    bool okc = cudaMemcpyAsync(dq, h_Q, bq, cudaMemcpyHostToDevice, st) == cudaSuccess;
    okc = okc && cudaMemcpyAsync(dk, h_K, bk, cudaMemcpyHostToDevice, st) == cudaSuccess;
    okc = okc && cudaMemcpyAsync(dv, h_V, bk, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (h_mask) okc = okc && cudaMemcpyAsync(dm, h_mask, T, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!okc) return SEKA_ERR_CUDA;
    stc = seka_attention_fwd(shape, dq, dk, dv, dO, h_lse ? reinterpret_cast<float*>(dl) : nullptr,
                             h_mask ? reinterpret_cast<const uint8_t*>(dm) : nullptr, U, alpha, gain, head_enable,
                             workspace, workspace_bytes, cuda_stream);
    if (stc != SEKA_OK) return stc;
    okc = cudaMemcpyAsync(h_O, dO, bq, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (h_lse) okc = okc && cudaMemcpyAsync(h_lse, dl, T * shape->n_q_heads * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    return okc ? SEKA_OK : SEKA_ERR_CUDA;
}
