// Decode-step attention over a cached, already edited key tensor (Algorithm 1: the hook edits the prompt's
// keys once, before generation; every generated token then attends to the whole cache).  One query token per
// sequence, so the step reads every cached key and value once and is bound by HBM bandwidth.
//
//   decode_split_kernel   one CTA per (sequence, KV head, chunk of cached tokens): a producer warp streams
//                         64-token K and V tiles through a ring of shared-memory stages with TMA; four
//                         consumer warps take 16 tokens of each stage, form the scores of the whole query
//                         group (query heads of the KV head padded to the 16 rows of mma.sync m16n8k16),
//                         keep a private online softmax and accumulate P V in registers; the warps' states
//                         are merged in shared memory and written as one partial (m, l, unnormalised o).
//   decode_combine_kernel merges the partials of a (sequence, query head) and normalises.
#include <math.h>

#include "seka_kernels.h"

namespace seka {
namespace {

constexpr int DEC_STAGE_KEYS = 64;
constexpr int DEC_CONSUMERS = 4;                       // warps; each owns 16 tokens of a stage
constexpr int DEC_THREADS = (DEC_CONSUMERS + 1) * 32;  // + one producer warp
constexpr int DEC_MAX_GROUP = 16;                      // query heads per KV head (rows of one MMA)
constexpr int DEC_SM_COUNT = 148;                      // used for sizing the split only

template <int D>
struct DecSmem {
    static constexpr int NSTAGE = D == 128 ? 3 : 4;
    static constexpr int CTAS_PER_SM = D == 128 ? 2 : 3;
    static constexpr int TILE_BYTES = DEC_STAGE_KEYS * D * 2;      // K or V of one stage
    static constexpr int BLOCK_BYTES = DEC_STAGE_KEYS * 128;       // one [64 tokens x 64 elements] swizzled block
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int BAR_OFF = NSTAGE * STAGE_BYTES;
    static constexpr int MISC_OFF = BAR_OFF + 2 * NSTAGE * 8;
    static constexpr int BYTES = MISC_OFF + 16;
    static constexpr int DYN_BYTES = BYTES + 1024;                 // room to align the base to 1024 bytes
    static constexpr int MERGE_STRIDE = D + 2;                     // floats per row: o[D], m, l
    static_assert(DEC_CONSUMERS * 16 * MERGE_STRIDE * 4 <= NSTAGE * STAGE_BYTES, "merge area aliases the stages");
};

struct DecodeParams {
    const __nv_bfloat16* Q;     // [B, Hq, D]
    __nv_bfloat16* O;           // [B, Hq, D]
    float* lse;                 // [B, Hq] or null
    const int* cu_seqlens;
    int B, L, Hq, Hkv, G;
    int chunk, n_splits;        // cached tokens per CTA (a multiple of 64), chunks per sequence at max_seqlen
    float scale_log2;
    float* part_o;              // [B, Hkv, n_splits, G, D] unnormalised outputs
    float* part_ml;             // [B, Hkv, n_splits, G, 2] running maximum (log2 domain) and sum
    int* status;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
// D[16 x 8] += A[16 x 16] B[16 x 8], bf16 operands, fp32 accumulation
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// HALF: the query group has at most 8 heads, so rows 8..15 of every MMA are padding and their softmax is skipped.
template <int D, bool HALF>
__global__ void __launch_bounds__(DEC_THREADS, DecSmem<D>::CTAS_PER_SM)
decode_split_kernel(const __grid_constant__ CUtensorMap tk, const __grid_constant__ CUtensorMap tv,
                    const DecodeParams p) {
    using SL = DecSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + SL::BAR_OFF);
    uint64_t* empty = full + SL::NSTAGE;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::MISC_OFF);

    const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int seq0, Lb;
    if (p.cu_seqlens != nullptr) { seq0 = p.cu_seqlens[b]; Lb = p.cu_seqlens[b + 1] - seq0; }
    else { seq0 = b * p.L; Lb = p.L; }
    const int k_begin = split * p.chunk;
    if (k_begin >= Lb) return;                              // the whole CTA leaves before any barrier exists
    const int k_end = min(Lb, k_begin + p.chunk);
    const int n_stage = (k_end - k_begin + DEC_STAGE_KEYS - 1) / DEC_STAGE_KEYS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SL::NSTAGE; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], DEC_CONSUMERS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    const int G = p.G;
    const int r0 = lane >> 2, cq = (lane & 3) * 2;          // accumulator rows r0 and r0 + 8, columns cq, cq + 1
    float o[D / 8][4];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
#pragma unroll
    for (int j = 0; j < D / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

    if (warp == DEC_CONSUMERS) {
        // ------------------------------------------------ producer: one lane streams the K and V tiles
        if (lane == 0) {
            tma_prefetch_desc(&tk);
            tma_prefetch_desc(&tv);
            int issued = 0;
            bool ok = true;
            for (int i = 0; i < n_stage; ++i) {
                const int s = i % SL::NSTAGE, round = i / SL::NSTAGE;
                if (round > 0 && !mbar_wait(&empty[s], (uint32_t)(round - 1) & 1u, abort_flag, p.status, 60)) { ok = false; break; }
                uint8_t* kt = smem + s * SL::STAGE_BYTES;
                mbar_expect_tx(&full[s], SL::STAGE_BYTES);
                const int row = seq0 + k_begin + i * DEC_STAGE_KEYS;
#pragma unroll
                for (int blk = 0; blk < D / 64; ++blk) {
                    tma_load_3d(kt + blk * SL::BLOCK_BYTES, &tk, &full[s], blk * 64, hkv, row);
                    tma_load_3d(kt + SL::TILE_BYTES + blk * SL::BLOCK_BYTES, &tv, &full[s], blk * 64, hkv, row);
                }
                issued = i + 1;
            }
            if (!ok || *abort_flag) {
                // a wait ran out somewhere: let the copies already issued land before the CTA's shared memory is released
                const int first = issued > SL::NSTAGE ? issued - SL::NSTAGE : 0;
                for (int i = first; i < issued; ++i) {
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(&full[i % SL::NSTAGE], (uint32_t)(i / SL::NSTAGE) & 1u) &&
                           global_timer_ns() - t0 < kWaitLimitNs) { }
                }
            }
        }
    } else {
        // ------------------------------------------------ consumers
        // A fragments of the query group (rows = query heads of this KV head, zero beyond the group), kept in registers
        uint32_t qa[D / 16][4];
        {
            const __nv_bfloat16* qb = p.Q + ((size_t)b * p.Hq + (size_t)hkv * G) * D;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const int c = kk * 16 + cq;
                qa[kk][0] = r0 < G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)r0 * D + c) : 0u;
                qa[kk][2] = r0 < G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)r0 * D + c + 8) : 0u;
                if (!HALF) {
                    qa[kk][1] = r0 + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)(r0 + 8) * D + c) : 0u;
                    qa[kk][3] = r0 + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)(r0 + 8) * D + c + 8) : 0u;
                } else {
                    qa[kk][1] = 0u; qa[kk][3] = 0u;
                }
            }
        }
        // ldmatrix source rows of this lane inside the warp's 16 tokens of a stage
        const int key_k = 16 * warp + (lane & 7) + ((lane >> 4) << 3);         // K: matrices 2, 3 hold tokens 8..15
        const int key_v = 16 * warp + (lane & 7) + (((lane >> 3) & 1) << 3);   // V: matrices 1, 3 hold tokens 8..15
        const uint32_t k_row = (uint32_t)key_k * 128u, v_row = (uint32_t)key_v * 128u;
        const uint32_t k_sel = (uint32_t)((lane >> 3) & 1), v_sel = (uint32_t)(lane >> 4);
        const uint32_t smem_base = smem_u32(smem);

        for (int i = 0; i < n_stage; ++i) {
            const int s = i % SL::NSTAGE;
            if (!mbar_wait(&full[s], (uint32_t)(i / SL::NSTAGE) & 1u, abort_flag, p.status, 61)) break;
            const uint32_t kt = smem_base + (uint32_t)(s * SL::STAGE_BYTES), vt = kt + SL::TILE_BYTES;

            // scores of the group against the warp's 16 tokens: two 16 x 8 tiles
            float sc[2][4];
#pragma unroll
            for (int t = 0; t < 2; ++t) { sc[t][0] = sc[t][1] = sc[t][2] = sc[t][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t chunk = (uint32_t)((kk & 3) * 2) + k_sel;
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kt + (uint32_t)((kk >> 2) * SL::BLOCK_BYTES) + k_row + (((chunk ^ (uint32_t)key_k) & 7u) << 4), b0, b1, b2, b3);
                mma_16816(sc[0], qa[kk], b0, b1);
                mma_16816(sc[1], qa[kk], b2, b3);
            }
            // tokens beyond the end of the chunk (ragged tail; they may belong to the next sequence) get no weight
            const int base = k_begin + i * DEC_STAGE_KEYS + 16 * warp;
            if (base + 16 > k_end) {
#pragma unroll
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (base + 8 * t + cq + (e & 1) >= k_end) sc[t][e] = -INFINITY;
            }
            // online softmax, private to the warp; the row sums stay per thread until the end
            float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            const float mn0 = fmaxf(m0, mx0 * p.scale_log2);
            const float ms0 = mn0 == -INFINITY ? 0.f : mn0;
            const float f0 = fast_exp2(m0 - ms0);
            float mn1 = -INFINITY, ms1 = 0.f, f1 = 1.f;
            if (!HALF) {
                float mx1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                mn1 = fmaxf(m1, mx1 * p.scale_log2);
                ms1 = mn1 == -INFINITY ? 0.f : mn1;
                f1 = fast_exp2(m1 - ms1);
            }
            const bool moved = (mn0 != m0) || (!HALF && mn1 != m1);
            if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
                for (int j = 0; j < D / 8; ++j) {
                    o[j][0] *= f0; o[j][1] *= f0;
                    if (!HALF) { o[j][2] *= f1; o[j][3] *= f1; }
                }
            }
            m0 = mn0; m1 = mn1;
            uint32_t pa[4];
            {
                const float p00 = fast_exp2(fmaf(sc[0][0], p.scale_log2, -ms0)), p01 = fast_exp2(fmaf(sc[0][1], p.scale_log2, -ms0));
                const float p10 = fast_exp2(fmaf(sc[1][0], p.scale_log2, -ms0)), p11 = fast_exp2(fmaf(sc[1][1], p.scale_log2, -ms0));
                l0 = fmaf(l0, f0, (p00 + p01) + (p10 + p11));
                pa[0] = pack_bf16(p00, p01); pa[2] = pack_bf16(p10, p11);
                if (!HALF) {
                    const float q00 = fast_exp2(fmaf(sc[0][2], p.scale_log2, -ms1)), q01 = fast_exp2(fmaf(sc[0][3], p.scale_log2, -ms1));
                    const float q10 = fast_exp2(fmaf(sc[1][2], p.scale_log2, -ms1)), q11 = fast_exp2(fmaf(sc[1][3], p.scale_log2, -ms1));
                    l1 = fmaf(l1, f1, (q00 + q01) + (q10 + q11));
                    pa[1] = pack_bf16(q00, q01); pa[3] = pack_bf16(q10, q11);
                } else {
                    pa[1] = 0u; pa[3] = 0u;
                }
            }
            // o[16 x D] += P[16 x 16 tokens] V[16 tokens x D]
#pragma unroll
            for (int jp = 0; jp < D / 16; ++jp) {
                const uint32_t chunk = (uint32_t)((jp & 3) * 2) + v_sel;
                uint32_t b0, b1, b2, b3;
                ldsm_x4_trans(vt + (uint32_t)((jp >> 2) * SL::BLOCK_BYTES) + v_row + (((chunk ^ (uint32_t)key_v) & 7u) << 4), b0, b1, b2, b3);
                mma_16816(o[2 * jp], pa, b0, b1);
                mma_16816(o[2 * jp + 1], pa, b2, b3);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }

    // ---------------------------------------------------- merge the four warps' states, write the partial
    __syncthreads();                                        // every stage has been consumed (or the CTA has aborted)
    if (*abort_flag) return;
    float* mg = reinterpret_cast<float*>(smem);             // [warp][16 rows][D + 2]
    if (warp < DEC_CONSUMERS) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        if (!HALF) {
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        }
        float* row0 = mg + ((size_t)warp * 16 + r0) * SL::MERGE_STRIDE;
        if (r0 < G) {
#pragma unroll
            for (int j = 0; j < D / 8; ++j) { row0[8 * j + cq] = o[j][0]; row0[8 * j + cq + 1] = o[j][1]; }
            if ((lane & 3) == 0) { row0[D] = m0; row0[D + 1] = l0; }
        }
        if (!HALF && r0 + 8 < G) {
            float* row1 = row0 + 8 * SL::MERGE_STRIDE;
#pragma unroll
            for (int j = 0; j < D / 8; ++j) { row1[8 * j + cq] = o[j][2]; row1[8 * j + cq + 1] = o[j][3]; }
            if ((lane & 3) == 0) { row1[D] = m1; row1[D + 1] = l1; }
        }
    }
    __syncthreads();
    const size_t item = ((size_t)b * p.Hkv + hkv) * p.n_splits + split;
    for (int idx = threadIdx.x; idx < G * D; idx += DEC_THREADS) {
        const int g = idx / D, c = idx - g * D;
        float mw[DEC_CONSUMERS], M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_CONSUMERS; ++w) { mw[w] = mg[((size_t)w * 16 + g) * SL::MERGE_STRIDE + D]; M = fmaxf(M, mw[w]); }
        float acc = 0.f, lsum = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_CONSUMERS; ++w) {
            const float f = mw[w] == -INFINITY ? 0.f : fast_exp2(mw[w] - M);
            acc = fmaf(mg[((size_t)w * 16 + g) * SL::MERGE_STRIDE + c], f, acc);
            lsum = fmaf(mg[((size_t)w * 16 + g) * SL::MERGE_STRIDE + D + 1], f, lsum);
        }
        p.part_o[(item * G + g) * D + c] = acc;
        if (c == 0) { p.part_ml[(item * G + g) * 2] = M; p.part_ml[(item * G + g) * 2 + 1] = lsum; }
    }
}

// One CTA per (sequence, query head), one thread per output element.
__global__ void decode_combine_kernel(const DecodeParams p, int D) {
    const int b = blockIdx.x / p.Hq, hq = blockIdx.x - b * p.Hq;
    const int hkv = hq / p.G, g = hq - hkv * p.G;
    const int c = threadIdx.x;
    const int Lb = p.cu_seqlens != nullptr ? p.cu_seqlens[b + 1] - p.cu_seqlens[b] : p.L;
    const int ns = (Lb + p.chunk - 1) / p.chunk;            // chunks that held cached tokens
    const size_t item0 = ((size_t)b * p.Hkv + hkv) * p.n_splits;
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, p.part_ml[((item0 + s) * p.G + g) * 2]);
    float acc = 0.f, l = 0.f;
    for (int s = 0; s < ns; ++s) {
        const float ms = p.part_ml[((item0 + s) * p.G + g) * 2];
        const float f = ms == -INFINITY ? 0.f : fast_exp2(ms - M);
        l = fmaf(p.part_ml[((item0 + s) * p.G + g) * 2 + 1], f, l);
        acc = fmaf(p.part_o[((item0 + s) * p.G + g) * D + c], f, acc);
    }
    const bool any = ns > 0 && l > 0.f;
    p.O[((size_t)b * p.Hq + hq) * D + c] = __float2bfloat16(any ? acc / l : 0.f);
    if (p.lse != nullptr && c == 0)
        p.lse[(size_t)b * p.Hq + hq] = any ? (M + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

struct DecodePlan {
    int chunk, n_splits;
    size_t ml_off, ml_bytes, o_off, o_bytes, total;
};

// Chunks of cached tokens.  A CTA has a fixed cost (query fragments, the merge of its warps, its partial), so chunks
// are long: about three waves of CTAs over the SMs, at least 1024 tokens each.  Where that would leave SMs without
// work (few sequences), the chunks shrink until one wave is full, down to 256 tokens.
DecodePlan decode_plan(const seka_shape* s) {
    DecodePlan d;
    const int G = s->n_q_heads / s->n_kv_heads;
    const long long pairs = (long long)s->batch * s->n_kv_heads;
    const int slots = DEC_SM_COUNT * (s->head_dim == 128 ? DecSmem<128>::CTAS_PER_SM : DecSmem<64>::CTAS_PER_SM);
    const long long want = pairs > 0 ? (3LL * slots + pairs - 1) / pairs : 1;    // splits that would give 3 waves
    const long long fill = pairs > 0 ? (slots + pairs - 1) / pairs : 1;          // splits that fill one wave
    long long chunk = (s->max_seqlen + want - 1) / want;
    if (chunk < 1024) {
        chunk = (s->max_seqlen + fill - 1) / fill;
        if (chunk > 1024) chunk = 1024;
        if (chunk < 256) chunk = 256;
    }
    chunk = (chunk + DEC_STAGE_KEYS - 1) / DEC_STAGE_KEYS * DEC_STAGE_KEYS;
    d.chunk = (int)chunk;
    d.n_splits = s->max_seqlen > 0 ? (s->max_seqlen + d.chunk - 1) / d.chunk : 1;
    const size_t items = (size_t)(pairs > 0 ? pairs : 0) * d.n_splits * G;
    d.ml_off = kStatusBytes;
    d.ml_bytes = align_up(items * 2 * sizeof(float) + 16, 256);
    d.o_off = d.ml_off + d.ml_bytes;
    d.o_bytes = align_up(items * s->head_dim * sizeof(float) + 16, 256);
    d.total = d.o_off + d.o_bytes;
    return d;
}

seka_status validate_decode(const seka_shape* s) {
    seka_status st = validate_shape(s);
    if (st != SEKA_OK) return st;
    if (s->dtype != SEKA_BF16) return SEKA_ERR_UNSUPPORTED;
    if (s->n_q_heads / s->n_kv_heads > DEC_MAX_GROUP) return SEKA_ERR_UNSUPPORTED;
    if (s->batch > 65535 || s->n_kv_heads > 65535) return SEKA_ERR_UNSUPPORTED;
    return SEKA_OK;
}

template <int D, bool HALF>
seka_status launch_split(const CUtensorMap& tk, const CUtensorMap& tv, const DecodeParams& p, cudaStream_t st) {
    using SL = DecSmem<D>;
    // the attribute belongs to the function on the current device: set on every call (a cheap driver call), so that
    // several devices or host threads need no bookkeeping here
    if (cudaFuncSetAttribute(decode_split_kernel<D, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)SL::DYN_BYTES) != cudaSuccess) return SEKA_ERR_CUDA;
    dim3 grid((unsigned)p.n_splits, (unsigned)p.Hkv, (unsigned)p.B);
    decode_split_kernel<D, HALF><<<grid, DEC_THREADS, SL::DYN_BYTES, st>>>(tk, tv, p);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

}  // namespace
}  // namespace seka

extern "C" size_t seka_decode_workspace_bytes(const seka_shape* shape) {
    if (seka::validate_decode(shape) != SEKA_OK) return 0;
    return seka::decode_plan(shape).total;
}

extern "C" seka_status seka_decode_attention(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                             void* O, float* lse, void* workspace, size_t workspace_bytes,
                                             void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_decode(shape);
    if (stc != SEKA_OK) return stc;
    if (shape->batch == 0) return SEKA_OK;
    const long long T = shape_total_tokens(shape);
    if (Q == nullptr || O == nullptr || (T > 0 && (K == nullptr || V == nullptr))) return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15) return SEKA_ERR_INVALID_ARG;
    const DecodePlan plan = decode_plan(shape);
    if (workspace == nullptr || workspace_bytes < plan.total) return SEKA_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255) return SEKA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int D = shape->head_dim, Hkv = shape->n_kv_heads;

    DecodeParams p;
    p.Q = static_cast<const __nv_bfloat16*>(Q); p.O = static_cast<__nv_bfloat16*>(O); p.lse = lse;
    p.cu_seqlens = shape->cu_seqlens;
    p.B = shape->batch; p.L = shape->max_seqlen; p.Hq = shape->n_q_heads; p.Hkv = Hkv; p.G = shape->n_q_heads / Hkv;
    p.chunk = plan.chunk; p.n_splits = plan.n_splits;
    const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.part_ml = reinterpret_cast<float*>(ws + plan.ml_off);
    p.part_o = reinterpret_cast<float*>(ws + plan.o_off);
    p.status = reinterpret_cast<int*>(ws);

    if (T > 0 && shape->max_seqlen > 0) {
        CUtensorMap tk, tv;
        if (!make_tile_map(&tk, K, D, Hkv, T, DEC_STAGE_KEYS) || !make_tile_map(&tv, V, D, Hkv, T, DEC_STAGE_KEYS))
            return SEKA_ERR_CUDA;
        const bool half = p.G <= 8;
        seka_status s2 = D == 128 ? (half ? launch_split<128, true>(tk, tv, p, st) : launch_split<128, false>(tk, tv, p, st))
                                  : (half ? launch_split<64, true>(tk, tv, p, st) : launch_split<64, false>(tk, tv, p, st));
        if (s2 != SEKA_OK) return s2;
    }
    decode_combine_kernel<<<(unsigned)(p.B * p.Hq), D, 0, st>>>(p, D);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}
