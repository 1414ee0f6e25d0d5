// Small preparation kernels: dense edit operators and per-tile highlight flags for the fused kernel,
// highlight-mask compaction, fp32 -> bf16 input conversion.
#include "seka_kernels.h"
#include "seka_route.cuh"

namespace seka {

// Operand preparation of the fused kernel, one launch.  The fused kernel stages every key tile that holds a highlighted
// token from a side buffer of edited keys (Eq. 5: the edited logit is q.k' with k' = k + g P k); this launch writes it:
//   blocks [0, n_flag):        one block per sequence: a flag per 128-key tile (does it hold a highlighted token?), the
//                              sequence's first such tile, and per KV head whether it is steered and whether the fused
//                              kernel multiplies the low parts too (see lo_needed);
//   blocks [n_flag, +n_a):     (only with `route.alpha_out`) one block per (sequence, KV head): the routing coefficients
//                              of Eq. 6, from the last token's query, for the caller;
//   the remaining n_x blocks:  a KV head each (n_x is a multiple of Hkv); together the warps of a head's blocks walk the
//                              tokens of every (sequence, key tile) pair that holds a highlighted token, a warp per token:
//                                  k' = k + g_b sum_m alpha_{b,h,m} U_m[h] (U_m[h]^T k)   (highlighted tokens; k otherwise)
//                              in fp32 (the contraction order of Algorithm 1's hook: first U^T k, then back through U),
//                              written as a high and a low bf16 part into one row of `X` [T, Hkv, 2 d]: high parts at
//                              columns [0, d), low parts at [d, 2 d) (only where the fused kernel reads them).  With
//                              `route.sigma` set these blocks compute the coefficients of Eq. 6 themselves, so that
//                              AdaSEKA needs no launch of its own before the forward.
// Plain fp32 multiply-adds on purpose: warp-level mma.sync gets little from this GPU's tensor cores (measured: about
// ten cycles per m16n8k16 and SM), the two bf16 parts it needs for fp32 accuracy triple the products, and it cannot
// skip the tokens that are not highlighted.
struct RouteArgs {
    const void* Q; int q_is_f32; const float* sigma; int k_route; int Hq; float* alpha_out;
};

constexpr int PREP_THREADS = 256;
constexpr int HOT_CAP = 2048;  // (sequence, tile) pairs looked at per round of the edited-key blocks
constexpr int ALPHA_CAP = 2048; // routed coefficients a block can hold (sequences x experts)
__device__ __forceinline__ size_t align_up_dev(size_t x, size_t a) { return (x + a - 1) / a * a; }

// two fp32 values -> their high bf16 parts and their low bf16 parts, packed in pairs
__device__ __forceinline__ void split_pair(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
    hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
    lo = pack_bf16(x - __bfloat162float(xh), y - __bfloat162float(yh));
}

template <int D>
__global__ void __launch_bounds__(PREP_THREADS, 2)
prep_steering_kernel(const __grid_constant__ CUtensorMap tmK, int* status, const float* __restrict__ U, const float* __restrict__ alpha,
                     const float* __restrict__ gain, const uint8_t* __restrict__ head_enable,
                     const uint8_t* __restrict__ mask, const int* __restrict__ cu_seqlens,
                     __nv_bfloat16* __restrict__ X, uint8_t* __restrict__ tile_hot, int* __restrict__ first_hot,
                     uint8_t* __restrict__ bh_info, int B, int L, int Hkv, int r, int M, int n_tiles, int n_flag,
                     int n_a, int n_x, const RouteArgs route) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    extern __shared__ __align__(16) unsigned char prep_sm[];
    if ((int)blockIdx.x < n_flag) {
        // ------------------------------------------------------------ flags of one sequence
        const int b = blockIdx.x;
        const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
        const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
        __shared__ int first_s;
        if (tid == 0) first_s = 0x7fffffff;
        __syncthreads();
        int first = 0x7fffffff;
        for (int t = warp; t < n_tiles; t += PREP_THREADS / 32) {
            bool any = false;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int pos = t * 128 + q * 32 + lane;
                any = any || (pos < Lb && mask[seq0 + pos] != 0);
            }
            any = __any_sync(0xffffffffu, any);
            if (lane == 0) tile_hot[(size_t)b * n_tiles + t] = any ? 1 : 0;
            if (any && t < first) first = t;
        }
        if (lane == 0 && first != 0x7fffffff) atomicMin(&first_s, first);
        const float g = gain[b];
        for (int h = tid; h < Hkv; h += PREP_THREADS) {
            const bool on = g != 0.f && (head_enable == nullptr || head_enable[h] != 0);
            const float amax = route.sigma != nullptr ? 1.f : alpha_max_of(alpha, (size_t)b * Hkv + h, M);
            bh_info[(size_t)b * Hkv + h] = (on ? 1 : 0) | ((on && lo_needed(g, amax)) ? 2 : 0);
        }
        __syncthreads();
        if (tid == 0) first_hot[b] = first_s;
        return;
    }
    if ((int)blockIdx.x < n_flag + n_a) {
        // ------------------------------------------------------------ routing coefficients for the caller
        const int bh = blockIdx.x - n_flag, b = bh / Hkv, h = bh % Hkv;
        const double* a = route_group(route.Q, route.q_is_f32, U, route.sigma, cu_seqlens, L, route.Hq, Hkv, D, r, M,
                                      route.k_route, b, h, reinterpret_cast<double*>(prep_sm));
        for (int m = tid; m < M; m += PREP_THREADS) route.alpha_out[(size_t)bh * M + m] = (float)a[m];
        return;
    }
    // ---------------------------------------------------------------- edited keys of one KV head, on tcgen05
    // The block keeps the edit operator of its head in shared memory as the B operand of a tensor-core product, as a
    // high and a low bf16 part (so that K W is fp32-accurate):  one expert: W = U U^T, and g_b alpha_{b,h} is applied to
    // the product per token;  several experts: W = g_b sum_m alpha_{b,h,m} U_m U_m^T, rebuilt when the sequence changes.
    // It walks a contiguous share of the head's (sequence, tile) pairs that hold a highlighted token: TMA stages the key
    // tile (two stages: the next tile lands while this one is worked on), one thread issues K W into tensor memory, the
    // eight warps add it to the highlighted rows (half a row per thread), split k' into its two bf16 parts (the high
    // parts in place in the staged tile, the low parts straight to global memory) and write the high parts of all
    // rows out, 16 bytes per lane with the lanes of a row adjacent.
    const int kb = blockIdx.x - n_flag - n_a;
    const int h = kb % Hkv, slot = kb / Hkv, n_slots = n_x / Hkv;
    if (head_enable != nullptr && head_enable[h] == 0) return;
    constexpr int NS = 1;                 // one key stage: two blocks share an SM instead of a block prefetching
    constexpr uint32_t TILE = (D / 64) * 128 * 128, PBLK = D * 128, PMAT = (D / 64) * PBLK;
    constexpr uint32_t TMEM_COLS = 2 * D;
    const int Rt = r * M;
    const bool routed = route.sigma != nullptr;
    const bool tc_build = D == 128 && M == 1 && r <= 64;      // U U^T on the tensor core (see build_W_tc)
    // dynamic shared memory (1024-byte aligned): key stages | W high, low | a chunk of U^T | routing scratch and coefficients
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(prep_sm) + 1023) & ~uintptr_t(1023));
    uint8_t* sW = smem + NS * TILE;
    float* ut = reinterpret_cast<float*>(sW + 2 * PMAT);        // staged chunk of U^T: [32][D + 4]
    unsigned char* tail = sW + 2 * PMAT + (tc_build ? 0 : 32 * (D + 4) * 4);       // (no chunk of U^T with the tensor-core build)
    float* alpha_s = reinterpret_cast<float*>(tail + (routed ? align_up_dev(route_smem_bytes(D, M, route.k_route), 16) : 0));
    __shared__ __align__(8) uint64_t bars[NS + 3];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_s;
    __shared__ unsigned char row_hl[NS][128];
    uint64_t* full = bars;            // [NS] key tile landed
    uint64_t* done = bars + NS;       // [2]  K W of a tile is in column set c
    uint64_t* built = bars + NS + 2;  // [1]  U U^T is in tensor memory
    volatile int* abort_flag = &abort_s;
    if (tid == 0) {
        for (int i = 0; i < NS; ++i) mbar_init(full + i, 1);
        mbar_init(done + 0, 1); mbar_init(done + 1, 1); mbar_init(built, 1);
        abort_s = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(&tmem_holder, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    constexpr uint32_t IDESC = umma_idesc_bf16(D, false);
    constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
    const uint32_t dKd = umma_desc_lo(smem_u32(smem), 16), dWd = umma_desc_lo(smem_u32(sW), 16);

    if (routed) {
        // Eq. 6 for every sequence (the whole block works on one at a time)
        for (int b = 0; b < B; ++b) {
            const double* a = route_group(route.Q, route.q_is_f32, U, route.sigma, cu_seqlens, L, route.Hq, Hkv, D, r, M,
                                          route.k_route, b, h, reinterpret_cast<double*>(tail));
            for (int m = tid; m < M; m += PREP_THREADS) alpha_s[b * M + m] = (float)a[m];
            __syncthreads();
        }
    }
    auto coef = [&](int b, int m) -> float {
        return routed ? alpha_s[b * M + m] : (alpha != nullptr ? alpha[((size_t)b * Hkv + h) * M + m] : 1.f);
    };
    // W (both parts) into shared memory in the operand layout: [D x 64] blocks of 128-byte rows, 128-byte swizzle.
    // U is staged 32 columns at a time, transposed (ut[kk][i] = U_m[i][kk0 + kk]: read coalesced, then every read
    // below is a row of ut); a thread forms PR rows x 16 columns of  W[n][k] = sum_j a_j U[n][j] U[k][j],  j = m r + kk,
    // its 16 columns being two groups of 8 (one 16-byte unit of the operand each), 64 apart.
    constexpr int UTP = D + 4;            // row pitch (floats) of ut: rows stay 16-byte aligned, transposed writes spread over banks
    auto build_W = [&](int b_for) {       // b_for < 0: plain U U^T (one expert)
        constexpr int PR = D * D / (PREP_THREADS * 16);
        constexpr int CG = D / 16;                       // column groups: thread g takes columns 8 g .. and D/2 + 8 g ..
        const int n0 = (tid / CG) * PR, kA = (tid % CG) * 8, kB = D / 2 + kA;
        float acc[PR][16];
#pragma unroll
        for (int p = 0; p < PR; ++p)
#pragma unroll
            for (int q = 0; q < 16; ++q) acc[p][q] = 0.f;
        const float gb = b_for >= 0 ? gain[b_for] : 1.f;
        for (int m = 0; m < M; ++m) {
            const float am = b_for >= 0 ? gb * coef(b_for, m) : 1.f;
            const float* Um = U + ((size_t)m * Hkv + h) * D * r;
            for (int kk0 = 0; kk0 < r; kk0 += 32) {
                const int kn = min(32, r - kk0);
                __syncthreads();
                {   // 32 D values, D / 8 per thread: all loads first, so that their latencies overlap
                    constexpr int NL = 32 * D / PREP_THREADS;
                    float v[NL];
                    const int kk = tid & 31;
#pragma unroll
                    for (int q = 0; q < NL; ++q) {
                        const int i = (tid >> 5) + q * (PREP_THREADS / 32);
                        v[q] = kk < kn ? __ldg(Um + (size_t)i * r + kk0 + kk) : 0.f;
                    }
#pragma unroll
                    for (int q = 0; q < NL; ++q) ut[kk * UTP + (tid >> 5) + q * (PREP_THREADS / 32)] = v[q];
                }
                __syncthreads();
#pragma unroll 2
                for (int kk = 0; kk < kn; ++kk) {
                    const float* row = ut + kk * UTP;
                    float un[PR], uk[16];
#pragma unroll
                    for (int p = 0; p < PR; ++p) un[p] = am * row[n0 + p];
#pragma unroll
                    for (int q4 = 0; q4 < 2; ++q4) {
                        const float4 a4 = *reinterpret_cast<const float4*>(row + kA + 4 * q4);
                        const float4 b4 = *reinterpret_cast<const float4*>(row + kB + 4 * q4);
                        uk[4 * q4] = a4.x; uk[4 * q4 + 1] = a4.y; uk[4 * q4 + 2] = a4.z; uk[4 * q4 + 3] = a4.w;
                        uk[8 + 4 * q4] = b4.x; uk[8 + 4 * q4 + 1] = b4.y; uk[8 + 4 * q4 + 2] = b4.z; uk[8 + 4 * q4 + 3] = b4.w;
                    }
#pragma unroll
                    for (int p = 0; p < PR; ++p)
#pragma unroll
                        for (int q = 0; q < 16; ++q) acc[p][q] = fmaf(un[p], uk[q], acc[p][q]);
                }
            }
        }
#pragma unroll
        for (int p = 0; p < PR; ++p) {
            uint32_t hi[8], lo[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) split_pair(acc[p][2 * q], acc[p][2 * q + 1], hi[q], lo[q]);
#pragma unroll
            for (int u8 = 0; u8 < 2; ++u8) {
                const int k0 = u8 ? kB : kA;
                uint8_t* dst = sW + (k0 >> 6) * PBLK + sw128_offset(n0 + p, k0 & 63);
                *reinterpret_cast<uint4*>(dst) = make_uint4(hi[4 * u8], hi[4 * u8 + 1], hi[4 * u8 + 2], hi[4 * u8 + 3]);
                *reinterpret_cast<uint4*>(dst + PMAT) = make_uint4(lo[4 * u8], lo[4 * u8 + 1], lo[4 * u8 + 2], lo[4 * u8 + 3]);
            }
        }
        fence_proxy_async();           // read next by the tensor core
    };

    // One expert, rank <= 64, head_dim 128: W = U U^T on the tensor core.  U (two bf16 parts) is written into the space
    // of W's low part (overwritten only after the product has finished) as two K-major operand tiles [128 x 64],
    // columns beyond the rank zero up to the next multiple of 16; hi.hi + hi.lo + lo.hi accumulate in tensor memory (column set 0); every thread then
    // reads half a row of the product, splits it and writes it where build_W would.
    uint32_t n_build = 0;
    auto build_W_tc = [&]() -> bool {
        const int r16 = (r + 15) / 16 * 16;
        uint8_t* t_hi = sW + PMAT;                  // [128 x 64] bf16, 128-byte swizzle: where the low part of W goes afterwards
        uint8_t* t_lo = sW + PMAT + 128 * 128;
        const float* Uh = U + (size_t)h * D * r;
        for (int e0 = 0; e0 < D * r16; e0 += PREP_THREADS * 8) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int e = e0 + q * PREP_THREADS + tid, i = e / r16, kk = e - i * r16;
                v[q] = (e < D * r16 && kk < r) ? __ldg(Uh + (size_t)i * r + kk) : 0.f;
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int e = e0 + q * PREP_THREADS + tid, i = e / r16, kk = e - i * r16;
                if (e < D * r16) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(v[q]);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(v[q] - __bfloat162float(hi));
                    const uint32_t off = sw128_offset(i, kk & ~7) + (kk & 7) * 2;
                    *reinterpret_cast<__nv_bfloat16*>(t_hi + off) = hi;
                    *reinterpret_cast<__nv_bfloat16*>(t_lo + off) = lo;
                }
            }
        }
        fence_proxy_async();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint32_t dhi = umma_desc_lo(smem_u32(t_hi), 16), dlo = umma_desc_lo(smem_u32(t_lo), 16);
            uint32_t acc = 0;
            for (int ks = 0; ks < r16 / 16; ++ks) {
                const uint32_t off = (uint32_t)(ks * 32) >> 4;
                umma_ss(tmem_base, dhi + off, DESC_HI, dhi + off, DESC_HI, IDESC, acc); acc = 1;
                umma_ss(tmem_base, dhi + off, DESC_HI, dlo + off, DESC_HI, IDESC, 1u);
                umma_ss(tmem_base, dlo + off, DESC_HI, dhi + off, DESC_HI, IDESC, 1u);
            }
            umma_commit(built);
        }
        bool good = mbar_wait(built, n_build & 1, abort_flag, status, 72);
        ++n_build;
        good = __syncthreads_and(good);
        if (!good) return false;
        tc_fence_after();
        const int row = tid & 127, half = tid >> 7;
#pragma unroll 1
        for (int cb = half * (D / 64); cb < (half + 1) * (D / 64); ++cb) {
            uint32_t v[32];
            tmem_ld32(t_lane + cb * 32, v);
            tmem_wait_ld_on(v);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2)
                    split_pair(__uint_as_float(v[q * 8 + 2 * e2]), __uint_as_float(v[q * 8 + 2 * e2 + 1]), hi[e2], lo[e2]);
                const int col = cb * 32 + q * 8;
                uint8_t* dst = sW + (col >> 6) * PBLK + sw128_offset(row, col & 63);
                *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(dst + PMAT) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
        tc_fence_before();
        fence_proxy_async();           // read next by the tensor core
        __syncthreads();
        return true;
    };

    // The (sequence, tile) pairs that hold a highlighted token, HOT_CAP candidates at a time: every block finds them for
    // itself (eight lanes per pair, 16 mask bytes each), so that the walk below only meets tiles with work.
    __shared__ int hot_list[HOT_CAP];
    __shared__ unsigned char hot_flag[HOT_CAP];
    __shared__ int warp_cnt[PREP_THREADS / 32];
    const int n_pairs = B * n_tiles;
    uint32_t n_load = 0, n_mma = 0;       // tiles loaded / multiplied so far (stage, column set and phases)
    int built_for = -2;                   // sequence W was built for (-1: plain U U^T, -2: nothing yet)
    bool ok = true;
    for (int p0 = 0; p0 < n_pairs && ok; p0 += HOT_CAP) {
        __syncthreads();
        const int p1 = min(n_pairs, p0 + HOT_CAP);
        for (int i = tid; i < HOT_CAP; i += PREP_THREADS) hot_flag[i] = 0;
        __syncthreads();
        for (int pp0 = p0; pp0 < p1; pp0 += PREP_THREADS / 8) {
            const int pp = pp0 + (tid >> 3), part = tid & 7;
            bool any = false;
            if (pp < p1) {
                const int b = pp / n_tiles, t = pp - b * n_tiles;
                const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
                const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
                const int pos0 = t * 128 + part * 16;
                if (gain[b] != 0.f && pos0 < Lb) {
                    const uint8_t* mp = mask + seq0 + pos0;
                    if (pos0 + 16 <= Lb && (reinterpret_cast<uintptr_t>(mp) & 15) == 0) {
                        const uint4 w = *reinterpret_cast<const uint4*>(mp);
                        any = (w.x | w.y | w.z | w.w) != 0;
                    } else {
                        for (int q = 0; q < 16; ++q) any = any || (pos0 + q < Lb && mp[q] != 0);
                    }
                }
            }
            any = __any_sync(0xffu << (lane & 24), any);
            if (part == 0 && pp < p1) hot_flag[pp - p0] = any ? 1 : 0;
        }
        __syncthreads();
        // the pairs in order (the same list in every block: the blocks of a head share it out by position)
        constexpr int PER = HOT_CAP / PREP_THREADS;
        int cnt = 0;
#pragma unroll
        for (int q = 0; q < PER; ++q) cnt += hot_flag[tid * PER + q];
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) warp_cnt[warp] = incl;
        __syncthreads();
        int base = incl - cnt, n_hot = 0;
#pragma unroll
        for (int w = 0; w < PREP_THREADS / 32; ++w) { if (w < warp) base += warp_cnt[w]; n_hot += warp_cnt[w]; }
#pragma unroll
        for (int q = 0; q < PER; ++q)
            if (hot_flag[tid * PER + q]) {
                const int pp = p0 + tid * PER + q, b = pp / n_tiles, t = pp - b * n_tiles;
                hot_list[base++] = b | (t << 16);
            }
        __syncthreads();

        // this block's contiguous share of the list
        const int i0 = (int)((long long)slot * n_hot / n_slots), i1 = (int)((long long)(slot + 1) * n_hot / n_slots);
        auto load_tile = [&](int i) {      // thread 0: key tile of list entry i into the next stage
            const int e = hot_list[i], b = e & 0xffff, t = e >> 16;
            const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
            const uint32_t st = n_load % NS;
            mbar_expect_tx(full + st, TILE);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) tma_load_3d(smem + st * TILE + c * (128 * 128), &tmK, full + st, c * 64, h, seq0 + t * 128);
        };
        for (int i = i0; i < i1 && ok; ++i) {
            const int e = hot_list[i], b = e & 0xffff, t = e >> 16;
            const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
            const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
            const float g = gain[b];
            const uint32_t st = n_mma % NS, cs = n_mma & 1;
            // the operator for this tile (the previous tile is through: every iteration ends with a barrier)
            const int want = M == 1 ? -1 : b;
            // the key tile starts to land (the stage is free: the previous tile is through)
            if (tid == 0) load_tile(i);
            ++n_load;
            if (built_for != want) {
                if (tc_build) { ok = build_W_tc(); if (!ok) break; } else build_W(want);
                built_for = want;
            }
            // the highlight flags of the tile's rows
            if (tid < 128) {
                const int kpos = t * 128 + tid;
                row_hl[st][tid] = (kpos < Lb && mask[seq0 + kpos] != 0) ? 1 : 0;
            }
            __syncthreads();               // W and the flags are in place
            ok = mbar_wait(full + st, ((n_mma / NS) & 1), abort_flag, status, 70);
            if (ok && tid == 0) {
                tc_fence_after();
                const uint32_t kd = dKd + st * (TILE >> 4);
#pragma unroll
                for (int part = 0; part < 2; ++part)
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t offk = ((uint32_t)(ks >> 2) * (128 * 128) + (uint32_t)(ks & 3) * 32) >> 4;
                        const uint32_t offw = ((uint32_t)part * PMAT + (uint32_t)(ks >> 2) * PBLK + (uint32_t)(ks & 3) * 32) >> 4;
                        umma_ss(tmem_base + cs * D, kd + offk, DESC_HI, dWd + offw, DESC_HI, IDESC, (ks > 0 || part) ? 1u : 0u);
                    }
                umma_commit(done + cs);
            }
            if (ok) ok = mbar_wait(done + cs, (n_mma >> 1) & 1, abort_flag, status, 71);
            ok = __syncthreads_and(ok);
            if (!ok) break;
            tc_fence_after();
            ++n_mma;
            // k' = k + c (K W)[row] for highlighted rows; high parts in place, low parts to global memory
            const float amax = routed ? 1.f : alpha_max_of(alpha, (size_t)b * Hkv + h, M);
            const bool with_lo = lo_needed(g, amax) || t < kLoTiles;     // what the fused kernel reads (see lo_needed)
            const float c = M == 1 ? g * coef(b, 0) : 1.f;
            const int row = tid & 127, half = tid >> 7;
            const bool hl = row_hl[st][row] != 0;
            const int kpos = t * 128 + row;
            const bool valid = kpos < Lb;
            uint8_t* sK = smem + st * TILE;
            __nv_bfloat16* xlo = X + ((size_t)(seq0 + (valid ? kpos : 0)) * Hkv + h) * (2 * D) + D;
            const bool warp_hl = __any_sync(0xffffffffu, hl);
#pragma unroll 1
            for (int cb = half * (D / 64); cb < (half + 1) * (D / 64); ++cb) {
                uint32_t v[32];
                if (warp_hl) { tmem_ld32(t_lane + cs * D + cb * 32, v); tmem_wait_ld_on(v); }      // warp-wide: every lane takes part
                uint4 lo4[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) lo4[q] = make_uint4(0u, 0u, 0u, 0u);
                if (hl) {
                    uint4* ptr[4];
                    uint4 kv[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {      // 8 elements = one 16-byte unit of the swizzled row; reads before writes
                        const int col = cb * 32 + q * 8;
                        ptr[q] = reinterpret_cast<uint4*>(sK + (col >> 6) * (128 * 128) + sw128_offset(row, col & 63));
                        kv[q] = *ptr[q];
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t* w = reinterpret_cast<uint32_t*>(&kv[q]);
                        uint32_t* l = reinterpret_cast<uint32_t*>(&lo4[q]);
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            const float2 k2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e2]));
                            split_pair(fmaf(c, __uint_as_float(v[q * 8 + 2 * e2]), k2.x), fmaf(c, __uint_as_float(v[q * 8 + 2 * e2 + 1]), k2.y), w[e2], l[e2]);
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) *ptr[q] = kv[q];
                }
                if (with_lo && valid) {
                    uint4* dst = reinterpret_cast<uint4*>(xlo + cb * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q) dst[q] = lo4[q];
                }
                __syncwarp();      // all lanes together again before the next warp-wide load
            }
            tc_fence_before();
            __syncthreads();
            // the high parts of all rows of the sequence go out: D / 8 lanes per row, 16 bytes each; 16 rows per warp
            constexpr int LPR = D / 8, RPI = 32 / LPR;
#pragma unroll 1
            for (int q = 0; q < 16 / RPI; ++q) {
                const int rr = warp * 16 + q * RPI + lane / LPR, col = (lane % LPR) * 8;
                if (t * 128 + rr < Lb) {
                    const uint4 val = *reinterpret_cast<const uint4*>(sK + (col >> 6) * (128 * 128) + sw128_offset(rr, col & 63));
                    *reinterpret_cast<uint4*>(X + ((size_t)(seq0 + t * 128 + rr) * Hkv + h) * (2 * D) + col) = val;
                }
            }
            __syncthreads();        // the stage, the flags and the columns are reused
        }
    }
    // a load that was armed may still be in flight after an abort: let it land before the shared memory is released
    if (!ok && tid == 0 && n_load > n_mma) {
        int dummy = 0;
        mbar_wait(full + n_mma % NS, (n_mma / NS) & 1, &dummy, nullptr, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// Operand preparation of the stand-alone edit, one launch:
//   blocks [0, n_p):   a 32 x 32 tile of the projector P[m][h] = U_m[h] U_m[h]^T (bf16 [D x D], as a high and a low
//                      part: [M, Hkv] matrices of high parts, then as many of low parts); gain and routing
//                      coefficients are applied per row when dK is added, so this does not depend on the batch;
//   blocks [n_p, ...): one warp per (sequence, 128-key tile): flag, and the tiles that hold a highlighted token
//                      appended to `hot_list` (any order).
// (for the fused forward) also the first highlighted tile of every sequence (atomic minimum: `first_hot` starts large)
// and the steering byte of every (sequence, KV head): bit 0 steered, bit 1 the fused kernel multiplies the low parts too
struct SteerInfoArgs {
    int* first_hot; uint8_t* bh_info; const float* gain; const float* alpha; const uint8_t* head_enable;
};

__global__ void prep_edit_kernel(const float* __restrict__ U, const uint8_t* __restrict__ mask,
                                 const int* __restrict__ cu_seqlens, __nv_bfloat16* __restrict__ P,
                                 uint8_t* __restrict__ tile_hot, int* __restrict__ hot_list, int* __restrict__ hot_count,
                                 int B, int L, int Hkv, int D, int r, int M, int n_tiles, int n_p, int n_flag,
                                 const SteerInfoArgs info, const RouteArgs route) {
    const int tid = threadIdx.x;
    if ((int)blockIdx.x >= n_p + n_flag) {
        // ------------------------------------------------------------ (routed call) Eq. 6 for one (sequence, KV head), with the
        // routine adaseka_route uses; the block also writes the steering byte of its pair, which needs the coefficients
        extern __shared__ double route_sm[];
        const int bh = (int)blockIdx.x - n_p - n_flag, b = bh / Hkv, h = bh % Hkv;
        const double* a = route_group(route.Q, route.q_is_f32, U, route.sigma, cu_seqlens, L, route.Hq, Hkv, D, r, M,
                                      route.k_route, b, h, route_sm);
        for (int m = tid; m < M; m += blockDim.x) route.alpha_out[(size_t)bh * M + m] = (float)a[m];
        if (tid == 0 && info.bh_info != nullptr) {
            const float g = info.gain[b];
            const bool on = g != 0.f && (info.head_enable == nullptr || info.head_enable[h] != 0);
            float amax = 0.f;
            for (int m = 0; m < M; ++m) amax = fmaxf(amax, fabsf((float)a[m]));
            info.bh_info[bh] = (on ? 1 : 0) | ((on && lo_needed(g, amax)) ? 2 : 0);
        }
        return;
    }
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
            if (any && info.first_hot != nullptr) atomicMin(info.first_hot + b, t);
        }
        if (info.bh_info != nullptr && t == 0 && route.sigma == nullptr) {
            const float g = info.gain[b];
            for (int h = lane; h < Hkv; h += 32) {
                const bool on = g != 0.f && (info.head_enable == nullptr || info.head_enable[h] != 0);
                const float amax = alpha_max_of(info.alpha, (size_t)b * Hkv + h, M);
                info.bh_info[(size_t)b * Hkv + h] = (on ? 1 : 0) | ((on && lo_needed(g, amax)) ? 2 : 0);
            }
        }
    }
}

// Item table of the fused kernel for packed variable-length batches: the items of decode_item whose tiles lie beyond
// their sequence are dropped, order kept.  One block per row slot (block 0: the last, heaviest row); where a block's
// items start follows from the sequence lengths alone, so the blocks do not talk to each other: a sequence of n_t row
// tiles has R = n_t (tiles A and B are two heads) or ceil(n_t / 2) (two row tiles) row slots, row slot `row` keeps the
// sequences with R > row, and the rows before it in the table hold hs * sum_b max(0, R_b - row - 1) items.
__global__ void __launch_bounds__(1024)
build_items_varlen_kernel(const Sched sc, const int* __restrict__ cu, const uint8_t* __restrict__ bh_info,
                          ItemRecord* __restrict__ items, int* __restrict__ count) {
    __shared__ long long red_s[32];
    __shared__ int pre_s[1024];
    __shared__ int warp_tot[32];
    __shared__ long long base_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
    const int row = sc.rs - 1 - (int)blockIdx.x;
    auto rows_of = [&](int b) -> int {
        const int n_t = (cu[b + 1] - cu[b] + 127) / 128;
        return sc.pair_heads ? n_t : (n_t + 1) / 2;
    };
    // items of the rows above this one (they come first), and, in block 0, of all rows
    long long before = 0, all = 0;
    for (int b = tid; b < sc.B; b += blockDim.x) {
        const int R = rows_of(b);
        before += R > row + 1 ? R - row - 1 : 0;
        all += R;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        all += __shfl_xor_sync(0xffffffffu, all, o);
    }
    if (lane == 0) red_s[wid] = before;
    __syncthreads();
    if (tid == 0) {
        long long t = 0;
        for (int q = 0; q < nw; ++q) t += red_s[q];
        base_s = t * sc.hs;
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        if (lane == 0) red_s[wid] = all;
        __syncthreads();
        if (tid == 0) {
            long long t = 0;
            for (int q = 0; q < nw; ++q) t += red_s[q];
            *count = (int)(t * sc.hs);
        }
    }
    // this row: the sequences that reach it, 1024 at a time, keep their order
    for (int b0 = 0; b0 < sc.B; b0 += blockDim.x) {
        const int b = b0 + tid;
        const bool keep = b < sc.B && rows_of(b) > row;
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_tot[wid] = __popc(bal);
        __syncthreads();
        int off = 0, tot = 0;
        for (int q = 0; q < nw; ++q) { if (q < wid) off += warp_tot[q]; tot += warp_tot[q]; }
        pre_s[tid] = keep ? off + __popc(bal & ((1u << lane) - 1)) : -1;
        const long long base = base_s;
        __syncthreads();
        const int n_b = sc.B - b0 < (int)blockDim.x ? sc.B - b0 : (int)blockDim.x;
        for (int c = tid; c < n_b * sc.hs; c += blockDim.x) {
            const int bi = c / sc.hs, slot = c - bi * sc.hs;
            const int pos = pre_s[bi];
            if (pos < 0) continue;
            ItemRecord r;
            decode_item(sc, (long long)blockIdx.x * sc.per + (long long)(b0 + bi) * sc.hs + slot, cu, r);
            r.steer = bh_info != nullptr ? (int)bh_info[(r.bh & 0xffff) * sc.Hkv + (r.bh >> 16)] : 0;
            items[base + (long long)pos * sc.hs + slot] = r;
        }
        __syncthreads();
        if (tid == 0) base_s = base + (long long)tot * sc.hs;
        __syncthreads();
    }
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

// fp32 -> bf16 copies of Q, K and V in one launch (groups of four values; the three tensors one after another)
struct ConvertArgs { const float4* in[3]; uint2* out[3]; size_t n4[3]; };
__global__ void convert_f32_bf16_kernel(const ConvertArgs a) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
    for (int t = 0; t < 3; ++t) {
        if (i < a.n4[t]) {
            const float4 v = a.in[t][i];
            a.out[t][i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
            return;
        }
        i -= a.n4[t];
    }
}

static size_t route_bytes_aligned(int D, int M, int k_route) { return align_up(route_smem_bytes(D, M, k_route), 16); }

// dynamic shared memory of prep_steering_kernel: the routing scratch (blocks that route), then the staged chunk of U
// in both layouts (blocks that form edited keys)
size_t prep_steering_smem(const seka_shape* sh, bool routed, int k_route) {
    const int D = sh->head_dim;
    const size_t tile = (size_t)(D / 64) * 128 * 128, pmat = (size_t)D * D * 2;
    const bool tc_build = D == 128 && sh->n_experts == 1 && sh->rank <= 64;      // as in the kernel: no staged chunk of U^T
    const size_t route = routed ? route_bytes_aligned(D, sh->n_experts, k_route) + (size_t)ALPHA_CAP * 4 : 0;
    return 1024 + tile + 2 * pmat + (tc_build ? 0 : (size_t)32 * (D + 4) * 4) + route;
}

seka_status launch_prep_steering(const seka_shape* sh, const SteerPlan& plan, const void* K16, const float* U,
                                 const float* alpha, const float* gain, const uint8_t* head_enable, const uint8_t* mask,
                                 void* X, uint8_t* tile_hot, int* first_hot, uint8_t* bh_info, int* status, int n_tiles,
                                 cudaStream_t st, const void* Q_route, const float* sigma, int k_route, float* alpha_out) {
    (void)plan;
    const int D = sh->head_dim, Hkv = sh->n_kv_heads;
    const bool routed = sigma != nullptr;
    if (routed && (long long)sh->batch * sh->n_experts > ALPHA_CAP) return SEKA_ERR_UNSUPPORTED;
    const int n_flag = sh->batch;
    const int n_a = (routed && alpha_out != nullptr) ? sh->batch * Hkv : 0;
    int n_sm = 0;
    if (!device_info(&n_sm)) return SEKA_ERR_CUDA;
    // blocks per KV head for the edited keys: one wave of the device (shared and tensor memory decide how many blocks
    // fit an SM), at most one per (sequence, tile)
    const size_t smem = prep_steering_smem(sh, routed, k_route);
    if (smem > 200 * 1024) return SEKA_ERR_UNSUPPORTED;
    // (about 10.5 KB of static shared memory per block on top; the register file holds two blocks)
    const int per_sm = (227 * 1024) / (smem + 11 * 1024) >= 2 ? 2 : 1;
    // (one wave: a block that had to wait for a free SM would finish a whole block-time later)
    long long per_head = ((long long)per_sm * n_sm - n_flag - n_a) / Hkv;
    const long long pairs = (long long)sh->batch * n_tiles;
    if (per_head > pairs) per_head = pairs;
    if (per_head < 1) per_head = 1;
    const long long n_x = per_head * Hkv;
    if (n_flag + n_a + n_x > 0x7fffffffLL) return SEKA_ERR_UNSUPPORTED;
    RouteArgs route{Q_route, sh->dtype == SEKA_F32 ? 1 : 0, sigma, k_route, sh->n_q_heads, alpha_out};
    CUtensorMap tk;
    if (!make_tile_map(&tk, K16, D, Hkv, shape_total_tokens(sh), 128)) return SEKA_ERR_CUDA;
    auto kern = D == 128 ? prep_steering_kernel<128> : prep_steering_kernel<64>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return SEKA_ERR_CUDA;
    kern<<<(unsigned)(n_flag + n_a + n_x), PREP_THREADS, smem, st>>>(
        tk, status, U, alpha, gain, head_enable, mask, sh->cu_seqlens,
        static_cast<__nv_bfloat16*>(X), tile_hot, first_hot, bh_info, sh->batch, sh->max_seqlen,
        Hkv, sh->rank, sh->n_experts, n_tiles, n_flag, n_a, (int)n_x, route);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

seka_status launch_prep_edit(const seka_shape* sh, const float* U, const uint8_t* mask, void* P, uint8_t* tile_hot, int n_tiles,
                             int* hot_list, int* hot_count, cudaStream_t st, int* first_hot, uint8_t* bh_info, const float* gain,
                             const float* alpha, const uint8_t* head_enable, const void* Q_route, const float* sigma,
                             int k_route, float* alpha_out) {
    const int D = sh->head_dim, tiles = D / 32;
    const int n_p = sh->n_experts * sh->n_kv_heads * tiles * tiles;
    const int n_flag = (sh->batch * n_tiles + 7) / 8;
    const int n_r = sigma != nullptr ? sh->batch * sh->n_kv_heads : 0;
    const size_t smem = sigma != nullptr ? route_smem_bytes(D, sh->n_experts, k_route) : 0;
    if (smem > 40 * 1024 &&      // beside 8 KB of static shared memory; very wide banks of rank-1 experts: up to 66 KB
        cudaFuncSetAttribute(prep_edit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SEKA_ERR_CUDA;
    cudaMemsetAsync(hot_count, 0, sizeof(int), st);
    if (first_hot != nullptr) cudaMemsetAsync(first_hot, 0x7f, sizeof(int) * sh->batch, st);      // a large value per sequence
    SteerInfoArgs info{first_hot, bh_info, gain, alpha, head_enable};
    RouteArgs route{Q_route, sh->dtype == SEKA_F32 ? 1 : 0, sigma, k_route, sh->n_q_heads, alpha_out};
    prep_edit_kernel<<<n_p + n_flag + n_r, 256, smem, st>>>(U, mask, sh->cu_seqlens, static_cast<__nv_bfloat16*>(P), tile_hot, hot_list,
                                                            hot_count, sh->batch, sh->max_seqlen, sh->n_kv_heads, D, sh->rank,
                                                            sh->n_experts, n_tiles, n_p, n_flag, info, route);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

void launch_build_items(const Sched& sc, const int* cu, const uint8_t* bh_info, ItemRecord* items, int* count,
                        cudaStream_t st) {
    if (sc.rs <= 0) return;
    build_items_varlen_kernel<<<(unsigned)sc.rs, 1024, 0, st>>>(sc, cu, bh_info, items, count);
    ++g_launches;
}

void launch_compact_mask(const uint8_t* mask, int T, int* list, int* count, cudaStream_t st) {
    cudaMemsetAsync(count, 0, sizeof(int), st);
    if (T == 0) return;
    compact_mask_kernel<<<(T + 255) / 256, 256, 0, st>>>(mask, T, list, count);
    ++g_launches;
}

void launch_convert_bf16(const float* Q, void* q16, size_t nq, const float* K, void* k16, const float* V, void* v16, size_t nk,
                         cudaStream_t st) {
    ConvertArgs a;      // head_dim is a multiple of 4, so the element counts are too
    a.in[0] = reinterpret_cast<const float4*>(Q); a.out[0] = reinterpret_cast<uint2*>(q16); a.n4[0] = nq / 4;
    a.in[1] = reinterpret_cast<const float4*>(K); a.out[1] = reinterpret_cast<uint2*>(k16); a.n4[1] = nk / 4;
    a.in[2] = reinterpret_cast<const float4*>(V); a.out[2] = reinterpret_cast<uint2*>(v16); a.n4[2] = nk / 4;
    const size_t n4 = a.n4[0] + a.n4[1] + a.n4[2];
    if (n4 == 0) return;
    convert_f32_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(a);
    ++g_launches;
}

}  // namespace seka
