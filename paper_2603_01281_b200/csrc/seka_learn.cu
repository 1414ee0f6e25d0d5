// Offline spectral learning of the projections (Section 3.1, Eq. 2-3, first loop of Algorithm 1) and the
// head-selection distance of Section 3.4, for all (layer, KV head) slots of a model in one call.
//
//   learn_cov_kernel      Omega+ = h^T h+ / n and Omega- = h^T h- / n.  The contraction runs over tokens, so the
//                         key embeddings are read exactly once (three bf16 tensors [n, slots, d]); at 2 d / 3 FLOP
//                         per byte the pass is bound by HBM bandwidth but needs the tensor cores to keep up.
//                         Persistent CTAs, an item = (group of 128 columns, chunk of tokens): a producer warp
//                         streams 128-token tiles of h, h+, h- with TMA through two stages; one thread issues
//                         tcgen05 products with BOTH operands MN-major (the token axis is the contraction) into two
//                         128 x 128 accumulators in tensor memory; four warps drain the finished accumulators of
//                         item i while item i + 1 accumulates in the other half of tensor memory.
//   learn_reduce_kernel   sums the per-chunk partials in chunk order, scales by 1 / n.
//   learn_dist_kernel     D = mean over the answer tokens of ||h+ - h-||_2, per slot (fixed summation order).
//   learn_svd_kernel      one CTA per matrix: one-sided Jacobi (Hestenes) in fp64 on the columns of Omega held in
//                         shared memory; every pair of columns meets once per sweep (ordering by recursive halving,
//                         four lanes per pair, one column of each pair resident in registers); on convergence the
//                         column norms are the singular values and the normalised columns the left singular
//                         vectors; sorted descending; the rank of Eq. 3 from the sorted values.
#include <math.h>

#include "seka_kernels.h"

namespace seka {
namespace {

// ------------------------------------------------------------------------------------ cross-covariances
constexpr int LC_THREADS = 192;                 // warp 0 producer, warp 1 MMA issuer, warps 2..5 drain
constexpr int LC_TOK = 128;                     // tokens per stage
constexpr int LC_NS = 2;
constexpr uint32_t LC_BLK = 128 * 128;          // [128 tokens x 64 columns] block, 128-byte swizzle
constexpr uint32_t LC_TILE = 2 * LC_BLK;        // 128 columns of one tensor
constexpr uint32_t LC_STAGE = 3 * LC_TILE;      // h, h+, h-
constexpr uint32_t LC_BARS = LC_NS * LC_STAGE;  // full[2], empty[2], acc_full[2], acc_free[2]
constexpr uint32_t LC_MISC = LC_BARS + 8 * 8;
constexpr uint32_t LC_DYN_BYTES = LC_MISC + 16 + 1024;
constexpr uint32_t LC_TMEM_COLS = 512;          // two sets of (Omega+, Omega-) accumulators

struct LearnCovParams {
    float* part;            // [n_chunks][slots][2][d][d]
    int n_tokens, n_groups, d, slots, chunk_tokens, n_chunks;
    int* status;
};

__device__ __forceinline__ bool lc_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int where) {
    const bool ok = mbar_wait(bar, parity, abort_flag, status, where);
    return __all_sync(0xffffffffu, ok);
}

// bf16 x bf16 -> fp32, M = N = 128, A and B both MN-major (their contraction axis, the tokens, is the slow one)
constexpr uint32_t LC_IDESC = umma_idesc_bf16(128, true) | (1u << 15);

__global__ void __launch_bounds__(LC_THREADS, 1)
learn_cov_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmP,
                 const __grid_constant__ CUtensorMap tmN, const LearnCovParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + LC_BARS);
    uint64_t* full = bars;              // [2] the three tiles of a stage have landed
    uint64_t* empty = bars + 2;         // [2] the products that read the stage have finished
    uint64_t* acc_full = bars + 4;      // [2] every product of an item has finished: its accumulators can be read
    uint64_t* acc_free = bars + 6;      // [2] four drain-warp arrivals: the accumulators have been read
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + LC_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + LC_MISC + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(p.status) != 0)) return;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 1); mbar_init(acc_full + i, 1); mbar_init(acc_free + i, 4); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmH); tma_prefetch_desc(&tmP); tma_prefetch_desc(&tmN);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, LC_TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int n_items = p.n_groups * p.n_chunks;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        uint32_t n_push = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int g = item % p.n_groups, c = item / p.n_groups;
            const int t0 = c * p.chunk_tokens, t1 = min(p.n_tokens, t0 + p.chunk_tokens);
            const int n_tiles = (t1 - t0 + LC_TOK - 1) / LC_TOK;
            for (int t = 0; t < n_tiles; ++t) {
                const uint32_t s = n_push % LC_NS;
                if (n_push >= LC_NS) {
                    ok = lc_wait(empty + s, ((n_push / LC_NS) - 1) & 1, abort_flag, p.status, 70);
                    if (!ok) break;
                }
                if (lane == 0) {
                    uint8_t* st = smem + s * LC_STAGE;
                    mbar_expect_tx(full + s, LC_STAGE);
                    const int row = t0 + t * LC_TOK;            // rows beyond the last token are filled with zeros
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
                        tma_load_3d(st + blk * LC_BLK, &tmH, full + s, blk * 64, g, row);
                        tma_load_3d(st + LC_TILE + blk * LC_BLK, &tmP, full + s, blk * 64, g, row);
                        tma_load_3d(st + 2 * LC_TILE + blk * LC_BLK, &tmN, full + s, blk * 64, g, row);
                    }
                }
                __syncwarp();
                ++n_push;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
        const uint32_t d0 = umma_desc_lo(smem_u32(smem), LC_BLK);
        uint32_t n_pop = 0, it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int c = item / p.n_groups;
            const int t0 = c * p.chunk_tokens, t1 = min(p.n_tokens, t0 + p.chunk_tokens);
            const int n_tiles = (t1 - t0 + LC_TOK - 1) / LC_TOK;
            const uint32_t set = it & 1;
            if (it >= 2) {
                ok = lc_wait(acc_free + set, ((it >> 1) - 1) & 1, abort_flag, p.status, 71);
                if (!ok) break;
            }
            for (int t = 0; t < n_tiles; ++t) {
                const uint32_t s = n_pop % LC_NS;
                ok = lc_wait(full + s, (n_pop / LC_NS) & 1, abort_flag, p.status, 72);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t dh = d0 + s * (LC_STAGE >> 4), dp = dh + (LC_TILE >> 4), dn = dp + (LC_TILE >> 4);
                    const uint32_t acc = tmem_base + set * 256;
#pragma unroll
                    for (int ks = 0; ks < LC_TOK / 16; ++ks) {        // 16 tokens per product: 16 rows x 128 B further on
                        const uint32_t off = (uint32_t)ks * (2048 >> 4);
                        const uint32_t accumulate = (t > 0 || ks > 0) ? 1u : 0u;
                        umma_ss(acc, dh + off, DESC_HI, dp + off, DESC_HI, LC_IDESC, accumulate);
                        umma_ss(acc + 128, dh + off, DESC_HI, dn + off, DESC_HI, LC_IDESC, accumulate);
                    }
                    umma_commit(empty + s);
                    if (t == n_tiles - 1) umma_commit(acc_full + set);
                }
                __syncwarp();
                ++n_pop;
            }
        }
    } else {
        // ------------------------------------------------------------ drain: accumulators -> per-chunk partials
        const int q = warp & 3;                                        // the quarter of tensor-memory lanes this warp may read
        const int row = q * 32 + lane;
        uint32_t it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int g = item % p.n_groups, c = item / p.n_groups;
            const uint32_t set = it & 1;
            ok = lc_wait(acc_full + set, (it >> 1) & 1, abort_flag, p.status, 73);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + set * 256;
#pragma unroll 1
            for (int sign = 0; sign < 2; ++sign) {
#pragma unroll 1
                for (int c4 = 0; c4 < 4; ++c4) {
                    float* dst;
                    if (p.d == 128) {
                        dst = p.part + ((((size_t)c * p.slots + g) * 2 + sign) * 128 + row) * 128 + c4 * 32;
                    } else {
                        // two heads of 64 columns share the product: only the diagonal blocks are cross-covariances
                        const int hd = q >> 1;
                        if ((c4 >> 1) != hd) continue;                 // the same for the whole warp
                        dst = p.part + ((((size_t)c * p.slots + 2 * g + hd) * 2 + sign) * 64 + (row & 63)) * 64 + (c4 & 1) * 32;
                    }
                    uint32_t v[32];
                    tmem_ld32(t_lane + sign * 128 + c4 * 32, v);
                    tmem_wait_ld_on(v);
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        reinterpret_cast<float4*>(dst)[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                                                        __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free + set);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, LC_TMEM_COLS);
    }
}

// omega[sign][slot][i][j] = sum over chunks (in order) of the partials, divided by the number of tokens
__global__ void learn_reduce_kernel(const float* __restrict__ part, float* __restrict__ omega_pos,
                                    float* __restrict__ omega_neg, int slots, int d, int n_chunks, float inv_n) {
    const size_t per = (size_t)d * d, total = (size_t)slots * 2 * per;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    float acc = 0.f;
    for (int c = 0; c < n_chunks; ++c) acc += part[(size_t)c * total + idx];
    const size_t slot = idx / (2 * per), rest = idx % (2 * per);
    float* out = rest < per ? omega_pos : omega_neg;
    out[slot * per + rest % per] = acc * inv_n;
}

// ------------------------------------------------------------------------------------ head-selection distance
// Block b takes a range of tokens; every slot has one owner (a fixed group of lanes of one warp), which keeps the
// slot's running sum in shared memory: one writer per slot, fixed order.
constexpr int LD_THREADS = 256;
__global__ void learn_dist_kernel(const __nv_bfloat16* __restrict__ hp, const __nv_bfloat16* __restrict__ hn,
                                  const uint8_t* __restrict__ answer, int n, int slots, int d, int tokens_per_block,
                                  float* __restrict__ part_sum, int* __restrict__ part_count) {
    extern __shared__ float acc[];                  // [slots]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int s = threadIdx.x; s < slots; s += LD_THREADS) acc[s] = 0.f;
    __syncthreads();
    const int t0 = blockIdx.x * tokens_per_block, t1 = min(n, t0 + tokens_per_block);
    int count = 0;
    for (int t = t0; t < t1; ++t) {
        if (answer != nullptr && answer[t] == 0) continue;
        ++count;
        // A row (one token of one slot) is d / 8 lanes of 16 bytes, so one warp load covers 2 (d = 128) or 4 (d = 64)
        // neighbouring slots: 512 contiguous bytes.  Four such loads per tensor are in flight before the sums.
        const int lpr = d / 8, rpw = 32 / lpr;              // lanes per row, rows per warp load
        const int sub = lane / lpr;
        const int n_q = (slots + rpw - 1) / rpw;
        for (int q0 = warp; q0 < n_q; q0 += 4 * (LD_THREADS / 32)) {
            float ss[4];
            uint4 a4[4], b4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int sl = (q0 + u * (LD_THREADS / 32)) * rpw + sub;
                a4[u] = make_uint4(0u, 0u, 0u, 0u); b4[u] = a4[u];
                if (q0 + u * (LD_THREADS / 32) < n_q && sl < slots) {
                    const size_t off = ((size_t)t * slots + sl) * d + (size_t)(lane % lpr) * 8;
                    a4[u] = *reinterpret_cast<const uint4*>(hp + off);
                    b4[u] = *reinterpret_cast<const uint4*>(hn + off);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t* aw = reinterpret_cast<const uint32_t*>(&a4[u]);
                const uint32_t* bw = reinterpret_cast<const uint32_t*>(&b4[u]);
                float acc2 = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[e]));
                    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[e]));
                    const float dx = a.x - b.x, dy = a.y - b.y;
                    acc2 = fmaf(dx, dx, fmaf(dy, dy, acc2));
                }
                ss[u] = acc2;
            }
            for (int o = lpr / 2; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < 4; ++u) ss[u] += __shfl_xor_sync(0xffffffffu, ss[u], o);
            }
            if (lane % lpr == 0) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int sl = (q0 + u * (LD_THREADS / 32)) * rpw + sub;
                    if (q0 + u * (LD_THREADS / 32) < n_q && sl < slots) acc[sl] += sqrtf(ss[u]);
                }
            }
        }
    }
    __syncthreads();
    for (int s = threadIdx.x; s < slots; s += LD_THREADS) part_sum[(size_t)blockIdx.x * slots + s] = acc[s];
    if (threadIdx.x == 0) part_count[blockIdx.x] = count;
}

// One CTA per slot: thread i adds the partials of blocks i, i + 256, ... in order, then thread 0 adds the 256 sums in order.
__global__ void learn_dist_reduce_kernel(const float* __restrict__ part_sum, const int* __restrict__ part_count,
                                         int n_blocks, int slots, float* __restrict__ D) {
    __shared__ double tot[256];
    __shared__ long long cnt[256];
    const int s = blockIdx.x, i = threadIdx.x;
    double t = 0.0;
    long long c = 0;
    for (int b = i; b < n_blocks; b += 256) { t += (double)part_sum[(size_t)b * slots + s]; c += part_count[b]; }
    tot[i] = t; cnt[i] = c;
    __syncthreads();
    if (i == 0) {
        double tt = 0.0;
        long long cc = 0;
        for (int k = 0; k < 256; ++k) { tt += tot[k]; cc += cnt[k]; }
        D[s] = cc > 0 ? (float)(tt / (double)cc) : 0.f;
    }
}

// ------------------------------------------------------------------------------------ SVD (one-sided Jacobi, fp64)
constexpr int SV_LP = 4;                        // lanes that share a column pair: eight pairs per warp
constexpr int SV_PAD = 4;                       // doubles of padding per column (32 bytes: the eight 32-byte pieces a warp
                                                // touches in neighbouring columns fall on different banks)
constexpr int SV_THREADS = 64 * SV_LP;          // 64 pairs per round at head_dim 128
constexpr int SV_MAX_SWEEPS = 60;

// One CTA per (sign, slot).  G (column-major, fp64, shared memory) starts as Omega; plane rotations from the right
// make its columns mutually orthogonal: Omega V = U S.  Outputs: U [d x d] row-major with the singular vectors as
// columns, S descending, and the smallest k with sum_{i<=k} S_i >= gamma * sum_i S_i (Eq. 3).
__global__ void __launch_bounds__(SV_THREADS, 1)
learn_svd_kernel(const float* __restrict__ omega_pos, const float* __restrict__ omega_neg, int slots, int d, float gamma,
                 float* __restrict__ U_pos, float* __restrict__ U_neg, float* __restrict__ S_pos, float* __restrict__ S_neg,
                 int* __restrict__ k_pos, int* __restrict__ k_neg, int* __restrict__ sweeps_out) {
    extern __shared__ double sv_sm[];
    const int ldg = d + SV_PAD;             // column stride: the pad staggers neighbouring columns over the banks
    double* G = sv_sm;                      // [d][ldg], column j at G + j * ldg
    double* sig = G + (size_t)d * ldg;      // [d]
    int* order = reinterpret_cast<int*>(sig + d);   // [d]: position of column j in the sorted output
    __shared__ int rotated;
    __shared__ double pr[64], scl[128], iscl[128], scale;
    __shared__ float nrm2[128];
    const int sign = blockIdx.x / slots, slot = blockIdx.x % slots;
    const float* om = (sign == 0 ? omega_pos : omega_neg) + (size_t)slot * d * d;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = SV_THREADS / 32;
    for (int idx = tid; idx < d * d; idx += SV_THREADS) {
        const int i = idx / d, j = idx - i * d;     // Omega[i][j], coalesced read
        G[(size_t)j * ldg + i] = (double)om[idx];
    }
    __syncthreads();
    // scale the matrix to unit largest entry (squares of column norms stay far from under- and overflow)
    {
        double mx = 0.0;
        for (int idx = tid; idx < d * d; idx += SV_THREADS) mx = fmax(mx, fabs(G[(size_t)(idx / d) * ldg + idx % d]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) pr[warp] = mx;
        __syncthreads();
        if (tid == 0) {
            double m2 = 0.0;
            for (int w = 0; w < n_warps; ++w) m2 = fmax(m2, pr[w]);
            scale = m2;
        }
        __syncthreads();
        const double inv = scale > 0.0 ? 1.0 / scale : 0.0;
        for (int idx = tid; idx < d * d; idx += SV_THREADS) G[(size_t)(idx / d) * ldg + idx % d] *= inv;
        __syncthreads();
    }
    constexpr int RPL = 128 / SV_LP;                // rows per lane at d = 128 (d = 64 uses the first half)
    const int per_lane = d / SV_LP;
    const int n_pairs = d / 2;
    // Scaled (fast) rotations: column j of the matrix is scl[j] * g_j with g_j the stored column.  A rotation
    //   A' = c (A - t B),  B' = c (B + t A)   becomes   g_a' = g_a - (t s_b / s_a) g_b,  g_b' = g_b + (t s_a / s_b) g_a
    // (two multiply-adds per row instead of four operations) with s_a' = c s_a, s_b' = c s_b; the reciprocals are
    // tracked too (1 / c = (1 + t^2) c), so no division is needed for the ratios.  The scales are folded back into
    // the columns at the start of every sweep (c >= 1 / sqrt 2 per rotation, 127 rotations per sweep at most).
    //
    // Ordering of a sweep (every pair of columns meets once, d - 1 rounds of d / 2 disjoint pairs): level l cuts
    // the columns into blocks of 2 m, m = d / 2, d / 4, ..., 1; in round r of the level the i-th column of the first
    // half of a block meets the ((i + r) mod m)-th column of its second half.  A group of SV_LP lanes owns one
    // first-half column for the whole level and keeps it in registers; only the second-half columns go through
    // shared memory (read, rotated, written back in place), and there is one barrier per round, since every group
    // works out its own rotation.
    //
    // What bounds the kernel is the fp64 pipe (one warp instruction every 8-11 cycles per scheduler on this part),
    // so the aim is few fp64 warp instructions per round: several pairs share a warp (the scalar work of a rotation
    // is then issued once for all of them), the tangent and the squared norms are fp32, only what decides the
    // orthogonality of the result stays fp64.
    for (int j = tid; j < d; j += SV_THREADS) { scl[j] = 1.0; iscl[j] = 1.0; }
    const int grp = lane / SV_LP, lg = lane % SV_LP;
    const int hw = (32 / SV_LP) * warp + grp;       // pair slot of a round
    const bool active = hw < n_pairs;
    int sweep = 0;
    for (; sweep < SV_MAX_SWEEPS; ++sweep) {
        if (tid == 0) rotated = 0;
        __syncthreads();
        // fold the scales, and the squared column norms, exact at the start of every sweep; inside the sweep they
        // follow the rotations (A' . A' = A . A - t A . B,  B' . B' = B . B + t A . B) in fp32: they only feed the
        // tangent.  A pair then costs one inner product.
        for (int j = warp; j < d; j += n_warps) {
            const double sj = scl[j];
            double ss = 0.0;
            for (int i = lane; i < d; i += 32) {
                const double v = G[(size_t)j * ldg + i] * sj;
                G[(size_t)j * ldg + i] = v;
                ss = fma(v, v, ss);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            __syncwarp();
            if (lane == 0) { nrm2[j] = (float)ss; scl[j] = 1.0; iscl[j] = 1.0; }
        }
        __syncthreads();
        for (int m = n_pairs; m >= 1; m >>= 1) {
            // the resident column of this group for the level, with its scale, reciprocal scale and squared norm
            const int blk = hw / m, idx = hw - blk * m;
            const int ca = blk * 2 * m + idx;
            double x[RPL];
            double sa = 1.0, isa = 1.0;
            float aa = 0.f, saf = 1.f;
            if (active) {
                const double* ga = G + (size_t)ca * ldg;
#pragma unroll
                for (int e = 0; e < RPL; ++e)
                    if (e < per_lane) x[e] = ga[lg + SV_LP * e];
                sa = scl[ca]; isa = iscl[ca]; aa = nrm2[ca]; saf = (float)sa;
            }
            for (int r = 0; r < m; ++r) {
                if (active) {
                    int ib = idx + r;
                    if (ib >= m) ib -= m;
                    const int cb = blk * 2 * m + m + ib;
                    double* gb = G + (size_t)cb * ldg;
                    double y[RPL];
                    double dsum[4] = {0.0, 0.0, 0.0, 0.0};      // four chains: dependent fp64 operations are slow
#pragma unroll
                    for (int e = 0; e < RPL; ++e) {
                        if (e < per_lane) {
                            y[e] = gb[lg + SV_LP * e];
                            dsum[e & 3] = fma(x[e], y[e], dsum[e & 3]);
                        }
                    }
                    double dot = (dsum[0] + dsum[1]) + (dsum[2] + dsum[3]);
#pragma unroll
                    for (int o = SV_LP / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);   // within the group
                    // every lane of the group holds the same sums and works out the same rotation
                    const double sb = scl[cb], isb = iscl[cb];
                    const float bb = nrm2[cb];
                    // The tangent of the rotation angle needs no more than single precision: an error eps in t leaves
                    // eps times the old inner product behind, which the next sweep removes; the rotation itself stays
                    // exact because the same t goes into both columns and into the scales.
                    const float ab = saf * (float)sb * (float)dot;
                    float tf = 0.f;
                    // |cos| > 1e-13 (well above the rounding noise of the inner product), as a product of ratios so
                    // that columns of very different size neither overflow nor underflow the test
                    if (aa > 0.f && bb > 0.f && (ab / aa) * (ab / bb) > 1e-26f) {
                        const float df = bb - aa, t2ab = 2.f * ab;
                        const float mf = fmaxf(fabsf(df), fabsf(t2ab));
                        const float dn = df / mf, tn = t2ab / mf;
                        tf = (dn >= 0.f ? tn : -tn) / (fabsf(dn) + sqrtf(fmaf(dn, dn, tn * tn)));
                    }
                    if (tf != 0.f) {                    // the same decision on all lanes of the group
                        // the cosine: one Newton step in fp64 from an fp32 seed
                        const double t = (double)tf;
                        const double t2 = fma(t, t, 1.0);
                        const double c0 = (double)rsqrtf(fmaf(tf, tf, 1.f));
                        const double cs = c0 * fma(-0.5 * t2, c0 * c0, 1.5), ics = t2 * cs;
                        const double ta = t * sb * isa, tb = t * sa * isb;
#pragma unroll
                        for (int e = 0; e < RPL; ++e) {
                            if (e < per_lane) {
                                const double xo = x[e];
                                x[e] = fma(-ta, y[e], xo);
                                gb[lg + SV_LP * e] = fma(tb, xo, y[e]);
                            }
                        }
                        if (lg == 0) {
                            scl[cb] = cs * sb; iscl[cb] = isb * ics; nrm2[cb] = bb + tf * ab;
                            rotated = 1;
                        }
                        sa *= cs; isa *= ics; saf = (float)sa; aa = fmaxf(aa - tf * ab, 0.f);
                    }
                }
                __syncthreads();                        // the second-half columns change hands
            }
            // the level ends: the resident columns go back
            if (active) {
                double* ga = G + (size_t)ca * ldg;
#pragma unroll
                for (int e = 0; e < RPL; ++e)
                    if (e < per_lane) ga[lg + SV_LP * e] = x[e];
                if (lg == 0) { scl[ca] = sa; iscl[ca] = isa; nrm2[ca] = aa; }
            }
            __syncthreads();
        }
        if (rotated == 0) break;                    // a whole sweep without a rotation: the columns are orthogonal
        __syncthreads();
    }
    // fold the scales of the last sweep
    for (int j = warp; j < d; j += n_warps) {
        const double sj = scl[j];
        for (int i = lane; i < d; i += 32) G[(size_t)j * ldg + i] *= sj;
    }
    __syncthreads();
    // singular values = column norms
    for (int j = warp; j < d; j += n_warps) {
        double ss = 0.0;
        for (int i = lane; i < d; i += 32) ss = fma(G[(size_t)j * ldg + i], G[(size_t)j * ldg + i], ss);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) sig[j] = sqrt(ss);           // of the scaled matrix; the scale goes back on at the output
    }
    __syncthreads();
    // descending order (ties: the earlier column first)
    for (int j = tid; j < d; j += SV_THREADS) {
        int r = 0;
        for (int i = 0; i < d; ++i) r += (sig[i] > sig[j] || (sig[i] == sig[j] && i < j)) ? 1 : 0;
        order[j] = r;
    }
    __syncthreads();
    float* Uo = (sign == 0 ? U_pos : U_neg) + (size_t)slot * d * d;
    float* So = (sign == 0 ? S_pos : S_neg) + (size_t)slot * d;
    for (int idx = tid; idx < d * d; idx += SV_THREADS) {
        const int i = idx / d, j = idx - i * d;     // component i of column j
        const double s = sig[j];
        Uo[(size_t)i * d + order[j]] = s > 0.0 ? (float)(G[(size_t)j * ldg + i] / s) : 0.f;
    }
    for (int j = tid; j < d; j += SV_THREADS) So[order[j]] = (float)(sig[j] * scale);
    __syncthreads();
    if (tid == 0) {
        // Eq. 3 on the sorted values, in fp64
        double* sorted = G;                         // the matrix has been written out: reuse its first d entries
        for (int j = 0; j < d; ++j) sorted[order[j]] = sig[j];
        double total = 0.0;
        for (int j = 0; j < d; ++j) total += sorted[j];
        double run = 0.0;
        int k = d;
        for (int j = 0; j < d; ++j) {
            run += sorted[j];
            if (run >= (double)gamma * total) { k = j + 1; break; }
        }
        (sign == 0 ? k_pos : k_neg)[slot] = k;
        if (sweeps_out != nullptr) sweeps_out[blockIdx.x] = sweep;
    }
}

struct LearnPlan {
    int n_groups, chunk_tokens, n_chunks, dist_tokens, dist_blocks;
    size_t part_off, part_bytes, dsum_off, dsum_bytes, dcnt_off, dcnt_bytes, sweeps_off, sweeps_bytes, total;
};

seka_status validate_learn(const seka_learn_shape* s) {
    if (s == nullptr) return SEKA_ERR_INVALID_ARG;
    if (s->n_tokens <= 0 || s->n_slots <= 0) return SEKA_ERR_INVALID_ARG;
    if (!(s->gamma > 0.f) || !(s->gamma <= 1.f)) return SEKA_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128) return SEKA_ERR_UNSUPPORTED;
    if (s->head_dim == 64 && (s->n_slots & 1)) return SEKA_ERR_UNSUPPORTED;       // heads of 64 are processed in pairs
    if ((long long)s->n_tokens * s->n_slots > 0x7fffffffLL) return SEKA_ERR_UNSUPPORTED;
    return SEKA_OK;
}

// Chunks of tokens: a few items per SM so that the accumulator drain of one item hides under the next, but long
// enough (>= 2048 tokens) that the partials stay small next to the embeddings.
LearnPlan learn_plan(const seka_learn_shape* s) {
    LearnPlan pl;
    const int d = s->head_dim;
    pl.n_groups = d == 128 ? s->n_slots : s->n_slots / 2;
    long long want = (4LL * 148 + pl.n_groups - 1) / pl.n_groups;          // chunks that give about 4 items per SM
    if (want < 1) want = 1;
    long long chunk = (s->n_tokens + want - 1) / want;
    if (chunk < 2048) chunk = 2048;
    chunk = (chunk + LC_TOK - 1) / LC_TOK * LC_TOK;
    pl.chunk_tokens = (int)chunk;
    pl.n_chunks = (int)((s->n_tokens + chunk - 1) / chunk);
    pl.dist_tokens = 8;
    pl.dist_blocks = (s->n_tokens + pl.dist_tokens - 1) / pl.dist_tokens;
    if (pl.dist_blocks > 8192) { pl.dist_tokens = (s->n_tokens + 8191) / 8192; pl.dist_blocks = (s->n_tokens + pl.dist_tokens - 1) / pl.dist_tokens; }
    pl.part_off = kStatusBytes;
    pl.part_bytes = align_up((size_t)pl.n_chunks * s->n_slots * 2 * d * d * sizeof(float), 256);
    pl.dsum_off = pl.part_off + pl.part_bytes;
    pl.dsum_bytes = align_up((size_t)pl.dist_blocks * s->n_slots * sizeof(float), 256);
    pl.dcnt_off = pl.dsum_off + pl.dsum_bytes;
    pl.dcnt_bytes = align_up((size_t)pl.dist_blocks * sizeof(int), 256);
    pl.sweeps_off = pl.dcnt_off + pl.dcnt_bytes;
    pl.sweeps_bytes = align_up((size_t)2 * s->n_slots * sizeof(int), 256);
    pl.total = pl.sweeps_off + pl.sweeps_bytes;
    return pl;
}

}  // namespace
}  // namespace seka

extern "C" size_t seka_learn_workspace_bytes(const seka_learn_shape* shape) {
    if (seka::validate_learn(shape) != SEKA_OK) return 0;
    return seka::learn_plan(shape).total;
}

extern "C" seka_status seka_learn_projections(const seka_learn_shape* shape, const void* h, const void* h_pos,
                                              const void* h_neg, const uint8_t* answer_tokens,
                                              float* omega_pos, float* omega_neg, float* U_pos, float* U_neg,
                                              float* S_pos, float* S_neg, int32_t* k_pos, int32_t* k_neg, float* D,
                                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
    using namespace seka;
    seka_status stc = validate_learn(shape);
    if (stc != SEKA_OK) return stc;
    if (!h || !h_pos || !h_neg || !omega_pos || !omega_neg || !U_pos || !U_neg || !S_pos || !S_neg || !k_pos || !k_neg || !D)
        return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)h | (uintptr_t)h_pos | (uintptr_t)h_neg | (uintptr_t)omega_pos | (uintptr_t)omega_neg) & 15) return SEKA_ERR_INVALID_ARG;
    const LearnPlan pl = learn_plan(shape);
    if (!workspace || workspace_bytes < pl.total || ((uintptr_t)workspace & 255)) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    const int d = shape->head_dim, slots = shape->n_slots, n = shape->n_tokens;

    // per-device facts: looked up per device; function attributes set on every call (they belong to the current device)
    int n_sm = 0;
    if (!device_info(&n_sm)) return SEKA_ERR_CUDA;
    if (cudaFuncSetAttribute(learn_cov_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LC_DYN_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(learn_svd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(sizeof(double) * (128 * (128 + SV_PAD) + 128) + sizeof(int) * 128)) != cudaSuccess)
        return SEKA_ERR_CUDA;

    // cross-covariances: columns in groups of 128 (one head of 128, or two neighbouring heads of 64)
    CUtensorMap tmH, tmP, tmN;
    if (!make_tile_map(&tmH, h, 128, pl.n_groups, n, LC_TOK) || !make_tile_map(&tmP, h_pos, 128, pl.n_groups, n, LC_TOK) ||
        !make_tile_map(&tmN, h_neg, 128, pl.n_groups, n, LC_TOK))
        return SEKA_ERR_CUDA;
    LearnCovParams p;
    p.part = reinterpret_cast<float*>(ws + pl.part_off);
    p.n_tokens = n; p.n_groups = pl.n_groups; p.d = d; p.slots = slots;
    p.chunk_tokens = pl.chunk_tokens; p.n_chunks = pl.n_chunks; p.status = reinterpret_cast<int*>(ws);
    const int n_items = pl.n_groups * pl.n_chunks;
    learn_cov_kernel<<<n_items < n_sm ? n_items : n_sm, LC_THREADS, LC_DYN_BYTES, st>>>(tmH, tmP, tmN, p);
    ++g_launches;
    const size_t total = (size_t)slots * 2 * d * d;
    learn_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(p.part, omega_pos, omega_neg, slots, d, pl.n_chunks, 1.f / (float)n);
    ++g_launches;

    // head-selection distance
    float* dsum = reinterpret_cast<float*>(ws + pl.dsum_off);
    int* dcnt = reinterpret_cast<int*>(ws + pl.dcnt_off);
    learn_dist_kernel<<<pl.dist_blocks, LD_THREADS, slots * sizeof(float), st>>>(
        static_cast<const __nv_bfloat16*>(h_pos), static_cast<const __nv_bfloat16*>(h_neg), answer_tokens, n, slots, d,
        pl.dist_tokens, dsum, dcnt);
    ++g_launches;
    learn_dist_reduce_kernel<<<slots, 256, 0, st>>>(dsum, dcnt, pl.dist_blocks, slots, D);
    ++g_launches;

    // SVD of every Omega, rank rule
    const size_t sv_smem = sizeof(double) * ((size_t)d * (d + SV_PAD) + d) + sizeof(int) * d;
    learn_svd_kernel<<<2 * slots, SV_THREADS, sv_smem, st>>>(omega_pos, omega_neg, slots, d, shape->gamma, U_pos, U_neg,
                                                           S_pos, S_neg, k_pos, k_neg, reinterpret_cast<int*>(ws + pl.sweeps_off));
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}
