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

// ---------------------------------------------------------------- bf16 tensors: one 128-token tile per step, on tcgen05
//
// A CTA (8 warps) takes a contiguous run of the (KV head, highlighted tile) pairs, head-major, so that the projector
// P[m][h] = U_m U_m^T (two bf16 parts, resident in shared memory) changes rarely: TMA stages the [128 x D] key tile,
// the tensor core forms K P_m in tensor memory (two products per expert), every thread adds
// g_b sum_m alpha_{b,h,m} (K P_m)[row] to half of its row in shared memory if the row is highlighted, and the warps
// then write the highlighted rows out, 16 bytes per lane with the lanes of a row next to each other.
// Unhighlighted rows are never written.  Two CTAs share an SM (96 KB of shared memory and M * D tensor-memory
// columns each), so the loads, products and stores of different tiles overlap.
constexpr uint32_t EBLK = 128 * 128;        // one [128 x 64] bf16 block

// all lanes of a warp wait on the same barrier and then agree on the outcome
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int where) {
    const bool ok = mbar_wait(bar, parity, abort_flag, status, where);
    return __all_sync(0xffffffffu, ok);
}
constexpr int EDIT_THREADS = 256;

template <int D>
struct EditSmem {
    static constexpr uint32_t TILE = (D / 64) * EBLK;
    static constexpr uint32_t PBLK = D * 128;
    static constexpr uint32_t PMAT = (D / 64) * PBLK;       // one D x D bf16 matrix
    static constexpr uint32_t K = 0;
    static constexpr uint32_t P = K + TILE;                 // high part, then low part
    static constexpr uint32_t FLAGS = P + 2 * PMAT;
    static constexpr uint32_t BARS = FLAGS + 128;
    static constexpr uint32_t MISC = BARS + 16;
    static constexpr uint32_t DYN_BYTES = MISC + 16 + 1024;
};

// SIDE: as in the pipelined kernel below, k' of every row of the tile that lies inside its sequence goes to the side
// buffer of the fused forward (rows of 2 D bf16: high parts, then low parts where the fused kernel reads them).
template <int D, bool SIDE>
__global__ void __launch_bounds__(EDIT_THREADS)
edit_tiles_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmP,
                  __nv_bfloat16* __restrict__ K_out, const uint8_t* __restrict__ mask, const float* __restrict__ alpha,
                  const float* __restrict__ gain, const uint8_t* __restrict__ head_enable,
                  const int* __restrict__ cu_seqlens, const int* __restrict__ hot_list, const int* __restrict__ hot_count,
                  int* status, int L, int Hkv, int M, int n_tiles, uint32_t tmem_cols) {
    using SL = EditSmem<D>;
    constexpr int NBLK = D / 64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + SL::K;
    uint8_t* flags = smem + SL::FLAGS;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + SL::BARS);
    uint64_t* done = full + 1;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + SL::MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::MISC + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row = tid & 127, half = tid >> 7;      // key row of the tile, and which half of its columns this thread updates
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(status) != 0)) return;

    if (tid == 0) {
        mbar_init(full, 1); mbar_init(done, 1);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmP);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    constexpr uint32_t IDESC = umma_idesc_bf16(D, false);
    constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
    const uint32_t dK = umma_desc_lo(smem_u32(sK), 16), dP = umma_desc_lo(smem_u32(smem + SL::P), 16);

    const int n_hot = *hot_count;
    const long long n_work = (long long)n_hot * Hkv;
    const long long per = (n_work + gridDim.x - 1) / gridDim.x;
    const long long w0 = (long long)blockIdx.x * per, w1 = w0 + per < n_work ? w0 + per : n_work;
    uint32_t n_full = 0, n_done = 0;
    int resident = -1;          // (m, h) pair whose projector is in shared memory: m * Hkv + h
    bool ok = true;
    for (long long idx = w0; idx < w1 && ok; ++idx) {
        const int h = (int)(idx / n_hot), tile = hot_list[idx % n_hot];
        const int b = tile / n_tiles, t = tile % n_tiles;
        const float g = gain[b];
        if (g == 0.f || (head_enable != nullptr && head_enable[h] == 0)) continue;      // same for the whole CTA
        const int seq0 = cu_seqlens ? cu_seqlens[b] : b * L;
        const int Lb = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0;
        const int kpos = t * 128 + row;
        const bool hl = kpos < Lb && mask[seq0 + kpos] != 0;
        if (half == 0) flags[row] = hl ? 1 : 0;
        const int nvalid = Lb - t * 128 < 128 ? Lb - t * 128 : 128;
        const bool with_lo = SIDE && (lo_needed(g, alpha_max_of(alpha, (size_t)b * Hkv + h, M)) || t < kLoTiles);
        for (int m = 0; m < M && ok; ++m) {
            const bool load_p = resident != m * Hkv + h;
            if (m == 0 || load_p) {
                if (tid == 0) {
                    mbar_expect_tx(full, (m == 0 ? SL::TILE : 0u) + (load_p ? 2 * SL::PMAT : 0u));
                    if (m == 0) {
#pragma unroll
                        for (int c = 0; c < NBLK; ++c) tma_load_3d(sK + c * EBLK, &tmK, full, c * 64, h, seq0 + t * 128);
                    }
                    if (load_p) {
#pragma unroll
                        for (int part = 0; part < 2; ++part)
#pragma unroll
                            for (int c = 0; c < NBLK; ++c)
                                tma_load_3d(smem + SL::P + part * SL::PMAT + c * SL::PBLK, &tmP, full, c * 64, 0,
                                            ((part * M + m) * Hkv + h) * D);
                    }
                }
                resident = m * Hkv + h;
                ok = mbar_wait(full, n_full & 1, abort_flag, status, 60);
                ++n_full;
                ok = __syncthreads_and(ok);
                if (!ok) break;
            }
            if (tid == 0) {
                tc_fence_after();
                // the high and the low part of the projector accumulate into the same columns
#pragma unroll
                for (int part = 0; part < 2; ++part)
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t offk = ((uint32_t)(ks >> 2) * EBLK + (uint32_t)(ks & 3) * 32) >> 4;
                        const uint32_t offp = ((uint32_t)part * SL::PMAT + (uint32_t)(ks >> 2) * SL::PBLK + (uint32_t)(ks & 3) * 32) >> 4;
                        umma_ss(tmem_base + (uint32_t)m * D, dK + offk, DESC_HI, dP + offp, DESC_HI, IDESC, (ks > 0 || part) ? 1u : 0u);
                    }
                umma_commit(done);
            }
            ok = mbar_wait(done, n_done & 1, abort_flag, status, 61);       // the projector may be replaced, K P_m may be read
            ++n_done;
            ok = __syncthreads_and(ok);
        }
        if (!ok) break;
        tc_fence_after();
        // this thread's half row: k' = k + g sum_m alpha_m (K P_m)[row]
        // (the tensor-memory loads are warp-wide instructions: every lane of a warp that has a highlighted row
        // takes part in them, only the update of the row itself depends on the lane's own flag)
        const bool warp_hl = __any_sync(0xffffffffu, hl);
        if (warp_hl || with_lo) {
            const bool side_lo = with_lo && row < nvalid;
            __nv_bfloat16* xlo = K_out + ((size_t)(seq0 + t * 128 + (row < nvalid ? row : 0)) * Hkv + h) * (2 * D) + D;
#pragma unroll 1
            for (int c = half * (D / 64); c < (half + 1) * (D / 64); ++c) {
                float dk[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) dk[e] = 0.f;
                for (int m = 0; m < M && warp_hl; ++m) {
                    const float cm = g * (alpha != nullptr ? alpha[((size_t)b * Hkv + h) * M + m] : 1.f);
                    uint32_t v[32];
                    tmem_ld32(t_lane + (uint32_t)m * D + c * 32, v);
                    tmem_wait_ld_on(v);
#pragma unroll
                    for (int e = 0; e < 32; ++e) dk[e] = fmaf(cm, __uint_as_float(v[e]), dk[e]);
                }
                uint4 lo4[4];
                if (SIDE) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) lo4[q] = make_uint4(0u, 0u, 0u, 0u);
                }
                if (hl) {
                    uint4* ptr[4];
                    uint4 kv[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {      // 8 elements = one 16-byte unit of the swizzled row; reads before writes
                        const int col = c * 32 + q * 8;
                        ptr[q] = reinterpret_cast<uint4*>(sK + (col >> 6) * EBLK + sw128_offset(row, col & 63));
                        kv[q] = *ptr[q];
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t* w = reinterpret_cast<uint32_t*>(&kv[q]);
                        uint32_t* l = reinterpret_cast<uint32_t*>(&lo4[q]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 k2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e]));
                            const float x0 = k2.x + dk[q * 8 + 2 * e], x1 = k2.y + dk[q * 8 + 2 * e + 1];
                            w[e] = pack_bf16(x0, x1);
                            if (SIDE) {        // the low parts: what the rounding above dropped
                                const float2 h2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e]));
                                l[e] = pack_bf16(x0 - h2.x, x1 - h2.y);
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) *ptr[q] = kv[q];
                }
                if (SIDE && side_lo) {
                    uint4* dst = reinterpret_cast<uint4*>(xlo + c * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q) dst[q] = lo4[q];
                }
                __syncwarp();      // all lanes together again before the next warp-wide load
            }
        }
        tc_fence_before();
        __syncthreads();
        // write the highlighted rows out: D / 8 lanes per row, 16 bytes each; 16 rows per warp
        constexpr int LPR = D / 8, RPI = 32 / LPR;
#pragma unroll 1
        for (int i = 0; i < 16 / RPI; ++i) {
            const int r = warp * 16 + i * RPI + lane / LPR, col = (lane % LPR) * 8;
            if (SIDE ? r < nvalid : flags[r] != 0) {
                const uint4 v = *reinterpret_cast<const uint4*>(sK + (col >> 6) * EBLK + sw128_offset(r, col & 63));
                *reinterpret_cast<uint4*>(K_out + ((size_t)(seq0 + t * 128 + r) * Hkv + h) * (SIDE ? 2 * D : D) + col) = v;
            }
        }
        __syncthreads();        // the tile and the flags are reused by the next step
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ---------------------------------------------------------------- single projector (plain SEKA): the same work as a pipeline
//
// One persistent CTA per SM with three roles, so that several key tiles are in flight per SM and the tensor-core
// product of one tile runs under the drain and write-out of the one before:
//   warp 8   producer: walks this CTA's run of (KV head, highlighted tile) pairs, stages key tiles through a ring of
//            NS shared-memory stages by TMA, writes the rows' highlight flags and the tile's coordinates beside them,
//            and (re)loads the projector when the head changes (after the ring has drained);
//   warp 9   MMA issuer: K P (two bf16 parts) into one of two sets of tensor-memory columns;
//   warps 0-7  drain: half a key row per thread, k' = k + c (K P)[row] into the staged tile for highlighted rows,
//            then the highlighted rows go out 16 bytes per lane; the stage and the columns are handed back.
constexpr int EP_THREADS = 320;

struct EpMeta { int tok0, h, valid, p_gen; float c; int nvalid, with_lo, pad; };     // per stage: first token, head, end marker, projector generation, g * alpha, rows inside the sequence, low parts wanted (side mode)

template <int D>
struct EpSmem {
    static constexpr uint32_t TILE = (D / 64) * EBLK;
    static constexpr uint32_t PBLK = D * 128;
    static constexpr uint32_t PMAT = (D / 64) * PBLK;
    static constexpr int NS = D == 128 ? 4 : 8;             // key tiles in flight per SM
    static constexpr uint32_t K = 0;                        // NS stages
    static constexpr uint32_t P = K + NS * TILE;            // high part, then low part
    static constexpr uint32_t FLAGS = P + 2 * PMAT;         // NS x 128 bytes
    static constexpr uint32_t META = FLAGS + NS * 128;      // NS x 32 bytes
    static constexpr uint32_t BARS = META + NS * 32;        // full[NS], free[NS], mma_done[2], cols_free[2], p_full, meet[2]
    static constexpr uint32_t NBARS = 2 * NS + 7;
    static constexpr uint32_t MISC = BARS + NBARS * 8;
    static constexpr uint32_t DYN_BYTES = MISC + 16 + 1024;
};

// SIDE: instead of rewriting the highlighted rows of the key tensor, write k' of every row of the tile that lies inside
// its sequence into the side buffer of the fused forward, rows of 2 D bf16: high parts [0, D), low parts [D, 2 D) (the low
// parts only where the fused kernel reads them: see lo_needed; zero for rows that are not highlighted).
template <int D, bool SIDE>
__global__ void __launch_bounds__(EP_THREADS, 1)
edit_tiles_pipe_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmP,
                       __nv_bfloat16* __restrict__ K_out, const uint8_t* __restrict__ mask, const float* __restrict__ alpha,
                       const float* __restrict__ gain, const uint8_t* __restrict__ head_enable,
                       const int* __restrict__ cu_seqlens, const int* __restrict__ hot_list, const int* __restrict__ hot_count,
                       int* status, int L, int Hkv, int n_tiles) {
    using SL = EpSmem<D>;
    constexpr int EP_NS = SL::NS;
    constexpr int NBLK = D / 64;
    constexpr uint32_t TMEM_COLS = 2 * D < 32 ? 32 : 2 * D;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::BARS);
    uint64_t* full = bars;                     // [NS]  tile landed (TMA bytes) and flags / coordinates written (producer)
    uint64_t* freeb = full + EP_NS;            // [NS]  8 drain-warp arrivals: the stage may be refilled
    uint64_t* mma_done = freeb + EP_NS;        // [2]   K P of a tile is in column set c
    uint64_t* cols_free = mma_done + 2;        // [2]   8 drain-warp arrivals: column set c has been read
    uint64_t* p_full = cols_free + 2;          // [1]   projector landed
    uint64_t* meetb = p_full + 1;              // [2]   8 drain-warp arrivals: all rows of the tile are updated
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + SL::MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::MISC + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(status) != 0)) return;

    if (tid == 0) {
        for (int i = 0; i < EP_NS; ++i) { mbar_init(full + i, 2); mbar_init(freeb + i, 8); }
        for (int i = 0; i < 2; ++i) { mbar_init(mma_done + i, 1); mbar_init(cols_free + i, 8); mbar_init(meetb + i, 8); }
        mbar_init(p_full, 1);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmP);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 8) {
        // ------------------------------------------------------------ producer
        const int n_hot = *hot_count;
        const long long n_work = (long long)n_hot * Hkv;
        const long long per = (n_work + gridDim.x - 1) / gridDim.x;
        long long w0 = (long long)blockIdx.x * per;
        if (w0 > n_work) w0 = n_work;                 // a CTA without work still pushes the end marker
        const long long w1 = w0 + per < n_work ? w0 + per : n_work;
        uint32_t n_push = 0;      // stages filled so far
        int p_gen = 0, cur_h = -1;
        bool ok = true;
        // What a work unit needs from global memory (its entry of the list, the sequence bounds, gain, coefficient) is a
        // chain of dependent loads; one lane per unit fetches it for 32 units at a time, and the highlight flags of a
        // tile are requested one tile ahead, so that the ring is not fed at the pace of memory round trips.
        uint8_t fl_next[4] = {0, 0, 0, 0};
        bool have_next = false;
        for (long long base = w0; base <= w1 && ok; base += 32) {
            int h_l = 0, t_l = 0, seq0_l = 0, Lb_l = 0, lo_l = 0, skip_l = 1;
            float c_l = 0.f;
            {
                const long long my = base + lane;
                if (my < w1) {
                    h_l = (int)(my / n_hot);
                    const int tile = hot_list[my % n_hot];
                    const int b = tile / n_tiles;
                    t_l = tile % n_tiles;
                    const float g = gain[b];
                    const float a = alpha != nullptr ? alpha[(size_t)b * Hkv + h_l] : 1.f;
                    skip_l = (g == 0.f || (head_enable != nullptr && head_enable[h_l] == 0)) ? 1 : 0;
                    c_l = g * a;
                    seq0_l = cu_seqlens ? cu_seqlens[b] : b * L;
                    Lb_l = (cu_seqlens ? cu_seqlens[b + 1] : (b + 1) * L) - seq0_l;
                    lo_l = (SIDE && (lo_needed(g, fabsf(a)) || t_l < kLoTiles)) ? 1 : 0;
                }
            }
            const int n_here = (int)((w1 - base + 1) < 32 ? (w1 - base + 1) : 32);      // units of this batch, end marker included
            auto flags_of = [&](int k, uint8_t (&f)[4]) {      // highlight flags of unit k of the batch (4 rows per lane)
                const int seq0 = __shfl_sync(0xffffffffu, seq0_l, k), t = __shfl_sync(0xffffffffu, t_l, k), Lb = __shfl_sync(0xffffffffu, Lb_l, k);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int kpos = t * 128 + q * 32 + lane;
                    f[q] = (kpos < Lb && mask[seq0 + kpos] != 0) ? 1 : 0;
                }
            };
            for (int k = 0; k < n_here && ok; ++k) {
                const long long idx = base + k;
                const bool last = idx >= w1;                    // one more stage after the work: the end marker
                const int h = __shfl_sync(0xffffffffu, h_l, k), t = __shfl_sync(0xffffffffu, t_l, k);
                const int seq0 = __shfl_sync(0xffffffffu, seq0_l, k), Lb = __shfl_sync(0xffffffffu, Lb_l, k);
                const int with_lo = __shfl_sync(0xffffffffu, lo_l, k), skip = __shfl_sync(0xffffffffu, skip_l, k);
                const float c = __shfl_sync(0xffffffffu, c_l, k);
                uint8_t fl_cur[4] = {0, 0, 0, 0};
                if (!last) {
                    if (have_next) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) fl_cur[q] = fl_next[q];
                    } else {
                        flags_of(k, fl_cur);
                    }
                }
                // the flags of the next unit of the batch are requested now and used in the next trip
                have_next = k + 1 < n_here && base + k + 1 < w1;
                if (have_next) flags_of(k + 1, fl_next);
                if (!last) {
                    if (skip) continue;
                    if (h != cur_h) {
                        // the projector changes: every tile of the old head must be through the tensor core (here: the
                        // whole ring handed back), then the new one is loaded
                        for (uint32_t q = n_push >= EP_NS ? n_push - EP_NS : 0; q < n_push && ok; ++q)
                            ok = warp_wait(freeb + q % EP_NS, (q / EP_NS) & 1, abort_flag, status, 62);
                        if (!ok) break;
                        if (lane == 0) {
                            mbar_expect_tx(p_full, 2 * SL::PMAT);
#pragma unroll
                            for (int part = 0; part < 2; ++part)
#pragma unroll
                                for (int cb = 0; cb < NBLK; ++cb)
                                    tma_load_3d(smem + SL::P + part * SL::PMAT + cb * SL::PBLK, &tmP, p_full, cb * 64, 0, (part * Hkv + h) * D);
                        }
                        __syncwarp();
                        cur_h = h; ++p_gen;
                    }
                }
                const uint32_t s = n_push % EP_NS;
                if (n_push >= EP_NS) {
                    ok = warp_wait(freeb + s, ((n_push / EP_NS) - 1) & 1, abort_flag, status, 63);
                    if (!ok) break;
                }
                uint8_t* fl = smem + SL::FLAGS + s * 128;
                if (!last) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) fl[q * 32 + lane] = fl_cur[q];
                }
                if (lane == 0) {
                    EpMeta* m = reinterpret_cast<EpMeta*>(smem + SL::META + s * 32);
                    m->tok0 = seq0 + t * 128; m->h = h; m->valid = last ? 0 : 1; m->p_gen = p_gen; m->c = c;
                    m->nvalid = Lb - t * 128 < 128 ? Lb - t * 128 : 128;
                    m->with_lo = last ? 0 : with_lo;
                    if (!last) {
                        mbar_expect_tx(full + s, SL::TILE);
#pragma unroll
                        for (int cb = 0; cb < NBLK; ++cb) tma_load_3d(smem + SL::K + s * SL::TILE + cb * EBLK, &tmK, full + s, cb * 64, h, seq0 + t * 128);
                    } else {
                        mbar_arrive(full + s);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(full + s);       // second arrival: flags and coordinates are in place
                ++n_push;
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t IDESC = umma_idesc_bf16(D, false);
        constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
        const uint32_t dK = umma_desc_lo(smem_u32(smem + SL::K), 16), dP = umma_desc_lo(smem_u32(smem + SL::P), 16);
        int seen_gen = 0;
        bool ok = true;
        for (uint32_t n = 0; ok; ++n) {
            const uint32_t s = n % EP_NS, cset = n & 1;
            ok = warp_wait(full + s, (n / EP_NS) & 1, abort_flag, status, 64);
            if (!ok) break;
            const EpMeta m = *reinterpret_cast<const EpMeta*>(smem + SL::META + s * 32);
            if (!m.valid) break;
            if (m.p_gen != seen_gen) {
                ok = warp_wait(p_full, (uint32_t)(m.p_gen - 1) & 1, abort_flag, status, 65);
                if (!ok) break;
                seen_gen = m.p_gen;
            }
            if (n >= 2) {
                ok = warp_wait(cols_free + cset, ((n >> 1) - 1) & 1, abort_flag, status, 66);
                if (!ok) break;
            }
            tc_fence_after();
            if (lane == 0) {
                const uint32_t kd = dK + s * (SL::TILE >> 4);
#pragma unroll
                for (int part = 0; part < 2; ++part)
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t offk = ((uint32_t)(ks >> 2) * EBLK + (uint32_t)(ks & 3) * 32) >> 4;
                        const uint32_t offp = ((uint32_t)part * SL::PMAT + (uint32_t)(ks >> 2) * SL::PBLK + (uint32_t)(ks & 3) * 32) >> 4;
                        umma_ss(tmem_base + cset * D, kd + offk, DESC_HI, dP + offp, DESC_HI, IDESC, (ks > 0 || part) ? 1u : 0u);
                    }
                umma_commit(mma_done + cset);
            }
            __syncwarp();
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------ drain and write-out
        const int row = tid & 127, half = tid >> 7;
        const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        bool ok = true;
        for (uint32_t n = 0; ok; ++n) {
            const uint32_t s = n % EP_NS, cset = n & 1;
            ok = warp_wait(full + s, (n / EP_NS) & 1, abort_flag, status, 67);
            if (!ok) break;
            const EpMeta m = *reinterpret_cast<const EpMeta*>(smem + SL::META + s * 32);
            if (!m.valid) break;
            uint8_t* sK = smem + SL::K + s * SL::TILE;
            const uint8_t* fl = smem + SL::FLAGS + s * 128;
            const bool hl = fl[row] != 0;
            ok = warp_wait(mma_done + cset, (n >> 1) & 1, abort_flag, status, 68);
            if (!ok) break;
            tc_fence_after();
            // (the tensor-memory loads are warp-wide: every lane takes part, only the row update depends on the flag)
            const bool side_lo = SIDE && m.with_lo != 0 && row < m.nvalid;
            __nv_bfloat16* xlo = K_out + ((size_t)(m.tok0 + (row < m.nvalid ? row : 0)) * Hkv + m.h) * (2 * D) + D;
            if (__any_sync(0xffffffffu, hl) || (SIDE && m.with_lo != 0)) {
                const bool warp_hl = __any_sync(0xffffffffu, hl);
#pragma unroll 1
                for (int c = half * (D / 64); c < (half + 1) * (D / 64); ++c) {
                    uint32_t v[32];
                    if (warp_hl) { tmem_ld32(t_lane + cset * D + c * 32, v); tmem_wait_ld_on(v); }
                    uint4 lo4[4];
                    if (SIDE) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) lo4[q] = make_uint4(0u, 0u, 0u, 0u);
                    }
                    if (hl) {
                        uint4* ptr[4];
                        uint4 kv[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {      // 8 elements = one 16-byte unit of the swizzled row; reads before writes
                            const int col = c * 32 + q * 8;
                            ptr[q] = reinterpret_cast<uint4*>(sK + (col >> 6) * EBLK + sw128_offset(row, col & 63));
                            kv[q] = *ptr[q];
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t* w = reinterpret_cast<uint32_t*>(&kv[q]);
                            uint32_t* l = reinterpret_cast<uint32_t*>(&lo4[q]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 k2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e]));
                                const float x0 = fmaf(m.c, __uint_as_float(v[q * 8 + 2 * e]), k2.x), x1 = fmaf(m.c, __uint_as_float(v[q * 8 + 2 * e + 1]), k2.y);
                                w[e] = pack_bf16(x0, x1);
                                if (SIDE) {        // the low parts: what the rounding above dropped
                                    const float2 h2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e]));
                                    l[e] = pack_bf16(x0 - h2.x, x1 - h2.y);
                                }
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) *ptr[q] = kv[q];
                    }
                    if (side_lo) {
                        uint4* dst = reinterpret_cast<uint4*>(xlo + c * 32);
#pragma unroll
                        for (int q = 0; q < 4; ++q) dst[q] = lo4[q];
                    }
                    __syncwarp();      // all lanes together again before the next warp-wide load
                }
            }
            // the columns are read: the next product may use them; all rows updated: the tile may be written out
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(cols_free + cset); mbar_arrive(meetb + cset); }
            ok = warp_wait(meetb + cset, (n >> 1) & 1, abort_flag, status, 69);
            if (!ok) break;
            constexpr int LPR = D / 8, RPI = 32 / LPR;
#pragma unroll 1
            for (int i = 0; i < 16 / RPI; ++i) {
                const int r = warp * 16 + i * RPI + lane / LPR, col = (lane % LPR) * 8;
                if (SIDE ? r < m.nvalid : fl[r] != 0) {
                    const uint4 v = *reinterpret_cast<const uint4*>(sK + (col >> 6) * EBLK + sw128_offset(r, col & 63));
                    *reinterpret_cast<uint4*>(K_out + ((size_t)(m.tok0 + r) * Hkv + m.h) * (SIDE ? 2 * D : D) + col) = v;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(freeb + s);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int D>
static seka_status launch_edit_tiles(const seka_shape* s, const WorkspaceLayout& w, const void* K_in, void* K_out,
                                     const uint8_t* mask, const float* U, const float* alpha, const float* gain,
                                     const uint8_t* he, char* ws, cudaStream_t st) {
    using SL = EditSmem<D>;
    // per-device facts: looked up per device; function attributes set on every call (they belong to the current device)
    int n_sm = 0;
    if (!device_info(&n_sm)) return SEKA_ERR_CUDA;
    if (cudaFuncSetAttribute(edit_tiles_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SL::DYN_BYTES) != cudaSuccess)
        return SEKA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws);
    void* P = ws + w.w_off;
    uint8_t* tile_hot = reinterpret_cast<uint8_t*>(ws + w.hot_off);
    int* hot_list = reinterpret_cast<int*>(ws + w.list_off);
    if (launch_prep_edit(s, U, mask, P, tile_hot, w.n_tiles, hot_list, status + 2, st) != SEKA_OK) return SEKA_ERR_CUDA;
    const int T = shape_total_tokens(s), Hkv = s->n_kv_heads, M = s->n_experts;
    CUtensorMap tk, tp;
    if (!make_tile_map(&tk, K_in, D, Hkv, T) || !make_tile_map(&tp, P, D, 1, (long long)2 * M * Hkv * D, D)) return SEKA_ERR_CUDA;
    if (M == 1) {
        using PL = EpSmem<D>;
        if (cudaFuncSetAttribute(edit_tiles_pipe_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PL::DYN_BYTES) != cudaSuccess)
            return SEKA_ERR_CUDA;
        const long long work = (long long)s->batch * w.n_tiles * Hkv;
        const unsigned gridp = (unsigned)(work < (long long)n_sm ? work : (long long)n_sm);
        edit_tiles_pipe_kernel<D, false><<<gridp, EP_THREADS, PL::DYN_BYTES, st>>>(tk, tp, static_cast<__nv_bfloat16*>(K_out), mask, alpha, gain, he,
                                                                          s->cu_seqlens, hot_list, status + 2, status, s->max_seqlen,
                                                                          Hkv, w.n_tiles);
        ++g_launches;
        return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
    }
    uint32_t cols = 32;
    while (cols < (uint32_t)(M * D)) cols *= 2;
    const int per_sm = (int)(512 / cols) < 2 ? (int)(512 / cols) : 2;          // tensor memory and shared memory per SM
    const long long work_max = (long long)s->batch * w.n_tiles * Hkv;
    const long long want = (long long)n_sm * per_sm;
    const unsigned grid = (unsigned)(work_max < want ? work_max : want);
    edit_tiles_kernel<D, false><<<grid, EDIT_THREADS, SL::DYN_BYTES, st>>>(tk, tp, static_cast<__nv_bfloat16*>(K_out), mask, alpha, gain, he,
                                                         s->cu_seqlens, hot_list, status + 2, status, s->max_seqlen, Hkv, M,
                                                         w.n_tiles, cols);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

template <int D>
static seka_status stage_keys_pipe_t(const seka_shape* s, const WorkspaceLayout& w, const void* K16, void* X,
                                     const uint8_t* mask, const float* U, const float* alpha, const float* gain,
                                     const uint8_t* he, char* ws, cudaStream_t st, const void* Q_route, const float* sigma,
                                     int k_route) {
    using PL = EpSmem<D>;
    int n_sm = 0;
    if (!device_info(&n_sm)) return SEKA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws);
    void* P = ws + w.w_off;
    uint8_t* tile_hot = reinterpret_cast<uint8_t*>(ws + w.hot_off);
    int* hot_list = reinterpret_cast<int*>(ws + w.list_off);
    // routed call: `alpha` is where the preparation launch writes the coefficients (read by the tile kernel after it)
    if (launch_prep_edit(s, U, mask, P, tile_hot, w.n_tiles, hot_list, status + 2, st, reinterpret_cast<int*>(ws + w.first_off),
                         reinterpret_cast<uint8_t*>(ws + w.info_off), gain, alpha, he, Q_route, sigma, k_route,
                         const_cast<float*>(alpha)) != SEKA_OK)
        return SEKA_ERR_CUDA;
    const int T = shape_total_tokens(s), Hkv = s->n_kv_heads, M = s->n_experts;
    CUtensorMap tk, tp;
    if (!make_tile_map(&tk, K16, D, Hkv, T) || !make_tile_map(&tp, P, D, 1, (long long)2 * M * Hkv * D, D)) return SEKA_ERR_CUDA;
    if (M > 1) {
        // a bank of experts: one product pair per expert into its own tensor-memory columns, two CTAs per SM
        using SL = EditSmem<D>;
        if (cudaFuncSetAttribute(edit_tiles_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SL::DYN_BYTES) != cudaSuccess)
            return SEKA_ERR_CUDA;
        uint32_t cols = 32;
        while (cols < (uint32_t)(M * D)) cols *= 2;
        const int per_sm = (int)(512 / cols) < 2 ? (int)(512 / cols) : 2;
        const long long work_max = (long long)s->batch * w.n_tiles * Hkv, want = (long long)n_sm * per_sm;
        const unsigned grid_b = (unsigned)(work_max < want ? work_max : want);
        edit_tiles_kernel<D, true><<<grid_b, EDIT_THREADS, SL::DYN_BYTES, st>>>(tk, tp, static_cast<__nv_bfloat16*>(X), mask, alpha, gain, he,
                                                                              s->cu_seqlens, hot_list, status + 2, status, s->max_seqlen,
                                                                              Hkv, M, w.n_tiles, cols);
        ++g_launches;
        return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
    }
    if (cudaFuncSetAttribute(edit_tiles_pipe_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PL::DYN_BYTES) != cudaSuccess)
        return SEKA_ERR_CUDA;
    const long long work = (long long)s->batch * w.n_tiles * Hkv;
    const unsigned grid = (unsigned)(work < (long long)n_sm ? work : (long long)n_sm);
    edit_tiles_pipe_kernel<D, true><<<grid, EP_THREADS, PL::DYN_BYTES, st>>>(tk, tp, static_cast<__nv_bfloat16*>(X), mask, alpha, gain, he,
                                                                           s->cu_seqlens, hot_list, status + 2, status, s->max_seqlen,
                                                                           Hkv, w.n_tiles);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

seka_status launch_stage_keys_pipe(const seka_shape* s, const WorkspaceLayout& w, const void* K16, void* X,
                                   const uint8_t* mask, const float* U, const float* alpha, const float* gain,
                                   const uint8_t* head_enable, char* ws, cudaStream_t st, const void* Q_route,
                                   const float* sigma, int k_route) {
    return s->head_dim == 128 ? stage_keys_pipe_t<128>(s, w, K16, X, mask, U, alpha, gain, head_enable, ws, st, Q_route, sigma, k_route)
                              : stage_keys_pipe_t<64>(s, w, K16, X, mask, U, alpha, gain, head_enable, ws, st, Q_route, sigma, k_route);
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
    if (!workspace || workspace_bytes < w.edit_total) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    int* status = reinterpret_cast<int*>(ws);
    int* list = reinterpret_cast<int*>(ws + w.list_off);
    const size_t esz = shape->dtype == SEKA_F32 ? 4 : 2;
    if (K_out != K_in) {
        const size_t bytes = (size_t)T * shape->n_kv_heads * shape->head_dim * esz;
        if (cudaMemcpyAsync(K_out, K_in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SEKA_ERR_CUDA;
    }
    // bf16 tensors go through the tensor-core tile kernel (the projector products of all experts have to fit
    // into tensor memory); fp32 tensors, and banks too large for that, take the fp32 row kernel
    if (shape->dtype == SEKA_BF16 && (long long)shape->n_experts * shape->head_dim <= 512 && ((uintptr_t)workspace & 255) == 0) {
        if (shape->head_dim == 128)
            return launch_edit_tiles<128>(shape, w, K_in, K_out, mask, U, alpha, gain, head_enable, ws, st);
        return launch_edit_tiles<64>(shape, w, K_in, K_out, mask, U, alpha, gain, head_enable, ws, st);
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
