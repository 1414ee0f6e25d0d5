// Fused SEKA / AdaSEKA steered causal GQA attention forward for sm_100a.
//
// One CTA (16 warps) owns two tiles of 128 queries that share a KV head ("A" and "B": two query heads of
// one group at the same rows, or two consecutive row tiles of one head when the group size is odd) and
// walks the key tiles 0 .. diagonal.  Warp roles:
//   warp 0        TMA producer: Q tiles and the edit operator W once, then K and V tiles (128-byte swizzle)
//                 through two shared-memory rings, throttled by "empty" mbarriers the tensor core signals;
//   warp 1        MMA issuer: S_x = Q_x K'^T and O_x += P_x V on tcgen05 with all accumulators in tensor
//                 memory (S_A, S_B, O_A, O_B = 512 columns); P_x is read from tensor memory.  For a staged
//                 K tile that holds highlighted tokens of a steered head it first issues dK = K W into the
//                 score columns of the tile that will use K first (they are idle just then);
//   warps 12-15   key editors: read dK from tensor memory and add it, for highlighted rows only, to the
//                 staged tile in place: k' = k + g * sum_m alpha_m U_m U_m^T k (Section 2 / Section 3.3, hook
//                 of Algorithm 1/2) with W = g * sum_m alpha_m U_m U_m^T prepared per (sequence, KV head);
//   warps 4-7 / 8-11  softmax of tile A / B, one query row per thread: causal mask on the diagonal
//                 tile, online softmax in base 2 with a lazily updated running maximum, P written
//                 back as bf16 over the consumed score columns, O rescaled in tensor memory only when
//                 the maximum moved by more than 2^8; final normalisation and store.
// While one tile's softmax runs, the tensor core works on the other tile.  Neither K' nor the score
// matrix ever reaches global memory; K and V are read only.  Every wait is bounded: a wait that runs
// out raises the CTA's abort flag, every role leaves its loop, and the status word reports it.
// The edit runs on tcgen05 like everything else: warp-level mma.sync is starved by a busy tcgen05 pipe
// (it gets roughly one slot per UMMA), and its unrolled code evicts the other roles' loops from the
// instruction cache.
#include <math.h>

#include "seka_kernels.h"

#ifndef SEKA_POLY_PAIR_MASK
#define SEKA_POLY_PAIR_MASK 0x0000u
#endif

namespace seka {

struct AttnParams {
    void* O;
    float* lse;
    const uint8_t* mask;
    const float* gain;
    const uint8_t* head_enable;
    const int* cu_seqlens;
    const uint8_t* tile_hot;      // [B, n_qt]: key tile holds a highlighted token
    int* status;
    int B, L, Hq, Hkv, n_qt;
    const ItemRecord* items;   // item table (built by the preparation kernel), heaviest first
    const int* n_items;        // its length (device word)
    long long n_items_max;
    int steer;
    int pair_heads;       // 1: the two tiles of an item are two query heads of one KV group; 0: two consecutive row tiles
    float scale_log2;
};

constexpr int BM = 128, BN = 128;
constexpr int NTHREADS = 512;
constexpr uint32_t BLK_BYTES = 128 * 128;   // one [128 x 64] bf16 block
constexpr float LAZY_RESCALE_LOG2 = 8.0f;   // the running maximum is only raised when it moved by more than this
// registers per thread after the roles split (the CTA owns the whole register file: 4 x 128 x (80+184+184+64) = 64 Ki)
constexpr int REGS_CTRL = 80, REGS_SOFTMAX = 184, REGS_EDIT = 64;
// which of the 16 element pairs of every 32-key chunk take the polynomial exp2 instead of the special-function unit
constexpr uint32_t POLY_PAIR_MASK = SEKA_POLY_PAIR_MASK;

template <int D>
struct SmemLayout {
    // K and V ring depth: head_dim 128 leaves room for two stages beside the 32 KB edit operator, head_dim 64 for three
    static constexpr int NK = D == 128 ? 2 : 3;
    static constexpr uint32_t TILE = (D / 64) * BLK_BYTES;
    static constexpr uint32_t WBLK = D * 128;              // one [D x 64] block of W
    static constexpr uint32_t Q = 0;                       // 2 tiles
    static constexpr uint32_t K = Q + 2 * TILE;            // NK stages
    static constexpr uint32_t V = K + NK * TILE;           // NK stages
    static constexpr uint32_t W = V + NK * TILE;           // D x D bf16
    static constexpr uint32_t BARS = W + (D / 64) * WBLK;  // mbarriers
    static constexpr uint32_t NBARS = 3 + 2 * NK + 8 + 3;
    static constexpr uint32_t MISC = BARS + NBARS * 8;     // tmem holder, abort flag
    static constexpr uint32_t ITEMS = MISC + 16;           // one 32-byte item record per warp
    static constexpr uint32_t TOTAL = ITEMS + 16 * 32;
    static constexpr uint32_t DYN_BYTES = TOTAL + 1024;    // slack for the 1024-byte alignment
};

// One 128-row query tile of a CTA: query head, tile index within the sequence, number of key tiles it attends
// to (the last of them is the diagonal tile); n == 0 means the tile lies beyond the sequence.
struct TileWork { int hq, qt, n; };

// all lanes of a warp wait on the same barrier and then agree on the outcome
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int where) {
    const bool ok = mbar_wait(bar, parity, abort_flag, status, where);
    return __all_sync(0xffffffffu, ok);
}

// true in exactly one lane of a fully active warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^x for a pair of arguments on the FMA pipe: x = n + f with n = round(x), f in [-1/2, 1/2];
// 2^f by a cubic fitted to relative error 7.5e-5 (far below the bf16 rounding of P), 2^n by adding n
// to the exponent field.  Arguments below -126 (masked scores) give a value below 2^-125.
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.f;      // 1.5 * 2^23: adding it rounds to an integer in the low mantissa bits
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
    float2 q = __ffma2_rn(f, make_float2(0.05517167f, 0.05517167f), make_float2(0.24261113f, 0.24261113f));
    q = __ffma2_rn(q, f, make_float2(0.69326097f, 0.69326097f));
    q = __ffma2_rn(q, f, make_float2(0.99992806f, 0.99992806f));
    float2 r;
    r.x = __int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23));
    r.y = __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23));
    return r;
}

template <typename OutT> __device__ __forceinline__ void store_chunk32(OutT* dst, const uint32_t (&v)[32], float inv);
template <> __device__ __forceinline__ void store_chunk32<__nv_bfloat16>(__nv_bfloat16* dst, const uint32_t (&v)[32], float inv) {
    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int c = 0; c < 4; ++c)
        d4[c] = make_uint4(pack_bf16(__uint_as_float(v[8 * c]) * inv, __uint_as_float(v[8 * c + 1]) * inv),
                           pack_bf16(__uint_as_float(v[8 * c + 2]) * inv, __uint_as_float(v[8 * c + 3]) * inv),
                           pack_bf16(__uint_as_float(v[8 * c + 4]) * inv, __uint_as_float(v[8 * c + 5]) * inv),
                           pack_bf16(__uint_as_float(v[8 * c + 6]) * inv, __uint_as_float(v[8 * c + 7]) * inv));
}
template <> __device__ __forceinline__ void store_chunk32<float>(float* dst, const uint32_t (&v)[32], float inv) {
    float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int c = 0; c < 8; ++c)
        d4[c] = make_float4(__uint_as_float(v[4 * c]) * inv, __uint_as_float(v[4 * c + 1]) * inv,
                            __uint_as_float(v[4 * c + 2]) * inv, __uint_as_float(v[4 * c + 3]) * inv);
}

// Adds dK (fp32, tensor memory, one key row per lane) to this thread's row of a staged K tile for the 32-column
// chunks [c0, c1); rows whose flag is clear are left alone.  The tensor-memory loads are warp-wide: every lane
// takes part in them whatever its flag.  The four 16-byte units of a chunk are read before any is written back
// (a store followed by a load of the same array would keep the updates strictly in sequence).
__device__ __forceinline__ void drain_edit(uint32_t tE, uint8_t* sK, int row, bool hl, int c0, int c1) {
#pragma unroll 1
    for (int c = c0; c < c1; ++c) {
        uint32_t dk[32];
        tmem_ld32(tE + c * 32, dk);
        tmem_wait_ld_on(dk);
        if (hl) {
            uint4* ptr[4];
            uint4 kv[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {      // 8 elements = one 16-byte unit of the swizzled row
                const int col = c * 32 + q * 8;
                ptr[q] = reinterpret_cast<uint4*>(sK + (col >> 6) * (128 * 128) + sw128_offset(row, col & 63));
                kv[q] = *ptr[q];
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t* w = reinterpret_cast<uint32_t*>(&kv[q]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 k2 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[e]));
                    const float2 s2 = __fadd2_rn(k2, make_float2(__uint_as_float(dk[q * 8 + 2 * e]), __uint_as_float(dk[q * 8 + 2 * e + 1])));
                    w[e] = pack_bf16(s2.x, s2.y);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) *ptr[q] = kv[q];
        }
        __syncwarp();      // all lanes together again before the next warp-wide load
    }
}

// One unit of work of a CTA: two 128-row query tiles that share a KV head of one sequence.
struct Item {
    int b, hkv, seq0, Lb;
    int hqA, hqB, qtA, qtB;     // query head and row-tile index of tile A / B
    int nA, nB, n_kv;           // key tiles of A / B (0: the tile lies beyond the sequence) and of the item
    bool steer;
};

template <int D, typename OutT, bool TABLE>
__global__ void __launch_bounds__(NTHREADS, 1)
seka_attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW,
                     const AttnParams p) {
    using SL = SmemLayout<D>;
    constexpr int NK = SL::NK;
    constexpr int NBLK = D / 64;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0, COL_O = 256;     // S_x at COL_S + 128 x, O_x at COL_O + D x
    // head_dim 64 leaves 128 columns unused: dK of a highlighted key tile gets columns of its own there and is
    // formed while the previous step's P V runs; head_dim 128 has to borrow the idle score columns of a tile
    constexpr bool EDIT_OWN_COLS = (D == 64);
    constexpr uint32_t COL_E = 384;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL::BARS);
    uint64_t* q_full = bars;                 // [2]   TMA bytes landed
    uint64_t* k0_full = q_full + 2;          // [1]   first key tile of the item landed
    uint64_t* kv_full = k0_full + 1;         // [NK]  V(t) and K(t+1) landed (they are loaded as a pair)
    uint64_t* kv_free = kv_full + NK;        // [NK]  one event per step: the tensor core is done with K(j+1) and V(j)
    uint64_t* s_full = kv_free + NK;         // [2]   scores of tile x are in tensor memory
    uint64_t* p_full = s_full + 2;           // [2]   4 softmax-warp arrivals (O_x rescaled, keys 0-95 of P_x written) + 1 from the operand relay
    uint64_t* p_last = p_full + 2;           // [2]   4 softmax-warp arrivals: keys 96-127 of P_x written
    uint64_t* o_full = p_last + 2;           // [2]   last P V of tile x finished
    uint64_t* w_full = o_full + 2;           // [1]   edit operator landed
    uint64_t* e_full = w_full + 1;           // [1]   dK = K W of the current highlighted tile is in tensor memory
    uint64_t* k_edited = e_full + 1;         // [1]   4 editor-warp + 4 softmax-warp arrivals: the staged tile now holds K'
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + SL::MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SL::MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // an earlier launch (or CTA) gave up on this workspace: all threads agree on leaving
    if (__syncthreads_or(*reinterpret_cast<volatile int*>(p.status) != 0)) return;

    // The CTA is persistent: it walks its share of the items (heaviest first; odd rounds run the CTAs in
    // reverse so that the shares come out even).  Every role goes through the same sequence of items by itself.
    // Fixed-length batches decode the item from its index; packed variable-length batches, where many index
    // slots are empty (row tiles beyond a short sequence), read a table from which those were dropped.
    const int n_items = TABLE ? *p.n_items : (int)p.n_items_max;
    auto item_index = [&](int round) -> int {
        const int G = (int)gridDim.x;
        const long long idx = (long long)round * G + ((round & 1) ? (G - 1 - (int)blockIdx.x) : (int)blockIdx.x);
        return idx < n_items ? (int)idx : -1;
    };
    // (table) the record of the next item is copied into a per-warp slot of shared memory while the current item
    // runs, so that no registers are held for it; lane 0 issues the copy and waits for it
    int round = 0, idx_next = TABLE ? item_index(0) : 0;
    auto prefetch = [&]() {
        if (TABLE && idx_next >= 0 && lane == 0) {
            const uint32_t dst = smem_u32(smem + SL::ITEMS + warp * 32);
            const ItemRecord* rec = p.items + idx_next;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(rec) : "memory");
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst + 16), "l"(reinterpret_cast<const char*>(rec) + 16) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    };
    prefetch();
    auto next_item = [&](Item& it) -> bool {
        if (TABLE) {
            if (idx_next < 0) return false;
            const uint8_t* slot = smem + SL::ITEMS + warp * 32;
            if (lane == 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
            const int4 raw0 = *reinterpret_cast<const int4*>(slot), raw1 = *reinterpret_cast<const int4*>(slot + 16);
            it.seq0 = raw0.x; it.Lb = raw0.y; it.b = raw0.z; it.hkv = raw0.w;
            it.hqA = raw1.x & 0xffff; it.hqB = raw1.x >> 16;
            it.qtA = raw1.y & 0xffff; it.qtB = raw1.y >> 16;
            it.nA = raw1.z & 0xffff; it.nB = raw1.z >> 16;
            it.steer = raw1.w != 0;
            __syncwarp();            // every lane has read the slot before it is refilled
            idx_next = item_index(++round);
            prefetch();
        } else {
            const int idx = item_index(round++);
            if (idx < 0) return false;
            if (p.pair_heads) {
                const int per_qt = p.B * (p.Hq >> 1);
                const int qt = p.n_qt - 1 - (int)((unsigned)idx / (unsigned)per_qt);
                const int rem = (int)((unsigned)idx % (unsigned)per_qt);
                it.b = rem / (p.Hq >> 1);
                const int hp = rem % (p.Hq >> 1);
                it.hqA = 2 * hp; it.hqB = 2 * hp + 1;
                it.qtA = it.qtB = qt;
            } else {
                const int per_qt = p.B * p.Hq;
                const int qt2 = ((p.n_qt + 1) >> 1) - 1 - (int)((unsigned)idx / (unsigned)per_qt);
                const int rem = (int)((unsigned)idx % (unsigned)per_qt);
                it.b = rem / p.Hq;
                it.hqA = it.hqB = rem % p.Hq;
                it.qtA = 2 * qt2; it.qtB = 2 * qt2 + 1;
            }
            it.hkv = it.hqA / (p.Hq / p.Hkv);
            it.seq0 = it.b * p.L;       // fixed length: every slot holds work (tile B of the last odd pair may not)
            it.Lb = p.L;
            it.nA = it.qtA * BM < it.Lb ? it.qtA + 1 : 0;
            it.nB = it.qtB * BM < it.Lb ? it.qtB + 1 : 0;
            it.steer = p.steer && p.gain[it.b] != 0.f && (p.head_enable == nullptr || p.head_enable[it.hkv] != 0);
        }
        it.n_kv = max(it.nA, it.nB);
        return true;
    };

    if (tid == 0) {
        mbar_init(q_full + 0, 1); mbar_init(q_full + 1, 1); mbar_init(k0_full, 1);
        for (int i = 0; i < NK; ++i) { mbar_init(kv_full + i, 1); mbar_init(kv_free + i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(s_full + i, 1); mbar_init(p_full + i, 5); mbar_init(p_last + i, 4); mbar_init(o_full + i, 1); }
        mbar_init(w_full, 1); mbar_init(e_full, 1); mbar_init(k_edited, 8);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    // Running counts shared by all roles (each keeps its own copy; they advance identically):
    //   ev   kv_free events so far (n_kv + 1 per item: after the first score products, then after every step)
    //   pr   V/K pairs so far (n_kv per item); pair t of an item uses V stage (pr + t) % NK and K stage (pr + t + 1) % NK
    //   cA/cB  steps of tile A / B so far (phases of s_full, p_full, p_last)
    Item it;

    if (warp < 4) {
        reg_dec<REGS_CTRL>();
        // The control warps run their loops with all 32 lanes and elect one lane only around the issuing
        // instructions: addresses, descriptors and barrier phases then stay warp-uniform values.
        const bool leader = elect_one();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            uint32_t ev = 0, pr = 0, n_it = 0, n_qb = 0;
            int prev_n = 0;
            bool ok = true;
            while (ok && next_item(it)) {
                // Q, W and the first K of an item may land once the last score product of the previous item is
                // done (event n_kv - 1 of that item), its V/K pairs once its last step is done (event n_kv)
                if (n_it > 0) {
                    const uint32_t e = ev - 2;
                    ok = warp_wait(kv_free + e % NK, (e / NK) & 1, abort_flag, p.status, 12);
                    if (!ok) break;
                }
                if (leader) {
                    mbar_expect_tx(q_full + 0, SL::TILE);
#pragma unroll
                    for (int c = 0; c < NBLK; ++c)
                        tma_load_3d(smem + SL::Q + c * BLK_BYTES, &tmQ, q_full + 0, c * 64, it.hqA, it.seq0 + it.qtA * BM);
                    if (it.nB > 0) {
                        mbar_expect_tx(q_full + 1, SL::TILE);
#pragma unroll
                        for (int c = 0; c < NBLK; ++c)
                            tma_load_3d(smem + SL::Q + SL::TILE + c * BLK_BYTES, &tmQ, q_full + 1, c * 64, it.hqB, it.seq0 + it.qtB * BM);
                    }
                    mbar_expect_tx(k0_full, SL::TILE);
#pragma unroll
                    for (int c = 0; c < NBLK; ++c)
                        tma_load_3d(smem + SL::K + (pr % NK) * SL::TILE + c * BLK_BYTES, &tmK, k0_full, c * 64, it.hkv, it.seq0);
                    if (it.steer) {
                        mbar_expect_tx(w_full, NBLK * SL::WBLK);
#pragma unroll
                        for (int c = 0; c < NBLK; ++c)
                            tma_load_3d(smem + SL::W + c * SL::WBLK, &tmW, w_full, c * 64, 0, (it.b * p.Hkv + it.hkv) * D);
                    }
                }
                __syncwarp();
                if (n_it > 0) {
                    const uint32_t e = ev - 1;
                    ok = warp_wait(kv_free + e % NK, (e / NK) & 1, abort_flag, p.status, 13);
                    if (!ok) break;
                }
                // V(t) and K(t+1) travel as a pair: both of their stages are released by the same event, the end
                // of step t - NK of the MMA issuer (event t - NK + 1 of this item)
#pragma unroll 1
                for (int t = 0; t < it.n_kv; ++t) {
                    if (t >= NK - 1) {
                        const uint32_t e = ev + (uint32_t)(t - NK + 1);
                        ok = warp_wait(kv_free + e % NK, (e / NK) & 1, abort_flag, p.status, 10);
                        if (!ok) break;
                    }
                    if (leader) {
                        const bool more = t + 1 < it.n_kv;
                        uint64_t* bar = kv_full + (pr + t) % NK;
                        mbar_expect_tx(bar, more ? 2 * SL::TILE : SL::TILE);
#pragma unroll
                        for (int c = 0; c < NBLK; ++c)
                            tma_load_3d(smem + SL::V + ((pr + t) % NK) * SL::TILE + c * BLK_BYTES, &tmV, bar, c * 64, it.hkv, it.seq0 + t * BN);
                        if (more) {
#pragma unroll
                            for (int c = 0; c < NBLK; ++c)
                                tma_load_3d(smem + SL::K + ((pr + t + 1) % NK) * SL::TILE + c * BLK_BYTES, &tmK, bar, c * 64, it.hkv,
                                            it.seq0 + (t + 1) * BN);
                        }
                    }
                    __syncwarp();
                }
                ev += it.n_kv + 1; pr += it.n_kv; ++n_it; prev_n = it.n_kv;
                if (it.nB > 0) ++n_qb;
            }
            (void)prev_n; (void)n_qb;
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            constexpr uint32_t IDESC_S = umma_idesc_bf16(BN, false);
            constexpr uint32_t IDESC_PV = umma_idesc_bf16(D, true);
            constexpr uint32_t IDESC_E = umma_idesc_bf16(D, false);
            constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
            const uint32_t dQ = umma_desc_lo(smem_u32(smem + SL::Q), 16), dK = umma_desc_lo(smem_u32(smem + SL::K), 16);
            const uint32_t dV = umma_desc_lo(smem_u32(smem + SL::V), BLK_BYTES);
            const uint32_t dW = umma_desc_lo(smem_u32(smem + SL::W), 16);
            uint32_t ev = 0, pr = 0, n_it = 0, n_qb = 0, n_w = 0, n_ob[2] = {0, 0};
            uint32_t cx[2] = {0, 0};      // steps of tile A / B so far
            uint32_t n_hot = 0;           // highlighted tiles edited so far (phase of e_full / k_edited)
            bool ok = true;
            auto commit = [&](uint64_t* bar) {
                if (leader) umma_commit(bar);
                __syncwarp();
            };
            while (ok && next_item(it)) {
                const uint8_t* hot_g = p.tile_hot + (size_t)it.b * p.n_qt;
                bool w_seen = false;
                // Before the first score product of key tile j (by tile x): if the tile holds highlighted tokens,
                // dK = K W goes into the score columns of tile x (idle between P_x V and the next S_x), the editors
                // add it to the staged tile, and only then may the tile be multiplied.
                auto edit_K = [&](int x, int j, bool is_hot) {
                    if (!is_hot) return;
                    if (!w_seen) { ok = warp_wait(w_full, n_w & 1, abort_flag, p.status, 31); w_seen = true; }
                    if (!ok) return;
                    const uint32_t kd = dK + ((pr + (uint32_t)j) % NK) * (SL::TILE >> 4);
                    const uint32_t dst = tmem_base + (EDIT_OWN_COLS ? COL_E : COL_S + 128 * x);
                    tc_fence_after();
                    if (leader) {
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            const uint32_t offk = ((uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32) >> 4;
                            const uint32_t offw = ((uint32_t)(ks >> 2) * SL::WBLK + (uint32_t)(ks & 3) * 32) >> 4;
                            umma_ss(dst, kd + offk, DESC_HI, dW + offw, DESC_HI, IDESC_E, ks > 0 ? 1u : 0u);
                        }
                        umma_commit(e_full);
                    }
                    __syncwarp();
                };
                // ... and the wait for the rows to be updated, kept apart: with columns of its own the product can be
                // issued a good while before the edited tile is needed
                auto edit_done = [&]() {
                    ok = warp_wait(k_edited, n_hot & 1, abort_flag, p.status, 32);
                    ++n_hot;
                };
                auto issue_S = [&](int x, int j) {
                    const uint32_t kd = dK + ((pr + (uint32_t)j) % NK) * (SL::TILE >> 4), qd = dQ + (uint32_t)x * (SL::TILE >> 4);
                    const uint32_t dst = tmem_base + COL_S + 128 * x;
                    tc_fence_after();
                    if (leader) {
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            // 16 elements along the contraction = 32 bytes inside a 64-element block
                            const uint32_t off = ((uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32) >> 4;
                            umma_ss(dst, qd + off, DESC_HI, kd + off, DESC_HI, IDESC_S, ks > 0 ? 1u : 0u);
                        }
                        umma_commit(s_full + x);
                    }
                    __syncwarp();
                };
                // P V of tile x and key tile j, key blocks [ks0, ks1) of 16 keys (2048 bytes of the V tile, 8 columns of P)
                auto issue_PV = [&](int x, int j, int ks0, int ks1, bool last) {
                    const uint32_t vd = dV + ((pr + (uint32_t)j) % NK) * (SL::TILE >> 4);
                    const uint32_t dst = tmem_base + COL_O + D * x, src = tmem_base + COL_S + 128 * x;
                    tc_fence_after();
                    if (leader) {
#pragma unroll
                        for (int ks = 0; ks < BN / 16; ++ks)
                            if (ks >= ks0 && ks < ks1)
                                umma_ts(dst, src + (uint32_t)ks * 8, vd + (uint32_t)ks * (2048 >> 4), DESC_HI, IDESC_PV,
                                        (j > 0 || ks > 0) ? 1u : 0u);
                        if (last) umma_commit(o_full + x);
                    }
                    __syncwarp();
                };
                const int nA = it.nA, nB = it.nB, n_kv = it.n_kv;
                // highlight flags of key tiles 0 and 1 (later ones are fetched one step ahead of their use)
                bool hot_cur = it.steer && hot_g[0] != 0;
                bool hot_nxt = it.steer && n_kv > 1 && hot_g[1] != 0;
                // One thread issues for both tiles, in a fixed order (A then B in every step): the in-order tensor
                // pipe then keeps the two tiles half a period apart (softmax of one tile under the MMAs of the other).
                ok = warp_wait(q_full + 0, n_it & 1, abort_flag, p.status, 20);
                if (ok && nB > 0) ok = warp_wait(q_full + 1, n_qb & 1, abort_flag, p.status, 21);
                if (ok) ok = warp_wait(k0_full, n_it & 1, abort_flag, p.status, 22);
                if (ok && hot_cur) { edit_K(0, 0, true); if (ok) edit_done(); }
                if (ok) {
                    issue_S(0, 0);
                    if (nB > 0) issue_S(1, 0);
                    // The edit operator of this item is seen here at the latest, before the event that lets the
                    // producer load the next item's: a barrier that ran two phases ahead of its waiter would
                    // never look complete to it.
                    if (it.steer && !w_seen) { ok = warp_wait(w_full, n_w & 1, abort_flag, p.status, 35); w_seen = true; }
                    commit(kv_free + ev % NK);
                    ++ev;
                }
#pragma unroll 1
                for (int j = 0; j < n_kv && ok; ++j) {
                    const int j1 = j + 1;
                    const bool hot_j1 = hot_nxt;
                    hot_nxt = it.steer && j + 2 < n_kv && hot_g[j + 2] != 0;
                    // V of this step and K of the next have landed once p_full completes: the relay warp vouches
                    // for them there, so this warp has no waits of its own for operands (every wait here is a
                    // bubble in the tensor pipe: its queue is only a couple of MMAs deep)
                    if (j < nA) {
                        ok = warp_wait(p_full + 0, (cx[0] + j) & 1, abort_flag, p.status, 24);
                        if (!ok) break;
                        if (EDIT_OWN_COLS && hot_j1 && j1 < nA) edit_K(0, j1, true);      // K(j1) has landed (the relay vouches), P_A V hides the drain
                        if (!ok) break;
                        issue_PV(0, j, 0, 6, false);
                        ok = warp_wait(p_last + 0, (cx[0] + j) & 1, abort_flag, p.status, 28);
                        if (!ok) break;
                        issue_PV(0, j, 6, 8, j == nA - 1);
                        if (j1 < nA) {
                            if (hot_j1) {
                                if (!EDIT_OWN_COLS) edit_K(0, j1, true);
                                if (ok) edit_done();
                            }
                            if (!ok) break;
                            issue_S(0, j1);
                        }
                    }
                    if (j < nB) {
                        ok = warp_wait(p_full + 1, (cx[1] + j) & 1, abort_flag, p.status, 26);
                        if (!ok) break;
                        issue_PV(1, j, 0, 6, false);
                        ok = warp_wait(p_last + 1, (cx[1] + j) & 1, abort_flag, p.status, 29);
                        if (!ok) break;
                        issue_PV(1, j, 6, 8, j == nB - 1);
                    }
                    if (j1 < nB) {
                        if (j1 >= nA && hot_j1) {      // tile A does not use this key tile: B is its first user
                            edit_K(1, j1, true);
                            if (ok) edit_done();
                        }
                        if (!ok) break;
                        issue_S(1, j1);
                    }
                    commit(kv_free + ev % NK);      // K(j+1) and V(j) may be overwritten
                    ++ev;
                }
                pr += n_kv; cx[0] += nA; cx[1] += nB; ++n_it;
                if (nB > 0) ++n_qb;
                if (it.steer) ++n_w;
            }
            (void)n_ob;
        } else if (warp == 2) {
            // ------------------------------------------------------------ operand relay: "V(j) and K(j+1) have landed" as a
            // fifth arrival on p_full of step j, so that the MMA issuer waits on one barrier per hand-off
            uint32_t pr = 0, cx[2] = {0, 0};
            bool ok = true;
            while (ok && next_item(it)) {
#pragma unroll 1
                for (int j = 0; j < it.n_kv; ++j) {
                    const uint32_t g = pr + j;
                    ok = warp_wait(kv_full + g % NK, (g / NK) & 1, abort_flag, p.status, 23);
                    if (!ok) break;
                    if (lane == 0) {
                        if (j < it.nA) mbar_arrive(p_full + 0);
                        if (j < it.nB) mbar_arrive(p_full + 1);
                    }
                    __syncwarp();
                    // stay within the phase: the next arrival may only come after this phase has completed
                    if (j < it.nA) ok = warp_wait(p_full + 0, (cx[0] + j) & 1, abort_flag, p.status, 33);
                    if (ok && j < it.nB) ok = warp_wait(p_full + 1, (cx[1] + j) & 1, abort_flag, p.status, 34);
                    if (!ok) break;
                }
                pr += it.n_kv; cx[0] += it.nA; cx[1] += it.nB;
            }
        }
    } else if (warp >= 12) {
        // ------------------------------------------------------------ key editors: one key row of the staged tile per thread
        reg_dec<REGS_EDIT>();
        const int row = (warp - 12) * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)((warp - 12) * 32) << 16);
        uint32_t pr = 0, n_hot = 0;
        bool ok = true;
        while (ok && next_item(it)) {
            if (it.steer) {
                const uint8_t* hot_g = p.tile_hot + (size_t)it.b * p.n_qt;
#pragma unroll 1
                for (int j = 0; j < it.n_kv; ++j) {
                    if (hot_g[j] == 0) continue;
                    const int kpos = j * BN + row;
                    const bool hl = kpos < it.Lb && p.mask[it.seq0 + kpos] != 0;
                    ok = warp_wait(e_full, n_hot & 1, abort_flag, p.status, 30);
                    if (!ok) break;
                    ++n_hot;
                    tc_fence_after();
                    const uint32_t tE = t_lane + (EDIT_OWN_COLS ? COL_E : COL_S + 128 * (j < it.nA ? 0 : 1));
                    uint8_t* sK = smem + SL::K + ((pr + (uint32_t)j) % NK) * SL::TILE;
                    drain_edit(tE, sK, row, hl, 0, D / 64);      // the other half of the columns is taken by the idle softmax warps
                    fence_proxy_async();       // the rewritten rows are read next by the tensor core
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(k_edited);
                }
            }
            pr += it.n_kv;
        }
    } else {
        // ------------------------------------------------------------ softmax of tile x, one query row per thread
        reg_inc<REGS_SOFTMAX>();
        const int x = (warp - 4) >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t tS = t_lane + COL_S + 128 * x, tO = t_lane + COL_O + D * x;
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        uint32_t cX = 0, n_o = 0;       // steps and items of this tile so far
        uint32_t pr = 0, n_hot = 0;     // V/K pairs and highlighted key tiles so far (all items)
        bool ok = true;
        while (ok && next_item(it)) {
            const int nX = x ? it.nB : it.nA;
            const int hqX = x ? it.hqB : it.hqA, qtX = x ? it.qtB : it.qtA;
            const uint8_t* hot_g = p.tile_hot + (size_t)it.b * p.n_qt;
            // Every softmax warp waits for dK of EVERY highlighted key tile, in order, whether or not it helps to drain
            // it: a warp that skipped a phase of e_full could find its next phase "complete" while the skipped one is
            // still running (a parity wait only tells the current phase from the one before).  The waits cost nothing:
            // the scores a warp needs next are issued after the edit anyway.
            auto see_edit = [&](int j0, int j1) {
                for (int j = j0; j < j1 && ok; ++j) {
                    if (hot_g[j] == 0) continue;
                    ok = warp_wait(e_full, n_hot & 1, abort_flag, p.status, 38);
                    ++n_hot;
                }
            };
            if (nX == 0) {      // tile B lies beyond the sequence: only the counts move
                if (it.steer) see_edit(0, it.n_kv);
                pr += it.n_kv;
                if (!ok) break;
                continue;
            }
            float m_run = -INFINITY, l_run = 0.f;
#pragma unroll 1
            for (int j = 0; j < nX; ++j) {
                // Key tile j holds highlighted tokens and this tile is the first to use it: while waiting for its
                // scores anyway, these warps add the upper half of the columns of dK to the staged K tile (the
                // key editors take the lower half).  Every softmax warp counts the highlighted tiles.
                if (it.steer && hot_g[j] != 0) {
                    ok = warp_wait(e_full, n_hot & 1, abort_flag, p.status, 36 + x);
                    if (!ok) break;
                    if ((j < it.nA ? 0 : 1) == x) {
                        const int kpos = j * BN + row;
                        const bool hl = kpos < it.Lb && p.mask[it.seq0 + kpos] != 0;
                        tc_fence_after();
                        drain_edit(EDIT_OWN_COLS ? t_lane + COL_E : tS, smem + SL::K + ((pr + (uint32_t)j) % NK) * SL::TILE, row, hl, D / 64, D / 32);
                        fence_proxy_async();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(k_edited);
                    }
                    ++n_hot;
                }
                ok = warp_wait(s_full + x, (cX + j) & 1, abort_flag, p.status, 40 + x);
                if (!ok) break;
                tc_fence_after();
                // the whole score row of this thread: 128 fp32 values in registers
                uint32_t v[128];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, reinterpret_cast<uint32_t(&)[32]>(v[32 * c]));
                tmem_wait_ld();
                if (j == nX - 1) {       // diagonal tile: keys after the query are masked
#pragma unroll
                    for (int e = 0; e < 128; ++e)
                        if (e > row) v[e] = 0xff800000u;
                }
                float mx[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    mx[q] = fmaxf(__uint_as_float(v[16 * q]), __uint_as_float(v[16 * q + 1]));
#pragma unroll
                    for (int e = 2; e < 16; e += 2) mx[q] = max3(mx[q], __uint_as_float(v[16 * q + e]), __uint_as_float(v[16 * q + e + 1]));
                }
                const float mx_all = fmaxf(max3(mx[0], mx[1], mx[2]), max3(mx[3], mx[4], max3(mx[5], mx[6], mx[7])));
                const float m_new = fmaxf(m_run, mx_all * p.scale_log2);
                // raise the running maximum only when it moved a lot; p may then exceed 1 (up to 2^8), which is harmless
                const bool raise = (m_new - m_run) > LAZY_RESCALE_LOG2;      // true on the first tile (m_run = -inf)
                const float factor = raise ? fast_exp2(m_run - m_new) : 1.f;
                if (raise) m_run = m_new;
                if (j > 0 && __any_sync(0xffffffffu, raise)) {
                    uint32_t o[32];
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        tmem_ld32(tO + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
                        tmem_st32(tO + c * 32, o);
                    }
                }
                const float2 nm2 = make_float2(-m_run, -m_run);
                float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk16[16];
#pragma unroll
                    for (int e2 = 0; e2 < 16; ++e2) {
                        const int e = 32 * c + 2 * e2;
                        const float2 arg = __ffma2_rn(make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), sc2, nm2);
                        float2 pe;
                        if ((POLY_PAIR_MASK >> e2) & 1u) {
                            pe = exp2_poly2(arg);
                        } else {
                            pe.x = fast_exp2(arg.x);
                            pe.y = fast_exp2(arg.y);
                        }
                        sum[e2 & 1] = __fadd2_rn(sum[e2 & 1], pe);
                        pk16[e2] = pack_bf16(pe.x, pe.y);
                    }
                    tmem_st16(tS + c * 16, pk16);     // P (bf16 pairs) over score columns that are already in registers
                    if (c == 2) {                     // keys 0-95 are in place: the tensor core may start on them
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(p_full + x);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_last + x);
                const float2 s2 = __fadd2_rn(sum[0], sum[1]);
                l_run = l_run * factor + (s2.x + s2.y);
            }
            cX += nX; pr += it.n_kv;
            if (ok) ok = warp_wait(o_full + x, n_o & 1, abort_flag, p.status, 44 + x);
            ++n_o;
            if (ok) {
                // final normalisation and store; the next item's first P_x (hence its first P_x V into these
                // columns) comes from these same threads, after they are done reading here
                tc_fence_after();
                const int qpos = qtX * BM + row;
                const bool valid = qpos < it.Lb;
                const size_t orow = (size_t)(it.seq0 + (valid ? qpos : 0)) * p.Hq + hqX;
                const float inv = 1.f / l_run;
                uint32_t o[32];
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
                    if (valid) store_chunk32<OutT>(static_cast<OutT*>(p.O) + orow * D + c * 32, o, inv);
                }
                if (valid && p.lse != nullptr) p.lse[orow] = (m_run + log2f(l_run)) * 0.6931471805599453f;
                tc_fence_before();
            }
            // highlighted tiles that only the other tile uses are seen too (after the output is on its way)
            if (it.steer && ok) see_edit(nX, it.n_kv);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (*abort_flag && lane == 0) {
            // let tile loads that may still be in flight land before the shared memory is released
            int dummy = 0;
            for (int i = 0; i < NK; ++i) { mbar_wait(kv_full + i, 0, &dummy, nullptr, 0); }
        }
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
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

// bf16 tensor [T, H, d] viewed as (d, H, T); tiles of 64 x 1 x box_rows with the 128-byte swizzle.
bool make_tile_map(CUtensorMap* m, const void* base, int d, int H, long long T, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)H * d * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, typename OutT, bool TABLE>
static seka_status launch_attn_t(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                 const CUtensorMap& tw, const AttnParams& p, cudaStream_t st) {
    using SL = SmemLayout<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(seka_attn_fwd_kernel<D, OutT, TABLE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)SL::DYN_BYTES) != cudaSuccess) return SEKA_ERR_CUDA;
        configured = true;
    }
    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm <= 0) { n_sm = 0; return SEKA_ERR_CUDA; }
    }
    // persistent CTAs, one per SM (the kernel needs the whole SM: all of tensor memory and most of shared memory)
    const unsigned grid = (unsigned)(p.n_items_max < (long long)n_sm ? p.n_items_max : (long long)n_sm);
    seka_attn_fwd_kernel<D, OutT, TABLE><<<grid, NTHREADS, SL::DYN_BYTES, st>>>(tq, tk, tv, tw, p);
    ++g_launches;
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

template <int D, typename OutT>
static seka_status launch_attn(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const CUtensorMap& tw, const AttnParams& p, cudaStream_t st) {
    return p.cu_seqlens != nullptr ? launch_attn_t<D, OutT, true>(tq, tk, tv, tw, p, st)
                                   : launch_attn_t<D, OutT, false>(tq, tk, tv, tw, p, st);
}

// The fused forward behind both entry points: coefficients either given (`alpha`, may be null) or, with `sigma`
// set, routed inside the preparation launch (Eq. 6) and reported through `alpha_out`.
static seka_status attention_fwd_impl(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                      void* O, float* lse, const uint8_t* mask, const float* U,
                                      const float* alpha, const float* sigma, int k_route, float* alpha_out,
                                      const float* gain, const uint8_t* head_enable,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    seka_status stc = validate_shape(shape);
    if (stc != SEKA_OK) return stc;
    const int T = shape_total_tokens(shape);
    if (T == 0 || shape->batch == 0 || shape->max_seqlen == 0) return SEKA_OK;
    if (!Q || !K || !V || !O) return SEKA_ERR_INVALID_ARG;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15) return SEKA_ERR_INVALID_ARG;
    const bool steer = mask != nullptr && U != nullptr;
    if (steer && !gain) return SEKA_ERR_INVALID_ARG;
    const WorkspaceLayout w = workspace_layout(shape);
    if (w.n_tiles > 32767 || shape->n_q_heads > 32767 || w.n_items_max > 0x7fffffffLL) return SEKA_ERR_UNSUPPORTED;   // item records pack 15-bit fields
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
    void* W = ws + w.w_off;
    uint8_t* tile_hot = reinterpret_cast<uint8_t*>(ws + w.hot_off);
    if (steer) launch_prep_steering(shape, U, alpha, gain, head_enable, mask, W, tile_hot, w.n_tiles, st, Q, sigma, k_route, alpha_out);

    CUtensorMap tq, tk, tv, tw;
    if (!make_tile_map(&tq, q16, D, Hq, T) || !make_tile_map(&tk, k16, D, Hkv, T) || !make_tile_map(&tv, v16, D, Hkv, T) ||
        !make_tile_map(&tw, W, D, 1, (long long)shape->batch * Hkv * D, D))
        return SEKA_ERR_CUDA;

    AttnParams p;
    p.O = O; p.lse = lse; p.mask = mask; p.gain = gain; p.head_enable = head_enable;
    p.cu_seqlens = shape->cu_seqlens; p.tile_hot = tile_hot; p.status = reinterpret_cast<int*>(ws);
    p.B = shape->batch; p.L = shape->max_seqlen; p.Hq = Hq; p.Hkv = Hkv;
    p.n_qt = w.n_tiles; p.steer = steer ? 1 : 0;
    ItemRecord* items = reinterpret_cast<ItemRecord*>(ws + w.item_off);
    if (shape->cu_seqlens != nullptr)
        launch_build_items(shape, w, steer, gain, head_enable, items, reinterpret_cast<int*>(ws) + 3, st);
    p.pair_heads = w.pair_heads;
    p.items = items; p.n_items = reinterpret_cast<int*>(ws) + 3; p.n_items_max = w.n_items_max;
    const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;

    if (D == 128) {
        return shape->dtype == SEKA_F32 ? launch_attn<128, float>(tq, tk, tv, tw, p, st)
                                        : launch_attn<128, __nv_bfloat16>(tq, tk, tv, tw, p, st);
    }
    return shape->dtype == SEKA_F32 ? launch_attn<64, float>(tq, tk, tv, tw, p, st)
                                    : launch_attn<64, __nv_bfloat16>(tq, tk, tv, tw, p, st);
}

}  // namespace seka

extern "C" seka_status seka_attention_fwd(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                          void* O, float* lse, const uint8_t* mask, const float* U,
                                          const float* alpha, const float* gain, const uint8_t* head_enable,
                                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return seka::attention_fwd_impl(shape, Q, K, V, O, lse, mask, U, alpha, nullptr, 0, nullptr, gain, head_enable,
                                    workspace, workspace_bytes, cuda_stream);
}

extern "C" seka_status seka_attention_fwd_routed(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                                 void* O, float* lse, const uint8_t* mask, const float* U,
                                                 const float* sigma, int32_t k_route, float* alpha_out,
                                                 const float* gain, const uint8_t* head_enable,
                                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (shape == nullptr || mask == nullptr || U == nullptr || sigma == nullptr) return SEKA_ERR_INVALID_ARG;
    if (k_route < 0 || k_route > shape->rank) return SEKA_ERR_INVALID_ARG;
    if (k_route == 0) k_route = shape->rank;
    return seka::attention_fwd_impl(shape, Q, K, V, O, lse, mask, U, nullptr, sigma, k_route, alpha_out, gain,
                                    head_enable, workspace, workspace_bytes, cuda_stream);
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
