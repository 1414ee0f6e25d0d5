// Fused SEKA / AdaSEKA steered causal GQA attention forward for sm_100a.
//
// The edited logit of Eq. 5 is q.k' = q.k + q.(g P k).  A small preparation launch leaves the edited keys k' of every
// key tile that holds a highlighted token in a side buffer as a high and a low bf16 part (see SteerPlan); this kernel
// stages such a tile from the high parts instead of from K and, where the gain is large enough for the rounding of k'
// to matter, extends the score product S = Q K'^T on the tensor core, in the same tensor-memory accumulator, by the
// contraction with the low parts, so that the logits are those of the fp32 k'.  The score matrix never reaches memory;
// K and V are read only.
//
// One CTA (16 warps) owns two tiles of 128 queries that share a KV head ("A" and "B": two query heads of one group at
// the same rows, or two consecutive row tiles of one head when the group size is odd) and walks the key tiles
// 0 .. diagonal.  Warp roles:
//   warp 0        TMA producer: Q tiles, then K (or edited-key) and V tiles (128-byte swizzle) through two
//                 shared-memory rings, throttled by "free" mbarriers the tensor core signals, and the low parts of
//                 edited tiles through a ring of their own;
//   warp 1        MMA issuer: S_x = Q_x K^T (+ the low-part steps) and O_x += P_x V on tcgen05 with all accumulators
//                 in tensor memory (S_A, S_B, O_A, O_B = 512 columns); P_x is read from tensor memory;
//   warp 2        operand relay: tells the issuer when the operands have landed, so that it waits on one barrier per
//                 hand-off;
//   warps 4-7 / 8-11  softmax of tile A / B, one query row per thread: causal mask on the diagonal tile, online
//                 softmax in base 2 with a lazily updated running maximum, P written back as bf16 over the consumed
//                 score columns, O rescaled in tensor memory only when the maximum moved by more than 2^8; final
//                 normalisation and store.
// (Warps 3 and 12-15 only give their registers to the softmax warps.)
// While one tile's softmax runs, the tensor core works on the other tile.  Every wait is bounded: a wait that runs
// out raises the CTA's abort flag, every role leaves its loop, and the status word reports it.
#include <math.h>

#include <mutex>

#include "seka_kernels.h"

#ifndef SEKA_POLY_PAIR_MASK
#define SEKA_POLY_PAIR_MASK 0x0000u
#endif

namespace seka {

struct AttnParams {
    void* O;
    float* lse;
    const uint8_t* bh_info;       // [B, Hkv]: bit 0 the keys of this (sequence, KV head) are edited, bit 1 with the low parts
    const uint8_t* tile_hot;      // [B, n_qt]: key tile holds a highlighted token
    const int* first_hot;         // [B]: first such tile of the sequence
    int* status;
    const ItemRecord* items;      // item table (packed batches), heaviest first
    const int* n_items;           // its length (device word)
    Sched sched;
    SteerPlan plan;
    int steer;
    float scale_log2;
};

constexpr int BM = 128, BN = 128;
constexpr int NTHREADS = 512;
constexpr uint32_t BLK_BYTES = 128 * 128;   // one [128 x 64] bf16 block
constexpr float LAZY_RESCALE_LOG2 = 8.0f;   // the running maximum is only raised when it moved by more than this
// registers per thread after the roles split (the CTA owns the whole register file: 4 x 128 x (80+184+184+64) = 64 Ki)
constexpr int REGS_CTRL = 80, REGS_SOFTMAX = 184, REGS_PROJ = 64;   // PROJ: the idle fourth warpgroup
// which of the 16 element pairs of every 32-key chunk take the polynomial exp2 instead of the special-function unit
constexpr uint32_t POLY_PAIR_MASK = SEKA_POLY_PAIR_MASK;
constexpr uint32_t SMEM_LIMIT = 227 * 1024;


// Shared memory of one CTA.  Tiles first (each a multiple of 1024 bytes), then barriers and per-warp item slots.
template <int D>
struct Geo {
    static constexpr int NK = D == 128 ? 2 : 3;                    // K and V ring depth
    static constexpr uint32_t TILE = (D / 64) * BLK_BYTES;         // a [128 x D] tile
    static constexpr int NXMAX = 3;                                // most stages of the key-side operand
    static constexpr uint32_t NBARS = 14 + 2 * NK + NXMAX;
    // shared-memory copy of the per-(sequence, KV head) steering bytes and the per-sequence first highlighted tile
    // (what fits beside the tiles; larger batches look them up in global memory)
    static constexpr int INFO_HEADS = D == 128 ? 768 : 4096, INFO_SEQS = D == 128 ? 64 : 512;
    static constexpr uint32_t INFO_BYTES = INFO_HEADS + INFO_SEQS * 4;
};

struct SmemPlan {
    uint32_t k, v, x, xb, bars, misc, items, info, total;
};

template <int D>
__host__ __device__ inline SmemPlan smem_plan(const SteerPlan& sp) {
    using G = Geo<D>;
    SmemPlan s;
    s.k = 2 * G::TILE;
    s.v = s.k + G::NK * G::TILE;
    s.x = s.v + G::NK * G::TILE;
    s.xb = sp.mode ? G::TILE : 0u;                                  // one stage of low parts: [128 x D]
    s.bars = s.x + (uint32_t)sp.nx * s.xb;
    s.misc = s.bars + ((G::NBARS * 8 + 15) & ~15u);                 // 16-byte aligned: the item slots are filled by 16-byte async copies
    s.items = s.misc + 32;
    s.info = s.items + 16 * 32;                                     // steering info of every (sequence, KV head), if it fits
    s.total = s.info + (sp.mode ? G::INFO_BYTES : 0u);
    return s;
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

// One unit of work of a CTA: two 128-row query tiles that share a KV head of one sequence.
struct Item {
    int b, hkv, seq0, Lb;
    int hqA, hqB, qtA, qtB;     // query head and row-tile index of tile A / B
    int nA, nB, n_kv;           // key tiles of A / B (0: the tile lies beyond the sequence) and of the item
    bool steer;                 // the keys of this (sequence, KV head) are edited
    bool hot_any;               // ... and one of the item's key tiles holds a highlighted token
    bool need_lo;               // ... and the low parts of the edited keys are multiplied too
};

template <int D, typename OutT, bool TABLE>
__global__ void __launch_bounds__(NTHREADS, 1)
seka_attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmX,
                     const __grid_constant__ AttnParams p) {
    using G = Geo<D>;
    constexpr int NK = G::NK;
    constexpr int NBLK = D / 64;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t COL_S = 0, COL_O = 256;     // S_x at COL_S + 128 x, O_x at COL_O + D x
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const SmemPlan sl = smem_plan<D>(p.plan);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sl.bars);
    uint64_t* q_full = bars;                 // [2]   Q tile landed
    uint64_t* k0_full = q_full + 2;          // [1]   first key tile of the item landed
    uint64_t* kv_full = k0_full + 1;         // [NK]  V(t) and K(t+1) landed (they are loaded as a pair)
    uint64_t* kv_free = kv_full + NK;        // [NK]  one event per step: the tensor core is done with K(j+1) and V(j)
    uint64_t* x_full = kv_free + NK;         // [3]   low parts of an edited tile landed
    uint64_t* s_full = x_full + G::NXMAX;    // [2]   scores of tile x are in tensor memory
    uint64_t* p_full = s_full + 2;           // [2]   4 softmax-warp arrivals (O_x rescaled, keys 0-95 of P_x written) + 1 from the relay
    uint64_t* p_last = p_full + 2;           // [2]   4 softmax-warp arrivals: keys 96-127 of P_x written
    uint64_t* o_full = p_last + 2;           // [2]   last P V of tile x finished
    uint64_t* o_drained = o_full + 2;        // [2]   4 softmax-warp arrivals: O_x of the item has been read
    uint64_t* start_full = o_drained + 2;    // [1]   relay: Q tiles and first key tile of the item landed
    uint64_t* drain = start_full + 1;        // [1]   every product issued has finished
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sl.misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sl.misc + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // an earlier launch (or CTA) gave up on this workspace: nothing is started (every role finds `ok` false)
    const bool dead = __syncthreads_or(*reinterpret_cast<volatile int*>(p.status) != 0);
    const int hook_skip = p.status[4];
    const uint64_t limit_ns = p.status[5] > 0 ? (uint64_t)p.status[5] * 1000ull : kWaitLimitNs;
    // steering info is kept in shared memory when it fits (a look-up per work item then costs no trip to the caches)
    const bool info_local = p.steer && p.sched.B * p.sched.Hkv <= G::INFO_HEADS && p.sched.B <= G::INFO_SEQS;
    uint8_t* info_bh = smem + sl.info;
    int* info_first = reinterpret_cast<int*>(smem + sl.info + G::INFO_HEADS);

    // all lanes of a warp wait on the same barrier and then agree on the outcome
    auto warp_wait = [&](uint64_t* bar, uint32_t parity, int where) -> bool {
        const bool ok = mbar_wait_limit(bar, parity, abort_flag, p.status, where, limit_ns);
        return __all_sync(0xffffffffu, ok);
    };

    // The CTA is persistent: it walks its share of the items (heaviest first; odd rounds run the CTAs in
    // reverse so that the shares come out even).  Every role goes through the same sequence of items by itself.
    // Fixed-length batches decode the item from its index; packed variable-length batches, where many index
    // slots are empty (row tiles beyond a short sequence), read a table from which those were dropped.
    const int n_items = TABLE ? *p.n_items : (int)p.sched.n_items_max;
    auto item_index = [&](int round) -> int {
        const int NG = (int)gridDim.x;
        const long long idx = (long long)round * NG + ((round & 1) ? (NG - 1 - (int)blockIdx.x) : (int)blockIdx.x);
        return idx < n_items ? (int)idx : -1;
    };
    // (table) the record of the next item is copied into a per-warp slot of shared memory while the current item
    // runs, so that no registers are held for it; lane 0 issues the copy and waits for it
    int round = 0, idx_next = TABLE ? item_index(0) : 0;
    auto prefetch = [&]() {
        if (TABLE && idx_next >= 0 && lane == 0) {
            const uint32_t dst = smem_u32(smem + sl.items + warp * 32);
            const ItemRecord* rec = p.items + idx_next;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(rec) : "memory");
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst + 16), "l"(reinterpret_cast<const char*>(rec) + 16) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    };
    prefetch();
    // `steering`: also look up whether the item's keys are edited (only the producer and the MMA issuer need to know)
    auto next_item = [&](Item& it, bool steering = false) -> bool {
        ItemRecord rec;
        if (TABLE) {
            if (idx_next < 0) return false;
            const uint8_t* slot = smem + sl.items + warp * 32;
            if (lane == 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
            const int4 raw0 = *reinterpret_cast<const int4*>(slot), raw1 = *reinterpret_cast<const int4*>(slot + 16);
            rec.seq0 = raw0.x; rec.Lb = raw0.y; rec.bh = raw0.z; rec.hq = raw0.w;
            rec.qt = raw1.x; rec.n = raw1.y; rec.steer = raw1.z;
            __syncwarp();            // every lane has read the slot before it is refilled
            idx_next = item_index(++round);
            prefetch();
        } else {
            const int idx = item_index(round++);
            if (idx < 0) return false;
            decode_item(p.sched, idx, nullptr, rec);
            const int b = rec.bh & 0xffff, hkv = rec.bh >> 16;
            rec.steer = (steering && p.steer) ? (int)(info_local ? info_bh[b * p.sched.Hkv + hkv] : __ldg(p.bh_info + b * p.sched.Hkv + hkv)) : 0;
        }
        it.seq0 = rec.seq0; it.Lb = rec.Lb; it.b = rec.bh & 0xffff; it.hkv = rec.bh >> 16;
        it.hqA = rec.hq & 0xffff; it.hqB = rec.hq >> 16;
        it.qtA = rec.qt & 0xffff; it.qtB = rec.qt >> 16;
        it.nA = rec.n & 0xffff; it.nB = rec.n >> 16;
        it.n_kv = max(it.nA, it.nB);
        it.steer = steering && (rec.steer & 1) != 0 && p.plan.mode != 0;
        it.hot_any = it.steer && (info_local ? info_first[it.b] : __ldg(p.first_hot + it.b)) < it.n_kv;
        it.need_lo = it.hot_any && ((rec.steer & 2) != 0 || it.n_kv <= kLoTiles);
        return true;
    };

    if (tid == 0) {
        mbar_init(q_full + 0, 1); mbar_init(q_full + 1, 1); mbar_init(k0_full, 1);
        for (int i = 0; i < NK; ++i) { mbar_init(kv_full + i, 1); mbar_init(kv_free + i, 1); }
        for (int i = 0; i < G::NXMAX; ++i) mbar_init(x_full + i, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full + i, 1); mbar_init(p_full + i, 5); mbar_init(p_last + i, 4); mbar_init(o_full + i, 1);
            mbar_init(o_drained + i, 4);
        }
        mbar_init(start_full, 1); mbar_init(drain, 1);
        *abort_flag = dead ? 1 : 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
        if (p.plan.mode) tma_prefetch_desc(&tmX);
    }
    __syncwarp();
    if (warp == 0) { tmem_alloc(tmem_holder, TMEM_COLS); tmem_relinquish(); }
    // steering info into shared memory
    if (info_local) {
        for (int i = tid; i < p.sched.B * p.sched.Hkv; i += NTHREADS) info_bh[i] = p.bh_info[i];
        for (int i = tid; i < p.sched.B; i += NTHREADS) info_first[i] = p.first_hot[i];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    // Running counts shared by all roles (each keeps its own copy; they advance identically):
    //   n_it   items so far (phases of start_full, q_full[0], k0_full)
    //   n_o[x] items that had a tile x so far (phases of o_full, o_drained)
    //   n_qb   items with a tile B so far (phase of q_full[1])
    //   n_hot  edited key tiles whose low parts were loaded / used so far, over all items (stage and phase of x_full)
    //   ev     kv_free events so far (n_kv + 1 per item: after the first score products, then after every step);
    //          event j of an item covers the score products of its key tile j
    //   pr     V/K pairs so far (n_kv per item); pair t of an item uses V stage (pr + t) % NK and K stage (pr + t + 1) % NK
    //   cx[x]  steps of tile x so far (phases of s_full, p_full, p_last)
    Item it;

    if (warp < 4) {
        reg_dec<REGS_CTRL>();
        // The control warps run their loops with all 32 lanes and elect one lane only around the issuing
        // instructions: addresses, descriptors and barrier phases then stay warp-uniform values.
        const bool leader = elect_one();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer
            const int nx = p.plan.nx;
            const bool staged = p.plan.mode != 0;       // key tiles with highlighted tokens come from the side buffer
            uint32_t ev = 0, pr = 0, n_it = 0, n_qb = 0, n_hot = 0;
            uint32_t ev_seen = 0;            // events [0, ev_seen) are known to have completed
            uint32_t ev_hot[G::NXMAX] = {0, 0, 0};      // per stage of the key-side operand: event that releases it, + 1
            // parity + 1 of the last load armed on each barrier (0: none), for the teardown after an abort
            uint32_t armed_q[2] = {0, 0}, armed_k0 = 0, armed_kv[NK], armed_x[G::NXMAX] = {0, 0, 0};
#pragma unroll
            for (int i = 0; i < NK; ++i) armed_kv[i] = 0;
            bool ok = !dead;
            auto see_event = [&](uint32_t e, int where) {        // events complete in order
                if (e < ev_seen) return;
                ok = warp_wait(kv_free + e % NK, (e / NK) & 1, where);
                ev_seen = e + 1;
            };
            // low parts of the edited key tile j of the item (event `e` covers its score products) into the next stage
            auto load_x = [&](int j, uint32_t e) {
                uint32_t st = 0, prev = 0;
#pragma unroll
                for (int i = 0; i < G::NXMAX; ++i)
                    if ((int)(n_hot % (uint32_t)nx) == i) { st = i; prev = ev_hot[i]; ev_hot[i] = e + 1; }
                if (prev) see_event(prev - 1, 14);       // the tile that used this stage before is through the tensor core
                if (!ok) return;
                if (leader) {
                    mbar_expect_tx(x_full + st, sl.xb);
#pragma unroll
                    for (int c = 0; c < NBLK; ++c)
                        tma_load_3d(smem + sl.x + st * sl.xb + c * BLK_BYTES, &tmX, x_full + st, D + c * 64, it.hkv, it.seq0 + j * BN);
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < G::NXMAX; ++i)
                    if ((int)st == i) armed_x[i] = ((n_hot / (uint32_t)nx) & 1) + 1;
                ++n_hot;
            };
            while (ok && next_item(it, true)) {
                const uint8_t* hot_g = p.tile_hot + (size_t)it.b * p.sched.n_qt;
                // Q and the first K of an item may land once the last score product of the previous item is
                // done (event n_kv - 1 of that item), its V/K pairs once its last step is done (event n_kv)
                if (n_it > 0) {
                    see_event(ev - 2, 12);
                    if (!ok) break;
                }
                if (leader) {
                    mbar_expect_tx(q_full + 0, G::TILE);
#pragma unroll
                    for (int c = 0; c < NBLK; ++c)
                        tma_load_3d(smem + c * BLK_BYTES, &tmQ, q_full + 0, c * 64, it.hqA, it.seq0 + it.qtA * BM);
                    if (it.nB > 0) {
                        mbar_expect_tx(q_full + 1, G::TILE);
#pragma unroll
                        for (int c = 0; c < NBLK; ++c)
                            tma_load_3d(smem + G::TILE + c * BLK_BYTES, &tmQ, q_full + 1, c * 64, it.hqB, it.seq0 + it.qtB * BM);
                    }
                    mbar_expect_tx(k0_full, G::TILE);
                    const CUtensorMap* km0 = (staged && it.hot_any && hot_g[0] != 0) ? &tmX : &tmK;
#pragma unroll
                    for (int c = 0; c < NBLK; ++c)
                        tma_load_3d(smem + sl.k + (pr % NK) * G::TILE + c * BLK_BYTES, km0, k0_full, c * 64, it.hkv, it.seq0);
                }
                __syncwarp();
                armed_q[0] = (n_it & 1) + 1; armed_k0 = (n_it & 1) + 1;
                if (it.nB > 0) { armed_q[1] = (n_qb & 1) + 1; ++n_qb; }
                if (it.need_lo && hot_g[0] != 0) {
                    load_x(0, ev);
                    if (!ok) break;
                }
                if (n_it > 0) {
                    see_event(ev - 1, 13);
                    if (!ok) break;
                }
                // V(t) and K(t+1) travel as a pair: both of their stages are released by the same event, the end
                // of step t - NK of the MMA issuer (event t - NK + 1 of this item)
#pragma unroll 1
                for (int t = 0; t < it.n_kv; ++t) {
                    if (t >= NK - 1) {
                        see_event(ev + (uint32_t)(t - NK + 1), 10);
                        if (!ok) break;
                    }
                    const bool more = t + 1 < it.n_kv;
                    const bool hot_n = more && it.hot_any && hot_g[t + 1] != 0;
                    const uint32_t g = pr + (uint32_t)t;
                    // (test hook: one pair of the first item of CTA 0 is left out altogether, so that its wait runs out)
                    const bool skip = hook_skip > 0 && n_it == 0 && blockIdx.x == 0 && t + 1 == hook_skip;
                    if (leader && !skip) {
                        uint64_t* bar = kv_full + g % NK;
                        mbar_expect_tx(bar, more ? 2 * G::TILE : G::TILE);
#pragma unroll
                        for (int c = 0; c < NBLK; ++c)
                            tma_load_3d(smem + sl.v + (g % NK) * G::TILE + c * BLK_BYTES, &tmV, bar, c * 64, it.hkv, it.seq0 + t * BN);
                        if (more) {
                            const CUtensorMap* km = (staged && hot_n) ? &tmX : &tmK;
#pragma unroll
                            for (int c = 0; c < NBLK; ++c)
                                tma_load_3d(smem + sl.k + ((g + 1) % NK) * G::TILE + c * BLK_BYTES, km, bar, c * 64, it.hkv,
                                            it.seq0 + (t + 1) * BN);
                        }
                    }
                    __syncwarp();
                    if (!skip) {
#pragma unroll
                        for (int i = 0; i < NK; ++i)
                            if ((int)(g % NK) == i) armed_kv[i] = ((g / NK) & 1) + 1;
                    }
                    if (hot_n && it.need_lo) {
                        load_x(t + 1, ev + (uint32_t)(t + 1));
                        if (!ok) break;
                    }
                }
                ev += it.n_kv + 1; pr += it.n_kv; ++n_it;
            }
            if (*abort_flag) {
                // loads that were armed may still be in flight: let them land before the shared memory is released
                auto settle = [&](uint64_t* bar, uint32_t armed) {
                    if (armed) mbar_wait_limit(bar, armed - 1, nullptr, nullptr, 0, limit_ns);
                };
                settle(q_full + 0, armed_q[0]); settle(q_full + 1, armed_q[1]); settle(k0_full, armed_k0);
#pragma unroll
                for (int i = 0; i < NK; ++i) settle(kv_full + i, armed_kv[i]);
#pragma unroll
                for (int i = 0; i < G::NXMAX; ++i) settle(x_full + i, armed_x[i]);
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------ MMA issuer
            constexpr uint32_t IDESC_S = umma_idesc_bf16(BN, false);
            constexpr uint32_t IDESC_PV = umma_idesc_bf16(D, true);
            constexpr uint32_t DESC_HI = umma_desc_hi_sw128(1024);
            const uint32_t dQ = umma_desc_lo(smem_u32(smem), 16), dK = umma_desc_lo(smem_u32(smem + sl.k), 16);
            const uint32_t dX = umma_desc_lo(smem_u32(smem + sl.x), 16);
            const uint32_t dV = umma_desc_lo(smem_u32(smem + sl.v), BLK_BYTES);
            const uint32_t nx = p.plan.nx > 0 ? (uint32_t)p.plan.nx : 1u;
            uint32_t ev = 0, pr = 0, n_it = 0, n_hot = 0;
            uint32_t cx[2] = {0, 0};      // steps of tile A / B so far
            uint32_t n_o[2] = {0, 0};     // items that had a tile A / B so far
            bool ok = !dead;
            auto commit = [&](uint64_t* bar) {
                if (leader) umma_commit(bar);
                __syncwarp();
            };
            while (ok && next_item(it, true)) {
                const uint8_t* hot_g = p.tile_hot + (size_t)it.b * p.sched.n_qt;
                const int nA = it.nA, nB = it.nB, n_kv = it.n_kv;
                uint32_t x_stage = 0;      // stage that holds the low parts of the key tile being multiplied
                // the low parts of the next edited key tile have landed (once per tile, before its first use)
                auto see_x = [&]() {
                    x_stage = n_hot % nx;
                    ok = warp_wait(x_full + x_stage, (n_hot / nx) & 1, 32);
                    ++n_hot;
                };
                // scores of tile x against key tile j; `hot`: the tile is an edited one whose low parts are multiplied too
                auto issue_S = [&](int x, int j, bool hot) {
                    const uint32_t kd = dK + ((pr + (uint32_t)j) % NK) * (G::TILE >> 4), qd = dQ + (uint32_t)x * (G::TILE >> 4);
                    const uint32_t dst = tmem_base + COL_S + 128 * x;
                    tc_fence_after();
                    if (leader) {
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            // 16 elements along the contraction = 32 bytes inside a 64-element block
                            const uint32_t off = ((uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32) >> 4;
                            umma_ss(dst, qd + off, DESC_HI, kd + off, DESC_HI, IDESC_S, ks > 0 ? 1u : 0u);
                        }
                        if (hot) {        // ... + Q (k'_lo)^T
                            const uint32_t xd = dX + x_stage * (sl.xb >> 4);
#pragma unroll
                            for (int ks = 0; ks < D / 16; ++ks) {
                                const uint32_t off = ((uint32_t)(ks >> 2) * BLK_BYTES + (uint32_t)(ks & 3) * 32) >> 4;
                                umma_ss(dst, qd + off, DESC_HI, xd + off, DESC_HI, IDESC_S, 1u);
                            }
                        }
                        umma_commit(s_full + x);
                    }
                    __syncwarp();
                };
                // P V of tile x and key tile j, key blocks [ks0, ks1) of 16 keys (2048 bytes of the V tile, 8 columns of P)
                auto issue_PV = [&](int x, int j, int ks0, int ks1, bool last) {
                    const uint32_t vd = dV + ((pr + (uint32_t)j) % NK) * (G::TILE >> 4);
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
                // The O_x of the last item that had a tile x has been read.  Its phases count those items only, and each is
                // seen, in order, by the next item that has the tile: a warp that could arrive for items in which it has
                // nothing to do would run ahead, and a parity wait cannot tell a phase from the one two later.
                auto see_drained = [&]() {
                    if (n_o[0] > 0) ok = warp_wait(o_drained + 0, (n_o[0] - 1) & 1, 46);
                    if (ok && nB > 0 && n_o[1] > 0) ok = warp_wait(o_drained + 1, (n_o[1] - 1) & 1, 47);
                };
                // do key tiles 0 and 1 take the low-part steps? (later ones are looked up one step ahead of their use)
                const bool hot_cur = it.need_lo && hot_g[0] != 0;
                bool hot_nxt = it.need_lo && n_kv > 1 && hot_g[1] != 0;
                // One thread issues for both tiles, in a fixed order (A then B in every step): the in-order tensor
                // pipe then keeps the two tiles half a period apart (softmax of one tile under the MMAs of the other).
                ok = warp_wait(start_full, n_it & 1, 20);
                if (!ok) break;
                if (hot_cur) { see_x(); if (!ok) break; }
                issue_S(0, 0, hot_cur);
                if (nB > 0) issue_S(1, 0, hot_cur);
                commit(kv_free + ev % NK);
                ++ev;
                see_drained();          // before the item's first P V writes O_x again
                if (!ok) break;
#pragma unroll 1
                for (int j = 0; j < n_kv && ok; ++j) {
                    const int j1 = j + 1;
                    const bool hot_j1 = hot_nxt && j1 < n_kv;
                    hot_nxt = it.need_lo && j + 2 < n_kv && hot_g[j + 2] != 0;
                    bool x_seen = false;
                    // V of this step and K of the next have landed once p_full completes: the relay warp vouches
                    // for them there, so this warp has no waits of its own for operands (every wait here is a
                    // bubble in the tensor pipe: its queue is only a couple of MMAs deep)
                    if (j < nA) {
                        ok = warp_wait(p_full + 0, (cx[0] + j) & 1, 24);
                        if (!ok) break;
                        issue_PV(0, j, 0, 6, false);
                        ok = warp_wait(p_last + 0, (cx[0] + j) & 1, 28);
                        if (!ok) break;
                        issue_PV(0, j, 6, 8, j == nA - 1);
                        if (j1 < nA) {
                            if (hot_j1) { see_x(); x_seen = true; if (!ok) break; }
                            issue_S(0, j1, hot_j1);
                        }
                    }
                    if (j < nB) {
                        ok = warp_wait(p_full + 1, (cx[1] + j) & 1, 26);
                        if (!ok) break;
                        issue_PV(1, j, 0, 6, false);
                        ok = warp_wait(p_last + 1, (cx[1] + j) & 1, 29);
                        if (!ok) break;
                        issue_PV(1, j, 6, 8, j == nB - 1);
                    }
                    if (j1 < nB) {
                        if (hot_j1 && !x_seen) { see_x(); if (!ok) break; }      // tile A does not use this key tile
                        issue_S(1, j1, hot_j1);
                    }
                    commit(kv_free + ev % NK);      // K(j+1) and V(j) may be overwritten
                    ++ev;
                }
                pr += n_kv; cx[0] += nA; cx[1] += nB; ++n_it;
                ++n_o[0];
                if (nB > 0) ++n_o[1];
            }
        } else if (warp == 2) {
            // ------------------------------------------------------------ operand relay: "the operands have landed", once per
            // item for Q and the first K, and per step "V(j) and K(j+1) landed" as a fifth arrival on the
            // P hand-off barrier, so that the MMA issuer waits on one barrier per hand-off
            uint32_t pr = 0, n_it = 0, n_qb = 0, cx[2] = {0, 0};
            bool ok = !dead;
            while (ok && next_item(it)) {
                ok = warp_wait(q_full + 0, n_it & 1, 21);
                if (ok && it.nB > 0) { ok = warp_wait(q_full + 1, n_qb & 1, 22); ++n_qb; }
                if (ok) ok = warp_wait(k0_full, n_it & 1, 23);
                if (!ok) break;
                if (lane == 0) mbar_arrive(start_full);
                __syncwarp();
#pragma unroll 1
                for (int j = 0; j < it.n_kv; ++j) {
                    const uint32_t g = pr + j;
                    ok = warp_wait(kv_full + g % NK, (g / NK) & 1, 25);
                    if (!ok) break;
                    if (lane == 0) {
                        if (j < it.nA) mbar_arrive(p_full + 0);
                        if (j < it.nB) mbar_arrive(p_full + 1);
                    }
                    __syncwarp();
                    // stay within the phase: the next arrival may only come after this phase has completed
                    if (j < it.nA) ok = warp_wait(p_full + 0, (cx[0] + j) & 1, 33);
                    if (ok && j < it.nB) ok = warp_wait(p_full + 1, (cx[1] + j) & 1, 34);
                    if (!ok) break;
                }
                pr += it.n_kv; cx[0] += it.nA; cx[1] += it.nB; ++n_it;
            }
        }
    } else if (warp >= 12) {
        // (these warps only hand their registers to the softmax warps)
        reg_dec<REGS_PROJ>();
    } else {
        // ------------------------------------------------------------ softmax of tile x, one query row per thread
        reg_inc<REGS_SOFTMAX>();
        const int x = (warp - 4) >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t tS = t_lane + COL_S + 128 * x, tO = t_lane + COL_O + D * x;
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        uint32_t cX = 0, n_o = 0;       // steps and items of this tile so far
        bool ok = !dead;
        while (ok && next_item(it)) {
            const int nX = x ? it.nB : it.nA;
            const int hqX = x ? it.hqB : it.hqA, qtX = x ? it.qtB : it.qtA;
            float m_run = -INFINITY, l_run = 0.f;
#pragma unroll 1
            for (int j = 0; j < nX; ++j) {
                ok = warp_wait(s_full + x, (cX + j) & 1, 40 + x);
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
            if (!ok) break;
            cX += nX;
            if (nX > 0) {
                ok = warp_wait(o_full + x, n_o & 1, 44 + x);
                ++n_o;
                if (!ok) break;
                // final normalisation and store
                tc_fence_after();
                const int qpos = qtX * BM + row;
                const bool valid = qpos < it.Lb;
                const size_t orow = (size_t)(it.seq0 + (valid ? qpos : 0)) * p.sched.Hq + hqX;
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
                // O_x may be written again (the next item's first P V)
                __syncwarp();
                if (lane == 0) mbar_arrive(o_drained + x);
            }
        }
    }

    // ---------------------------------------------------------------- teardown (also after an abort)
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // every product issued has finished before tensor and shared memory are released
        if (elect_one()) umma_commit(drain);
        __syncwarp();
        mbar_wait_limit(drain, 0, nullptr, p.status, 90, limit_ns);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
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

// Per-device facts, looked up once per device (a process may drive several GPUs from several threads).
bool device_info(int* n_sm) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int sm_of[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (sm_of[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return false;
        sm_of[dev] = n;
    }
    *n_sm = sm_of[dev];
    return true;
}

struct TileMaps { CUtensorMap q, k, v, x; };

template <int D, typename OutT, bool TABLE>
static seka_status launch_attn_t(const TileMaps& tm, const AttnParams& p, cudaStream_t st) {
    const SmemPlan sl = smem_plan<D>(p.plan);
    const uint32_t dyn = sl.total + 1024;      // slack for the 1024-byte alignment
    if (dyn > SMEM_LIMIT) return SEKA_ERR_UNSUPPORTED;
    auto kern = seka_attn_fwd_kernel<D, OutT, TABLE>;
    // the attribute belongs to the function on the current device: set on every call (a cheap driver call), so that a
    // process that drives several devices, or calls from several threads, needs no bookkeeping here
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT) != cudaSuccess) return SEKA_ERR_CUDA;
    int n_sm = 0;
    if (!device_info(&n_sm)) return SEKA_ERR_CUDA;
    // persistent CTAs, one per SM (the kernel needs the whole SM: all of tensor memory and most of shared memory)
    const unsigned grid = (unsigned)(p.sched.n_items_max < (long long)n_sm ? p.sched.n_items_max : (long long)n_sm);
    if (grid == 0) return SEKA_OK;
    kern<<<grid, NTHREADS, dyn, st>>>(tm.q, tm.k, tm.v, tm.x, p);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? SEKA_OK : SEKA_ERR_CUDA;
}

template <int D, typename OutT>
static seka_status launch_attn(const TileMaps& tm, const AttnParams& p, bool table, cudaStream_t st) {
    return table ? launch_attn_t<D, OutT, true>(tm, p, st) : launch_attn_t<D, OutT, false>(tm, p, st);
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
    const int D = shape->head_dim, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads;
    const Sched sched = make_sched(shape);
    if (w.n_tiles > 32767 || Hq > 32767 || shape->batch > 65535 || sched.n_items_max > 0x7fffffffLL) return SEKA_ERR_UNSUPPORTED;   // item records pack 15/16-bit fields
    if (!workspace || workspace_bytes < w.total || ((uintptr_t)workspace & 255)) return SEKA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);

    const void *q16 = Q, *k16 = K, *v16 = V;
    if (shape->dtype == SEKA_F32) {
        const size_t nq = (size_t)T * Hq * D, nk = (size_t)T * Hkv * D;
        char* cq = ws + w.cvt_off;
        char* ck = cq + align_up(nq * 2, 256);
        char* cv = ck + align_up(nk * 2, 256);
        launch_convert_bf16(static_cast<const float*>(Q), cq, nq, static_cast<const float*>(K), ck, static_cast<const float*>(V), cv, nk, st);
        q16 = cq; k16 = ck; v16 = cv;
    }
    AttnParams p;
    p.plan = make_steer_plan(shape, steer);
    p.sched = sched;
    void* X = ws + w.x_off;
    uint8_t* tile_hot = reinterpret_cast<uint8_t*>(ws + w.hot_off);
    int* first_hot = reinterpret_cast<int*>(ws + w.first_off);
    uint8_t* bh_info = reinterpret_cast<uint8_t*>(ws + w.info_off);
    if (steer) {
        // The tile kernels of the stand-alone edit write the side buffer (two small launches; in a routed call further
        // blocks of the first one evaluate Eq. 6 with the routine of adaseka_route, so the coefficients, and with them
        // everything after, are those of route-then-forward bit for bit).  Banks too wide for tensor memory
        // (n_experts * head_dim > 512) take the one-launch preparation kernel.
        if ((long long)shape->n_experts * D <= 512) {
            const float* a = alpha;
            if (sigma != nullptr) a = alpha_out != nullptr ? alpha_out : reinterpret_cast<float*>(ws + w.alpha_off);
            stc = launch_stage_keys_pipe(shape, w, k16, X, mask, U, a, gain, head_enable, ws, st, Q, sigma, k_route);
        } else {
            stc = launch_prep_steering(shape, p.plan, k16, U, alpha, gain, head_enable, mask, X, tile_hot, first_hot, bh_info,
                                       reinterpret_cast<int*>(ws), w.n_tiles, st, Q, sigma, k_route, alpha_out);
        }
        if (stc != SEKA_OK) return stc;
    }

    TileMaps tm;
    if (!make_tile_map(&tm.q, q16, D, Hq, T, 128) || !make_tile_map(&tm.k, k16, D, Hkv, T, 128) ||
        !make_tile_map(&tm.v, v16, D, Hkv, T, 128))
        return SEKA_ERR_CUDA;
    tm.x = tm.k;      // never dereferenced without steering
    if (p.plan.mode != 0 && !make_tile_map(&tm.x, X, p.plan.xcols, Hkv, T, 128)) return SEKA_ERR_CUDA;

    p.O = O; p.lse = lse;
    p.tile_hot = tile_hot; p.first_hot = first_hot; p.bh_info = bh_info; p.status = reinterpret_cast<int*>(ws);
    p.steer = steer ? 1 : 0;
    ItemRecord* items = reinterpret_cast<ItemRecord*>(ws + w.item_off);
    const bool table = shape->cu_seqlens != nullptr;
    if (table) launch_build_items(sched, shape->cu_seqlens, steer ? bh_info : nullptr, items, reinterpret_cast<int*>(ws) + 3, st);
    p.items = items; p.n_items = reinterpret_cast<int*>(ws) + 3;
    const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;

    if (D == 128) {
        return shape->dtype == SEKA_F32 ? launch_attn<128, float>(tm, p, table, st)
                                        : launch_attn<128, __nv_bfloat16>(tm, p, table, st);
    }
    return shape->dtype == SEKA_F32 ? launch_attn<64, float>(tm, p, table, st)
                                    : launch_attn<64, __nv_bfloat16>(tm, p, table, st);
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

namespace seka {
// Per device: events that mark the end of the compute of each part of the last host-buffer call, and that call's
// geometry.  The next call's copies into the staging buffer wait for them instead of for the caller's stream, so its
// input copies run while the previous call's output is still on its way back.
struct HostPipeState {
    cudaEvent_t cmp[8] = {};
    bool made = false, valid = false;
    const void* staging = nullptr;
    int parts = 0;
    size_t tok_per = 0;
};
static std::mutex g_host_pipe_mutex;
static HostPipeState g_host_pipe[64];
}  // namespace seka

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
    const size_t rq = (size_t)shape->n_q_heads * shape->head_dim * esz, rk = (size_t)shape->n_kv_heads * shape->head_dim * esz;
    const size_t bq = T * rq, bk = T * rk;
    char* dq = static_cast<char*>(staging);
    char* dk = dq + align_up(bq, 256);
    char* dv = dk + align_up(bk, 256);
    char* dO = dv + align_up(bk, 256);
    char* dm = dO + align_up(bq, 256);
    char* dl = dm + align_up(T, 256);
    // Sequences are independent, so a fixed-length batch is cut into parts (one sequence each, at most eight) that go
    // through a three-stage pipeline: the inputs of part i + 1 are copied in (a second stream) while part i is computed
    // (the caller's stream) and the output of part i - 1 is copied out (a third stream); the two copy directions share
    // the link at full duplex.  A packed batch (cu_seqlens) runs as one part.
    int parts = 1;
    if (shape->cu_seqlens == nullptr && shape->batch > 1) {
        parts = shape->batch < 8 ? shape->batch : 8;
        while (shape->batch % parts) --parts;
    }
    const int seq_per = shape->batch / parts;
    const size_t tok_per = (size_t)seq_per * shape->max_seqlen;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_tail = nullptr, ev_in[8] = {}, ev_out = nullptr;
    bool okc = true;
    auto make_event = [&](cudaEvent_t* e) { okc = okc && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SEKA_ERR_CUDA;
    std::lock_guard<std::mutex> pipe_lock(g_host_pipe_mutex);
    HostPipeState& hs = g_host_pipe[dev];
    if (!hs.made) {
        for (int i = 0; i < 8; ++i) make_event(&hs.cmp[i]);
        if (!okc) return SEKA_ERR_CUDA;
        hs.made = true;
    }
    // The staging buffer of the call before may still be read by its kernels.  Same buffer cut the same way: part i
    // waits for that call's part i; anything else: for its last part.
    const bool same_cut = hs.valid && hs.staging == staging && hs.parts == parts && hs.tok_per == tok_per;
    const int prev_last = hs.valid ? hs.parts - 1 : -1;
    if (parts > 1) {
        okc = okc && cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess;
        okc = okc && cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess;
        make_event(&ev_tail); make_event(&ev_out);
        for (int i = 0; i < parts; ++i) make_event(&ev_in[i]);
    } else {
        s_in = st; s_out = st;
    }
    seka_shape part = *shape;
    part.batch = seq_per;
    part.total_tokens = shape->cu_seqlens ? shape->total_tokens : 0;
    for (int i = 0; i < parts && okc && stc == SEKA_OK; ++i) {
        const size_t t0 = (size_t)i * tok_per, nt = parts > 1 ? tok_per : T;
        if (parts > 1 && prev_last >= 0 && (same_cut || i == 0))
            okc = okc && cudaStreamWaitEvent(s_in, hs.cmp[same_cut ? i : prev_last], 0) == cudaSuccess;
        okc = okc && cudaMemcpyAsync(dq + t0 * rq, static_cast<const char*>(h_Q) + t0 * rq, nt * rq, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        okc = okc && cudaMemcpyAsync(dk + t0 * rk, static_cast<const char*>(h_K) + t0 * rk, nt * rk, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        okc = okc && cudaMemcpyAsync(dv + t0 * rk, static_cast<const char*>(h_V) + t0 * rk, nt * rk, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (h_mask) okc = okc && cudaMemcpyAsync(dm + t0, h_mask + t0, nt, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (parts > 1) okc = okc && cudaEventRecord(ev_in[i], s_in) == cudaSuccess && cudaStreamWaitEvent(st, ev_in[i], 0) == cudaSuccess;
        if (!okc) break;
        stc = seka_attention_fwd(&part, dq + t0 * rq, dk + t0 * rk, dv + t0 * rk, dO + t0 * rq,
                                 h_lse ? reinterpret_cast<float*>(dl) + t0 * shape->n_q_heads : nullptr,
                                 h_mask ? reinterpret_cast<const uint8_t*>(dm) + t0 : nullptr, U,
                                 alpha ? alpha + (size_t)i * seq_per * shape->n_kv_heads * shape->n_experts : nullptr,
                                 gain ? gain + (size_t)i * seq_per : nullptr, head_enable, workspace, workspace_bytes, cuda_stream);
        if (stc != SEKA_OK) break;
        okc = okc && cudaEventRecord(hs.cmp[i], st) == cudaSuccess;
        if (parts > 1) okc = okc && cudaStreamWaitEvent(s_out, hs.cmp[i], 0) == cudaSuccess;
        okc = okc && cudaMemcpyAsync(static_cast<char*>(h_O) + t0 * rq, dO + t0 * rq, nt * rq, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        if (h_lse) okc = okc && cudaMemcpyAsync(h_lse + t0 * shape->n_q_heads, reinterpret_cast<float*>(dl) + t0 * shape->n_q_heads,
                                                nt * shape->n_q_heads * 4, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    }
    if (parts > 1) {
        // the caller's stream ends behind the last copy out (and behind the copies in, if the loop stopped early)
        if (ev_out && s_out) { cudaEventRecord(ev_out, s_out); cudaStreamWaitEvent(st, ev_out, 0); }
        if (ev_tail && s_in) { cudaEventRecord(ev_tail, s_in); cudaStreamWaitEvent(st, ev_tail, 0); }
        // queued work keeps what it needs: destroying a stream or an event only drops the handle
        for (int i = 0; i < parts; ++i) if (ev_in[i]) cudaEventDestroy(ev_in[i]);
        if (ev_tail) cudaEventDestroy(ev_tail);
        if (ev_out) cudaEventDestroy(ev_out);
        if (s_in) cudaStreamDestroy(s_in);
        if (s_out) cudaStreamDestroy(s_out);
    }
    // a call that stopped early leaves the next one to wait for the whole stream instead
    hs.valid = okc && stc == SEKA_OK;
    hs.staging = staging; hs.parts = parts; hs.tok_per = tok_per;
    if (!hs.valid) cudaStreamSynchronize(st);
    if (stc != SEKA_OK) return stc;
    return okc ? SEKA_OK : SEKA_ERR_CUDA;
}
