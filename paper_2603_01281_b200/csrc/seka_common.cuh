// Shared device helpers for the sm_100a SEKA kernels: status word, bounded mbarrier
// waits, TMA tile loads, tcgen05 (UMMA + tensor memory) wrappers, descriptors.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <atomic>

#include "../../include/seka.h"

namespace seka {

// ---------------------------------------------------------------- workspace layout
// [0, 256)            status block: word 0 = seka_status, word 1 = where the wait gave up,
//                     word 2 = number of highlighted tokens found by the compaction pass,
//                     word 3 = number of work items in the item table of the fused kernel,
//                     word 4 = test hook: the producer of CTA 0 leaves out the load of this V/K pair (1-based) of its
//                              first item, so that a bounded wait runs out (0 = off),
//                     word 5 = limit of every device-side wait of the fused kernel in microseconds (0 = 2 s)
// [256, ...)          projector operands: the stand-alone edit keeps P[m][h] = U_m U_m^T here (two bf16 parts); the fused
//                     kernel does not use it
// then                one byte per (sequence, 128-key tile): the tile contains a highlighted token; then one int32
//                     per sequence: its first such tile; then one byte per (sequence, KV head): steered / low parts used
// then                item table of the fused kernel (32 bytes per unit, heaviest first)
// then                compacted highlighted-token list (int32 per token)
// then (fp32 inputs)  bf16 copies of Q, K, V
// then                edited keys of the fused kernel, bf16 [T, Hkv, 2 d] (high | low parts; only rows of tiles that
//                     hold a highlighted token are ever written or read)
constexpr size_t kStatusBytes = 256;

// How the fused kernel applies the edit (Eq. 5: logits = q.k + q.(g P k)) on a key tile that holds highlighted tokens:
// a preparation launch leaves k' = k + g sum_m alpha_m U_m U_m^T k (fp32-accurate) of the tile's tokens in a side
// buffer as a high and a low bf16 part (k' = hi + lo to about 2^-17; for a token that is not highlighted hi = k, lo = 0).
// The fused kernel stages such a tile from the high parts instead of from K, at no cost of its own, and where the gain
// is large enough for the bf16 rounding of k' to matter (see lo_needed) it extends the score product, in the same
// tensor-memory accumulator, by  S += Q (k'_lo)^T.  The low parts go through a small shared-memory ring of their own.
struct SteerPlan {
    int mode;            // 0: no steering, 1: steering
    int Rt;              // stacked rank M * r
    int xcols;           // bf16 columns of a side-buffer row: high parts [0, D), low parts [D, 2D)
    int nx;              // shared-memory stages of the low parts
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static inline int shape_total_tokens(const seka_shape* s) {
    return s->total_tokens > 0 ? s->total_tokens : s->batch * s->max_seqlen;
}

// head_dim 128 leaves 32 KB of shared memory beside the Q, K and V tiles: one stage of low parts
static inline SteerPlan make_steer_plan(const seka_shape* s, bool steer) {
    SteerPlan p;
    p.mode = steer ? 1 : 0; p.Rt = s->rank * s->n_experts;
    p.xcols = steer ? 2 * s->head_dim : 0;
    p.nx = steer ? (s->head_dim == 64 ? 3 : 1) : 0;
    return p;
}

// Is the low part of k' worth a second product?  One bf16 rounding of k' perturbs a logit by about
// eps = 2^-9 |q| |k'| / sqrt(3 d) in scaled units (1.2e-3 (1 + |g| a) for unit-variance inputs, a = largest |alpha|),
// and the output by about eps |v - o| sqrt(sum_j p_j^2).  Two cases take the low parts:
//   - |g| a > 1: the edited keys are far from unit variance and eps grows with them;
//   - query rows that see at most kLoTiles key tiles (512 keys): with few keys sqrt(sum p^2) is not small and the
//     tail of that noise reaches the stated 1e-2 on single elements (seen on a 35-key row at g = 1); these work items
//     are a few per cent of the steps of a long prompt.
// Everywhere else (long rows, |g| a <= 1) the noise is averaged over thousands of keys and stays several times
// below the rounding of P itself.
constexpr int kLoTiles = 4;
#if defined(__CUDACC__)
__host__ __device__
#endif
static inline bool lo_needed(float g, float alpha_max) { return fabsf(g) * alpha_max > 1.0f; }

// ---------------------------------------------------------------- schedule of the fused kernel
// An item is two 128-row query tiles "A" and "B" that share a KV head of one sequence: two query heads of one group at
// the same rows (even group size) or two consecutive row tiles of one head (odd group size).  Items are numbered
// heaviest first.
struct Sched {
    int B, L, Hq, Hkv, n_qt;
    int pair_heads;      // tiles A and B are two query heads (1) or two row tiles (0)
    int hs;              // head slots per sequence
    int rs;              // row slots
    int per;             // items per row slot
    long long n_items_max;
};

static inline Sched make_sched(const seka_shape* s) {
    Sched c;
    c.B = s->batch; c.L = s->max_seqlen; c.Hq = s->n_q_heads; c.Hkv = s->n_kv_heads;
    c.n_qt = (s->max_seqlen + 127) / 128;
    const int G = c.Hq / c.Hkv;
    c.pair_heads = (G % 2 == 0) ? 1 : 0;
    c.hs = c.pair_heads ? c.Hq / 2 : c.Hq;
    c.rs = c.pair_heads ? c.n_qt : (c.n_qt + 1) / 2;
    c.per = c.B * c.hs;
    c.n_items_max = (long long)c.per * c.rs;
    return c;
}

// One item (32 bytes in the item table).
struct __align__(16) ItemRecord {
    int seq0, Lb;           // first token and length of the sequence
    int bh;                 // sequence | KV head << 16
    int hq;                 // query head of tile A | of tile B << 16
    int qt;                 // row-tile index of tile A | of tile B << 16
    int n;                  // key tiles of tile A | of tile B << 16 (0: the tile lies beyond the sequence)
    int steer;              // bit 0: the keys of this (sequence, KV head) are edited; bit 1: with the low part of k'
    int pad;
};

#if defined(__CUDACC__)
#define SEKA_HD __host__ __device__ __forceinline__
#else
#define SEKA_HD inline
#endif

// Item `idx`; false if both tiles lie beyond the sequence.
SEKA_HD bool decode_item(const Sched& c, long long idx, const int* cu, ItemRecord& r) {
    const int row = c.rs - 1 - (int)(idx / c.per), rem = (int)(idx % c.per);
    const int b = rem / c.hs, slot = rem % c.hs;
    int hqA, hqB, qtA, qtB;
    if (c.pair_heads) { hqA = 2 * slot; hqB = 2 * slot + 1; qtA = qtB = row; }
    else { hqA = hqB = slot; qtA = 2 * row; qtB = 2 * row + 1; }
    const int hkv = hqA / (c.Hq / c.Hkv);
    r.seq0 = cu ? cu[b] : b * c.L;
    r.Lb = (cu ? cu[b + 1] : (b + 1) * c.L) - r.seq0;
    const int nA = qtA * 128 < r.Lb ? qtA + 1 : 0, nB = qtB * 128 < r.Lb ? qtB + 1 : 0;
    r.bh = b | (hkv << 16);
    r.hq = hqA | (hqB << 16); r.qt = qtA | (qtB << 16); r.n = nA | (nB << 16);
    r.steer = 0; r.pad = 0;
    return nA > 0;
}

struct WorkspaceLayout {
    size_t w_off, w_bytes;            // projector operands (see above)
    size_t hot_off, hot_bytes;        // uint8 [B, ceil(max_seqlen / 128)], then int32 [B]
    size_t first_off;                 // the int32 [B] inside the hot region
    size_t info_off;                  // uint8 [B, Hkv] inside the hot region: bit 0 steered, bit 1 with the low parts
    size_t item_off, item_bytes;      // ItemRecord [n_items_max]
    size_t list_off, list_bytes;      // int32 [total_tokens]
    size_t cvt_off, cvt_bytes;        // bf16 copies of Q, K, V (fp32 inputs only)
    size_t x_off, x_bytes;            // edited keys of the fused kernel
    size_t alpha_off;                 // fp32 [B, Hkv, M]: routing coefficients of a routed call that does not ask for them
    size_t edit_total;                // what the stand-alone edit needs (everything before the edited keys)
    size_t total;
    int n_tiles;                      // key tiles per sequence = ceil(max_seqlen / 128)
};

static inline WorkspaceLayout workspace_layout(const seka_shape* s) {
    WorkspaceLayout w;
    const size_t T = (size_t)shape_total_tokens(s);
    const int D = s->head_dim;
    const SteerPlan plan = make_steer_plan(s, true);
    w.n_tiles = (s->max_seqlen + 127) / 128;
    w.w_off = kStatusBytes;
    w.w_bytes = align_up((size_t)2 * s->n_experts * s->n_kv_heads * D * D * 2, 1024);
    w.hot_off = w.w_off + w.w_bytes;
    w.first_off = w.hot_off + align_up((size_t)s->batch * w.n_tiles + 1, 256);
    w.info_off = w.first_off + align_up((size_t)s->batch * 4 + 4, 256);
    w.hot_bytes = (w.info_off - w.hot_off) + align_up((size_t)s->batch * s->n_kv_heads + 1, 256);
    const Sched sc = make_sched(s);
    w.item_off = w.hot_off + w.hot_bytes;
    w.item_bytes = align_up((size_t)sc.n_items_max * 32 + 32, 256);
    w.list_off = w.item_off + w.item_bytes;
    w.list_bytes = align_up(T * 4 + 4, 256);
    w.cvt_off = w.list_off + w.list_bytes;
    w.cvt_bytes = 0;
    if (s->dtype == SEKA_F32)
        w.cvt_bytes = align_up(T * s->n_q_heads * D * 2, 256) + 2 * align_up(T * s->n_kv_heads * D * 2, 256);
    w.edit_total = w.cvt_off + w.cvt_bytes;
    w.x_off = align_up(w.edit_total, 1024);
    w.x_bytes = align_up(T * s->n_kv_heads * plan.xcols * 2, 1024);
    w.alpha_off = w.x_off + w.x_bytes;
    w.total = w.alpha_off + align_up((size_t)s->batch * s->n_kv_heads * s->n_experts * 4 + 4, 256);
    return w;
}

extern std::atomic<unsigned long long> g_launches;   // kernels launched by this library in this process

// ---------------------------------------------------------------- small device utilities
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Records the first device-side failure in the workspace status block.
__device__ __forceinline__ void report_timeout(int* status, int where) {
    if (status != nullptr && atomicCAS(status, (int)SEKA_OK, (int)SEKA_ERR_TIMEOUT) == (int)SEKA_OK)
        status[1] = where;
}

// largest |alpha| of a (sequence, KV head); 1 without coefficients (all ones, or routed: Eq. 6 normalises to 1)
__device__ __forceinline__ float alpha_max_of(const float* __restrict__ alpha, size_t bh, int M) {
    if (alpha == nullptr) return 1.f;
    float a = 0.f;
    for (int m = 0; m < M; ++m) a = fmaxf(a, fabsf(alpha[bh * M + m]));
    return a;
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One poll of an mbarrier phase.  The plain form returns at once either way (about 40 cycles when the phase
// has completed).  The parked form, if the phase has not completed, lets the hardware park the thread until it
// completes or about kPollNs have passed: a parked thread takes no issue slots from the warps that share its
// scheduler, but the form costs about twice as much when the phase has already completed.
constexpr uint32_t kPollNs = 20000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(kPollNs) : "memory");
    return ok != 0;
}

// Bounded wait: gives up after kWaitLimitNs or as soon as another thread has raised the
// CTA's abort flag, records where, raises the flag and returns false.  The caller must
// then leave through its teardown path (no further waits succeed once the flag is up).
// A few plain polls first (most waits on the tensor pipe's critical path find their phase
// complete or nearly so), then parked ones.
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s; a whole launch takes milliseconds
constexpr int kPlainPolls = 8;

__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                int* status, int where, uint64_t limit_ns) {
#pragma unroll 1
    for (int i = 0; i < kPlainPolls; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    while (true) {
        if (mbar_try_wait_parked(bar, parity)) return true;
        // a parked poll came back empty-handed: that is rare (tens of microseconds have passed), so the flag
        // and the clock can be looked at every time
        if (abort_flag != nullptr && *abort_flag) return false;
        const uint64_t now = global_timer_ns();
        if (t0 == 0) {
            t0 = now;
        } else if (now - t0 > limit_ns) {
            if (abort_flag != nullptr) *abort_flag = 1;
            report_timeout(status, where);
            return false;
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int where) {
    return mbar_wait_limit(bar, parity, abort_flag, status, where, kWaitLimitNs);
}

// ---------------------------------------------------------------- TMA (bulk tensor loads, no multicast)
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 3-D tile load: coordinates are (element in head_dim, head, token); x must be a multiple of 8 (bf16).
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, uint64_t* bar,
                                            int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// generic-proxy writes to shared memory -> visible to the async proxy (UMMA / TMA)
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- tensor memory + UMMA
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_holder, uint32_t ncols) {   // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(smem_holder)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {        // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptors are passed as their two 32-bit halves: the high half is the same for
// every step of a tile and the low half only moves by a constant, so the issuing thread spends one add
// per operand and step.
// D[tmem] (+)= A[smem] * B[smem]; one thread issues.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                        uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; one thread issues.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival once every UMMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp reads lane (warp%4)*32 + t.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
// Waits for the tensor-memory loads of this thread; the registers of the load that is about to be used are
// named as operands so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld_on(uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// Shared-memory operand descriptor, 128-byte swizzle, tiles made of [rows x 64 bf16] blocks whose
// rows are 128 bytes and whose 8-row groups are 1024 bytes apart (what a TMA box {64, rows} writes).
//   K-major operand (Q, K, P): leading offset unused, stride offset = 1024 B between 8-row groups;
//     advancing 16 elements along the contraction adds 32 B to the start address.
//   MN-major operand (V as B of P*V): leading offset = distance between 64-column blocks,
//     stride offset = 1024 B between 8-row (contraction) groups; 16 contraction rows = 2048 B.
//   Low half: start address >> 4 (bits 0-13) and leading offset >> 4 (bits 16-29); moving the start by
//   `bytes` adds bytes >> 4.  High half: stride offset >> 4 (bits 0-13), descriptor version 1 for sm_100
//   (bit 14), 128-byte swizzle (value 2 in bits 29-31).
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
    return ((smem_addr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t umma_desc_hi_sw128(uint32_t sbo_bytes) {
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// Byte offset of element (row, col) inside a [rows x 64 bf16] block written with the 128-byte swizzle.
__device__ __forceinline__ uint32_t sw128_offset(int row, int col) {
    return (uint32_t)(row * 128 + ((((col >> 3) ^ row) & 7) << 4) + ((col & 7) << 1));
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

#endif  // __CUDACC__

}  // namespace seka
