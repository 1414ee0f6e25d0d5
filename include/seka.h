/*
 * seka.h -- C ABI of the B200 (sm_100a) SEKA / AdaSEKA steered-attention library.
 *
 * The library computes prefill causal grouped-query attention in which the keys
 * of highlighted tokens are spectrally edited before the scores are formed:
 *     k' = k + g * P k,   P = U U^T                    (SEKA,    Section 2 / Eq. 7)
 *     P = sum_m alpha_m U_m U_m^T                      (AdaSEKA, Section 3.3)
 * with the routing coefficients alpha of Eq. 6, applied only where the per-token
 * highlight mask is set and only on selected KV heads (Section 3.4), the edited
 * keys feeding a causal softmax attention with scores q.k'/sqrt(d) (Section 2).
 *
 * Conventions shared by every entry point
 *  - Pointers are DEVICE pointers unless the name starts with `h_`. The caller owns
 *    every buffer; the library keeps none and allocates no device memory.  Process state it
 *    does keep: the launch counter of seka_launch_count (atomic), the SM count of each
 *    device it has been called on, the driver entry point for tensor maps, the per-device
 *    address of the built-in scratch of seka_edit_keys_static, and eight events per device
 *    that order the staging buffer of seka_attention_fwd_host between calls (all behind
 *    mutexes; calls may come from several host threads and for several devices).
 *  - Tensors are packed token-major: Q [T, Hq, d], K and V [T, Hkv, d], O [T, Hq, d],
 *    mask [T] (non-zero = highlighted), T = total_tokens, rows contiguous, base
 *    pointers 16-byte aligned.  Sequence b owns tokens cu_seqlens[b] .. cu_seqlens[b+1]-1;
 *    with cu_seqlens == NULL every sequence has max_seqlen tokens (the [B, L, H, d]
 *    layout of the hook in Algorithm 1).
 *  - Query head hq reads KV head hq / (Hq / Hkv).
 *  - U is fp32 [M, Hkv, d, r] (columns assumed orthonormal but used as stored: the
 *    kernels compute U (U^T k)).  alpha is fp32 [B, Hkv, M] or NULL (all ones).
 *    gain is fp32 [B] (any sign, zero allowed).  head_enable is uint8 [Hkv] or NULL
 *    (all heads steered).
 *  - The two-projector edit of Eq. 4, k' = k + (g+ P+ k + g- P- k) / 2 with P+ from the leading k+ vectors and
 *    P- from the vectors after the leading k- ones (Eq. 2), is the same blend with two "experts":
 *    U_1 = U+[:, :k+], U_2 = U-[:, k-:] (zero-padded to a common r), alpha = (g+/2, g-/2), gain = 1.
 *  - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*).
 *    Argument errors are returned before anything is launched.  A device-side wait
 *    that runs out (every wait in the kernels is bounded) records SEKA_ERR_TIMEOUT in
 *    the first word of `workspace`; seka_poll_status reads it.
 *  - Causal, forward only, queries and keys of equal length.  head_dim is 64 or 128.
 */
#ifndef SEKA_H_
#define SEKA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SEKA_OK = 0,
    SEKA_ERR_INVALID_ARG = 1,   /* null pointer, bad size, misaligned buffer */
    SEKA_ERR_UNSUPPORTED = 2,   /* shape outside what the kernels cover */
    SEKA_ERR_WORKSPACE = 3,     /* workspace missing or smaller than seka_workspace_bytes */
    SEKA_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed */
    SEKA_ERR_TIMEOUT = 5        /* a bounded device-side wait ran out */
} seka_status;

typedef enum { SEKA_F32 = 0, SEKA_BF16 = 1 } seka_dtype;

typedef struct {
    int32_t batch;              /* number of sequences B (>= 0) */
    int32_t max_seqlen;         /* L, or max_b L_b when cu_seqlens is given */
    int32_t total_tokens;       /* T; 0 means batch * max_seqlen (only valid without cu_seqlens) */
    int32_t n_q_heads;          /* Hq, a multiple of n_kv_heads */
    int32_t n_kv_heads;         /* Hkv */
    int32_t head_dim;           /* d: 64 or 128 */
    int32_t rank;               /* r: columns stored per expert, 1 .. d */
    int32_t n_experts;          /* M >= 1 */
    int32_t dtype;              /* seka_dtype of Q, K, V, O */
    float   softmax_scale;      /* 0 means 1/sqrt(head_dim) (Section 2) */
    const int32_t* cu_seqlens;  /* device int32 [B+1], or NULL for fixed length */
} seka_shape;

/* Bytes of scratch the calls below need for this shape (host-only, launches nothing). */
size_t seka_workspace_bytes(const seka_shape* shape);

/*
 * Key-editing hook of Algorithm 1 / Algorithm 2 on a key tensor in HBM (for example a
 * KV cache): K_out[t, h, :] = K_in[t, h, :] + gain[b] * sum_m alpha[b,h,m] U_m (U_m^T K_in[t,h,:])
 * for highlighted tokens t of enabled heads h; every other row of K_out equals K_in
 * bit for bit.  K_out may alias K_in (in place: only edited rows are written).
 * fp32 tensors are edited in fp32 arithmetic; bf16 tensors accumulate in fp32 and round
 * once.  Uses `workspace` for the compacted list of highlighted tokens.
 */
seka_status seka_edit_keys(const seka_shape* shape, const void* K_in, void* K_out,
                           const uint8_t* mask, const float* U, const float* alpha,
                           const float* gain, const uint8_t* head_enable,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * AdaSEKA routing, Eq. 6 / Algorithm 2: from the query of each sequence's LAST token,
 *   s_m = sum_{k < k_route} (q . U_m[:, k]) * sigma_m[k],   alpha_m = s_m / max_m' |s_m'|
 * per (sequence, KV head); q is the sum of the query heads of that KV head's group; all
 * s_m zero gives alpha = 0.  sigma is fp32 [M, Hkv, r]; k_route in 1..r, 0 means r.
 * alpha_out is fp32 [B, Hkv, M].
 */
seka_status adaseka_route(const seka_shape* shape, const void* Q, const float* U,
                          const float* sigma, int32_t k_route, float* alpha_out,
                          void* cuda_stream);

/*
 * Fused steered attention (Algorithm 1/2 hook + the attention it feeds, Eq. 4-5 in the
 * single-projector form): O = softmax_causal(Q K'^T * scale) V with K' the edited keys;
 * the score matrix is never written to memory, K and V are not modified.  The edited
 * keys of the 128-token key tiles that hold a highlighted token (and of no others) are
 * formed once per call, in fp32, by a preparation launch into `workspace` as a high and
 * a low bf16 part; the attention kernel stages those tiles from there instead of from K
 * and adds the contraction with the low parts where it matters (gain x coefficient above
 * 1 in magnitude, and every query row that sees at most 512 keys), so the logits follow
 * the fp32 edited keys there and one bf16 rounding of them elsewhere.
 * O has the dtype of the inputs.  With dtype SEKA_F32 the inputs are rounded to bf16
 * on the way in (the contraction runs on bf16 tensor cores, fp32 accumulation).
 * lse, if not NULL, receives log sum_j exp(score_ij) as fp32 [T, Hq].
 * mask == NULL or U == NULL means no steering (plain causal attention).
 */
seka_status seka_attention_fwd(const seka_shape* shape, const void* Q, const void* K,
                               const void* V, void* O, float* lse,
                               const uint8_t* mask, const float* U, const float* alpha,
                               const float* gain, const uint8_t* head_enable,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * AdaSEKA in one call (Algorithm 2): seka_attention_fwd with the routing coefficients of Eq. 6 computed by further
 * blocks of the library's operand-preparation launch instead of by a separate adaseka_route call (one launch fewer).
 * sigma and k_route are those of adaseka_route; the result equals adaseka_route followed by seka_attention_fwd bit
 * for bit.  alpha_out, if not NULL, receives the coefficients (fp32 [B, Hkv, M]); without it they live in the
 * workspace.  mask, U and sigma are required.
 */
seka_status seka_attention_fwd_routed(const seka_shape* shape, const void* Q, const void* K,
                                      const void* V, void* O, float* lse,
                                      const uint8_t* mask, const float* U, const float* sigma,
                                      int32_t k_route, float* alpha_out,
                                      const float* gain, const uint8_t* head_enable,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Same computation as seka_attention_fwd for callers whose tensors live in HOST memory
 * (pinned memory makes the copies asynchronous): h_Q, h_K, h_V, h_mask are copied to
 * `staging` (device, seka_host_staging_bytes(shape) bytes, 256-byte aligned), the
 * fused kernel runs, and O (and lse if h_lse != NULL) is copied back to h_O.  The result
 * is complete when the work queued on `cuda_stream` is.  A fixed-length batch is cut by
 * sequence into up to eight parts that are copied in, computed and copied out as a
 * pipeline (the call creates two more streams and a few events for its duration and
 * releases them before it returns); a packed batch goes through in one piece.  The host
 * input buffers are read from the moment of the call on: they must hold their data when
 * the call is made, and the copies in do NOT wait for work queued on `cuda_stream`
 * earlier (so the input copies of one call overlap the output copies of the call before
 * it).  What they do wait for is the previous host-buffer call's kernels on this device,
 * which may still be reading a staging buffer; the library keeps eight events per device
 * for that.  `staging` belongs to the call until `cuda_stream` has passed it; two calls
 * that overlap in time need a staging buffer and a workspace each.  Because its copies
 * run on streams of its own that do not start from `cuda_stream`, this entry point must
 * not be called while `cuda_stream` is being captured into a graph.  U, alpha, gain,
 * head_enable stay device pointers (they are per-model or per-prompt constants).
 */
size_t seka_host_staging_bytes(const seka_shape* shape);
seka_status seka_attention_fwd_host(const seka_shape* shape, const void* h_Q, const void* h_K,
                                    const void* h_V, void* h_O, float* h_lse,
                                    const uint8_t* h_mask, const float* U, const float* alpha,
                                    const float* gain, const uint8_t* head_enable,
                                    void* staging, size_t staging_bytes,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * seka_edit_keys without a workspace, for callers that cannot allocate device memory.  (The paper
 * has no counterpart for this entry point: it exists for the integration, not for the method.)
 *
 * Some hosts of this library may not call cudaMalloc at the point where the key cache has to be
 * edited: an inference server that hands its whole memory budget to a pre-sized KV-cache pool at
 * start-up, a plug-in that runs inside another framework's stream callback, or code that has
 * already frozen its allocator.  seka_edit_keys needs a scratch buffer (the compacted list of
 * highlighted tokens) that such a caller has nowhere to get.  This variant keeps that scratch in
 * a fixed array inside the library's device image instead; it takes the same tensors, minus
 * the workspace, and computes the same edit: in fp32 arithmetic with one rounding to the
 * tensor's type (for bf16 tensors seka_edit_keys uses a tensor-core kernel whose result can
 * differ from this one in the last bf16 place).
 *
 *  - Limit: total tokens <= SEKA_STATIC_MAX_TOKENS.  A larger shape is refused with
 *    SEKA_ERR_UNSUPPORTED before anything is launched; use seka_edit_keys with a workspace there.
 *  - Cost: every GPU that loads the library holds the array (4 * SEKA_STATIC_MAX_TOKENS + 256
 *    bytes) until the process exits, whether or not this entry point is ever called.  The
 *    kernel behind it (a warp per highlighted token, plain multiply-adds) is several times
 *    slower on large caches than the pipelined kernel of seka_edit_keys.
 *  - The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *    The first call on each device looks up the array's device address (once, with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on one device share the one array.  Its contents are whatever the previous call
 *    left; the call clears what it needs (the list counter) on `cuda_stream` first.  Two calls
 *    that may overlap on the GPU (different streams, or different host threads without ordering)
 *    race on the array: serialise them, or give the overlapping ones seka_edit_keys with
 *    separate workspaces.
 */
#define SEKA_STATIC_MAX_TOKENS 262144
seka_status seka_edit_keys_static(const seka_shape* shape, const void* K_in, void* K_out,
                                  const uint8_t* mask, const float* U, const float* alpha,
                                  const float* gain, const uint8_t* head_enable, void* cuda_stream);

/*
 * One decode step over a cached key tensor whose highlighted keys have already been edited (Algorithm 1 runs the
 * hook once, "before generation": seka_edit_keys in place on the prompt's keys; every generated token then
 * attends to the whole cache with the score of Section 2).  For sequence b and query head h
 *     O[b, h, :] = sum_j softmax_j(Q[b, h, :] . K[t_j, h / (Hq/Hkv), :] * scale) V[t_j, h / (Hq/Hkv), :]
 * over the cached tokens t_j of sequence b (all of them: the new token's own key and value are the last
 * cached row).  Q and O are bf16 [B, Hq, d] (one query token per sequence); K and V are the packed caches
 * [T, Hkv, d] described above; lse, if not NULL, receives fp32 [B, Hq] (natural log).  A sequence without
 * cached tokens gets O = 0 and lse = -inf.  K and V are read once and never written.
 * Only SEKA_BF16, at most 16 query heads per KV head and at most 65535 sequences (SEKA_ERR_UNSUPPORTED
 * otherwise); rank and n_experts of the shape are not used.  `workspace` holds the per-chunk partial results:
 * seka_decode_workspace_bytes(shape) bytes, 256-byte aligned, its first 256 bytes the status block that
 * seka_reset_status / seka_poll_status read.
 */
size_t seka_decode_workspace_bytes(const seka_shape* shape);
seka_status seka_decode_attention(const seka_shape* shape, const void* Q, const void* K, const void* V,
                                  void* O, float* lse, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);

/*
 * Offline spectral learning of the projections (Section 3.1, Eq. 2-3; first loop of Algorithm 1) and the
 * head-selection distance of Section 3.4, for every (layer, KV head) slot of a model in one call.
 *   h, h_pos, h_neg   bf16 [n_tokens, n_slots, head_dim]: neutral / positive / negative key embeddings, token-major
 *   answer_tokens     uint8 [n_tokens] (non-zero = the token counts for D) or NULL (all tokens)
 * Per slot s (all outputs device fp32 unless noted, written by this call):
 *   omega_pos[s], omega_neg[s]  [d, d] row-major: Omega+ = h^T h+ / n, Omega- = h^T h- / n  (bf16 products, fp32 sums)
 *   U_pos[s], U_neg[s]          [d, d] row-major, COLUMNS = left singular vectors of Omega+ / Omega-, singular values
 *                               descending (the layout seka_edit_keys / seka_attention_fwd take as U with rank = d;
 *                               P+ of Eq. 2 uses columns [0, k_pos), P- columns [k_neg, d)); computed in fp64 from the
 *                               fp32 Omega by one-sided Jacobi; a singular vector is defined up to its sign; columns
 *                               of exactly zero singular value are returned as zeros
 *   S_pos[s], S_neg[s]          [d] singular values
 *   k_pos[s], k_neg[s]          int32: the smallest k with sum_{i<=k} S_i >= gamma * sum_i S_i (Eq. 3), decided in fp64
 *   D[s]                        mean over the answer tokens of ||h+_t - h-_t||_2 (Section 3.4); 0 without answer tokens
 * head_dim is 64 or 128 (64 needs an even number of slots: neighbouring heads share a tensor-core product).
 * `workspace`: seka_learn_workspace_bytes(shape) bytes, 256-byte aligned, first 256 bytes the status block.
 */
typedef struct {
    int32_t n_tokens;           /* n >= 1 */
    int32_t n_slots;            /* number of (layer, KV head) pairs */
    int32_t head_dim;           /* d: 64 or 128 */
    float   gamma;              /* variance threshold of Eq. 3, in (0, 1] */
} seka_learn_shape;
size_t seka_learn_workspace_bytes(const seka_learn_shape* shape);
seka_status seka_learn_projections(const seka_learn_shape* shape, const void* h, const void* h_pos,
                                   const void* h_neg, const uint8_t* answer_tokens,
                                   float* omega_pos, float* omega_neg, float* U_pos, float* U_neg,
                                   float* S_pos, float* S_neg, int32_t* k_pos, int32_t* k_neg, float* D,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The first 256 bytes of a workspace are its status block (int32 words): word 0 the status, word 1 a code for the
 * wait that gave up.  Two more words are read by the fused forward and are there for tests of the failure path:
 * word 4 (non-zero n: CTA 0 leaves out the load of the n-th V/K pair of its first work item, so that a wait runs out)
 * and word 5 (limit of every device-side wait of that launch in microseconds; 0 means 2 s).  A launch on a workspace
 * whose status is not SEKA_OK does nothing.
 * seka_reset_status clears the whole block (async on the stream); call it once before first use of a workspace.
 */
seka_status seka_reset_status(void* workspace, void* cuda_stream);
/* Synchronises the stream and returns the device status word (SEKA_OK if no wait ran out). */
seka_status seka_poll_status(const void* workspace, void* cuda_stream);

const char* seka_status_string(seka_status status);

/* Number of kernels this library has launched in this process (for benchmark accounting). */
uint64_t seka_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SEKA_H_ */
