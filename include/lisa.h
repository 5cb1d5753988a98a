/*
 * lisa.h -- C ABI of the LiSA shared-layer attention library for NVIDIA B200 (sm_100a).
 *
 * LiSA (arXiv 2408.01890, Sec. 5.1) replaces a layer's Q K^T by
 *     A_n = Integrate( Align(A_{n-1}), A_Delta ),   A_Delta = Q' K'^T / sqrt(r)      (Eq. 3-4)
 * where A_{n-1} are the previous layer's pre-softmax scores (already scaled by
 * 1/sqrt(d_k), Eq. 2), Align is a tiny FFN over the head axis applied at every
 * (query, key) position, and Q', K' are low-rank (r << d_k) projections.  The
 * layer then applies the causal softmax and multiplies by its own V (Eq. 1).
 *
 * Conventions that hold for every entry point
 *   - Returns a lisa_status_t.  Never throws, never aborts.  Unless an entry
 *     point says otherwise it allocates and frees no device memory and does not
 *     synchronise: it validates on the host, then enqueues kernels on the
 *     caller's stream.  (The prefill of a shared layer also runs one small kernel
 *     on a stream of the library's own, created on first use per device; it is
 *     forked from the caller's stream and joined back into it by events inside
 *     the same call, so to the caller all work is ordered on the stream it gave.)
 *     On any error nothing is launched and outputs are untouched.
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte
 *     aligned, and must stay valid until the enqueued work has finished.
 *     Descriptor structs and the `links` array are HOST memory, read only
 *     during the call.
 *   - Activations are [B, N, H, x] with x (d or r) contiguous; strides are in
 *     elements.  Scores handed between decode layers are [B, Hq, L_cap], fp32 unless the call says bf16.
 *   - Grouped-query attention: query head h reads key/value head h / (Hq/Hkv).
 *   - Scratch memory comes from the caller: ask lisa_workspace_bytes() for the
 *     size and pass a buffer of at least that size (may be NULL when 0).
 *   - Supported ranges: d in {32, 64, 128}; 1 <= r <= 32; Hq <= 64, Hq % Hkv == 0;
 *     m <= 256; chain_len <= 8.  Outside them: LISA_ERR_UNSUPPORTED.
 */
#ifndef LISA_H_
#define LISA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* lisa_stream_t; /* a cudaStream_t (NULL = the default stream) */

typedef enum lisa_status_t {
    LISA_OK = 0,
    LISA_ERR_INVALID_ARG = 1, /* NULL where data is required, bad size/stride/alignment, wrong struct_size */
    LISA_ERR_UNSUPPORTED = 2, /* well-formed but outside the supported ranges above */
    LISA_ERR_WORKSPACE = 3,   /* workspace missing or smaller than lisa_workspace_bytes() */
    LISA_ERR_CUDA = 4,        /* a CUDA call failed; the code is kept for lisa_last_cuda_error() */
    LISA_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (reported by lisa_check) */
} lisa_status_t;

typedef enum lisa_dtype_t { LISA_F32 = 0, LISA_BF16 = 1 } lisa_dtype_t;
typedef enum lisa_act_t { LISA_ACT_NONE = 0, LISA_ACT_RELU = 1, LISA_ACT_SILU = 2 } lisa_act_t;

/* Eq. 4's Integrate.  ADD: A_n = FFN(A_{n-1}) + A_Delta.  CONCAT (Sec. 5.1, "An overview of LiSA"):
 * A_n = FFN([A_{n-1}; A_Delta]) with the two halves stacked on the head axis in that order, so W1 has
 * 2*Hq rows.  PLUS: no FFN, A_n = A_{n-1} + A_Delta (the variant for models pre-trained with sharing). */
typedef enum lisa_integrate_t { LISA_INTEGRATE_ADD = 0, LISA_INTEGRATE_CONCAT = 1, LISA_INTEGRATE_PLUS = 2 } lisa_integrate_t;

typedef enum lisa_cache_kind_t { LISA_CACHE_STANDARD = 0, LISA_CACHE_SHARED = 1 } lisa_cache_kind_t;
typedef enum lisa_op_t {
    LISA_OP_ANCHOR = 0, LISA_OP_SHARED_PREFILL = 1, LISA_OP_SHARED_DECODE = 2, LISA_OP_SHARED_PREFILL_CHAIN = 3,
    LISA_OP_SHARED_PREFILL_CARRY = 4
} lisa_op_t;

/* A strided view of an activation tensor [B, N, H, x]; x contiguous. */
typedef struct lisa_tensor {
    void* ptr;        /* device */
    int32_t dtype;    /* lisa_dtype_t */
    int32_t reserved; /* 0 */
    int64_t stride_b; /* elements */
    int64_t stride_n;
    int64_t stride_h;
} lisa_tensor;

/* One shared layer ("link") of a chain: the difference-compensation operands (Eq. 3) and the
 * attention-heads alignment FFN (Sec. 5.1).  Weights are row-major, row = input unit:
 *   w1 [h_in, m]   h_in = Hq (ADD) or 2*Hq (CONCAT);  b1 [m] or NULL
 *   w2 [m, Hq], b2 [Hq] or NULL                       (ffn_layers == 2)
 *   ffn_layers == 1: y = W1^T x + b1 with m == Hq, no activation, w2/b2 ignored (the LiSA_SL variant)
 *   integrate == PLUS: all four ignored.
 * For a two-layer FFN: y = W2^T act(W1^T x + b1) + b2. */
typedef struct lisa_link {
    lisa_tensor qp; /* Q' [B, N, Hq, r]   (decode: [B, 1, Hq, r], the new token's) */
    lisa_tensor kp; /* K' [B, N, Hkv, r]  (decode: ignored, K' is read from the cache) */
    const void* w1;
    const void* b1;
    const void* w2;
    const void* b2;
    int32_t w_dtype; /* lisa_dtype_t of w1,b1,w2,b2 */
    int32_t r;
    int32_t m;
    int32_t act;        /* lisa_act_t */
    int32_t integrate;  /* lisa_integrate_t */
    int32_t ffn_layers; /* 1 or 2 */
} lisa_link;

/* The cache of one layer (Sec. 2.2, KV cache; Sec. 5.2: a shared layer caches the low-rank keys K_LR in place of K).
 *   STANDARD: k = K   [B][Hkv][L_cap][d]
 *   SHARED:   k = K'^T [B][Hkv][r][L_cap]   (position contiguous, so r needs no padding)
 *   both:     v = V   [B][Hkv][L_cap][d]
 * L_cap must be a multiple of 8.  Memory is the caller's; lisa_kvcache_bytes() gives the sizes. */
typedef struct lisa_kvcache_layer {
    int32_t kind;  /* lisa_cache_kind_t */
    int32_t dtype; /* lisa_dtype_t */
    int32_t B;
    int32_t Hkv;
    int32_t L_cap;
    int32_t d;
    int32_t r; /* SHARED only */
    int32_t reserved;
    void* k;
    void* v;
} lisa_kvcache_layer;

/* The cache of a whole stack of layers: one lisa_kvcache_layer per layer, all carved out of ONE caller-owned device
 * buffer (Sec. 5.2: standard layers keep K and V, shared layers K_LR and V; the layers of a model differ only in kind).
 * lisa_kvcache_total_bytes gives the size of that buffer, lisa_kvcache_init fills in the per-layer descriptors
 * (host-only: no device work, nothing is cleared); layer l's k and v then live at 256-byte aligned offsets of `base`.
 * `layers[l]` can be handed to the attention entry points; lisa_kvcache_append_layer is lisa_kvcache_append on layer l. */
#define LISA_MAX_LAYERS 128
typedef struct lisa_kvcache_desc {
    size_t struct_size; /* sizeof(lisa_kvcache_desc) */
    int32_t n_layers;   /* 1..LISA_MAX_LAYERS */
    int32_t dtype;      /* lisa_dtype_t */
    int32_t B, Hkv, L_cap, d;
    int32_t r;          /* low rank of the shared layers */
    int32_t reserved;
    const int32_t* kinds; /* host array [n_layers] of lisa_cache_kind_t */
} lisa_kvcache_desc;
typedef struct lisa_kvcache {
    int32_t n_layers;
    int32_t reserved;
    lisa_kvcache_layer layers[LISA_MAX_LAYERS];
} lisa_kvcache;

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_anchor -- standard causal attention (Eq. 1-2), the layer whose scores a chain starts from.
 * Prefill (cache == NULL): q [B,Nq,Hq,d], k, v [B,Nq,Hkv,d]; o[b,i,h,:] = sum_{j<=i} softmax_j(q_i.k_j/sqrt(d)) v_j.
 * Decode  (cache != NULL, Nq == 1): the new token's q against a STANDARD cache that already holds the
 *   new token's K and V.  The context length of sequence b is seq_lens[b] (device int32 [B]) with
 *   1 <= seq_lens[b] <= L, or L for every sequence when seq_lens is NULL; L <= L_cap.
 *   If out_scores != NULL the pre-softmax row q.k_j/sqrt(d), j < length, is written there (fp32, or bf16 when
 *   scores_dtype says so) for the following shared layer (entries beyond the length are left untouched).
 * o has q's shape.  Workspace: lisa_workspace_bytes(LISA_OP_ANCHOR, args, &n). */
typedef struct lisa_anchor_args {
    size_t struct_size; /* sizeof(lisa_anchor_args) */
    int32_t B, Nq, Hq, Hkv, d;
    int32_t L; /* decode: context length (upper bound of seq_lens when those are given) */
    lisa_tensor q, k, v, o;
    const lisa_kvcache_layer* cache;
    const int32_t* seq_lens;
    void* out_scores; /* decode only; [B, Hq, >= length], fp32 or (scores_dtype == LISA_BF16) bf16 */
    int64_t scores_stride_b, scores_stride_h;
    void* workspace;
    size_t workspace_bytes;
    int32_t scores_dtype; /* lisa_dtype_t of out_scores: LISA_F32 (0, the default) or LISA_BF16 */
    int32_t reserved;
} lisa_anchor_args;
lisa_status_t lisa_attn_anchor(const lisa_anchor_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_shared_prefill -- a shared layer at chain depth c = chain_len over a whole prompt
 * (Sec. 5.1, Eq. 3-4, then Eq. 1).  The N x N x Hq scores of the whole prompt are not kept: they are recomputed
 * tile by tile (the tensor-core kernels hold a strip of query rows of them in the workspace at a time)
 * from the anchor's q0 [B,N,Hq,d], k0 [B,N,Hkv,d] and links[0..c-1] (links[c-1] is this layer's own,
 * the earlier ones belong to the shared layers between the anchor and this one), masked causally AFTER
 * the last link, soft-maxed and multiplied by this layer's v [B,N,Hkv,d].  o [B,N,Hq,d].
 * chain_len == 0 degenerates to lisa_attn_anchor on (q0,k0,v). */
typedef struct lisa_shared_prefill_args {
    size_t struct_size;
    int32_t B, N, Hq, Hkv, d, chain_len;
    lisa_tensor q0, k0, v, o;
    const lisa_link* links; /* host array [chain_len] */
    void* workspace;
    size_t workspace_bytes;
} lisa_shared_prefill_args;
lisa_status_t lisa_attn_shared_prefill(const lisa_shared_prefill_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_shared_prefill_chain -- prefill of ALL shared layers that hang off one anchor, in one pass
 * (Sec. 5.1: each shared layer takes the scores of the layer before it, so the layers at depth 1..c of
 * a chain compute nested prefixes of the same sequence A_1, ..., A_c of Eq. 4).
 * For k = 0..chain_len-1: o[k] is exactly what lisa_attn_shared_prefill returns for chain_len = k+1 with
 * v = v[k]: softmax(mask(A_{k+1})) . v[k].  The anchor scores and every link's difference are computed once
 * instead of once per layer that needs them.  v and o are host arrays of chain_len tensor descriptors
 * ([B,N,Hkv,d] and [B,N,Hq,d], device memory); the o[k] must not overlap one another.
 * Workspace: lisa_workspace_bytes(LISA_OP_SHARED_PREFILL_CHAIN, args, &n).  Shapes outside the tensor-core
 * kernels' range run layer by layer through lisa_attn_shared_prefill with the same results.
 * Errors as lisa_attn_shared_prefill; on error nothing is launched. */
typedef struct lisa_shared_prefill_chain_args {
    size_t struct_size;
    int32_t B, N, Hq, Hkv, d, chain_len; /* chain_len >= 1 */
    lisa_tensor q0, k0;
    const lisa_link* links;  /* host array [chain_len] */
    const lisa_tensor* v;    /* host array [chain_len] */
    const lisa_tensor* o;    /* host array [chain_len] */
    void* workspace;
    size_t workspace_bytes;
} lisa_shared_prefill_chain_args;
lisa_status_t lisa_attn_shared_prefill_chain(const lisa_shared_prefill_chain_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_shared_prefill_carry -- a shared layer over a whole prompt that takes the scores of the layer before it
 * from memory, as Sec. 5.1 states the method (layer n aligns the scores A_{n-1} of the layer directly before it), instead of
 * recomputing them from the anchor: the cost of a layer no longer grows with its depth in the chain, so runs of many
 * consecutive shared layers (the appendix's configurations have runs of 15 and 27) cost the same per layer as the first.
 * The price is memory: `scores` holds A_n for the whole prompt, lisa_prefill_scores_bytes(B, N, Hq) =
 * B * Hq * ceil128(N)^2 * 2 bytes (fp16, a blocked layout private to the library; 17.2 GB for B 4, N 8192, 32 heads).
 *   layer   the layer as for lisa_attn_shared_prefill with chain_len == 1: links[0] is this layer's own link, v and o its
 *           own; q0 and k0 are read only when `first` (otherwise they may be zeroed descriptors)
 *   first   1: this is the shared layer right after the anchor: A_0 = q0.k0^T/sqrt(d) is written into `scores` first;
 *           0: `scores` holds A_{n-1} as the previous call left it (same B, N, Hq)
 *   keep    1: A_n = Integrate(Align(A_{n-1}), D_n), unmasked, is left in `scores` for the next shared layer;
 *           0: last layer of its chain, the contents of `scores` are unspecified afterwards
 * o is exactly what lisa_attn_shared_prefill returns for the whole chain up to this layer, up to the rounding of the
 * carried scores to fp16 (which the recomputing path applies between links as well).
 * Tensor-core shapes only (d = 128, bf16, r <= 32; 32 heads with any Integrate, 40 heads with the adding ones; hidden
 * width up to 256): others LISA_ERR_UNSUPPORTED.  Workspace: lisa_workspace_bytes(LISA_OP_SHARED_PREFILL_CARRY, args, &n).  `scores` must be
 * 256-byte aligned.  On error nothing is launched. */
typedef struct lisa_shared_prefill_carry_args {
    size_t struct_size;
    lisa_shared_prefill_args layer;
    void* scores;
    size_t scores_bytes;
    int32_t first, keep;
} lisa_shared_prefill_carry_args;
size_t lisa_prefill_scores_bytes(int32_t B, int32_t N, int32_t Hq);
lisa_status_t lisa_attn_shared_prefill_carry(const lisa_shared_prefill_carry_args* args, lisa_stream_t stream);
/* The same call with the layer's tensors, weights and `o` in HOST memory, like lisa_attn_shared_prefill_host (dense layout,
 * strides ignored, workspace fields ignored); `scores` stays DEVICE memory.  q0 and k0 are staged only when `first`.
 * device_arena: at least lisa_carry_host_arena_bytes() bytes, 256-byte aligned.  Synchronises the stream before returning. */
lisa_status_t lisa_attn_shared_prefill_carry_host(const lisa_shared_prefill_carry_args* host_args, void* device_arena,
                                                  size_t arena_bytes, lisa_stream_t stream);
lisa_status_t lisa_carry_host_arena_bytes(const lisa_shared_prefill_carry_args* host_args, size_t* bytes);

/* The same call with every tensor, weight and `o` in HOST memory (dense [B,N,H,x] layout, strides
 * ignored; workspace fields ignored).  Inputs are staged into `device_arena` (device memory of at least
 * lisa_host_arena_bytes(), 256-byte aligned), the layer runs, `o` is copied back and the stream is
 * synchronised before returning.  On the tensor-core path the copies overlap the layer: q0, k0 and v come in, and o goes
 * back, one strip of query rows at a time on streams of the library's own (created on first use, joined into `stream`
 * before the call returns) while other strips compute; this needs pinned host memory to take effect, pageable memory
 * works but serialises. */
lisa_status_t lisa_attn_shared_prefill_host(const lisa_shared_prefill_args* host_args, void* device_arena,
                                            size_t arena_bytes, lisa_stream_t stream);
lisa_status_t lisa_host_arena_bytes(const lisa_shared_prefill_args* host_args, size_t* bytes);

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_shared_decode -- one decode step of a shared layer (Sec. 5.2, decoding stage).
 * prev_scores: the previous layer's fp32 score row [B,Hq,>=length]; link.qp the new token's Q' [B,1,Hq,r];
 * cache: a SHARED layer already holding the new token's K' and V; length = seq_lens[b] (<= L) or L.
 * For each cached position j < length: A[:,j] = Integrate(Align(prev[:,j]), q'.K'_j/sqrt(r)); then softmax
 * over j and the product with V.  o [B,1,Hq,d].  out_scores ([B,Hq,>=length], may be NULL, must not alias prev_scores)
 * receives A for the next shared layer.
 * Score rows are fp32 by default.  With scores_dtype == LISA_BF16 both rows are bf16 (2 bytes per entry, the size
 * Sec. 5.2 counts for the row): every hand-off between layers then rounds the scores to 8 mantissa bits (relative
 * 2^-9), on top of which the layer computes exactly as before. */
typedef struct lisa_shared_decode_args {
    size_t struct_size;
    int32_t B, Hq, L;
    int32_t scores_dtype; /* lisa_dtype_t of prev_scores AND out_scores: LISA_F32 (0, the default) or LISA_BF16 */
    const void* prev_scores;
    int64_t prev_stride_b, prev_stride_h;
    lisa_link link;
    const lisa_kvcache_layer* cache;
    const int32_t* seq_lens; /* device int32 [B] or NULL */
    lisa_tensor o;
    void* out_scores;
    int64_t scores_stride_b, scores_stride_h;
    void* workspace;
    size_t workspace_bytes;
} lisa_shared_decode_args;
lisa_status_t lisa_attn_shared_decode(const lisa_shared_decode_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_attn_shared_decode_static -- lisa_attn_shared_decode without caller-provided scratch.
 * (The paper has no counterpart to this entry point; it exists for integration reasons only.)
 *
 * Who needs it: callers that cannot obtain device memory at the moment they need to decode.  Typical cases
 * are a serving process whose memory manager claimed the whole GPU at start-up (so cudaMalloc fails or
 * fragments its pool), code running where an allocation would stall the device (cudaMalloc and cudaFree
 * synchronise it), and hosts that forbid allocator calls inside their latency-critical loop.  For them the
 * split-K partials live in a fixed array that is part of the library image: LISA_STATIC_SCRATCH_BYTES bytes
 * of device memory are held on every GPU that loads the library, until the process exits.
 *
 * Same arguments, results and errors as lisa_attn_shared_decode, except:
 *   - args->workspace and args->workspace_bytes are ignored;
 *   - if the step needs more than LISA_STATIC_SCRATCH_BYTES of scratch (lisa_workspace_bytes(
 *     LISA_OP_SHARED_DECODE, ...) tells how much) nothing is launched and LISA_ERR_WORKSPACE is returned;
 *     use the regular entry point with your own buffer for such sizes;
 *   - it calls no allocation routine of any kind, on the host or on the device.
 * The first call on each device looks up the array's device address (a host-side call, made with that device
 * current).  Make that first call outside of any stream capture.
 * All calls on a device share the one array, and it keeps whatever the previous call left there.  Nothing in
 * it has to start at zero: each call fully rewrites every entry it later reads.  Two calls whose kernels may
 * run at the same time on one GPU (different streams, or different host threads) race on the array and give
 * wrong results; order them on one stream or with events. */
#define LISA_STATIC_SCRATCH_BYTES (8u << 20)
lisa_status_t lisa_attn_shared_decode_static(const lisa_shared_decode_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_project -- the projections either side of the attention (Eq. 1: H W^V_i per head, and Concat(.) W^O; Eq. 3:
 * H W^Q_LR, H W^K_LR): C = X . W with X [B,N,1,d_in] (rows of d_in contiguous values; stride_h is ignored) and
 * W [d_in, n_out] row-major (row = input unit, as the paper writes H W), fp32 accumulation.  The n_out columns of C are
 * the concatenation [outputs[0] | outputs[1] | ...]: output o receives H_o * x_o consecutive columns, column h*x_o + j
 * of its block going to element [b, n, h, j] of its tensor (any strides, so a block can be written straight into the
 * layout its consumer reads: Q' and K' for lisa_attn_shared_prefill, K'/V rows for lisa_kvcache_append, a flat
 * [B,N,1,d_model] row for W^O).  One call with W = [W^Q_LR | W^K_LR | W^V] projects a shared layer's three operands at once.
 * bf16 X, W and outputs with 16-byte aligned rows run on the tensor cores; fp32 and odd shapes on a general kernel.
 * No workspace.  1 <= n_outputs <= 4. */
typedef struct lisa_project_output {
    lisa_tensor t; /* [B, N, H, x] */
    int32_t H;
    int32_t x;
} lisa_project_output;
typedef struct lisa_project_args {
    size_t struct_size;
    int32_t B, N, d_in, n_outputs;
    lisa_tensor x;   /* [B, N, 1, d_in] */
    const void* w;   /* [d_in, sum_o H_o * x_o], row-major, device */
    int32_t w_dtype; /* lisa_dtype_t; must equal x.dtype */
    int32_t reserved;
    lisa_project_output outputs[4];
} lisa_project_args;
lisa_status_t lisa_project(const lisa_project_args* args, lisa_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * lisa_kvcache_append -- write n_new new positions into a layer's cache (Sec. 2.2; Sec. 5.2: a shared layer
 * caches K_LR in place of K).  k_or_kp: [B,n_new,Hkv,d] for a STANDARD layer, [B,n_new,Hkv,r] (K') for a SHARED one,
 * which is stored transposed.  v: [B,n_new,Hkv,d].  Row t of sequence b lands at position
 * seq_lens_before[b] + t (device int32 [B]; NULL = position 0).  Positions that would fall at or beyond
 * L_cap are dropped and counted: lisa_check() then reports LISA_ERR_INVALID_ARG. */
lisa_status_t lisa_kvcache_append(const lisa_kvcache_layer* layer, const lisa_tensor* k_or_kp, const lisa_tensor* v,
                                  const int32_t* seq_lens_before, int32_t n_new, lisa_stream_t stream);

/* lisa_kvcache_append on layer `layer` of a multi-layer cache (LISA_ERR_INVALID_ARG if there is no such layer). */
lisa_status_t lisa_kvcache_append_layer(const lisa_kvcache* cache, int32_t layer, const lisa_tensor* k_or_kp, const lisa_tensor* v,
                                        const int32_t* seq_lens_before, int32_t n_new, lisa_stream_t stream);

/* Host-only helpers (no device work). */

/* Bytes of the one buffer that backs every layer of `desc` (each k and v rounded up to 256 bytes), and the carving of
 * such a buffer (`base`: device memory, 256-byte aligned, at least that many bytes) into `cache`. */
lisa_status_t lisa_kvcache_total_bytes(const lisa_kvcache_desc* desc, size_t* bytes);
lisa_status_t lisa_kvcache_init(const lisa_kvcache_desc* desc, void* base, size_t base_bytes, lisa_kvcache* cache);

/* Bytes of the k and v buffers of a cache layer (fields k, v ignored).  For one SHARED layer with 2-byte
 * elements, k_bytes is smaller than a STANDARD layer's by B*Hkv*L_cap*(d-r)*2, the saving of Sec. 5.2. */
lisa_status_t lisa_kvcache_bytes(const lisa_kvcache_layer* layer, size_t* k_bytes, size_t* v_bytes);

/* Scratch bytes the given call needs; `args` is the call's argument struct (data pointers are not read). */
lisa_status_t lisa_workspace_bytes(int32_t op, const void* args, size_t* bytes);

/* Synchronises `stream` and reports device-side conditions recorded since the last call: a dropped cache
 * append (LISA_ERR_INVALID_ARG) or a bounded wait that ran out (LISA_ERR_TIMEOUT); LISA_ERR_CUDA if the
 * stream itself reports an error. */
lisa_status_t lisa_check(lisa_stream_t stream);

int lisa_last_cuda_error(void);             /* the cudaError_t of the last LISA_ERR_CUDA on this thread, else 0 */
const char* lisa_status_string(int status); /* static string */
int lisa_version(void);                     /* major*1000 + minor */

#ifdef __cplusplus
}
#endif
#endif /* LISA_H_ */
