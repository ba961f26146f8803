/*
 * kvcar.h -- C ABI of the KV-CAR decode hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA, attention over a paged KV cache
 * that stores per-layer autoencoder latents of K and V instead of K and V, plus
 * a per-layer/per-head table that lets a head read the adjacent lower layer's
 * cached K or V and store nothing (paper: Sec. "Network Architecture"; Eq. 1 for
 * the attention itself; Eq. 3 for the cache-size model).
 *
 * Conventions
 *   - Every call returns a kvcar_status; nothing throws or aborts across the ABI.
 *     kvcar_last_error() gives a human-readable reason for the last failure.
 *   - "HOST" / "DEVICE" beside a pointer says where the memory lives.
 *   - All DEVICE memory is owned by the caller: the library reports the sizes it
 *     needs (kvcar_required_bytes), receives three buffers (kvcar_bind_memory)
 *     and never allocates or frees device memory itself.  Buffers must be
 *     256-byte aligned and must outlive the context.
 *   - Kernels are launched on the cudaStream_t the caller passes (as void*; 0 is
 *     the default stream).  Calls are asynchronous with respect to the device;
 *     host-side bookkeeping (page table mirror, sequence lengths) is updated
 *     immediately, so all calls on one context must use one stream or be
 *     ordered by the caller.
 *   - Element type of q/k/v/out and of the cache rows is config.storage
 *     (float or bfloat16); all accumulation is fp32.
 *   - Matrices are row-major; autoencoder weights are [out][in].
 *   - There is no CPU fallback: without a CUDA device the launching calls fail
 *     with KVCAR_ERR_CUDA.
 */
#ifndef KVCAR_H
#define KVCAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvcar_ctx kvcar_ctx;

typedef enum {
    KVCAR_OK = 0,
    KVCAR_ERR_INVALID_ARG = 1,   /* bad pointer, index, size or alignment            */
    KVCAR_ERR_STATE = 2,         /* call not allowed in the context's current state  */
    KVCAR_ERR_OOM_PAGES = 3,     /* page pool exhausted; nothing was changed         */
    KVCAR_ERR_WORKSPACE = 4,     /* bound buffers too small for the request          */
    KVCAR_ERR_UNSUPPORTED = 5,   /* shape outside what the kernels handle            */
    KVCAR_ERR_CUDA = 6,          /* a CUDA runtime/driver call failed                */
    KVCAR_ERR_DEVICE_TIMEOUT = 7,/* a bounded device-side wait ran out               */
    KVCAR_ERR_GUARD = 8          /* kvcar_debug_check found memory it guards altered */
} kvcar_status;

typedef enum { KVCAR_F32 = 0, KVCAR_BF16 = 1 } kvcar_dtype;
typedef enum { KVCAR_K = 0, KVCAR_V = 1 } kvcar_which;

/* kernel families (kvcar_set_kernel) */
typedef enum {
    KVCAR_KERNEL_AUTO = 0,    /* tensor-core kernel where the shape allows, else generic */
    KVCAR_KERNEL_GENERIC = 1, /* fp32-FMA kernels (any supported shape, both dtypes)     */
    KVCAR_KERNEL_TENSOR = 2,  /* tcgen05/TMEM fused kernel (bf16 storage only)           */
    KVCAR_KERNEL_RAW = 3      /* reported only: streaming kernel AUTO picks for a layer
                                 whose K and V are all stored raw (no autoencoder)       */
} kvcar_kernel;

/* flags of kvcar_decode_attention */
#define KVCAR_INCLUDE_CURRENT_EXACT 1u /* also attend to the current token through its exact K/V */
#define KVCAR_ABSORBED 2u /* K side through the absorbed last decoder layer (see kvcar_decode_attention) */
#define KVCAR_ABSORBED_V 4u /* with KVCAR_ABSORBED: the V side too */

#define KVCAR_MAX_BATCH 512    /* sequences per launching call   */
#define KVCAR_MAX_KV_HEADS 32
#define KVCAR_MAX_Q_HEADS 128
#define KVCAR_MAX_HEAD_DIM 128

typedef struct {
    int32_t n_layers;
    int32_t n_q_heads;         /* query heads; multiple of n_kv_heads (grouped-query attention) */
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t page_tokens;       /* tokens per cache page                                          */
    int32_t max_seqs;          /* sequence ids are 0 .. max_seqs-1                               */
    int32_t max_pages;         /* physical pages shared by all sequences (and all layers)       */
    int32_t max_pages_per_seq; /* longest sequence = max_pages_per_seq * page_tokens tokens     */
    int32_t storage;           /* kvcar_dtype of q/k/v/out and of cache rows                    */
    int32_t latent_quant;      /* 0: latent rows in the storage type.  1: int8 latent rows (Sec.
                                  "Quantization", Eq. 4), one scale and one zero-point (fp32 each)
                                  per cached row, kept beside the codes; needs bf16 storage, an
                                  autoencoder on every (layer, K/V) that stores heads, and latent
                                  widths that are multiples of 16                                */
} kvcar_config;

/*
 * One autoencoder (encoder + decoder) for the K or the V of one layer, as the
 * paper describes it (Sec. "Network Architecture"): FC(in_dim -> hidden),
 * BatchNorm over the hidden features with stored statistics, LeakyReLU,
 * FC(hidden -> latent); the decoder mirrors it (latent -> hidden -> in_dim).
 * in_dim must equal (#heads the layer stores for this K/V) * head_dim: the
 * autoencoder spans exactly the heads that are cached (a reused head is never
 * encoded).  All pointers are HOST float arrays, read during the call only.
 * *_bn is [4][hidden] = gamma, beta, running mean, running variance.
 */
typedef struct {
    int32_t in_dim, hidden, latent;
    float leaky_slope, bn_eps;
    const float *enc_w1, *enc_b1, *enc_bn, *enc_w2, *enc_b2; /* [hidden][in_dim], [hidden], [4][hidden], [latent][hidden], [latent] */
    const float *dec_w1, *dec_b1, *dec_bn, *dec_w2, *dec_b2; /* [hidden][latent], [hidden], [4][hidden], [in_dim][hidden], [in_dim] */
} kvcar_ae;

/* ---- set-up ------------------------------------------------------------- */

/* Create a context (host bookkeeping only; touches no device).  Errors:
 * INVALID_ARG for non-positive sizes, n_q_heads not a multiple of n_kv_heads, or
 * limits above the KVCAR_MAX_* constants. */
kvcar_status kvcar_create(const kvcar_config *cfg, kvcar_ctx **out_ctx);
kvcar_status kvcar_destroy(kvcar_ctx *ctx);

/*
 * Cross-layer head reuse (Sec. "Network Architecture", last paragraph: chosen K
 * and V heads of a layer read the corresponding head of the layer below instead
 * of caching their own).  src_k/src_v: HOST int32 [n_layers * n_kv_heads]; entry
 * (layer, head) is -1 if the head keeps its own cache rows, else the index of
 * the head of layer-1 whose cached K (resp. V) it reads.  Chains are legal and
 * resolve transitively.  Layer 0 must be all -1.  Only before kvcar_bind_memory
 * (ERR_STATE after) and before any kvcar_set_autoencoder.  Default: all -1.
 */
kvcar_status kvcar_set_reuse_map(kvcar_ctx *ctx, const int32_t *src_k, const int32_t *src_v);

/*
 * Install the autoencoder of (layer, which).  A (layer, which) without one
 * stores the raw rows of its stored heads (uncompressed layer).  Only before
 * kvcar_bind_memory.  Errors: INVALID_ARG if in_dim does not match the stored
 * heads or a pointer is NULL.
 */
kvcar_status kvcar_set_autoencoder(kvcar_ctx *ctx, int32_t layer, int32_t which, const kvcar_ae *ae);

/* Sizes (bytes) of the three DEVICE buffers the context needs:
 * pool = all cache pages of all layers + the current-token rows;
 * weights = packed autoencoder weights and per-layer tables;
 * workspace = page table, sequence lengths, split-KV partial results, staging. */
kvcar_status kvcar_required_bytes(kvcar_ctx *ctx, size_t *pool, size_t *weights, size_t *workspace);

/* Hand over the three DEVICE buffers (256-byte aligned, at least the required
 * sizes), upload weights and tables on `stream`, and freeze the reuse map and
 * autoencoders.  Must be called once, with the target device current. */
kvcar_status kvcar_bind_memory(kvcar_ctx *ctx, void *pool, size_t pool_bytes, void *weights, size_t weights_bytes,
                               void *workspace, size_t workspace_bytes, void *stream);

/* Choose the kernel family used by the launching calls (default AUTO). */
kvcar_status kvcar_set_kernel(kvcar_ctx *ctx, int32_t kernel);

/* ---- sequences and pages -------------------------------------------------- */

/* Open / close a sequence id (0 <= seq < max_seqs).  Closing returns its pages:
 * the page released last is handed out first; a fresh pool hands out 0,1,2,... */
kvcar_status kvcar_seq_open(kvcar_ctx *ctx, int32_t seq);
kvcar_status kvcar_seq_close(kvcar_ctx *ctx, int32_t seq);

/* Make sure pages exist for positions seq_len .. seq_len+n_tokens-1 of each
 * listed sequence (pages are taken in list order).  All or nothing: on
 * ERR_OOM_PAGES no page has been taken.  Host-side only; the device copy of the
 * page table is brought up to date by the next launching call. */
kvcar_status kvcar_reserve(kvcar_ctx *ctx, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens);

/* ---- the hot path --------------------------------------------------------- */

/*
 * Encoder + append (Sec. "Network Architecture": the new token's key and value
 * vectors go through the layer's encoder right after they are produced, and the
 * resulting 1 x d latent rows are what the cache stores).
 * k, v: DEVICE [n_seqs][n_tokens][n_kv_heads*head_dim] new rows (all heads;
 * columns of reused heads are ignored).  For each sequence the stored heads'
 * slices are encoded (or copied, for an uncompressed layer), rounded to the
 * storage type and written at logical positions seq_len .. seq_len+n_tokens-1
 * (pages are reserved first; on ERR_OOM_PAGES nothing is written).  The last
 * token's exact rows are also kept as the layer's "current token".  seq_len is
 * NOT changed: call kvcar_advance once per step after all layers.
 * seqs: HOST int32 [n_seqs], distinct open sequences, n_seqs <= KVCAR_MAX_BATCH.
 */
kvcar_status kvcar_encode_append(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                 int32_t n_tokens, const void *k, const void *v, void *stream);

/*
 * kvcar_encode_append on the tensor cores, for many tokens per sequence (cache
 * prefill): same arguments, same rows written, same current-token rows (Sec.
 * "Network Architecture", the encoder of the appended key and value vectors).
 * The two fully connected layers run as tiled bf16 products with fp32
 * accumulation, so the hidden activations pass through bf16 between them
 * (kvcar_encode_append keeps them in fp32): a latent may differ from that
 * call's by a few bf16 steps of the row's scale.  Only bf16 storage, 64-wide
 * heads, and layers whose K and V both have an autoencoder with hidden and
 * latent widths that are multiples of 16 (else KVCAR_ERR_UNSUPPORTED, nothing
 * written).  Other errors as kvcar_encode_append.
 */
kvcar_status kvcar_encode_append_tensor(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                        int32_t n_tokens, const void *k, const void *v, void *stream);

/* seq_len += n_tokens for the listed sequences (host mirror now, device copy in
 * stream order). */
kvcar_status kvcar_advance(kvcar_ctx *ctx, const int32_t *seqs, int32_t n_seqs, int32_t n_tokens, void *stream);

/*
 * Decoder + attention (Sec. "Network Architecture": the cached latent rows are
 * expanded back to full-width K and V by the layer's two decoders and joined with
 * the current token's exact key and value vectors; Eq. 1 per head).
 * q: DEVICE [n_seqs][n_q_heads][head_dim]; out: DEVICE, same shape.
 * For each sequence and query head i (KV head g = i / (n_q_heads/n_kv_heads)):
 * resolve g through the reuse table for K and for V separately, restore the
 * root layer's cached rows 0 .. seq_len-1 with that layer's decoder, take the
 * head's 64-wide slice, and compute softmax(q K^T / sqrt(head_dim)) V.  With
 * KVCAR_INCLUDE_CURRENT_EXACT the exact current-token K/V written by this
 * step's kvcar_encode_append of the root layer joins the attended set.
 * A sequence with nothing to attend to yields zeros.
 * KVCAR_ABSORBED: the decoder ends in a plain fully connected layer (Sec.
 * "Network Architecture": FC, BatchNorm, LeakyReLU, FC, nothing after it), so
 * a head's score q.k' with k' = W4_h a + b4_h equals a.(W4_h^T q) + q.b4_h,
 * where a is the token's activated hidden vector: the restored K rows are then
 * never formed.  The same result up to rounding (W4_h^T q is rounded to the
 * storage type once per sequence and head); honoured by the tensor-core kernel
 * for K when the launch fills the machine, ignored (plain form computed) by
 * every other kernel.  KVCAR_ABSORBED_V (only together with KVCAR_ABSORBED): the
 * same for V, sum_t p_t v'_t = W4_h (sum_t p_t a_t) + b4_h sum_t p_t: a tile
 * hands on sum_t p_t a_t (m values per query head) and the last layer is applied
 * once per sequence and head when the tiles are merged; the probabilities enter
 * that product rounded to the storage type.  For at most 32 query heads and
 * hidden layers whose feature chunks fit one accumulator buffer (576 columns with
 * up to 16 query heads, 512 with up to 32); ignored elsewhere.
 */
kvcar_status kvcar_decode_attention(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                    const void *q, void *out, uint32_t flags, void *stream);

/*
 * One decode step of one layer in one call: kvcar_encode_append (n_tokens = 1)
 * of k, v followed by kvcar_decode_attention of q, same arguments, same
 * results, all DEVICE buffers.  Because the cached rows that the decoder reads
 * do not depend on the row the encoder appends (Sec. "Network Architecture":
 * the restored (l-1) x D matrices are concatenated with the current token's
 * exact vectors, which enter only when the tiles are merged), the library runs
 * the tile kernel on a stream of its own, forked from `stream` at the call and
 * joined back before the merge, beside the encoder's launches.  On return all
 * work is enqueued and ordered after what `stream` held at the call and before
 * what is enqueued on it afterwards.
 * Errors as for the two calls; on KVCAR_ERR_OOM_PAGES nothing is written.
 */
kvcar_status kvcar_step_layer(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs, const void *k,
                              const void *v, const void *q, void *out, uint32_t flags, void *stream);

/*
 * The same step for one layer with HOST buffers: copies k, v, q (each
 * n_tokens = 1) to the device, runs kvcar_step_layer, and copies `out`
 * back, all ordered on `stream`.  Returns
 * after enqueuing; synchronise the stream before reading out_host.  k, v
 * and q are gathered into one of eight page-locked slots of the context and
 * cross in a single copy (the call waits for the copy that used the slot eight
 * calls earlier), so k_host, v_host and q_host may be reused as soon as the
 * call returns; out_host should be page-locked for its copy to be asynchronous.
 */
kvcar_status kvcar_step_layer_host(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                   const void *k_host, const void *v_host, const void *q_host, void *out_host,
                                   uint32_t flags, void *stream);

/*
 * kvcar_decode_attention for callers that cannot obtain device memory for the
 * split-KV scratch.  (The paper has no counterpart to this call; it exists for
 * integration reasons only.)
 *
 * Who needs it: an inference server that gave its whole device budget to its
 * own arena at start-up and forbids driver allocations afterwards; a plugin
 * running under a host application that hands it input/output tensors but no
 * allocator; a latency-critical decode loop in which a cudaMalloc would stall
 * the device and may fail once memory is fragmented.  Such callers cannot grow
 * a workspace when a longer sequence needs more partial results.
 *
 * What it does: identical arithmetic and kernels to kvcar_decode_attention
 * (generic kernel family), except that the per-chunk partial results
 * (max, sum, weighted values) live in a fixed array inside the library image,
 * KVCAR_STATIC_SCRATCH_BYTES long, which every GPU that loads the library holds
 * until the process exits.  The call allocates and frees nothing, on the host
 * side of CUDA or through any library.  q and out are DEVICE buffers as in
 * kvcar_decode_attention.
 *
 * Limits and rules:
 *  - n_seqs * ceil(longest listed sequence / 128) * n_q_heads * (head_dim + 2)
 *    floats must fit in KVCAR_STATIC_SCRATCH_BYTES, else KVCAR_ERR_WORKSPACE
 *    and nothing is launched.
 *  - kvcar_bind_memory looks up the array's device address (set-up time, with
 *    the target device current; the first lookup on a device is when the driver
 *    sets the array's memory aside).  The call itself only reads that address.
 *    Contexts are used on the device they were bound on.
 *  - All contexts and streams of a process share the one array per device, and
 *    it keeps whatever the previous call left; every slot a call reads is
 *    written earlier in the same call, so nothing needs clearing, but two
 *    calls that overlap in time on one GPU race on it: keep such calls on one
 *    stream or order them yourself.
 */
#define KVCAR_STATIC_SCRATCH_BYTES (8u << 20)
kvcar_status kvcar_decode_attention_static(kvcar_ctx *ctx, int32_t layer, const int32_t *seqs, int32_t n_seqs,
                                           const void *q, void *out, uint32_t flags, void *stream);

/* ---- observability ---------------------------------------------------------- */

/* Reuse table resolution of (layer, kv_head): the layer and head whose cache
 * rows are read, and the 64-wide column slot of that head among the root
 * layer's stored heads (ascending head order). */
kvcar_status kvcar_debug_resolve(kvcar_ctx *ctx, int32_t layer, int32_t kv_head, int32_t which,
                                 int32_t *root_layer, int32_t *root_head, int32_t *slot);
/* Physical page and pool row of a logical token (must lie in a reserved page). */
kvcar_status kvcar_debug_locate(kvcar_ctx *ctx, int32_t seq, int32_t token, int32_t *page, int64_t *row);
kvcar_status kvcar_seq_len(kvcar_ctx *ctx, int32_t seq, int32_t *len);
/* Placement of one layer's K or V rows inside the pool buffer: byte offset of
 * row 0, bytes between rows, and elements per row (0 if the layer stores none). */
kvcar_status kvcar_pool_layout(kvcar_ctx *ctx, int32_t layer, int32_t which, size_t *offset, size_t *row_pitch,
                               int32_t *width);
/* int8 latent rows (config.latent_quant): byte offset, inside the pool buffer, of the layer's
 * [max_pages*page_tokens][2] fp32 array of (scale, zero-point) per cached row; the codes are at
 * kvcar_pool_layout's offset with a row pitch of `width` bytes.  Row r holds x ~ (code - zero-point) / scale. */
kvcar_status kvcar_pool_quant_layout(kvcar_ctx *ctx, int32_t layer, int32_t which, size_t *param_offset);
/* Bytes one cached token occupies over all layers: as configured, and with
 * neither autoencoders nor reuse (Eq. 3 per token and sequence). */
kvcar_status kvcar_cache_bytes_per_token(kvcar_ctx *ctx, double *compressed, double *uncompressed);
/* Algorithmic work of one kvcar_decode_attention call on `layer` per cached
 * token: cache bytes read and floating-point operations (decoder + attention),
 * following the reuse map (each distinct source layer's latent row is read whole
 * and passed through its first decoder layer once; of a raw row only the needed
 * heads' slices are read). */
kvcar_status kvcar_layer_work_per_token(kvcar_ctx *ctx, int32_t layer, double *bytes, double *flops);
/* The same count of floating-point operations for the KVCAR_ABSORBED form: on the K side the second decoder layer
 * (2 m 64 per needed head) and the 2 * 64 of q.k' per query head are replaced by 2 m per query head (the score taken
 * from the hidden vector); V side and bytes unchanged.  The per-sequence cost of W4_h^T q (m * 64 multiply-adds per
 * query head and call, not per token) is left out.  both_sides != 0: the count for KVCAR_ABSORBED | KVCAR_ABSORBED_V,
 * where the V side's second decoder layer and p.v' are likewise replaced by 2 m per query head (the per-sequence
 * W4_h product of the merge left out). */
kvcar_status kvcar_layer_work_absorbed(kvcar_ctx *ctx, int32_t layer, int32_t both_sides, double *flops);
/* Number of kernels the library has launched so far on this context. */
kvcar_status kvcar_launch_count(kvcar_ctx *ctx, int64_t *count);
/* Kernel family (kvcar_kernel: GENERIC, TENSOR or RAW) that kvcar_decode_attention will use
 * for `layer` under the current kvcar_set_kernel choice.  Only after kvcar_bind_memory. */
kvcar_status kvcar_layer_kernel(kvcar_ctx *ctx, int32_t layer, int32_t *kernel);
/* Synchronise `stream` and report any asynchronous CUDA error or device-side
 * bounded-wait timeout recorded since the last call. */
kvcar_status kvcar_sync_status(kvcar_ctx *ctx, void *stream);
const char *kvcar_last_error(kvcar_ctx *ctx);
/* Test hook for the device-side timeout path: enqueue a one-warp kernel that waits
 * on a barrier nothing ever completes, gives up after limit_ns (1 ns .. 1 s),
 * records a code in the context's status word and returns normally.  The next
 * kvcar_sync_status then reports KVCAR_ERR_DEVICE_TIMEOUT once.  Every bounded
 * wait of the fused kernel ends this way when it runs out (their limit is 2 s);
 * nothing traps and the context stays usable. */
kvcar_status kvcar_debug_expire_wait(kvcar_ctx *ctx, uint64_t limit_ns, void *stream);
/* Stand-in for a memory checker, callable at any point between steps.  The pool
 * buffer carries 256 guard bytes behind each of its regions (every layer's K and V
 * pool, their int8 row parameters, the per-layer current-token rows), filled with
 * a fixed byte by kvcar_bind_memory; no kernel has a reason to write them.  The
 * call brings the device tables up to date, waits for `stream`, reads the guards
 * and the device copies of the page table and sequence lengths back and compares
 * them with the fill byte and with the allocator's host-side tables.  Returns
 * KVCAR_OK, or KVCAR_ERR_GUARD with *what = 1 (guard byte altered; *where = byte
 * offset in the pool buffer), 2 (page-table entry; *where = sequence *
 * max_pages_per_seq + index) or 3 (sequence length; *where = sequence).  Host
 * pointers; synchronises the stream; not for the timed path. */
kvcar_status kvcar_debug_check(kvcar_ctx *ctx, void *stream, int32_t *what, int64_t *where);

/* ---- choosing the reuse map (Alg. 2, its first three steps) -------------------
 *
 * These calls need no context: they work on activations recorded by the caller.
 *
 * kvcar_head_l1_distance: the distance step of Alg. 2 (Sec. "Network
 * Architecture": an L1 norm between the same head's K, or V, matrices in two
 * adjacent layers, i.e. the sum of their absolute differences).
 * x: DEVICE [n_layers][n_rows][n_kv_heads * head_dim], storage type `storage`
 * (KVCAR_F32 / KVCAR_BF16), 16-byte aligned: the K (or the V) rows of one
 * mini-batch, n_rows = sequences x tokens.  dist: DEVICE float
 * [n_layers - 1][n_kv_heads]; dist[l-1][h] = mean over rows and over head h's
 * head_dim channels of |x[l] - x[l-1]| (the paper does not say whether the norm
 * is normalised; dividing by the element count lets mini-batches of different
 * sizes be averaged, as the text averages them - that average is the caller's).
 * scratch: DEVICE, at least kvcar_head_l1_scratch_bytes() bytes, 16-byte
 * aligned, contents irrelevant before and after.  Sums are taken in a fixed
 * order: the result is the same on every run.  head_dim * element size must be
 * a multiple of 16 bytes.  Errors: KVCAR_ERR_INVALID_ARG (pointers, alignment,
 * sizes), KVCAR_ERR_WORKSPACE (scratch too small), KVCAR_ERR_CUDA (launch).
 * Returns after enqueuing on `stream`.
 */
kvcar_status kvcar_head_l1_scratch_bytes(int32_t n_layers, int32_t n_kv_heads, int64_t n_rows, size_t *bytes);
kvcar_status kvcar_head_l1_distance(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t storage, const void *x,
                                    int64_t n_rows, void *scratch, size_t scratch_bytes, float *dist, void *stream);
/*
 * The selection step of Alg. 2 (heads whose distance to the layer below is small
 * enough read that layer's head instead of their own): the n_reuse heads
 * with the smallest distance reuse the same head of the layer below (the
 * paper's empirical threshold, given as a count; equal distances: lower layer,
 * then lower head, first).  dist: HOST float [n_layers - 1][n_kv_heads] (no NaN);
 * src: HOST int32 [n_layers * n_kv_heads], written in the form
 * kvcar_set_reuse_map takes (-1 = own data).  Host only, no GPU needed.
 */
kvcar_status kvcar_reuse_map_from_l1(const float *dist, int32_t n_layers, int32_t n_kv_heads, int32_t n_reuse,
                                     int32_t *src);

#ifdef __cplusplus
}
#endif
#endif /* KVCAR_H */
