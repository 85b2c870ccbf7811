/*
 * fa.h -- C ABI of the B200 (sm_100a) hybrid-KV decode path of FourierAttention.
 *
 * The cache of one attention layer keeps, per KV head,
 *   - the first l_init and the most recent l_local tokens in all head dims
 *     (Sec. 3.3, Eq.1),
 *   - for the tokens in between ("middle"), the context-sensitive dims
 *     D^ku / D^vu per token (K^mu, V^mu, Eq.2) and
 *   - the remaining dims D^kc / D^vc only as n_coef = 2k real coefficients of
 *     the translated Fourier basis along the token axis (K^mc, V^mc, Eq.3-4).
 *
 * fa_compress builds that cache from a prefilled K, V (Eq.1-3), fa_append
 * pushes one token and folds the token that leaves the local window into the
 * coefficients (Eq.5), fa_decode_attention computes softmax attention of one
 * query per head over the cache, rebuilding the compressed dims on the fly
 * without ever writing a dense K or V (Eq.6).
 *
 * Conventions for every call
 *   - All buffers are caller-owned DEVICE memory on the current device unless
 *     a parameter says "host".  The library allocates nothing and runs every
 *     kernel on the stream passed in (a cudaStream_t handed over as void*;
 *     NULL is the default stream).  Its only state on the device besides the
 *     caller's buffers is the fixed scratch array of fa_decode_attention_static.
 *   - Host threads may call concurrently (the few host-side caches are locked);
 *     calls that share a cache, a workspace or the static scratch must be
 *     ordered by the caller (same stream, or events).
 *   - Calls are asynchronous.  Argument errors are found on the host before
 *     anything is launched and returned as fa_status.  Conditions only the
 *     device can see (middle segment full) are written to cache->status and
 *     read back with fa_poll_status; a call that hits one changes nothing.
 *   - Device pointers must be 16-byte aligned.  Index arrays are int32,
 *     strictly ascending per head.
 *   - No call throws, aborts or traps.
 */
#ifndef FA_H_
#define FA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FA_OK = 0,
    FA_ERR_INVALID_ARG = 1,   /* NULL pointer, bad size, inconsistent layout       */
    FA_ERR_UNSUPPORTED = 2,   /* valid but outside what the kernels implement      */
    FA_ERR_CAPACITY = 3,      /* the middle segment would exceed max_mid / period  */
    FA_ERR_WORKSPACE = 4,     /* workspace pointer NULL / misaligned / too small   */
    FA_ERR_CUDA = 5,          /* a CUDA runtime call failed                        */
    FA_ERR_TIMEOUT = 6,       /* a bounded device-side wait gave up                */
    FA_ERR_INDEX = 7          /* index sets are not a sorted disjoint cover        */
} fa_status;

typedef enum { FA_F32 = 0, FA_BF16 = 1 } fa_dtype;

/* Reconstruction weights of Eq.6.  ORTHO: 1/T for the constant row, 2/T for
 * the others, which inverts Eq.3 exactly on the span of the basis over a full
 * period.  PAPER: the literal 1/k of Eq.6. */
typedef enum { FA_NORM_ORTHO = 0, FA_NORM_PAPER = 1 } fa_norm;

/* How fa_decode_attention evaluates the compressed dims.  DIRECT sums the
 * n_coef basis terms per token; FFT evaluates each residue class of tokens
 * (token index mod mid_classes) with one length period/mid_classes transform.
 * AUTO picks FFT when the layout allows it.  FFT runs as one kernel whenever
 * its shared-memory staging fits the layout: a cooperative launch whose CTAs
 * wait for one another while every (batch, KV head) can have a CTA resident at
 * once, one CTA per (batch, KV head) in waves past that; else as three kernels.
 * FFT_SPLIT always takes the three-kernel form.  AUTO also takes it when there
 * are more (batch, KV head) pairs than SMs and the last wave of the one-kernel
 * form would be nearly empty. */
typedef enum { FA_DECODE_AUTO = 0, FA_DECODE_DIRECT = 1, FA_DECODE_FFT = 2, FA_DECODE_FFT_SPLIT = 3 } fa_decode_algo;

/* Immutable description of one layer's cache. */
typedef struct fa_layout {
    int32_t batch;          /* B                                                        */
    int32_t n_q_heads;      /* H_q; query head g reads KV head g / (H_q / H_kv)         */
    int32_t n_kv_heads;     /* H_kv, divides H_q                                        */
    int32_t head_dim;       /* d, multiple of 8, <= 256                                 */
    int32_t n_full_k;       /* |D^ku|, 0..d, multiple of 8                              */
    int32_t n_full_v;       /* |D^vu|, 0..d, multiple of 8                              */
    int32_t n_coef;         /* M = 2k real coefficients (Eq.4), even, 2 <= M <= period  */
    int32_t period;         /* T of Eq.4; middle token j uses basis column j, j < T     */
    int32_t l_init;         /* Eq.1                                                     */
    int32_t l_local;        /* Eq.1                                                     */
    int32_t max_mid;        /* capacity of the middle segment in tokens, <= period      */
    int32_t mid_classes;    /* P >= 1: K^mu / V^mu are stored [P][ceil(max_mid/P)][n_full],
                               middle token j in class j % P at slot j / P; 1 = token-major */
    int32_t kv_dtype;       /* fa_dtype of K, V, q, out and of the cached K/V rows      */
    int32_t norm;           /* fa_norm                                                  */
    int32_t decode_algo;    /* fa_decode_algo                                           */
    float   softmax_scale;  /* logits = softmax_scale * q . k                           */
} fa_layout;

/* Device buffers of one layer's cache (sizes from fa_cache_sizes). */
typedef struct fa_cache {
    const int32_t* idx_full_k;  /* [H_kv][n_full_k]        D^ku                         */
    const int32_t* idx_comp_k;  /* [H_kv][d - n_full_k]    D^kc                         */
    const int32_t* idx_full_v;  /* [H_kv][n_full_v]        D^vu                         */
    const int32_t* idx_comp_v;  /* [H_kv][d - n_full_v]    D^vc                         */
    void*  k_init;              /* [B][H_kv][l_init][d]                                 */
    void*  v_init;
    void*  k_local;             /* [B][H_kv][l_local][d], a ring: oldest row at state.local_head */
    void*  v_local;
    void*  k_mid;               /* [B][H_kv][P][ceil(max_mid/P)][n_full_k]   K^mu       */
    void*  v_mid;               /* [B][H_kv][P][ceil(max_mid/P)][n_full_v]   V^mu.  In bf16
                                   caches the 8-dim (16-byte) chunks of a row are permuted: chunk c
                                   of slot a is stored at chunk c ^ x, x = (a>>2)&1 for 2 or 6 chunks
                                   per row, (a>>1)&3 for 4, a&7 for 8, 0 otherwise (bank-conflict-free
                                   shared-memory image for the tensor-core loads of the decode kernel) */
    float* coef_k;              /* [B][H_kv][M][d - n_full_k]  K^mc, raw sums of Eq.3   */
    float* coef_v;              /* [B][H_kv][M][d - n_full_v]  V^mc                     */
    int32_t* state;             /* [B][8]: n_init, n_local, n_mid, local_head, ticket, 3 spare */
    int32_t* status;            /* [4]: sticky fa_status word, then scratch counters    */
} fa_cache;

/* Bytes of every buffer of fa_cache, in the order of its fields. */
typedef struct fa_cache_sizes {
    size_t idx_full_k, idx_comp_k, idx_full_v, idx_comp_v;
    size_t k_init, v_init, k_local, v_local, k_mid, v_mid;
    size_t coef_k, coef_v, state, status;
} fa_cache_sizes;

/* Host only.  Checks the layout and fills *out.  INVALID_ARG / UNSUPPORTED on a bad layout. */
fa_status fa_cache_sizes_of(const fa_layout* layout, fa_cache_sizes* out);

/* Host only.  Bytes of workspace fa_decode_attention and fa_compress need for this layout
 * (the larger of the two).  The workspace is scratch whose contents need not survive
 * between calls, with one rule: its first 4 KiB hold barrier counters that must be zero
 * when a call starts.  Zero-fill a new workspace once (cudaMemset); every call that ends
 * without FA_ERR_TIMEOUT leaves the counters at zero again.  After FA_ERR_TIMEOUT
 * zero-fill it before the next call. */
fa_status fa_workspace_bytes(const fa_layout* layout, size_t* out);

/* Puts a workspace into the state the first call expects (zeroes its barrier counters): for a new
 * buffer, or after FA_ERR_TIMEOUT.  ws_bytes >= 4096.  Asynchronous on `stream`. */
fa_status fa_workspace_init(void* ws, size_t ws_bytes, void* stream);

/* Clears state and status (an empty cache: no tokens, zero coefficients). */
fa_status fa_cache_reset(const fa_layout* layout, fa_cache* cache, void* stream);

/* Checks on the device that, per KV head, idx_full_* and idx_comp_* are strictly ascending,
 * in range and together cover 0..d-1 exactly once (Eq.2's D^u, D^c).  Synchronises the
 * stream.  Returns FA_ERR_INDEX if they do not. */
fa_status fa_validate(const fa_layout* layout, const fa_cache* cache, void* stream);

/* Eq.1-3.  K, V: prefilled keys / values of L tokens, element (b, t, h, e) at
 * b*stride_b + t*stride_t + h*stride_h + e (strides in elements, multiples of 8), dtype
 * layout->kv_dtype.  Overwrites the whole cache: windows, K^mu / V^mu, coefficients
 * (basis column j = t - n_init for middle token t) and state.  n_init = min(L, l_init),
 * n_local = min(L - n_init, l_local), the rest is the middle.  FA_ERR_CAPACITY (host side)
 * if the middle exceeds max_mid.  ws / ws_bytes: workspace as sized by fa_workspace_bytes. */
fa_status fa_compress(const fa_layout* layout, fa_cache* cache, const void* K, const void* V,
                      int64_t stride_b, int64_t stride_t, int64_t stride_h, int32_t L,
                      void* ws, size_t ws_bytes, void* stream);

/* fa_compress with a choice of how the coefficients of Eq.3 are evaluated (flags, OR-ed together; 0 is fa_compress):
 *   FA_COMPRESS_ORDERED  the sums of Eq.3 do not depend on the order of execution, so two calls on the same input
 *                        give the same bits (the default splits the token axis over many CTAs and adds the partial
 *                        sums with floating-point atomics, whose order varies from run to run; this mode adds at
 *                        most two partial sums to a zeroed coefficient, and a two-term sum commutes);
 *   FA_COMPRESS_FFT      the coefficients are computed as the k lowest bins of the discrete Fourier transform of
 *                        each zero-extended token column (Sec. 3.3, Eq.3-4 without forming F): one length
 *                        period / mid_classes transform per residue class and column, fp32 throughout, always in a
 *                        fixed order.  Needs a power-of-two period and mid_classes with n_coef / 2 <=
 *                        period / mid_classes <= 2048; FA_ERR_UNSUPPORTED otherwise.
 * Everything else (arguments, what is written, errors) as for fa_compress. */
enum { FA_COMPRESS_ORDERED = 1, FA_COMPRESS_FFT = 2 };
fa_status fa_compress_ex(const fa_layout* layout, fa_cache* cache, const void* K, const void* V, int64_t stride_b,
                         int64_t stride_t, int64_t stride_h, int32_t L, uint32_t flags, void* ws, size_t ws_bytes,
                         void* stream);

/* Compression of the prefill of n_layers layers in one call (Eq.1-4 per layer): layer i gets what
 * fa_compress_ex(&layouts[i], &caches[i], K[i], V[i], stride_b, stride_t, stride_h, L, flags, ...) gives it (windows,
 * kept-dim rows and counters bit for bit; coefficients within the same tolerance: floating-point atomics).  layouts
 * and caches are HOST arrays of n_layers entries; K and V are HOST arrays of n_layers DEVICE pointers to the layers'
 * prefilled tensors, which share strides and length L.  The caches of different layers must not share memory.
 * Where every layer takes the tensor-core path on CTA pairs, the call enqueues all partition kernels and then all
 * contractions, each launched programmatically behind the one before: kernels of neighbouring layers overlap (the
 * small partition kernels run side by side, a contraction starts on the SMs that its predecessor's first CTAs to
 * finish leave) and every kernel waits for its predecessor before it ends, so that work enqueued behind the call
 * sees all layers complete.  Otherwise the layers are compressed one after the other.  All layers are checked on the
 * host before the first launch; returns the first error. */
fa_status fa_compress_layers(int32_t n_layers, const fa_layout* layouts, fa_cache* caches, const void* const* K,
                             const void* const* V, int64_t stride_b, int64_t stride_t, int64_t stride_h, int32_t L,
                             uint32_t flags, void* ws, size_t ws_bytes, void* stream);

/* fa_compress for a batch whose rows have different prompt lengths: row b is compressed from its
 * first lengths[b] tokens (HOST array of B entries, each 0 <= lengths[b] and within the capacity rule
 * of fa_compress; K / V rows beyond a row's length are not read).  Every row becomes what a one-row
 * fa_compress would make of it; fa_append, fa_decode_attention and fa_decode_step then work on the
 * ragged batch as on any other (the token counters are per batch row). */
fa_status fa_compress_ragged(const fa_layout* layout, fa_cache* cache, const void* K, const void* V,
                             int64_t stride_b, int64_t stride_t, int64_t stride_h, const int32_t* lengths,
                             void* ws, size_t ws_bytes, void* stream);

/* Eq.5.  k_new, v_new: [B][H_kv][d].  The token goes to the init window while that has
 * room, else to the local window; when the local window is full its oldest token leaves:
 * its D^u dims are appended to K^mu / V^mu and its D^c dims are added to the coefficients
 * with basis column j = n_mid.  If the middle is full nothing changes and FA_ERR_CAPACITY
 * is written to cache->status. */
fa_status fa_append(const fa_layout* layout, fa_cache* cache, const void* k_new, const void* v_new,
                    void* stream);

/* Eq.6.  q, out: [B][H_q][d].  Softmax attention (no mask) of every query head over
 * cat(init, middle, local) of its KV head, where the D^c dims of a middle token j are
 * sum_m w_m F[m][j] C[m][.]; evaluated as Phi (W C^K q) for the scores and
 * (p^T Phi) W C^V for the outputs.  Does not modify the cache.  An empty cache gives zeros. */
fa_status fa_decode_attention(const fa_layout* layout, const fa_cache* cache, const void* q, void* out,
                              void* ws, size_t ws_bytes, void* stream);

/* One decode step with device inputs (Eq.5 then Eq.6): the result and the cache afterwards are those
 * of fa_append(k_new, v_new) followed by fa_decode_attention(q).  Where the decode call is a single
 * fused kernel (see fa_decode_algo), the KV head's query heads fit one pass and a head is spread over
 * at least eight CTAs, the whole step is that ONE launch: every CTA applies the push to its own view of
 * the token counters, the CTA that meets a moved row in a tile (the new token's window row, the kept
 * dims of the row that leaves the local window) patches the tile in shared memory, f_j x^T is added
 * to each coefficient row as the kernel streams it (C^K before forming u, C^V before the output
 * product) and written back, so the coefficients cross the memory bus once per step instead of twice,
 * and the moved rows and the counters are written to the cache once every CTA that reads the old
 * ones is past them.  Otherwise the two calls are made one after the other (with few CTAs per head
 * the stand-alone append kernel, which spreads the coefficient update over the whole device, is the
 * faster way).  Same arguments, workspace rule and errors as those two calls (a full middle sets
 * FA_ERR_CAPACITY in cache->status and the step decodes the unchanged cache). */
fa_status fa_decode_step(const fa_layout* layout, fa_cache* cache, const void* q, const void* k_new,
                         const void* v_new, void* out, void* ws, size_t ws_bytes, void* stream);

/* One decoded token across n_layers layers (Eq.5 then Eq.6 per layer): layer i runs
 * fa_decode_step(&layouts[i], &caches[i], q[i], k_new[i], v_new[i], out[i], ws, ...) in order on
 * `stream`, with the same result and cache contents, bit for bit, as n_layers single calls.  layouts
 * and caches are HOST arrays of n_layers entries; q, k_new, v_new, out are HOST arrays of n_layers
 * DEVICE pointers ([B][H_q][d] / [B][H_kv][d] of that layer).  One workspace serves all layers (the
 * calls are ordered by the stream): ws_bytes must cover the largest fa_workspace_bytes of the layouts.
 * All layers are checked on the host before the first launch; after that the call only enqueues
 * kernels, so a whole token step can be captured in one CUDA graph (after one eager call).  Stops at,
 * and returns, the first error. */
fa_status fa_decode_step_layers(int32_t n_layers, const fa_layout* layouts, fa_cache* caches,
                                const void* const* q, const void* const* k_new, const void* const* v_new,
                                void* const* out, void* ws, size_t ws_bytes, void* stream);

/* One decode step with HOST inputs and outputs (Eq.5 then Eq.6): copies q [B][H_q][d] and
 * k_new, v_new [B][H_kv][d] from host memory (pinned for the copies to be asynchronous) into
 * `staging`, runs fa_decode_step, and copies the result to out_host
 * [B][H_q][d].  `staging` is caller-owned device memory of at least
 * fa_step_staging_bytes(layout) bytes; k_new_host == NULL skips the append.  Asynchronous on
 * `stream`: out_host is valid after the stream is synchronised.  Host buffers that the device can
 * address (pinned or registered memory, 16-byte aligned) are not copied by separate copy
 * operations: one small kernel in front of the step reads q, k_new, v_new over the bus into
 * `staging`, and the decode kernel writes its result rows straight into out_host.  The host input
 * buffers must not be written between the call and the completion of the step. */
fa_status fa_decode_step_host(const fa_layout* layout, fa_cache* cache, const void* q_host,
                              const void* k_new_host, const void* v_new_host, void* out_host,
                              void* staging, void* ws, size_t ws_bytes, void* stream);
size_t fa_step_staging_bytes(const fa_layout* layout);

/* Sec. 3.4, dimension selection.  Compresses and reconstructs EVERY dimension of the middle
 * segment of the prefilled K and V (Eq.3, then Eq.6's reconstruction with this layout's weights) and
 * ranks the dimensions of each KV head by mean squared reconstruction error, averaged over the batch
 * rows: the layout's n_full_k (n_full_v) dimensions with the LARGEST error are to be kept per token,
 * the others held as coefficients; among equal errors the lower index is compressed first.
 *   K, V, strides, L: as for fa_compress (the middle is what lies between the first l_init and
 *     the last l_local tokens; period, n_coef, max_mid, norm of the layout apply).
 *   idx_full_k [H_kv][n_full_k], idx_comp_k [H_kv][d - n_full_k], idx_full_v, idx_comp_v: DEVICE
 *     outputs, ascending, ready to be a cache's index sets.
 *   mse: optional DEVICE output [B][H_kv][2][d] (side 0 = K, 1 = V), the per-row mean squared errors.
 *   ws / ws_bytes: scratch of fa_select_workspace_bytes(layout) bytes, 256-byte aligned (it holds the
 *     coefficients of all dimensions).  head_dim must be 64, 128 or 256.
 * For bf16 tensors (head_dim 64 or 128, n_coef a multiple of 64, 16-byte aligned bases and strides) the
 * reconstruction runs on the tensor cores with the basis and the weighted coefficients rounded to bf16: a
 * dimension that its coefficients rebuild exactly still reports an error of about 1e-6 of its mean square.
 * Asynchronous on `stream`.  An empty middle gives zero errors (the lowest indices are compressed). */
fa_status fa_select_workspace_bytes(const fa_layout* layout, size_t* out);
fa_status fa_select_dims(const fa_layout* layout, const void* K, const void* V, int64_t stride_b, int64_t stride_t,
                         int64_t stride_h, int32_t L, int32_t* idx_full_k, int32_t* idx_comp_k, int32_t* idx_full_v,
                         int32_t* idx_comp_v, float* mse, void* ws, size_t ws_bytes, void* stream);

/* fa_decode_attention without a caller workspace.  (The paper has no counterpart: this is a
 * packaging variant of the same computation.)  It is meant for callers that cannot allocate
 * device memory when they reach this call: an engine that gave all of its HBM to its own pools
 * at start-up and hands plug-ins no scratch, or a decode loop in which cudaMalloc, which
 * synchronises the device, is not allowed.  The scratch is a fixed array of
 * fa_static_workspace_limit() bytes (8 MiB) built into the library; each GPU that loads the
 * library holds it until the process exits.  No call made here allocates or frees.
 *   - q, out, cache: exactly as for fa_decode_attention; the result is the same.
 *   - Layouts whose fa_workspace_bytes exceeds the limit are refused with FA_ERR_WORKSPACE
 *     before anything runs; use fa_decode_attention with your own workspace for those.
 *   - The first call on each device looks the array's device address up (with that device
 *     current); make that first call before any stream capture.
 *   - All calls on one GPU share the one array.  It keeps whatever the previous call left; each
 *     call starts by clearing the barrier counters in its first 4 KiB (a memset on `stream`), so
 *     a call that ended with FA_ERR_TIMEOUT does not poison the next one.  Two calls that overlap
 *     on the GPU (two streams, two threads) race on it: serialise them. */
fa_status fa_decode_attention_static(const fa_layout* layout, const fa_cache* cache, const void* q,
                                     void* out, void* stream);
size_t fa_static_workspace_limit(void);

/* Synchronises the stream and returns (then clears) the sticky device status word. */
fa_status fa_poll_status(const fa_cache* cache, void* stream);

/* Number of kernels one call launches for this layout (what = 0 compress, 1 append,
 * 2 decode, 3 decode step); for launch accounting by callers.  what >= 4 asks about the decode plan instead:
 * 4: 1 if fa_decode_attention runs the split build of the fused kernel for this layout, else 0;
 * 5: residue classes per batch of the transform kernel (0 for the direct kernel);
 * 6: CTAs per (batch, KV head, pass of query heads).  Unknown values of what return 0. */
int fa_launch_count(const fa_layout* layout, int what);

const char* fa_status_string(fa_status s);
int fa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FA_H_ */
