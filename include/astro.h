/*
 * astro.h -- C ABI of the rolling-KV chunk-attention library (sm_100a).
 *
 * One DiT layer's self-attention in the streaming scheme: the queries of a new
 * chunk of latent frames attend to a restricted context (S permanently kept
 * "sink" frames plus a sliding window of recent frames) and to the chunk itself.
 *
 * Conventions shared by every call
 *   - Every data pointer is a DEVICE pointer to memory the caller allocated and
 *     keeps alive; the library frees none of it.  The cache handle owns only
 *     host-side metadata.  Query outputs (int*, int64_t*) are HOST pointers.
 *   - Work is enqueued on the given CUDA stream (passed as void*, a cudaStream_t)
 *     and the call returns without synchronising.  Metadata changes take effect in
 *     call order.  Threads: calls that change a cache (append, evict, reset,
 *     set_state, destroy) must not run at the same time as any other call on that
 *     cache; calls that take it as const (the attention calls, query, get_state,
 *     key_segments, export) may be issued by several host threads at once on one
 *     handle -- the G candidates of a group decoding against one shared prefix --
 *     each with its own stream and output buffers.
 *   - bf16 tensors Q, O, K_chunk, V_chunk, dO, dQ, dK_chunk, dV_chunk are
 *     contiguous [batch, tokens, heads, head_dim].  LSE and delta are fp32
 *     [batch, heads, tokens].  Data pointers must be 16-byte aligned.
 *   - Functions return ASTRO_OK or an error code; they never throw or exit, and
 *     on an error the cache metadata is unchanged and nothing was launched.
 */
#ifndef ASTRO_H_
#define ASTRO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct astro_kvcache astro_kvcache_t; /* opaque, host side */

typedef enum {
  ASTRO_OK = 0,
  ASTRO_ERR_NULL = 1,      /* a required pointer is null */
  ASTRO_ERR_SHAPE = 2,     /* unsupported or inconsistent shape (head_dim not 64/128, batch mismatch, empty key set) */
  ASTRO_ERR_ALIGN = 3,     /* a data pointer is not 16-byte aligned */
  ASTRO_ERR_CAPACITY = 4,  /* append would hold more than S+L frames, or a buffer is too small */
  ASTRO_ERR_UNDERFLOW = 5, /* evict asks for more window frames than are held */
  ASTRO_ERR_ARCH = 6,      /* current device is not compute capability 10.x */
  ASTRO_ERR_CUDA = 7,      /* a CUDA runtime/driver call failed */
  ASTRO_ERR_TIMEOUT = 8    /* a bounded device-side wait ran out (see astro_last_device_status) */
} astro_status_t;

typedef struct {
  int cache_batch;      /* B_c: samples with their own cache; 1 = one shared frozen prefix for a group */
  int heads;            /* H */
  int head_dim;         /* D: 64 or 128 */
  int tokens_per_frame; /* T */
  int sink_frames;      /* S >= 0 */
  int window_frames;    /* L >= 1: slots of the sliding window */
} astro_kvcache_desc_t;

/* Bytes the caller must allocate for K (and the same again for V):
 * B_c * H * (S+L) * T * D * 2.  Returns 0 for an invalid descriptor. */
size_t astro_kvcache_storage_bytes(const astro_kvcache_desc_t* desc);

/* Sec. 3.2, "Rolling KV Cache with Frame Sinks": bind caller-allocated device
 * storage for the restricted context C_n (S sink frames + window of L frames),
 * so that resident KV memory is constant however long the video grows.
 * k_storage/v_storage: device, >= bytes_each each, 16-byte aligned; the layout
 * inside is private ([B_c, H, slot, T, D]).  The storage need not be initialised.
 * The cache starts empty.  *out receives the handle.  The call also encodes the
 * tensor maps of the storage (a host-only driver call; nothing is launched). */
astro_status_t astro_kvcache_create(const astro_kvcache_desc_t* desc, void* k_storage, void* v_storage,
                                    size_t bytes_each, astro_kvcache_t** out);

/* Frees the host-side handle only. */
astro_status_t astro_kvcache_destroy(astro_kvcache_t* cache);

/* Empties the cache (the next S appended frames become the new sink); storage is kept. */
astro_status_t astro_kvcache_reset(astro_kvcache_t* cache);

/* Sec. 3.3, "Streaming Long Tuning" (the forward pass accumulates the KV cache up
 * to the target step) and Sec. 3.2: store K and V of n_frames new frames.
 * k, v: device bf16 [B_c, n_frames*T, H, D].  The first S frames ever appended
 * fill the sink; later ones take the next free window slot.  The copy is
 * bit-exact.  There is no implicit eviction: ASTRO_ERR_CAPACITY if the cache
 * would hold more than S+L frames. */
astro_status_t astro_kvcache_append(astro_kvcache_t* cache, const void* k, const void* v, int n_frames,
                                    void* stream);

/* Sec. 3.2: the window keeps "the L most recent frames": drop the n_frames
 * oldest window frames.  Sink frames are never dropped.  The window is a ring,
 * so this advances an index and moves no bytes (the stream is unused today).
 * ASTRO_ERR_UNDERFLOW if n_frames exceeds the window frames held. */
astro_status_t astro_kvcache_evict(astro_kvcache_t* cache, int n_frames, void* stream);

/* Host-side state: frames held in the sink, in the window, and frames appended
 * since create/reset.  Any of the three HOST pointers may be null. */
astro_status_t astro_kvcache_query(const astro_kvcache_t* cache, int* sink_held, int* window_held,
                                   int64_t* frames_seen);

/* Checkpoint / resume.  The cache's whole state is the caller's storage plus this small record: a caller
 * that saves both (Sec. 3.3: the forward roll that accumulates the cache is the expensive part of a
 * training step) can later bind the saved bytes to a new handle with astro_kvcache_create and restore the
 * record with astro_kvcache_set_state.  HOST pointers.  set_state returns ASTRO_ERR_SHAPE if the record
 * does not fit the descriptor (counts out of range, window frames without a full sink). */
typedef struct {
  int sink_held;       /* frames in the sink slots */
  int window_head;     /* ring index of the oldest window frame, 0..L-1 */
  int window_held;     /* frames in the window ring */
  int64_t frames_seen; /* frames appended since create/reset */
} astro_kvcache_state_t;
astro_status_t astro_kvcache_get_state(const astro_kvcache_t* cache, astro_kvcache_state_t* state);
astro_status_t astro_kvcache_set_state(astro_kvcache_t* cache, const astro_kvcache_state_t* state);

/* Inspection aid (host only, launches nothing): the physical token ranges of the cache storage that an
 * attention call would walk in the cache's present state -- at most two, merged where adjacent, because the
 * window ring can be split by its wrap-around or by a hole left by evict -- followed by the chunk's own keys
 * when n_kc > 0.  HOST arrays of at least 3 entries each: first token, token count, and 1 for the chunk
 * segment / 0 for a cache segment.  *n_segments receives the number of entries written. */
astro_status_t astro_kvcache_key_segments(const astro_kvcache_t* cache, int n_kc, int* n_segments, int* first_token,
                                          int* token_count, int* from_chunk);

/* Inspection aid: write the held frames in logical order (sink frames, then
 * window oldest to newest) to k_out, v_out: device bf16 [B_c, held*T, H, D]. */
astro_status_t astro_kvcache_export(const astro_kvcache_t* cache, void* k_out, void* v_out, void* stream);

/* Sec. 3.2 (while the next clip is generated, attention is restricted to the cached
 * keys and values of the context C_n; G candidates decode against one shared prefix)
 * -- forward of chunk attention.  For every sample b, head h and chunk query i:
 *   keys/values = every token held in the cache (of sample b, or of the single
 *   shared cache when B_c = 1) followed by the n_kc chunk tokens;
 *   s_ij = scale * q_i . k_j;  LSE_i = ln sum_j exp(s_ij);  o_i = sum_j exp(s_ij - LSE_i) v_j.
 * q [batch, n_q, H, D], k_chunk/v_chunk [batch, n_kc, H, D] (may be null when
 * n_kc = 0), o [batch, n_q, H, D] bf16, lse [batch, H, n_q] fp32 (may be null).
 * cache may be null (no context).  n_q, n_kc are token counts and need not be
 * multiples of T or of any tile.  ASTRO_ERR_SHAPE if there is no key at all,
 * batch differs from B_c and B_c != 1, or scale is negative or not finite.
 * bf16 products, fp32 accumulation and softmax. */
astro_status_t astro_chunk_attn_fwd(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                    const void* v_chunk, int batch, int heads, int head_dim, int n_q,
                                    int n_kc, float scale, void* o, float* lse, void* stream);

/* Scratch bytes astro_chunk_attn_bwd needs (delta, fp32 [batch, H, n_q], rounded up). */
size_t astro_chunk_attn_bwd_workspace_bytes(int batch, int heads, int n_q, int head_dim);

/* Sec. 3.3, "Streaming Long Tuning": the KV cache of all preceding frames is
 * detached; gradients flow through the active window only.  Given dO and the
 * forward's O and LSE:
 *   p_ij = exp(s_ij - LSE_i); dp_ij = dO_i . v_j; delta_i = dO_i . o_i;
 *   ds_ij = p_ij (dp_ij - delta_i);
 *   dq_i = scale * sum over ALL keys of ds_ij k_j;
 *   dk_j = scale * sum_i ds_ij q_i and dv_j = sum_i p_ij dO_i for CHUNK keys only.
 * dq [batch, n_q, H, D], dk_chunk/dv_chunk [batch, n_kc, H, D], all bf16 written
 * from fp32 accumulators (dk_chunk/dv_chunk may be null when n_kc = 0).
 * workspace: device scratch of at least astro_chunk_attn_bwd_workspace_bytes(). */
astro_status_t astro_chunk_attn_bwd(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                    const void* v_chunk, const void* o, const float* lse, const void* d_o,
                                    int batch, int heads, int head_dim, int n_q, int n_kc, float scale,
                                    void* dq, void* dk_chunk, void* dv_chunk, void* workspace,
                                    size_t workspace_bytes, void* stream);

/* The three stages of astro_chunk_attn_bwd as calls of their own (same layouts, same checks); the
 * composite call is exactly delta, then dq, then dkv on one stream.  A caller that trains only the
 * query side can skip the last stage.
 *   delta: delta[b,h,i] = sum_d dO[b,i,h,d] * O[b,i,h,d], fp32 [batch, H, n_q] (device, 16-byte aligned).
 *   dq:    dQ over ALL keys (cache + chunk) from Q, dO, LSE, delta.
 *   dkv:   dK, dV of the chunk's own keys from Q, dO, LSE, delta (no cache involved: context is detached). */
astro_status_t astro_chunk_attn_bwd_delta(const void* o, const void* d_o, int batch, int heads, int head_dim,
                                          int n_q, float* delta, void* stream);
astro_status_t astro_chunk_attn_bwd_dq(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                       const void* v_chunk, const float* lse, const float* delta, const void* d_o,
                                       int batch, int heads, int head_dim, int n_q, int n_kc, float scale,
                                       void* dq, void* stream);
astro_status_t astro_chunk_attn_bwd_dkv(const void* q, const void* k_chunk, const void* v_chunk, const float* lse,
                                        const float* delta, const void* d_o, int batch, int heads, int head_dim,
                                        int n_q, int n_kc, float scale, void* dk_chunk, void* dv_chunk,
                                        void* stream);

/* Eq. 1, Eq. 2 and the selective KL term of Sec. 3.4 (Algorithm 2, "Policy loss on window"), fused with
 * the gradient for the current policy, over the velocity tensors of the active window:
 *   v+ = (1-beta) v_old + beta v_theta;  v- = (1+beta) v_old - beta v_theta;
 *   policy_i = r_i ||v+ - target||^2 + (1 - r_i) ||v- - target||^2;   kl_i = ||v_theta - v_ref||^2
 * per sample i, with ||.||^2 the plain sum of squares over the sample's `elems` elements, and
 *   grad = d/d v_theta of sum_i (w_policy_i policy_i + w_kl_i kl_i)
 * (the caller folds 1/elems, 1/batch, lambda_KL, the uncertainty mask and 1/|M| into the weights).
 * v_theta, v_old, v_ref, v_target, grad: device bf16 [batch, elems], 16-byte aligned, elems a multiple of 8.
 * r_tilde, w_policy, w_kl, policy_out, kl_out: device fp32 [batch].  v_ref and kl_out may be null together
 * (no KL term); w_policy null means 1, w_kl null means 0; grad may be null (losses only).  policy_out and
 * kl_out are overwritten.  fp32 arithmetic; the per-sample sums use atomics, so their last bits depend on
 * the order of the blocks. */
astro_status_t astro_nft_loss(const void* v_theta, const void* v_old, const void* v_ref, const void* v_target,
                              const float* r_tilde, const float* w_policy, const float* w_kl, int batch,
                              long long elems, float beta, float* policy_out, float* kl_out, void* grad,
                              void* stream);

/* The paper has no counterpart for this call: it exists for callers that must not allocate device
 * memory around the backward -- a training loop whose allocator is frozen after warm-up, a plug-in
 * that runs inside someone else's memory pool, a host thread that may not take the allocator's lock.
 * Such callers cannot provide the delta scratch that astro_chunk_attn_bwd asks for, so this variant
 * keeps it in a fixed device array inside the library instead: ASTRO_BWD_STATIC_MAX_ROWS fp32 values
 * (1 MiB), resident on every GPU that loads the library until the process exits.
 * Same inputs, outputs, layouts and results as astro_chunk_attn_bwd, without the workspace arguments.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.
 *   - ASTRO_ERR_CAPACITY if batch * heads * n_q exceeds ASTRO_BWD_STATIC_MAX_ROWS; nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on it.  Calls on one stream are safe.  The
 *     array keeps the previous call's delta; every element a call reads it has written first. */
#define ASTRO_BWD_STATIC_MAX_ROWS 262144
astro_status_t astro_chunk_attn_bwd_static(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                           const void* v_chunk, const void* o, const float* lse, const void* d_o,
                                           int batch, int heads, int head_dim, int n_q, int n_kc, float scale,
                                           void* dq, void* dk_chunk, void* dv_chunk, void* stream);

/* Every device-side wait in the kernels is bounded; one that runs out records a
 * code in a device status word instead of hanging.  This call synchronises the
 * current device, reads and clears that word: ASTRO_OK, or ASTRO_ERR_TIMEOUT
 * (then *detail, a HOST pointer that may be null, receives the raw word). */
astro_status_t astro_last_device_status(uint32_t* detail);

/* Self-test of that mechanism (the paper has no counterpart): enqueues a one-warp kernel that waits about a
 * millisecond on a barrier nothing will ever complete.  The kernel gives up, ends normally and leaves the
 * time-out in the status word, so the next astro_last_device_status returns ASTRO_ERR_TIMEOUT and the
 * context stays usable.  Nothing faults or hangs. */
astro_status_t astro_selftest_wait_timeout(void* stream);

/* Diagnostic switch (the paper has no counterpart).  The forward kernel first runs a fast pass in which a
 * query row keeps the maximum of its first key tile as its one reference exponent, and repeats a 128-query
 * tile with a running reference (the "safe pass") only if a row sum left the range fp32 can hold.
 *   mode 0  normal operation;
 *   mode 1  every later astro_chunk_attn_fwd of this process runs the safe pass only;
 *   mode 2  head_dim 128 calls run the CTA-pair kernel (two query tiles share every K/V tile through one
 *           tcgen05 cta_group::2 MMA); it has no safe pass of its own: a call whose rows would need one leaves
 *           a flag that astro_debug_pair_flag reads (and clears) after synchronising the device.
 * Results agree within the rounding of bf16 in every mode; the switch exists so that tests and benchmarks can
 * reach each code path on ordinary inputs.  Process-wide, not stream-ordered: it applies to calls made after it
 * returns.  ASTRO_ERR_SHAPE for any other mode. */
astro_status_t astro_debug_forward_mode(int mode);
astro_status_t astro_debug_pair_flag(int* flag);

/* Static, never null. */
const char* astro_status_string(astro_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* ASTRO_H_ */
