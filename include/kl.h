/*
 * kl -- kernel-looped transformer decode on one NVIDIA B200 (sm_100a).  C ABI.
 *
 * The library implements the decode step of a decoder-only transformer the way the paper
 * "Kernel Looping" (arXiv 2410.23668) schedules it: Embedding, L x Decoder, Classifier, Sampling
 * (Section 2, call-schedule figure).  In KL_MODE_LOOPED the L consecutive calls to the decoder-layer
 * kernel are one call to a persistent kernel with an outer loop over layers (Section 3.2, rules
 * (1)-(10)); in KL_MODE_PER_LAYER the same kernel body is launched once per layer, which is the
 * synchronisation-boundary schedule the transformation removes (Section 2, schedule (ii)); in
 * KL_MODE_PER_STAGE once per operator group of every layer (schedule (i)).
 *
 * Conventions
 *   - All pointers named *_d are DEVICE pointers, *_h are HOST pointers.  Nothing here allocates or frees
 *     device memory: the caller owns the weight arena, the scratch arena, the KV cache, token/position/logit
 *     buffers and the CUDA stream (passed as a void* holding a cudaStream_t; NULL = default stream).
 *   - Every function returns a kl_status (0 = KL_OK, negative = error); nothing throws, aborts or traps.
 *   - Calls on one handle must not overlap on the GPU (use one stream per handle).
 *   - Storage is bf16 for weights and KV cache; activations and all accumulation are fp32.
 */
#ifndef KL_H_
#define KL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kl_handle kl_handle;
typedef int32_t kl_status;

enum {
    KL_OK = 0,
    KL_ERR_INVALID_ARG = -1,       /* null pointer, bad enum, size mismatch */
    KL_ERR_UNSUPPORTED_SHAPE = -2, /* model or batch shape outside what the kernels cover */
    KL_ERR_NOT_LOADED = -3,        /* kl_decode_step before every tensor was loaded */
    KL_ERR_CUDA = -4,              /* a CUDA runtime call failed */
    KL_ERR_SYNC_TIMEOUT = -5,      /* a bounded device-side wait ran out (reported by kl_last_status) */
    KL_ERR_OUT_OF_RANGE = -6,      /* token >= vocab or position >= max_ctx seen on the device */
    KL_ERR_TOO_LARGE = -7          /* a size beyond the fixed capacity of kl_argmax_advance_static */
};

enum { KL_MODE_LOOPED = 0, KL_MODE_PER_LAYER = 1, KL_MODE_PER_STAGE = 2 };

/* Tensors accepted by kl_load_weights; all bf16, row-major [out_features, in_features] (gains: [hidden]). */
enum {
    KL_EMBED = 0,   /* [vocab, hidden]           layer = -1 */
    KL_WQ = 1,      /* [n_q_heads*head_dim, hidden] */
    KL_WK = 2,      /* [n_kv_heads*head_dim, hidden] */
    KL_WV = 3,      /* [n_kv_heads*head_dim, hidden] */
    KL_WO = 4,      /* [hidden, n_q_heads*head_dim] */
    KL_WGATE = 5,   /* [ffn, hidden] */
    KL_WUP = 6,     /* [ffn, hidden] */
    KL_WDOWN = 7,   /* [hidden, ffn] */
    KL_NORM1 = 8,   /* [hidden]  gain of the RMSNorm before attention */
    KL_NORM2 = 9,   /* [hidden]  gain of the RMSNorm before the MLP */
    KL_NORM_F = 10, /* [hidden]  final gain              layer = -1 */
    KL_LM_HEAD = 11,/* [vocab, hidden]                  layer = -1 */
    /* only for models created with KL_FLAG_QKV_BIAS: q, k, v = W a + b, the bias added before the rotation */
    KL_BQ = 12,     /* [n_q_heads*head_dim] */
    KL_BK = 13,     /* [n_kv_heads*head_dim] */
    KL_BV = 14,     /* [n_kv_heads*head_dim] */
    /* only for mixture-of-experts models (n_experts > 0) */
    KL_WROUTER = 15 /* [n_experts, hidden]  router of the layer's MLP; the experts' KL_WGATE / KL_WUP / KL_WDOWN are loaded
                       with kl_load_expert_weights */
};

/* kl_model_desc.flags: the q, k, v projections carry biases (KL_BQ, KL_BK, KL_BV must be loaded for every layer).
 * The paper's operator list has no such term; its Table 2 includes a 72B decoder that does. */
#define KL_FLAG_QKV_BIAS 1u
/* kl_model_desc.flags: keep the batch-1 kernels in their plain mode (weights consumed from the shared-memory ring).  By
 * default, shapes that allow it -- dense layers, head_dim 64 or 128, hidden, n_q_heads * head_dim and ffn multiples of
 * 2048, an input vector of ffn floats next to an eight-slot ring in shared memory -- run in stash mode: every weight
 * chunk moves on from its ring slot into tensor memory and is multiplied from there, which more than doubles what an SM
 * holds ahead of its consumers (the cross-layer weight prefetch of Section 2, deeper).  Both modes compute the same
 * function; their sums are taken in different orders.  The environment variable KL_STASH=0 acts as this flag for every
 * handle the process creates (for measurements that must not touch the caller's code).  No counterpart in the paper. */
#define KL_FLAG_NO_STASH 2u

/* Shapes the kernels cover (anything else: KL_ERR_UNSUPPORTED_SHAPE): head_dim 32, 64, 128 or 256; hidden and ffn
 * multiples of 8; n_q_heads a multiple of n_kv_heads with 1, 2, 4 or 8 query heads per kv head -- any group size up
 * to 8 (3 and 6 included) when head_dim is 64 or 128, where attention runs on the tensor-core loop; at most as many
 * kv heads as the device has SMs. */
typedef struct {
    uint32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    float rms_eps;    /* added to the mean of squares, inside the root */
    float rope_theta; /* RoPE base; pair (i, i + head_dim/2) rotates by position * theta^(-2i/head_dim) */
    uint32_t max_batch;
    uint32_t max_ctx; /* capacity of the KV cache in positions */
    uint32_t flags;   /* 0 or a combination of KL_FLAG_QKV_BIAS, KL_FLAG_NO_STASH */
    /* Mixture-of-experts MLP (the 8x7B decoder of the paper's Table 2 is of this kind; the paper's operator list has no
     * such term): n_experts > 0 gives every layer a router [n_experts, hidden] and n_experts MLPs of width ffn, of
     * which the top_k with the largest router logits (the lower index first among equals) process a token, weighted
     * by the softmax over those top_k logits.  0, 0 = dense MLP.  Limits: n_experts <= 16, top_k <= 4 and
     * top_k x (column pieces of the down projection) <= 20, i.e. top_k <= 2 at ffn 14336.  Such models decode batches
     * sequence after sequence (no tensor-core path), and KL_MODE_PER_STAGE keeps gate/up and down in one launch. */
    uint32_t n_experts, top_k;
} kl_model_desc;

/* Sizes of the two device arenas the caller must provide to kl_create (both 256-byte aligned).
 * weight_bytes holds the library's own copy of every tensor, grouped per layer (the [N x S] parameters that Eq. 3 /
 * Group(p) of Section 3.2 yields) and stored as one contiguous run per layer in the order the persistent kernel
 * streams it -- the second representation of grouped tensors that the end of Section 3.2 describes.
 * scratch_bytes holds activations, split-K attention partials, synchronisation counters, the status word and
 * staging buffers for the host-buffer entry point. */
kl_status kl_workspace_bytes(const kl_model_desc* desc, size_t* weight_bytes, size_t* scratch_bytes);

/* Creates a handle over caller-owned arenas (device pointers, sizes as reported by kl_workspace_bytes).
 * The handle is the merged kernel's parameter list of Section 3.2 (rules (2)-(5) and Eq. 3): per-layer tensors become
 * grouped parameters with a leading layer dimension and one constant layer stride, constants (shape, eps, RoPE base)
 * are kept once.  Several handles may be alive at once (one stream each).
 * Uses the current CUDA device.  The scratch arena is cleared synchronously.  *out is set on success only. */
kl_status kl_create(const kl_model_desc* desc, void* weight_arena_d, void* scratch_arena_d, kl_handle** out);

/* Copies one tensor into the weight arena (host or device source, any pageable/pinned/device memory), in the
 * library's streaming layout: slot `layer` of a grouped parameter (Section 3.2, rule (3): a grouped parameter is indexed
 * by the loop variable; the closing paragraph of that section: grouped tensors stored contiguously, in loop order).  `bytes` must equal the tensor's size.  layer = -1 for KL_EMBED, KL_NORM_F,
 * KL_LM_HEAD.  The copy is ordered on `stream`; the source may be released once the stream has passed it. */
kl_status kl_load_weights(kl_handle* h, int tensor, int layer, const void* src, size_t bytes, void* stream);

/* The same for one expert's matrix of a mixture-of-experts model: tensor = KL_WGATE, KL_WUP or KL_WDOWN, expert in
 * [0, n_experts).  In the looped kernel the experts' matrices are the one grouped parameter whose ADDRESS depends on an
 * activation (Section 3.2's grouping assumes addresses known up front): the weight stream of a layer's MLP starts when
 * the layer's router has run; everything else is requested ahead as for a dense model. */
kl_status kl_load_expert_weights(kl_handle* h, int tensor, int layer, int expert, const void* src, size_t bytes, void* stream);

/* Bytes of a KV cache for `batch` sequences: layout [n_layers][2 (K,V)][batch][n_kv_heads][max_ctx][head_dim]
 * bf16.  The cache is read, written and live after the call, i.e. element (6) {In, Live, Out} of the lattice of
 * Section 3.1: a grouped in/out parameter with a leading layer dimension (Eq. 3), sized as Table 1's KV column
 * (batch x context x layers x 2 x kv heads x head size x 2 bytes).  Cached keys are stored already rotated.  The cache is caller-owned and updated in place. */
size_t kl_kv_cache_bytes(const kl_handle* h, uint32_t batch);

/* KL_MODE_LOOPED (default): one persistent kernel runs all layers (4 launches per token with embedding, classifier
 * and sampling).  KL_MODE_PER_LAYER: one launch per layer (L + 3).  KL_MODE_PER_STAGE: one launch per operator group
 * of every layer -- QKV, attention, O, gate/up, down (5 L + 3): the three call schedules of Section 2, from the
 * same stage code.
 * Batches on the tensor-core path (kl_set_batched_path) have the same three schedules from one set of phase functions,
 * with identical results: KL_MODE_LOOPED = ONE cooperative launch per step (embedding, all layers, classifier; grid
 * barriers between the phases, the projections' weight stream running ahead of them), KL_MODE_PER_LAYER = that kernel
 * launched once per layer, KL_MODE_PER_STAGE = ten launches per layer joined by programmatic dependent launch
 * (kl_set_dependent_launch).  A handle on which kl_set_mode has never been called decodes batches on the per-operator
 * schedule, the fastest of the three on this GPU; after a call batches follow the mode like single sequences. */
kl_status kl_set_mode(kl_handle* h, int mode);

/* One decode step for `batch` sequences, asynchronous on `stream`.
 *   tokens_d[b]    token to embed (int32, < vocab)
 *   positions_d[b] number of valid cached positions of sequence b = index written by this step (< max_ctx);
 *                  attention covers positions 0..positions_d[b] inclusive
 *   kv_cache_d     cache in the layout above; row positions_d[b] of every layer is written
 *   logits_d       [batch, vocab] fp32, written
 * Sequences of a batch are independent (ragged positions are fine).  A batch of 2..32 sequences takes the
 * tensor-core path when the shape allows (kl_set_batched_path): every projection is one contraction for the whole
 * batch, the weights are streamed once per step.  Otherwise the sequences are decoded one after another by the
 * batch-1 kernels (weights streamed once per sequence).  Tokens and positions of the whole batch are checked before
 * anything is written: one bad entry makes the step a no-op for every sequence.
 * The step reads tokens and positions on the device and keeps its own step counter there, so a stream capture of
 * kl_decode_step + kl_argmax_advance can be replayed step after step (same buffers).
 * Merged-call argument rule of Section 3.2: weights (grouped, all layers) come from the handle, the hidden
 * state enters once (from the embedding) and leaves once (kl_read_hidden / the classifier), the KV cache is the
 * grouped in/out parameter.  Device-detected errors are reported by kl_last_status.  KL_ERR_OUT_OF_RANGE (a bad
 * token or position) is found before anything is written and makes the step a no-op.  KL_ERR_SYNC_TIMEOUT (a
 * bounded wait ran out in the middle of the step) leaves the step's logits, its cache row and the hidden state
 * undefined; the greedy entry points then leave tokens_d and positions_d as they were, and the next call starts a
 * new chain. */
kl_status kl_decode_step(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d,
                         float* logits_d, uint32_t batch, void* stream);

/* One greedy decode step, sampling included, on device buffers: decodes tokens_d at positions_d, writes the logits,
 * replaces tokens_d[b] by the next token (lowest index among the maxima) and adds one to positions_d[b].
 * For batch 1 this is ONE launch per token instead of the four of Section 2's looped schedule (embedding, looped
 * decoder, classifier, sampling): the classifier runs as one more stage of the persistent kernel, every CTA reduces
 * the logits rows it produced, and the last CTA to finish picks the token, advances the position, keeps the final
 * hidden state for kl_read_hidden and writes the next token's embedding, rotary table and step counter.  Calls are
 * therefore CHAINED: pass restart != 0 on the first call of a chain and whenever tokens_d / positions_d were changed
 * by anyone else, or another decode call was made on this handle, since the previous call (the embedding is then
 * computed from tokens_d first, one more launch);
 * restart = 0 continues the chain and must see the buffers as the previous call left them (when the handle knows
 * that there is no chain to continue -- first call, another decode call in between, another tokens_d -- it starts
 * one as if restart were set).  kl_set_mode does not
 * apply.  For batch > 1 the call is kl_decode_step followed by kl_argmax_advance, the step replayed from a CUDA graph
 * that the handle keeps per set of buffers (see kl_decode_step_host) unless `stream` is itself being captured.  When the new position reaches
 * max_ctx the status word is set to KL_ERR_OUT_OF_RANGE and the next step is a no-op. */
kl_status kl_decode_greedy(kl_handle* h, int32_t* tokens_d, int32_t* positions_d, void* kv_cache_d, float* logits_d,
                           uint32_t batch, int restart, void* stream);

/* n_tokens greedy steps in a row: after the call tokens_d / positions_d hold what n_tokens calls of kl_decode_greedy
 * would have left, and out_tokens_d[k * batch + b] (device, n_tokens * batch int32) the token sequence b picked after
 * step k.  logits_d holds the last step's logits.
 * For batch 1 the loop over the decoder layers (Section 3.3) is extended to a loop over TOKENS: one launch of the
 * persistent kernel decodes up to 256 consecutive tokens (longer runs are cut into launches of 256), with a small
 * launch before it that writes the rotary tables of the tokens' positions (position and step number advance inside the
 * kernel).
 * Inside the launch the CTA that finishes a token's sampling writes the next embedding while every other CTA already
 * holds the next token's first weight tiles: neither a launch boundary nor a pipeline restart between tokens.
 * The launch needs position + n_tokens <= max_ctx (checked on the device before anything is decoded: otherwise the
 * status word is set to KL_ERR_OUT_OF_RANGE and nothing is decoded).  restart as in kl_decode_greedy; the call continues and is
 * continued by chains of kl_decode_greedy on the same buffers.  For batch > 1 the call is a loop of kl_decode_greedy
 * with the picked tokens copied to out_tokens_d after every step. */
kl_status kl_decode_greedy_tokens(kl_handle* h, int32_t* tokens_d, int32_t* positions_d, void* kv_cache_d, float* logits_d,
                                  int32_t* out_tokens_d, uint32_t n_tokens, uint32_t batch, int restart, void* stream);

/* The same for one sequence with HOST buffers: decodes n_tokens (1..256) tokens starting from `token` at `position`,
 * copies the picked tokens to out_tokens_h (n_tokens int32) and synchronises `stream` before returning.  Always starts
 * a chain. */
kl_status kl_decode_greedy_tokens_host(kl_handle* h, int32_t token, int32_t position, void* kv_cache_d, int32_t* out_tokens_h,
                                       uint32_t n_tokens, void* stream);

/* Same step with HOST token / position / logit buffers: copies tokens and positions to the device, runs the
 * step, copies the logits back and synchronises `stream` before returning.  The KV cache stays on the device.
 * A step of the batched tensor-core path is a few hundred launches whose host cost would otherwise sit between two
 * synchronisations of every step; this entry point therefore captures it once per (kv_cache_d, batch) into a CUDA
 * graph on a stream of its own (nothing executes there) and replays the graph on `stream` afterwards -- same
 * kernels, same arguments, same results.  The graph is dropped by kl_set_batched_path, kl_set_wait_limit_ns and
 * kl_destroy; with kl_profile_enable active, or if the capture is refused, the step is launched kernel by kernel. */
kl_status kl_decode_step_host(kl_handle* h, const int32_t* tokens_h, const int32_t* positions_h, void* kv_cache_d,
                              float* logits_h, uint32_t batch, void* stream);

/* One greedy decode step with HOST buffers: tokens and positions in, the next token of every sequence out
 * (next_tokens_h[b] = lowest index among the maxima of sequence b's logits; Section 2's embedding, decoder,
 * classifier and sampling calls in one entry point).  Copies tokens and positions to the device, runs the step as
 * kl_decode_step_host does, samples on the device (kl_argmax_advance on the library's staging buffers), copies the
 * batch x 4 bytes of tokens back and synchronises `stream`.  The logits stay on the device. */
kl_status kl_decode_greedy_host(kl_handle* h, const int32_t* tokens_h, const int32_t* positions_h, void* kv_cache_d,
                                int32_t* next_tokens_h, uint32_t batch, void* stream);

/* Sampling block, the last of the four calls per token of Section 2's looped schedule (Embedding, looped Decoder,
 * Classifier, Sampling), as greedy sampling: tokens_d[b] = argmax_v logits_d[b, v] (lowest index on ties);
 * positions_d[b] += 1. */
kl_status kl_argmax_advance(kl_handle* h, const float* logits_d, int32_t* tokens_d, int32_t* positions_d,
                            uint32_t batch, void* stream);

/* The same sampling block for callers that cannot give the library any memory to work in and must not cause an
 * allocation: a sampler that runs on logits produced elsewhere and holds no kl_handle (so there is no scratch arena
 * to carve from), or a serving loop in which a device allocation would synchronise the device or fail because the
 * process has already committed all device memory to its own pools.  The paper has no counterpart of this entry
 * point; it describes the sampling block only as one of the calls around the looped decoder (Section 2).
 *
 * The per-block partial results and the completion tickets live in a fixed array that is part of the library
 * image (KL_STATIC_ARGMAX_MAX_BATCH sequences, about 130 KB per device); nothing is allocated or freed, here or
 * inside the CUDA runtime routines this call uses (a symbol-address query, a memset node and a kernel launch).
 *   logits_d    [batch, vocab] fp32 on the current device
 *   tokens_d    [batch] int32, written: argmax (lowest index on ties)
 *   positions_d [batch] int32, incremented
 *   batch       1..KL_STATIC_ARGMAX_MAX_BATCH; larger -> KL_ERR_TOO_LARGE, nothing is launched
 * The first call on a device looks up the array's address (with that device current): make that first call outside
 * any stream capture, before the latency-critical part of the program.  Every call on a device shares the one
 * array, which keeps whatever the previous call left; the call itself clears the tickets it is about to use, in
 * stream order.  Two calls that may run at the same time on one device (different streams, or different host
 * threads without ordering) would race on the array: order them. */
#define KL_STATIC_ARGMAX_MAX_BATCH 256
kl_status kl_argmax_advance_static(const float* logits_d, uint32_t vocab, int32_t* tokens_d, int32_t* positions_d,
                                   uint32_t batch, void* stream);

/* The hidden state is the loop-carried {In, Local} / {Local, Out} pair of the merged kernel: it lives in the kernel's
 * own buffers for all L iterations and is stored once after the loop (Section 3.2, rules (6) and (10)); this call
 * returns that single store.
 * Copies the hidden state after the last decoder layer (before the final RMSNorm) of the latest step:
 * hidden_d [batch, hidden] fp32; batch must be the latest step's. */
kl_status kl_read_hidden(kl_handle* h, float* hidden_d, uint32_t batch, void* stream);

/* No counterpart in the paper (its kernels report no errors): the bounded device-side waits and the range checks of
 * this library report through one status word.
 * Synchronises nothing: call after the stream has been synchronised.  Reads and clears the device status word
 * (KL_OK, KL_ERR_SYNC_TIMEOUT or KL_ERR_OUT_OF_RANGE).  The word is sticky: once a step has set it, every later
 * step on the handle is a no-op until this call has read (and thereby cleared) it. */
kl_status kl_last_status(kl_handle* h);

/* Number of kernels this handle has launched so far (for reporting). */
uint64_t kl_launch_count(const kl_handle* h);

/* Per-kernel timing for roofline reports.  kl_profile_enable creates `capacity` sets of CUDA events (no device
 * memory); from then on every kl_decode_step records events around its decoder launches and its classifier launch
 * on the caller's stream, into set (step index mod capacity).  capacity = 0 switches recording off and destroys
 * the events.  kl_profile_read (after the stream has been synchronised) returns, for the latest min(steps,
 * capacity) steps, the milliseconds between the first decoder launch and the end of the last one, and of the
 * classifier kernel; *n is in: room in the arrays, out: entries written. */
kl_status kl_profile_enable(kl_handle* h, uint32_t capacity);
kl_status kl_profile_read(kl_handle* h, uint32_t* n, float* decoder_ms, float* classifier_ms);

/* Stage timeline of the decoder kernel (the analogue of the paper's per-socket HBM-bandwidth trace, Section 4).
 * trace_d: DEVICE buffer of n_ctas * n_layers * n_stamps + 8192 * 4 uint64 (zero it first), or NULL to switch
 * tracing off; the three sizes are returned through the out pointers (each may be NULL).  While set, consumer
 * thread 0 of every CTA stores the GPU global timer (ns) at fixed points of every layer:
 *    0 layer entered (starts polling the hidden state)      8 thread 0 holds valid words of it
 *    1 input normalised                                     2 QKV rows of this CTA done
 *   14 attention prologue done (q, k, v polled, rotated)   15 this warp's ring chunks of the unit consumed
 *    3 partial result of the unit written                   5 thread 0's loads for the slice merge complete
 *    4 attention block done                                 6 attention output loaded
 *    7 O-projection rows done                              11 thread 0 holds valid words of x'
 *    9 x' normalised                                       10 gate/up rows done
 *   12 counter of the gate/up stage passed                 13 down-projection rows done
 * The trailing 8192 x 4 block logs the first 8192 ring chunks of CTA 0: [0] issue by the producer, [2] chunk seen
 * landed by its consumer warp, [1] dot product done, [3] results emitted.  Stamps of the latest step overwrite
 * earlier ones.  kl_decode_step and kl_decode_greedy (batch 1) both take the stage stamps; the chunk log is written by
 * kl_decode_step in the plain mode only. */
kl_status kl_set_trace(kl_handle* h, uint64_t* trace_d, uint32_t* n_ctas, uint32_t* n_layers, uint32_t* n_stamps);

/* Attention inner loop.  on = 1 (default when head_dim is 64 or 128): tensor-core loop (mma.sync on 128-byte
 * swizzled TMA boxes of the cache); on = 0: CUDA-core loop on linear copies (always used for other head sizes;
 * built for 1, 2, 4 and 8 query heads per kv head: KL_ERR_UNSUPPORTED_SHAPE for other group sizes, and for handles
 * in stash mode, whose kernels carry the tensor-core loop only -- create the model with KL_FLAG_NO_STASH to use
 * on = 0).  In stash mode the chunk log of kl_set_trace stays empty (stage stamps are taken). */
kl_status kl_set_tensor_core_attention(kl_handle* h, int on);

/* 1: the handle's batch-1 kernels run in stash mode (see KL_FLAG_NO_STASH), 0: plain mode, negative: h is null.  No
 * counterpart in the paper. */
int kl_stash_mode(const kl_handle* h);

/* Decode steps of a batch (batch > 1).  on = 1 (default when available): the tensor-core path -- every projection
 * of the step (QKV, O, gate/up, down, classifier) is one dense contraction for the whole batch on the tcgen05 tensor
 * cores (M = 128 weight rows x N = 64 = 32 sequences x (hi, lo bf16 halves of the fp32 input), fp32 accumulators in
 * TMEM), so the weights are streamed once per step instead of once per sequence -- at batch 32 the projections are
 * dense contractions (Table 1 of the paper); attention runs as one balanced stream of K|V chunks over all (sequence,
 * kv head) pairs.  kl_set_mode selects the call schedule of the step (see there).  on = 0: the batch-1 kernels in the mode of kl_set_mode, sequence after sequence.  Available when
 * max_batch is 2..32, head_dim is 64 or 128, hidden / q width / ffn are multiples of 8, every projection has at
 * least 128 rows and the driver exports cuTensorMapEncodeTiled; otherwise KL_ERR_UNSUPPORTED_SHAPE for on = 1. */
kl_status kl_set_batched_path(kl_handle* h, int on);

/* How the kernels of a batched step (ten per layer: the per-operator call schedule of Section 2) follow one
 * another.  on = 1 (default): programmatic dependent launch -- a kernel may start while its predecessor still runs,
 * sets itself up and requests weight tiles, and waits for the predecessor only before it touches the step's
 * buffers.  on = 0: plain stream order, every kernel starts when the one before it has ended.  Same results; the
 * switch exists so that the cost of the launch boundaries can be measured. */
kl_status kl_set_dependent_launch(kl_handle* h, int on);

/* Limit, in nanoseconds, of every device-side wait (tagged word, counter or mbarrier).  Default 2e9. */
kl_status kl_set_wait_limit_ns(kl_handle* h, uint64_t ns);

/* Test hook for the bounded waits: when stage >= 0 the results of that stage (0 QKV, 1 attention, 2 O, 3 gate/up,
 * 4 down) of layer 0 are published with a tag nobody waits for (stage 3: its counter is not incremented) on the
 * NEXT kl_decode_step only, so the waits on them run out and the step reports KL_ERR_SYNC_TIMEOUT.  No fault, trap
 * or endless loop is involved. */
kl_status kl_debug_skip_signal_once(kl_handle* h, int stage);

/* Test hook for the synchronisation protocol of the batch-1 persistent kernels (the tagged words and the counter that
 * replace kernel boundaries, Section 3.2): with seed != 0 and max_ns > 0 every CTA sleeps a pseudo-random time below
 * max_ns (at most 1 ms) whenever it enters a stage, a different one per (CTA, step, layer, stage), so that the CTAs
 * meet every exchange in a different order from step to step; the kernels then run in their instantiation with the
 * debug hooks compiled in.  Results must not change by a bit.  max_ns = 0 switches the hook off.  No counterpart in
 * the paper. */
kl_status kl_debug_set_jitter(kl_handle* h, uint32_t seed, uint32_t max_ns);

/* Test hook for the step numbers behind the tags.  Every decoded token takes one step number; the tags hold 28 bits of
 * (step x n_layers + layer), so after *wrap_at steps (about 2^28 / n_layers: 8.4 million tokens at 32 layers) the
 * library clears its tagged scratch areas at the next launch boundary and starts numbering again at 1 -- a tagged word
 * left over from the previous use of a number can therefore never be taken for a fresh one.  This call sets the
 * counter (device word; synchronous; the stream must be idle) so that a test can step across the wrap;
 * step = 0xffffffff only queries.  wrap_at may be NULL. */
kl_status kl_debug_set_step(kl_handle* h, uint32_t step, uint32_t* wrap_at);

const char* kl_status_string(kl_status s);

/* Releases host-side state only (the arenas belong to the caller). */
void kl_destroy(kl_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* KL_H_ */
