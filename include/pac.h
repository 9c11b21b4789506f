/*
 * pac.h - C ABI of the adapter-over-cache trainer (one GPU, sm_100a).
 *
 * The library trains the Parallel Adapters side network of PAC+ (arXiv
 * 2408.10746) from an activation cache: the frozen backbone's per-layer hidden
 * states b_1..b_L of every training sample, stored once, so that later epochs
 * never run the backbone (Section IV-B, "Activation Cache for Parallel
 * Adapters"; Section V-B, data-parallel fine-tuning of the adapters alone).
 *
 * Model (Section IV-A, "Parallel Adapters Architecture"), per token row, with
 * h_l the cached state of layer l (l = 1..L), adapter width r, a_0 = 0:
 *     u_l = h_l W_down^l                       down-projection, W_down^l in R^{d x r}
 *     z_l = lambda_l u_l + (1 - lambda_l) a_{l-1}     learnable scalar mix, lambda init 0.5
 *     a_l = phi(z_l)                           adapter body (ReLU or identity)
 *     y   = h_L + a_L W_up                     up-projection, summed with the backbone output
 * Heads: PAC_HEAD_MEANPOOL_CLS  logits = mean_s(y) W_head + b_head, loss = mean softmax
 * cross-entropy over the batch (head is trainable); PAC_HEAD_FROZEN_LM  logits = y W_lm^T
 * with a borrowed, frozen W_lm, loss = mean cross-entropy over all B*S positions.
 * Gradients reach the adapter parameters only; nothing is ever written toward the cache.
 *
 * Conventions
 *  - Every pointer argument says "host" or "device".  Device pointers are plain
 *    CUDA device addresses on the context's device.
 *  - Borrowed memory (cache, labels, LM head) must outlive the context and is never
 *    written.  Parameters, gradients, optimizer moments and scratch are owned by the
 *    context (allocated in pac_adapter_init, freed in pac_destroy).
 *  - Flat parameter layout (fp32), used by every get/set call:
 *        W_down[L][d][r] | lambda[L] | W_up[r][d] | W_head[d][C] | b_head[C]
 *    (the last two only with PAC_HEAD_MEANPOOL_CLS); with PAC_BODY_TRANSFORMER followed, for every
 *    layer l = 0..L-1, by  g1[r] | b1[r] | Wq[r][r] | Wk[r][r] | Wv[r][r] | Wo[r][r] | g2[r] | b2[r] |
 *    W1[r][f] | c1[f] | W2[f][r] | c2[r].
 *  - Every call returns a pac_status and never throws or aborts.  Arguments are
 *    checked on the host before any launch; on error no device state changes.
 *    pac_last_error() gives a message for the most recent failure on a context.
 *  - A context is not thread-safe.  All work is enqueued on the context's stream.
 *  - There is no CPU fallback: without a usable CUDA device pac_create fails.
 */
#ifndef PAC_H
#define PAC_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pac_ctx pac_ctx;

typedef enum {
    PAC_OK = 0,
    PAC_ERR_INVALID_ARG = 1,      /* null pointer, non-positive size, bad enum */
    PAC_ERR_BAD_STATE = 2,        /* call order: create -> cache_register -> adapter_init -> ... */
    PAC_ERR_SAMPLE_ID_RANGE = 3,  /* a sample id outside [0, N) */
    PAC_ERR_UNSUPPORTED = 4,      /* shape/dtype combination the kernels do not cover */
    PAC_ERR_NOMEM = 5,            /* device or pinned-host allocation failed */
    PAC_ERR_CUDA = 6,             /* a CUDA runtime/driver call failed */
    PAC_ERR_TIMEOUT = 7           /* a bounded device-side wait ran out */
} pac_status;

typedef enum { PAC_F32 = 0, PAC_BF16 = 1 } pac_dtype;
typedef enum { PAC_ACT_RELU = 0, PAC_ACT_IDENTITY = 1 } pac_act;
typedef enum { PAC_HEAD_MEANPOOL_CLS = 0, PAC_HEAD_FROZEN_LM = 1 } pac_head;
/* Adapter body (Section IV-A): the point-wise activation `act`, or one reduced-width transformer
 * encoder layer per adapter ("a lightweight version of the backbone"; Section VI-A: every weight and
 * hidden dimension 1/rho of the backbone's):
 *     x  = lambda_l u_l + (1 - lambda_l) a_{l-1};  n1 = LayerNorm(x);  q,k,v = n1 Wq, n1 Wk, n1 Wv
 *     x' = x + concat_h(softmax(q_h k_h^T / sqrt(r/H)) v_h) Wo;  n2 = LayerNorm(x')
 *     a_l = x' + relu(n2 W1 + c1) W2 + c2
 * (pre-norm, bidirectional attention over the S tokens of a sample, LayerNorm eps 1e-5 with gain and
 * bias, no dropout).  Classifier head only; it runs on the plain fp32 kernels. */
typedef enum { PAC_BODY_POINTWISE = 0, PAC_BODY_TRANSFORMER = 1 } pac_body;

typedef struct {
    int r;               /* adapter width (the paper's d / reduction factor) */
    int act;             /* pac_act */
    int head;            /* pac_head */
    int n_out;           /* classes C, or vocabulary size V for the LM head */
    float lambda_init;   /* 0.5 in the paper */
    int max_batch;       /* largest B any later call will pass */
    const void* lm_head; /* device, [V][d] bf16, borrowed, frozen; NULL for the classifier head */
    int body;            /* pac_body; 0 = point-wise */
    int n_heads;         /* transformer body: attention heads H (r a multiple of H) */
    int ffn_width;       /* transformer body: width f of the feed-forward layer (e.g. 4 r) */
} pac_adapter_cfg;

typedef struct { float lr, beta1, beta2, eps, weight_decay; } pac_adamw;

/* Options for pac_set_option. */
typedef enum {
    PAC_OPT_KERNEL_PATH = 0,  /* 0 = automatic: tensor-core path when the shape allows.  Its forward half
                                     (down-projections + classifier-head phase) runs as ONE launch per step for
                                     short sequences (bf16 cache, classifier head, S <= 128, r <= 64) when the
                                     batch's clusters all fit on the device at once; with enough 128-token
                                     tiles to fill the device (2 * B * ceil(S/128) >= SMs, r a multiple of 32 up
                                     to 128) the merge / activation chain runs in the epilogue of the
                                     down-projection kernel instead; otherwise two plain launches,
                                 1 = force the plain fp32-FMA kernels,
                                 2 = tensor-core path, forward half always as two plain launches,
                                 3 = tensor-core path, one-launch forward whenever the shape allows it,
                                 4 = tensor-core path, chain-in-epilogue forward whenever the shape allows it (with
                                     r > 64 and an even number of 128-token tiles its CTAs work in pairs that share
                                     each weight tile),
                                 5 = as 4, but never in CTA pairs;
                                 set before adapter_init */
    PAC_OPT_KERNEL_TIMING = 1 /* 0 = off (default), 1 = bracket the cache-stream kernels with events
                                 (pac_kernel_times), 2 = device-side timestamps of the two passes' stream
                                 phases on the tensor-core path (pac_stream_phase_times) */
} pac_option;

/* Creates a context on CUDA device `device`.  `cuda_stream` is a cudaStream_t to
 * enqueue all work on, or NULL for a stream the context creates and owns. */
pac_status pac_create(pac_ctx** out, int device, void* cuda_stream);
pac_status pac_destroy(pac_ctx* ctx);

/* Registers the activation cache (Section IV-B): dev_cache is a device array
 * [N][L][S][d] of `dtype`, row-major, 16-byte aligned, borrowed and read-only.
 * dev_labels is a device int32 array [N] (labels_per_sample = 1, classifier) or
 * [N][S] (labels_per_sample = S, LM targets), borrowed and read-only.
 * Re-registering is allowed before pac_adapter_init only. */
pac_status pac_cache_register(pac_ctx* ctx, const void* dev_cache, int dtype, long long N, int L, int S, int d,
                              const int* dev_labels, int labels_per_sample);

/* The same for a cache that does not fit (or should not occupy) device memory (Section V-B,
 * storage cost analysis: the cache is kept on storage and reloaded per micro-batch).  host_cache is
 * HOST memory, [N][L][S][d] of `dtype`, 16-byte aligned; host_labels is HOST int32 memory, [N] or
 * [N][S]; both borrowed and read-only until pac_destroy.  Page-locked memory (cudaHostAlloc /
 * cudaHostRegister) lets the reload overlap the computation; pageable memory works but every copy
 * then waits for the host.  pac_adapter_init allocates two device staging slots of max_batch
 * samples each (2 * max_batch * L*S*d elements).  Every call that takes host sample ids
 * (pac_train_step, pac_train_step_async, pac_train_epoch, pac_eval_logits, pac_gather) first copies
 * the slabs and labels of its ids into a slot, one contiguous copy per sample on a copy stream of
 * the context's own, and runs the same kernels on the slot; the copies of a step overlap the
 * kernels of the step before it, and the host runs at most two steps ahead of the copies.  Results
 * are bit-identical to those on a device-resident cache.  pac_train_epoch_dev (ids on the device)
 * returns PAC_ERR_UNSUPPORTED in this mode. */
pac_status pac_cache_register_host(pac_ctx* ctx, const void* host_cache, int dtype, long long N, int L, int S, int d,
                                   const int* host_labels, int labels_per_sample);

/* The same for a cache kept in a FILE (Section IV-B: the activations are recorded during the first
 * epoch; Section V-B, storage cost analysis: they live on storage and are reloaded per micro-batch).
 * `path` (host string) names a file written by pac_cache_writer_*: a 64-byte header (magic
 * "PACCACHE", version, dtype, N, L, S, d, labels_per_sample), the cache [N][L][S][d], then, at the next
 * multiple of 64 bytes, the int32 labels.
 * The file is mapped read-only until pac_destroy and then treated as a host-resident cache
 * (pageable memory: the copies of a step overlap the GPU work of the step before, the host waits for
 * the page cache / storage).  Errors: PAC_ERR_INVALID_ARG for a missing, truncated or foreign file,
 * PAC_ERR_NOMEM when the mapping fails, PAC_ERR_BAD_STATE after pac_adapter_init. */
pac_status pac_cache_register_file(pac_ctx* ctx, const char* path);

/* Writer side of a cache file: what the first epoch does with each sample's backbone activations
 * (Section IV-B).  create makes (or truncates) `path` for N samples of L x S x d elements of `dtype`
 * with labels_per_sample (1 or S) int32 labels each; store copies one sample - `slabs` is [L][S][d],
 * device memory when slabs_on_device != 0 (copied on cuda_stream, which the call waits for) or host
 * memory - and its labels (host) into place, in any order, any number of times; close flushes and
 * unmaps.  Samples never stored read as zeros.  The writer needs no pac_ctx; a backbone forward hands
 * it each layer stack as it is produced.  info reads a file's header (any pointer may be NULL).
 * Errors: PAC_ERR_INVALID_ARG (bad sizes, unopenable path, foreign file), PAC_ERR_SAMPLE_ID_RANGE,
 * PAC_ERR_NOMEM, PAC_ERR_CUDA (device copy failed, or a device source without a usable device). */
typedef struct pac_cache_writer pac_cache_writer;
pac_status pac_cache_writer_create(pac_cache_writer** out, const char* path, int dtype, long long N, int L, int S, int d,
                                   int labels_per_sample);
pac_status pac_cache_writer_store(pac_cache_writer* w, long long sample_id, const void* slabs, int slabs_on_device,
                                  const int* host_labels, void* cuda_stream);
pac_status pac_cache_writer_close(pac_cache_writer* w);
pac_status pac_cache_file_info(const char* path, int* dtype, long long* N, int* L, int* S, int* d, int* labels_per_sample);

/* Allocates parameters, gradients, AdamW moments and scratch for batches up to
 * cfg->max_batch and fills the parameters from `seed`:
 * W_down ~ N(0, 1/d), lambda = lambda_init, W_up = 0, W_head ~ N(0, 1/d), b_head = 0
 * (transformer bodies: LayerNorm gains 1, all biases 0, Wq, Wk, Wv, Wo, W1 ~ N(0, 1/r), W2 ~ N(0, 1/f):
 * the paper initialises them by pruning the backbone, whose weights are not part of this path)
 * (zero up-projection so the initial model equals backbone + head, the rationale of
 * Section IV-C).  Element i of the flat vector is a function of (seed, i) only.
 * For the classifier head this call also reads the last cached layer of every sample
 * once to store its token mean (a per-sample constant of the frozen backbone). */
pac_status pac_adapter_init(pac_ctx* ctx, const pac_adapter_cfg* cfg, unsigned long long seed);

/* One minibatch: gather cached states of sample_ids (host, B ints, duplicates allowed),
 * adapter forward, loss, adapter backward.  Overwrites the gradients; does not change
 * parameters.  If loss_out (host) is non-NULL the call waits for the stream and stores
 * the mean loss; if NULL the call returns as soon as the work is enqueued. */
pac_status pac_train_step(pac_ctx* ctx, const int* sample_ids, int B, float* loss_out);

/* One whole training step without waiting: pac_train_step on sample_ids (host, B ints) followed by
 * the AdamW update of pac_adam_step with `hp`, all enqueued on the context's stream; the call
 * returns as soon as that is done (it waits only when too many earlier steps' ids are still in
 * flight: 8, or 32 to 64 with the one-launch forward).  If loss_out is non-NULL the step's mean loss
 * arrives there once the step has run: loss_out is HOST memory that must stay valid until the next
 * pac_sync; read it after pac_sync.  Page-locked memory (cudaHostAlloc / cudaHostRegister) is written
 * by the last kernel of the step itself; other memory gets a copy behind the step.  With the one-launch
 * forward the ids are likewise taken by the kernels from a page-locked ring inside the library (the
 * step before fetches them into device memory when the host is already a call ahead, otherwise the
 * forward kernel reads them across the host link), so a step is three kernels back to back and
 * consecutive steps overlap as in pac_train_epoch_dev.  Errors of the arguments are reported at once,
 * device-side errors by the next pac_sync.  The step a caller loops over when the minibatches
 * are chosen on the host one at a time (Section IV-B: from the second epoch on a step needs
 * nothing but the cached activations of its samples). */
pac_status pac_train_step_async(pac_ctx* ctx, const int* sample_ids, int B, const pac_adamw* hp, float* loss_out);

/* pac_train_step without any wait and with the loss left on the device: the step is enqueued and
 * the call returns; the mean loss of the minibatch is written to *dev_loss (device, one float; NULL
 * keeps it in a buffer of the context).  The per-step call of data-parallel training (Section V-B:
 * every device trains on its share of the minibatch, then the devices combine the adapter
 * gradients): a collective enqueued behind this call on the context's stream reduces the gradient
 * buffer of pac_device_buffers in place, pac_adam_step follows, and the host reads losses once per
 * epoch instead of once per step. */
pac_status pac_train_step_dev_loss(pac_ctx* ctx, const int* sample_ids, int B, float* dev_loss);

/* Factor in (0, 1] that every optimizer update (pac_adam_step and the updates fused into
 * pac_train_step_async / pac_train_epoch*) applies to each gradient as it reads it; the gradient
 * buffer keeps its values.  1 by default.  With W data-parallel ranks whose gradient buffers hold the
 * SUM over ranks after an all-reduce, 1/W makes the update use the mean (Section V-B). */
pac_status pac_set_grad_scale(pac_ctx* ctx, float scale);

/* AdamW on the adapter parameters (and the classifier head) from the current gradients:
 * decoupled decay on W_down, W_up, W_head; none on lambda and b_head; bias-corrected
 * moments; step counter advances by one. */
pac_status pac_adam_step(pac_ctx* ctx, const pac_adamw* hp);

/* Forward only.  dev_out (device, fp32): [B][C] for the classifier head, [B][S][V] for
 * the LM head.  sample_ids is a host array. */
pac_status pac_eval_logits(pac_ctx* ctx, const int* sample_ids, int B, float* dev_out);

/* Cache gather alone: dev_out (device, cache dtype) [L][B][S][d] with
 * dev_out[l][b] = cache[sample_ids[b]][l], bit for bit.  sample_ids is a host array. */
pac_status pac_gather(pac_ctx* ctx, const int* sample_ids, int B, void* dev_out);

/* Runs train_step + adam_step for every consecutive B-slice of perm (host, n ids,
 * n a multiple of B) with one wait at the end.  losses_out (host, n/B floats) may be NULL. */
pac_status pac_train_epoch(pac_ctx* ctx, const int* perm, long long n, int B, const pac_adamw* hp,
                           float* losses_out);

/* The same with ids and losses resident on the device: dev_perm (device int32, n ids,
 * validated on the device: an out-of-range id is clamped into range, counted, and reported
 * as PAC_ERR_SAMPLE_ID_RANGE by the next pac_sync), dev_losses (device fp32, n/B, may be
 * NULL).  Returns without waiting. */
pac_status pac_train_epoch_dev(pac_ctx* ctx, const int* dev_perm, long long n, int B, const pac_adamw* hp,
                               float* dev_losses);

/* Checkpointing and inspection (host buffers of pac_param_count floats). */
pac_status pac_param_count(pac_ctx* ctx, long long* n);
pac_status pac_get_params(pac_ctx* ctx, float* host);
pac_status pac_set_params(pac_ctx* ctx, const float* host);
pac_status pac_get_grads(pac_ctx* ctx, float* host);
pac_status pac_get_opt_state(pac_ctx* ctx, float* m, float* v, long long* step);
pac_status pac_set_opt_state(pac_ctx* ctx, const float* m, const float* v, long long step);

/* Device addresses of the context's flat fp32 parameter and gradient vectors (pac_param_count
 * floats each, owned by the context, valid until pac_destroy).  For data-parallel training
 * (Section V-B: every device holds the adapter parameters, trains on its share of the minibatch
 * and the devices combine gradients): a collective library can reduce *dev_grads in place between
 * pac_train_step and pac_adam_step, and broadcast *dev_params once at the start.  After writing
 * to the parameters through this pointer call pac_params_changed() so that derived copies (the
 * bf16 weight shadow) are refreshed.  Order all accesses on the context's stream. */
pac_status pac_device_buffers(pac_ctx* ctx, float** dev_params, float** dev_grads);
pac_status pac_params_changed(pac_ctx* ctx);

pac_status pac_set_option(pac_ctx* ctx, int option, int value);
/* Per-kernel device times.  With PAC_OPT_KERNEL_TIMING = 1 the kernels of every later train
 * step are bracketed by CUDA events on the context's stream, in four groups:
 *   [0] down-projection u_l = h_l W_down^l over all layers (first pass over the cache)
 *   [1] merge/activation chain, head, loss and the reverse chain
 *   [2] dW_down = h_l^T du_l over all layers (second pass over the cache)
 *   [3] gradient finalisation (+ AdamW when fused into the step)
 * When the forward half runs as one kernel (pac_kernel_path() == "tensor+fused_forward") that
 * kernel is counted in group [0] and group [1] stays empty.  With the frozen LM head on the tensor
 * cores, group [1] is the logits GEMM (logits = y W_lm^T) and group [3] the dy GEMM
 * (dy = dlogits W_lm), each 2*B*S*V*d flop.
 * This call waits for the stream, then stores the summed milliseconds and the number of
 * bracketed launches since the last call in out_ms[4] and out_count[4] (host arrays).
 * At most 4096 brackets per group are kept between two calls. */
pac_status pac_kernel_times(pac_ctx* ctx, double* out_ms, long long* out_count);
/* Stream phases of the two passes over the cached activations (Section IV-B), timed on the device.
 * With PAC_OPT_KERNEL_TIMING = 2 every later launch of a tensor-core cache pass records, through
 * %globaltimer, the earliest time any of its CTAs issued its first cache copy and the latest time
 * any of its CTAs saw its last accumulator complete.  The difference is the time the minibatch's
 * slabs took to stream from memory through the tensor cores, without the kernel's launch, set-up
 * and (for the one-launch forward) its chain / head phase; the launch overlap between the kernels
 * of a step stays as it is without timing.  This call waits for the stream, then stores the summed
 * milliseconds and the number of timed launches since the last call in out_ms[2] / out_count[2]
 * (host arrays): [0] first pass (down-projections), [1] second pass (dW_down).  At most 1024
 * launches per pass are kept between two calls. */
pac_status pac_stream_phase_times(pac_ctx* ctx, double* out_ms, long long* out_count);
/* Number of kernels this context has launched so far. */
pac_status pac_launch_count(pac_ctx* ctx, long long* n);
/* Waits for the context's stream; reports device-side status words (bounded waits that
 * ran out, ids clamped by pac_train_epoch_dev). */
pac_status pac_sync(pac_ctx* ctx);
/* What a timeout means for the training state.  Every wait inside the pipeline kernels (on a copy, an
 * accumulator, a peer CTA) gives up after about a second, records PAC_ERR_TIMEOUT in the device status
 * words and lets its kernel finish without its results.  From that moment until the next pac_sync every
 * optimizer update (fused or pac_adam_step) finds the flag and leaves parameters, moments and gradients
 * untouched; pac_sync reports PAC_ERR_TIMEOUT once, clears the flag and takes the skipped updates off the
 * step counter.  Only the step in which the wait ran out can be half applied (when it was the second
 * pass that gave up, the head-side parameters of that step are already updated): restore the last
 * checkpoint (pac_set_params / pac_set_opt_state) after a PAC_ERR_TIMEOUT unless the timed-out call was
 * pac_selftest_wait_expiry.
 *
 * pac_selftest_wait_expiry exercises that path without breaking anything: one CTA allocates tensor
 * memory, waits limit_ns nanoseconds (1e3 .. 1e8) on a barrier nobody arrives at, and leaves the way the
 * pipeline kernels do after an abort.  The call waits for the stream; it returns PAC_OK when the wait
 * reported expiry, and the status word it set is then reported by the next pac_sync like any other
 * timeout.  The paper describes no failure handling for this path; this is the library's own contract. */
pac_status pac_selftest_wait_expiry(pac_ctx* ctx, unsigned long long limit_ns);
const char* pac_last_error(const pac_ctx* ctx);
/* Which kernels the next train step will use (valid after adapter_init): "simt", "tensor",
 * "tensor+fused_forward" when a batch of max_batch samples runs the down-projections
 * (Section IV-A) and the whole classifier-head phase as one launch per step, or
 * "tensor+chain_forward" when the merge / activation chain runs in the down-projection kernel's epilogue. */
const char* pac_kernel_path(const pac_ctx* ctx);

/* Block-wise absmax INT8 quantisation, Section IV-D, Eq. 1 (the paper applies it to the frozen
 * backbone's weights; here it is a stand-alone codec over any fp32 device array):
 *     c_j = 127 / absmax(block j),   q = round(c_j * x)  (fp32 arithmetic, ties to even)
 * for every block j of `block` consecutive elements (the last may be shorter); an all-zero block
 * gets c_j = 0 and codes 0.  dev_x: device, n floats, read-only.  dev_q: device, n int8 codes.
 * dev_c: device, ceil(n / block) quantisation constants.  Enqueued on cuda_stream (NULL: default
 * stream) of `device`; nothing is allocated.  Errors: PAC_ERR_INVALID_ARG for NULL pointers or
 * non-positive sizes, PAC_ERR_CUDA when the launch fails. */
pac_status pac_quantize_absmax(int device, void* cuda_stream, const float* dev_x, long long n, int block,
                               signed char* dev_q, float* dev_c);
/* Dequantisation, Eq. 2: dev_out[i] = dev_q[i] / c_j (0 where c_j == 0), fp32.  Same conventions. */
pac_status pac_dequantize_absmax(int device, void* cuda_stream, const signed char* dev_q, const float* dev_c, long long n,
                                 int block, float* dev_out);

/* Evaluation forward that allocates nothing (the paper has no counterpart; this is a
 * packaging variant of pac_eval_logits for the mean-pool classifier head).
 *
 * Who needs it: code that runs where device allocation is off limits - inside a host
 * application that has handed all device memory to its own pool, in a latency-critical serving
 * loop that must never hit the allocator's implicit synchronisation, or in a plugin that is only
 * given raw buffers.  Such callers cannot create a pac_ctx (pac_adapter_init allocates).
 *
 * The forward's intermediates (u_l and a_l for every layer, pooled vectors, a token mean of the
 * last cached layer for the B samples) live in one fixed array of PAC_STATIC_SCRATCH_BYTES
 * (8 MiB) that is part of the library image: every GPU that loads the library holds it until the
 * process exits.  A call is rejected with PAC_ERR_UNSUPPORTED when
 *     4 * (2*L*B*S*r + B*r + B*d + B) bytes (each block rounded up to 256) exceed that size.
 * The first call on a device looks up the array's device address; make that first call outside
 * any stream capture.  No call allocates or frees device or pinned memory.
 *
 * All calls on a device share the array.  Every part of it is rewritten before it is read, so a
 * call never sees the previous call's contents, but two calls whose kernels overlap on the GPU
 * (different streams, no ordering) race on it: order them.
 *
 * Arguments: device, cuda_stream (cudaStream_t or NULL for the default stream); dev_cache, dtype,
 * N, L, S, d as in pac_cache_register (device, read-only); dev_params: device, flat fp32 vector
 * in the layout W_down[L][d][r] | lambda[L] | W_up[r][d] | W_head[d][C] | b_head[C]; r, act
 * (pac_act), n_out = C; dev_sample_ids: device, B int32 ids (an id outside [0, N) is clamped
 * into range, not reported); dev_out: device, fp32 [B][C]; err / err_len: optional host buffer
 * that receives a message when the status is not PAC_OK.  The work is enqueued on the stream;
 * dev_out is valid once the stream has reached that point.  The call makes `device` current while
 * it runs and puts the caller's current device back before it returns.  Limits beside the scratch
 * size: L <= 65535, (d + C + 32) floats within 48 KB of shared memory. */
#define PAC_STATIC_SCRATCH_BYTES (8u << 20)
pac_status pac_eval_logits_static(int device, void* cuda_stream, const void* dev_cache, int dtype, long long N, int L,
                                  int S, int d, const float* dev_params, int r, int act, int n_out,
                                  const int* dev_sample_ids, int B, float* dev_out, char* err, int err_len);

#ifdef __cplusplus
}
#endif
#endif /* PAC_H */
