/*
 * lgc.h -- C ABI of the Learned Gradient Compression (LGC) per-step path for NVIDIA B200 (sm_100a).
 *
 * The library runs, for K data-parallel nodes held as K rows of buffers on ONE device, the
 * per-iteration compression pipeline of "Learned Gradient Compression for Distributed Deep
 * Learning" (arXiv 2103.08870): local accumulation with momentum correction, per-layer top-k
 * magnitude selection, gather, the autoencoder's encoder, the across-node combination of the
 * codes, the decoder, and the scatter back into a dense update while the sent entries leave the
 * residual buffers; plus one training step of the autoencoder.
 *
 * Conventions common to every entry point
 *  - Memory.  The caller owns every device byte: `state`, `scratch`, `params`, the gradients and
 *    the update.  The library allocates no device memory and frees none; `lgc_ctx` is its only
 *    host allocation (released by lgc_destroy).  Device pointers must be 16-byte aligned.
 *  - Streams.  All work is ordered by the stream given in lgc_config.stream (a cudaStream_t,
 *    NULL = the legacy default stream): when that stream has drained, everything a call
 *    enqueued has run.  Two calls fork onto streams of the library's own and join back before
 *    they return control of the ordering to that stream: lgc_topk of the parameter-server
 *    variant (small layers beside the large ones) and lgc_step_host (the upload).  Those streams
 *    and their events are created at the first such call and released by lgc_destroy.  Stage
 *    calls never synchronise; lgc_init, lgc_check and the host-pointer forms of the parameter
 *    accessors do.
 *  - Errors.  Every call returns an lgc_status; nothing aborts, throws or traps.  Argument and
 *    call-order errors are detected on the host before anything is enqueued.  Inconsistencies a
 *    kernel detects are recorded in a device word that lgc_check reads.
 *  - Layout.  A node's gradient is one flat fp32 vector of N = sum_l n_l elements, layers
 *    back to back in the order of `layer_numel`; K nodes are K such rows, row stride N.
 *    Indices are int32 offsets inside a row (N < 2^31); offsets across rows are 64 bit.
 *  - Call order inside one step:
 *        lgc_accumulate -> lgc_topk -> lgc_encode -> lgc_combine -> lgc_decode_scatter
 *    or, while the autoencoder is being trained (second phase of Section V-B):
 *        lgc_accumulate -> lgc_topk -> [lgc_ae_train_step] -> lgc_topk_scatter
 *    Any other order returns LGC_ERR_BAD_STATE and enqueues nothing.
 */
#ifndef LGC_H
#define LGC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lgc_ctx lgc_ctx; /* opaque, host side */

typedef enum {
    LGC_OK = 0,
    LGC_ERR_INVALID_ARG = 1,  /* null/misaligned pointer, size out of range */
    LGC_ERR_BAD_STATE = 2,    /* stage called out of order */
    LGC_ERR_WORKSPACE = 3,    /* a caller buffer is smaller than lgc_workspace_bytes says */
    LGC_ERR_UNSUPPORTED = 4,  /* configuration outside what the kernels are built for */
    LGC_ERR_CUDA = 5,         /* a CUDA runtime call failed; see lgc_last_error */
    LGC_ERR_DEVICE_CHECK = 6, /* a kernel recorded an inconsistency; see lgc_check */
    LGC_ERR_NO_MEMORY = 7     /* host allocation of the context failed */
} lgc_status;

typedef enum { LGC_VARIANT_RAR = 0, LGC_VARIANT_PS = 1 } lgc_variant;
/* CONV2: two stride-2 convolutions each way with (ae_c1, ae_c2) channels.  IDENTITY: no autoencoder.
 * CONV5: the autoencoder of the paper's Section IV-C (encoder filters 64/128/256/64/4, decoder filters
 * 4/32/64/128/32 and a 1x1 convolution, leaky ReLU); mu >= 31; ae_c1 / ae_c2 are ignored.
 * Parameter vector: per layer the weights then the bias, encoder conv1..conv5 (w[co][ci][tap])
 * then decoder deconv1..deconv5 (w[ci][co][tap]) and the final convolution; 216,729 floats for
 * the ring-allreduce variant.  Parameter server (Section IV-A): the encoder (172,996 floats), then
 * one decoder per node, whose final convolution has a 33rd weight, on the node's innovation, which
 * joins the decoder's 32 feature channels in front of that convolution (43,734 floats per decoder).
 * deconv1 has stride 1 and padding 1, the others stride 2 with the output padding that returns each
 * length to the one the mirrored encoder layer saw.  Codes are stored position-major:
 * code[K][L4][4].  Training: lgc_ae_train_step (ring-allreduce), lgc_ae_train_step_ps (parameter server). */
typedef enum { LGC_AE_CONV2 = 0, LGC_AE_IDENTITY = 1, LGC_AE_CONV5 = 2 } lgc_ae_kind;

/* Treatment of a layer (Section VI-A, "Experimental Setup": the first layer's gradient is sent as it is, the
 * last layer's top-magnitude values are sent without the autoencoder, the layers in between go through
 * top-k selection and the autoencoder).
 *   TOPK_AE   : accumulated, selected, and the kept values are part of the autoencoder's input.  The kept
 *               values of ALL such layers, in layer order, form the one vector g~_k in R^mu that is encoded.
 *   TOPK_ONLY : accumulated and selected like the others; the kept values bypass the autoencoder: the update
 *               gets their mean over the nodes at the leader's indices (ring-allreduce), or, parameter server,
 *               the node-ordered sum over the nodes that kept an index of value / K.  Sent entries leave u and v.
 *   DENSE     : no state and no selection: update = (((g_0 + g_1) + ...) + g_{K-1}) / K for every element of
 *               the layer, taken from the gradients of this step's lgc_accumulate when the scatter call runs. */
typedef enum { LGC_LAYER_TOPK_AE = 0, LGC_LAYER_TOPK_ONLY = 1, LGC_LAYER_DENSE = 2 } lgc_layer_mode;

/*
 * Problem description (Section V: K nodes, L layers, layer l has n_l elements).
 */
typedef struct {
    int32_t num_nodes;            /* K >= 1 */
    int32_t num_layers;           /* L >= 1 */
    const int64_t *layer_numel;   /* host array [L], each >= 1, sum N <= 2^31 - 1; copied by lgc_init */
    uint32_t density_ppm;         /* alpha of Section V-A in parts per million of n_l: 1000 = 0.1 %.
                                     k_l = clamp(floor((n_l * ppm + 500000) / 10^6), 1, n_l) */
    uint32_t innovation_permille; /* parameter-server variant: share of a layer's kept values that
                                     form the innovation (Algorithm 1: 100 = the top tenth);
                                     kI_l = clamp(floor((k_l * pm + 500) / 1000), 1, k_l) */
    float momentum;               /* m of the momentum correction (Section V-A); 0 = plain residual */
    int32_t variant;              /* lgc_variant: ring-allreduce (Algorithm 2) or parameter server (Algorithm 1) */
    int32_t ae_kind;              /* lgc_ae_kind; IDENTITY passes the kept values through unchanged */
    int32_t ae_c1, ae_c2;         /* channels of the two encoder convolutions: (8,4) or (16,8) */
    float adam_lr, adam_beta1, adam_beta2, adam_eps; /* lgc_ae_train_step; 0 selects 1e-3, 0.9, 0.999, 1e-8 */
    void *stream;                 /* cudaStream_t */
    int64_t grad_row_stride;      /* elements between consecutive nodes' rows of the `grads` argument of
                                     lgc_accumulate; 0 = N (rows back to back).  A larger stride lets a context
                                     work on a run of layers inside a longer flat gradient (Section VI-A: the first
                                     layer is sent dense and the last one without the autoencoder, so a model is
                                     served by one context per run of layers that are treated alike) */
    const uint8_t *layer_mode;    /* host array [L] of lgc_layer_mode, or NULL = every layer TOPK_AE; copied by
                                     lgc_init.  At least one layer must be TOPK_AE.  With DENSE layers the
                                     `grads` buffer of lgc_accumulate must stay valid and unchanged until this
                                     step's lgc_decode_scatter / lgc_topk_scatter has run on the stream (their
                                     elements are read then); k_l of a DENSE layer is 0 */
} lgc_config;

/* Sizes the caller must provide, in bytes.
 *   state   : velocity u and residual v, each K * N fp32 padded to a multiple of four
 *             (Section V-A; zeroed by lgc_init)
 *   scratch : indices, kept values, codes, selection work space, tables
 *   params  : autoencoder parameters followed by the two Adam moment vectors, each padded to a
 *             multiple of four floats (3 * ceil(P/4) * 4 fp32)
 * Returns LGC_ERR_INVALID_ARG / LGC_ERR_UNSUPPORTED for a configuration lgc_init would refuse. */
lgc_status lgc_workspace_bytes(const lgc_config *cfg, size_t *state_bytes, size_t *scratch_bytes,
                               size_t *params_bytes);

/* Builds the context, uploads the layer tables, zeroes `state`, the Adam moments and the work
 * space (Algorithm 1/2: the accumulated gradient starts at 0).  Autoencoder parameters are left
 * as found in `params` (set them with lgc_set_ae_params).  Synchronises the stream.
 * The three buffers are device memory of at least the sizes lgc_workspace_bytes reports and
 * must stay valid until lgc_destroy. */
lgc_status lgc_init(const lgc_config *cfg, void *state, size_t state_bytes, void *scratch,
                    size_t scratch_bytes, void *params, size_t params_bytes, lgc_ctx **out);

/* Frees the host context.  Touches no device memory.  NULL is allowed. */
lgc_status lgc_destroy(lgc_ctx *ctx);

/* Stage 1 -- Algorithm 1/2, local accumulation, with the momentum correction of Section V-A:
 *     u <- m * u + g (one fused rounding);  v <- v + u          for every node and element.
 * grads: device, fp32 [K][N], read only.
 * leader_hint (ring-allreduce only; ignored for the parameter server): the node that lgc_topk
 * will be given as leader in this step, or -1 if not known yet.  With a hint the kernel also
 * collects that node's selection candidates while it streams (against a threshold predicted from
 * the previous step and verified afterwards), which saves lgc_topk its reads of v.  The hint
 * never changes a result: a wrong or missing hint only makes lgc_topk do the reads itself. */
lgc_status lgc_accumulate(lgc_ctx *ctx, const float *grads, int32_t leader_hint);

/* Stages 2+3 -- Section V-A, Algorithm 1/2 (threshold, mask, concatenation): per layer the k_l
 * entries of largest |v| (equal magnitudes: the lower index wins), in ascending index order,
 * layers in order, then the gather of the kept values g~_k in R^mu for every node.
 * Ring-allreduce: only node `leader` selects and all nodes use its indices.
 * Parameter server: every node selects on its own; `leader` is ignored.
 * update_hint: NULL, or the device buffer (fp32 [N], 16-byte aligned) that this step's
 * lgc_decode_scatter / lgc_topk_scatter will be given.  With a hint the library clears that buffer
 * while the selection runs (spare thread blocks of the same launch), so that the scatter call
 * only writes the kept entries; the caller must leave the buffer alone from this call until the
 * scatter call has run.  A different buffer may still be passed later (it is then cleared there). */
lgc_status lgc_topk(lgc_ctx *ctx, int32_t leader, float *update_hint);

/* Stage 4a -- Section IV: g~^c_k = E_c(g~_k) for every node: Conv1d(1->c1, 3 taps, stride 2),
 * ReLU, Conv1d(c1->c2, 3 taps, stride 2), no padding. */
lgc_status lgc_encode(lgc_ctx *ctx);

/* Stage 4b -- across-node combination.
 * Ring-allreduce (Section IV-B / V-B.2): g~^avg = (1/K) sum_k g~^c_k, summed in node order.
 * Parameter server (Algorithm 1, Section V-B.1): the code of node `common_node` is kept as the
 * common representation; for every node the innovation g~^I_k keeps, per layer, the kI_l kept
 * values of largest magnitude (ties: lower position) and zero elsewhere. */
lgc_status lgc_combine(lgc_ctx *ctx, int32_t common_node);

/* Stage 5 -- Section V-B: decoding, scatter, and removal of the sent entries from u and v.
 * Ring-allreduce: g~^rec = D_c(g~^avg) (ConvTranspose1d(c2->c1), ReLU, ConvTranspose1d(c1->1),
 * output padding mirroring the encoder); update[idx[p]] = g~^rec[p], 0 elsewhere.
 * Parameter server: g~^rec_k = w0_k * D_c^k(g~^c) + w1_k * g~^I_k + b_k (the innovation joins
 * the decoder output through a 1x1 convolution); update = sum over k, in node order, of
 * g~^rec_k / K scattered at node k's own indices, 0 elsewhere.
 * update: device, fp32 [N], fully overwritten. */
lgc_status lgc_decode_scatter(lgc_ctx *ctx, float *update);

/* Second training phase (Section V-B, weights updated with the top-magnitude gradients): the dense
 * mean over nodes of the kept values, no autoencoder; sent entries leave u and v.
 * Valid after lgc_topk (and after lgc_ae_train_step / lgc_ae_train_step_ps).  update: device, fp32 [N]. */
lgc_status lgc_topk_scatter(lgc_ctx *ctx, float *update);

/* One training step of the autoencoder on the kept values of the last lgc_topk: ring-allreduce
 * reconstruction loss of Section IV-B scaled by 1/mu,
 *     loss = (1/mu) || D_c((1/K) sum_k E_c(g~_k)) - (1/K) sum_k g~_k ||^2,
 * analytic backward pass, Adam with bias correction.  Ring-allreduce variant, LGC_AE_CONV2 or
 * LGC_AE_CONV5 (whose forward pass and the two largest input-gradient products run on the tensor
 * cores as in lgc_encode, the rest of the backward pass on the fp32 pipes; gradient sums in fp64
 * over per-chunk fp32 partial sums).
 * loss_out: device fp32 scalar or NULL.  May be called several times after one lgc_topk. */
lgc_status lgc_ae_train_step(lgc_ctx *ctx, float *loss_out);

/* The same for the parameter-server autoencoder (Section IV-A): every node's kept values are
 * encoded; the code of `common_node` goes through all K decoders, each with its node's innovation;
 *     loss = lambda_rec * (1/mu) sum_k || g~_k - g~^rec_k ||^2
 *          + lambda_sim * (1/(c2 L2)) sum_k sum_{m != k} || E_c(g~_k) - E_c(g~_m) ||^2
 * (the paper's L_rec and L_sim, each divided by the number of entries it sums over per node),
 * analytic backward pass through the K decoders, their fusion scalars and the encoder, Adam.
 * Parameter-server variant, LGC_AE_CONV2 or LGC_AE_CONV5 (there the code has 4 L4 entries and the
 * innovation is the 33rd input of each decoder's last convolution; the K decoders are run, differentiated
 * and updated one after the other); valid after lgc_topk.  Overwrites the codes, the common code and
 * the innovations of the context.  loss_out: device fp32 scalar or NULL. */
lgc_status lgc_ae_train_step_ps(lgc_ctx *ctx, int32_t common_node, float lambda_rec, float lambda_sim,
                                float *loss_out);

/* Dense average of K rows (first training phase of Section V-B, and the layers Section VI-A leaves
 * uncompressed): update[j] = (((g_0[j] + g_1[j]) + ...) + g_{K-1}[j]) / K in fp32, for j < n.
 * grads: device, row k starts at grads + k * row_stride; update: device, n floats.  Needs no context;
 * enqueued on `stream` (a cudaStream_t). */
lgc_status lgc_dense_mean(const float *grads, int64_t row_stride, int32_t num_nodes, int64_t n, float *update,
                          void *stream);

/* Gives the current step up: whatever stage the context is in, the next call may be lgc_accumulate (or
 * lgc_step_host) again.  Nothing is enqueued and nothing is undone: if lgc_accumulate has run, u and v
 * hold this step's gradient and no entry of it has been sent or cleared, which is the state
 * Algorithm 1/2 has after a step that transmitted nothing (the gradient stays in the residual).
 * For callers that must drop a step after a failed stage or a change of plan.  lgc_step_host does the
 * same by itself when one of its stages fails. */
lgc_status lgc_abort_step(lgc_ctx *ctx);

/* Entropy coding of an index list (Section V-A: the transferred indices are DEFLATE-coded and
 * their rate counts in the compression ratio).  The ascending offsets of every layer become gaps
 * (the first counted from the layer's start, the others from the previous offset + 1), each gap
 * a little-endian base-128 varint; the bytes are written as one raw DEFLATE block (RFC 1951,
 * dynamic Huffman codes, literals only), which any inflate implementation decodes.
 * node: whose list (ring-allreduce: all nodes share the leader's; parameter server: 0 .. K-1).
 * stream_out: device, `capacity` bytes, 4-byte aligned, capacity a multiple of 4; zero-filled
 * beyond the stream.  sizes_out: device, two uint64: bytes of the DEFLATE stream and bytes of the
 * varint form.  If the stream is larger than the capacity only the sizes are valid.
 * Valid from lgc_topk until the next lgc_accumulate. */
lgc_status lgc_encode_indices(lgc_ctx *ctx, int32_t node, void *stream_out, size_t capacity, uint64_t *sizes_out);

/* The same coding for the positions of node `node`'s innovation (parameter server, Algorithm 1: the
 * node sends the top tenth of each layer's kept values, so the receiver must learn which of the
 * kept slots they are): per layer the ascending slots inside the layer's run of kept values, the
 * first gap counted from the run's first slot.  Same buffers, sizes and stream format as
 * lgc_encode_indices.  Valid between lgc_combine and lgc_decode_scatter. */
lgc_status lgc_encode_innovation_positions(lgc_ctx *ctx, int32_t node, void *stream_out, size_t capacity,
                                           uint64_t *sizes_out);

/* A whole compression step from host memory: uploads `host_grads` ([K][N], ideally pinned) to
 * `dev_grads`, runs the five stages, downloads the dense update to `host_update` ([N]).
 * The call returns without waiting; when the context's stream has drained, `host_update` is
 * complete.  `choice` is the leader (ring-allreduce) or the common node (parameter server), 0 .. K-1
 * for both variants.  All arguments are checked before anything is copied or enqueued: a refused call
 * leaves u, v and the context as they were.
 * The upload goes node by node over a stream of the library's own (created at the first call,
 * released by lgc_destroy), and each node's row is accumulated as soon as it has arrived, so
 * stage 1 hides under the transfer; the download stays on the context's stream.  The upload of
 * one call waits for the scatter of the previous lgc_step_host, not for that call's download:
 * back-to-back calls keep both directions of the bus busy.  From the moment of the call
 * `host_grads` and `dev_grads` belong to it: the upload does not wait for work the caller
 * queued on the context's stream after the previous lgc_step_host, so such work must not touch
 * `dev_grads`, and `host_grads` must already hold the gradients.  Results are bit for bit those
 * of the five stage calls. */
lgc_status lgc_step_host(lgc_ctx *ctx, const float *host_grads, float *dev_grads, float *dev_update,
                         float *host_update, int32_t choice);

/* Top-k by magnitude of ONE flat vector without any caller-provided work space.
 * (The paper has no counterpart; this serves callers of the library, not the method.)
 *
 * For callers that may not allocate device memory or hand over scratch: code running under a
 * fixed-footprint promise, plugins whose host owns the allocator and passes only inputs and
 * outputs, jobs on a device that is already full.  The selection's tables, radix histogram and
 * per-chunk counts live in a fixed array compiled into the library (about 60 KB, held by every
 * GPU that loads the library until the process exits), which caps the vector length at
 * LGC_NOALLOC_MAX_N elements.  The call itself performs no allocation of any kind.
 *
 *   v       : device, fp32 [n], read only          n : 1 .. LGC_NOALLOC_MAX_N
 *   k       : 1 .. n entries to keep               stream : cudaStream_t
 *   idx_out : device, int32 [k]; receives the offsets of the k entries of largest |v| (equal
 *             magnitudes: the lower index wins) in ascending order -- the same result lgc_topk
 *             gives for a single layer of n elements.
 * Returns LGC_ERR_UNSUPPORTED when n is above the maximum and LGC_ERR_INVALID_ARG for null
 * pointers or k outside 1..n; lgc_last_error(NULL) has the text.  Nothing is enqueued then.
 *
 * The first call on a device looks up the array's device address (once per device, with that
 * device current); make that first call before any stream capture begins.
 * All calls share the one array and it keeps the previous call's contents (the call clears what
 * must start at zero itself): two calls whose kernels overlap on the GPU -- different streams,
 * or different host threads -- race on it.  Serialise them. */
#define LGC_NOALLOC_MAX_N 16777216
lgc_status lgc_topk_noalloc(const float *v, int64_t n, int64_t k, int32_t *idx_out, void *stream);

/* The consistency checks of lgc_topk_noalloc's kernels (counts that must add up to k) are recorded
 * in a word of the built-in array, not in a context: lgc_check never reports them, this call does.
 * It waits for `stream`, reads the word of the current device (a four-byte copy to the host, no
 * allocation), returns LGC_OK or LGC_ERR_DEVICE_CHECK (text through lgc_last_error(NULL)) and clears
 * the record.  (No counterpart in the paper either.) */
lgc_status lgc_topk_noalloc_check(void *stream);

/* ---- inspection --------------------------------------------------------------------------- */

/* N, mu, encoder lengths L1 (after the first convolution) and L2 (code length per channel), and
 * the parameter count P.  Any output pointer may be NULL. */
lgc_status lgc_get_layout(const lgc_ctx *ctx, int64_t *N, int64_t *mu, int64_t *L1, int64_t *L2,
                          int64_t *param_count);

/* Host array [L] of k_l, owned by the context (0 for DENSE layers). */
const int64_t *lgc_keep_counts(const lgc_ctx *ctx);

/* Where the kept entries of each layer sit inside a row of `idx`.  A row has mu_all slots: first the mu
 * slots of the TOPK_AE layers, in layer order (these are the autoencoder's input, and what lgc_get_layout
 * reports as mu), then the slots of the TOPK_ONLY layers, in layer order.  Without a layer_mode array
 * mu_all = mu and the slots follow the layers.  first_slot: host array [L] owned by the context, -1 for DENSE
 * layers.  val_topk_only: device, fp32 [K][mu_all - mu], the kept values of the TOPK_ONLY layers (filled by
 * lgc_topk for the parameter server and by lgc_topk_scatter; NULL when there are none).  Any pointer may be NULL. */
lgc_status lgc_get_slots(const lgc_ctx *ctx, int64_t *mu_all, const int64_t **first_slot, float **val_topk_only);

/* Device pointers into the caller's buffers (any may be NULL):
 *   u, v    [K][N]                     idx   [S][mu_all] int32 (see lgc_get_slots), S = 1 (ring-allreduce) or K
 *   val     [K][mu] (filled by lgc_topk for the parameter server and the identity autoencoder,
 *           else by lgc_encode / lgc_ae_train_step / lgc_topk_scatter)
 *   code    [K][c2][L2] (identity: [K][mu])
 *   combined[c2][L2] (ring-allreduce: the mean; parameter server: the common code)
 *   inn     [K][mu] (parameter server) recon [S][mu] */
lgc_status lgc_get_buffers(const lgc_ctx *ctx, float **u, float **v, int32_t **idx, float **val,
                           float **code, float **combined, float **inn, float **recon);

/* Autoencoder parameters, flat fp32, tensors in this order (row major):
 *   enc.w1 [c1][1][3], enc.b1 [c1], enc.w2 [c2][c1][3], enc.b2 [c2],
 *   then per decoder: w1 [c2][c1][3], b1 [c1], w2 [c1][1][3], b2 [1]
 * (ring-allreduce: one decoder; parameter server: K decoders, each followed by its fusion
 * scalars w0, w1, b).  `src`/`dst` may be host or device memory; the copy is synchronous. */
lgc_status lgc_set_ae_params(lgc_ctx *ctx, const float *src, size_t count);
lgc_status lgc_get_ae_params(const lgc_ctx *ctx, float *dst, size_t count);

/* Waits for the stream and reports what kernels recorded: LGC_OK or LGC_ERR_DEVICE_CHECK
 * (code readable through lgc_last_error).  Clears the record. */
lgc_status lgc_check(lgc_ctx *ctx);

/* How the last lgc_topk got its entries: the number of (selecting row, layer) pairs with more
 * than 4096 elements; how many of them were finished from candidates collected during
 * lgc_accumulate (no further pass over v); the total and the largest number of candidates per
 * pair (the k_l selected entries are found among them; a pair finished from the data counts
 * with its length); and how many pairs were finished from the data itself (no usable lists, a
 * list overflow, too many candidates, or a prediction that was too high).  Any pointer may be
 * NULL.  Waits for the stream. */
lgc_status lgc_selection_stats(lgc_ctx *ctx, int64_t *large_segments, int64_t *served_by_accumulation,
                               int64_t *candidates_total, int64_t *candidates_max, int64_t *finished_from_data);

/* Number of kernels the library has enqueued from the calling thread since it was loaded
 * (all contexts); the benchmark reports the difference over its timed region. */
uint64_t lgc_kernel_launches(void);

const char *lgc_status_string(lgc_status s);
/* Text of the last failure recorded in `ctx`; with ctx == NULL, of the calling thread's last
 * failure that had no context (lgc_init).  Owned by the library, valid until the next call. */
const char *lgc_last_error(const lgc_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* LGC_H */
