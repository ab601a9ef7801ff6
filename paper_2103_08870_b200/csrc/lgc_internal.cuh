// Internal declarations shared by the translation units of liblgc: the host context, the work
// space carve-up, and one launcher prototype per kernel family.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "lgc.h"

namespace lgc {

constexpr int kSelChunk = 4096;    // elements per selection chunk: 256 threads x 16
constexpr int kSelThreads = 256;
constexpr int kSelPerThread = 16;
constexpr int kSelCandCap = 256;   // candidates a chunk's list holds; more than that and the segment is finished from the data
constexpr int kHistBins = 2048;    // first radix digit: 11 bits; the next two: 10 bits each
constexpr int kDenseChunk = 1024;  // elements of a dense (uncompressed) layer that one CTA averages over the nodes
constexpr int kSelGroup = 2048;    // chunks whose candidate lists one CTA compacts at a time; a segment of more chunks
                                   // than this has its groups compacted by CTAs of their own before it is finished

// One selection problem family: R rows of `data` (row stride in elements), each cut into the same
// segments; per segment the k entries of largest |x| are reported, ascending, as int32 offsets.
// All pointers are device memory.
struct SelectTables {
    int num_segments = 0;
    int num_small = 0;            // segments of at most kSelChunk elements
    int num_large = 0;
    int max_rows = 0;
    int64_t *seg_off = nullptr;   // [S] first element of the segment inside a row
    int32_t *seg_len = nullptr;   // [S]
    int32_t *seg_k = nullptr;     // [S]
    int32_t *seg_out = nullptr;   // [S] first output slot of the segment
    int32_t *small_ids = nullptr; // [num_small] segment ids
    int32_t *large_ids = nullptr; // [num_large] segment ids
    uint32_t *hist = nullptr;     // [rows][num_large][kHistBins], all zero between passes
    uint32_t *prefix = nullptr;   // [rows][num_large] key prefix found so far
    int32_t *k_rem = nullptr;     // [rows][num_large] entries still to find at the prefix

    // -- launch_select_multipass: chunks of kSelChunk elements counted from each segment's start
    int num_chunks = 0;
    int32_t *large_chunk0 = nullptr; // [num_large + 1] first chunk of each large segment
    int32_t *chunk_large = nullptr;  // [num_chunks] index into large_ids
    int2 *chunk_cnt = nullptr;       // [rows][num_chunks] (#key > T, #key == T), then exclusive prefix

    // -- launch_select: chunks are the intersections of a segment with the row's 4096-element tiles
    int num_tchunks = 0;
    int tiles_per_row = 0;
    int32_t *seg_large = nullptr;    // [S] index into large_ids, -1 for small segments
    int32_t *large_q0 = nullptr;     // [num_large] first tile the segment overlaps
    int32_t *large_order = nullptr;  // [num_large] indices into large_ids, longest segment first
    int num_group_jobs = 0;
    int2 *group_job = nullptr;       // [num_group_jobs] (index into large_ids, first chunk of the group), for the
                                     // segments of more than kSelGroup chunks
    int2 *job_range = nullptr;       // [rows][num_group_jobs] candidates before the group, candidates of the group
    int2 *job_cnt = nullptr;         // [rows][num_group_jobs] entries of the group above / at the k-th key
    int32_t *seg_wide = nullptr;     // [rows][num_large] the segment's selection was completed group by group
    int32_t *tchunk0 = nullptr;      // [num_large + 1] first tile-chunk of each large segment
    int32_t *tchunk_large = nullptr; // [num_tchunks] index into large_ids
    int4 *tile_desc = nullptr;       // [tiles_per_row] x: first segment the tile overlaps; y: the large segment that
                                     // covers the whole tile (-1: several segments, -2: no large one); z: its chunk;
                                     // w: 0 no dense element in the tile; one dense run [lo, hi) inside it: 1 + lo + (hi << 13);
                                     // several runs: -(1 + the first run's number)
    const int64_t *dense_rng = nullptr;  // [num_dense] (begin, end) of the row's runs of dense elements
    int num_dense = 0;
    int32_t *cand_cnt = nullptr;     // [rows][num_tchunks] candidates found in the chunk
    uint2 *cand = nullptr;           // [rows][num_tchunks][kSelCandCap] (key, position inside the tile), ascending position
    int32_t *seg_m = nullptr;        // [rows][num_large] candidates of the segment
    int32_t *seg_ticket = nullptr;   // [rows][num_large] chunks that have reported; zero between passes
    int32_t *seg_epoch = nullptr;    // [rows][num_large] step in which the two-pass path settled the segment
    int32_t *seg_path = nullptr;     // [rows][num_large] how the last selection got its entries (see lgc_selection_stats)
    uint32_t *last_key = nullptr;    // [rows][num_large] k-th key of the previous selection (0: none)
    uint32_t *lbkey = nullptr;       // [rows][num_large] key from which the next accumulation collects candidates (0: none)
    float2 *key_trend = nullptr;     // [rows][num_large] x: ln of the last ratio of consecutive k-th keys; y: how much that
                                     // ratio has jumped from step to step lately (decaying maximum)
    int64_t *comp_off = nullptr;     // [num_large + 1] first compact slot of each large segment
    int64_t comp_total = 0;          // compact slots per row
    uint32_t *comp_key = nullptr;    // [rows][comp_total] keys of the candidates, index order
    int32_t *comp_idx = nullptr;     // [rows][comp_total] their offsets inside the row
};

// Compact-array capacity of a large segment of n elements of which k are kept: above it the segment is
// finished by streaming over the data itself.  Candidates are the entries from a little below the k-th
// key upwards, a few times k in practice; ties can make them many more.
inline int64_t select_compact_capacity(int64_t n, int64_t k)
{
    const int64_t c = 64 * k > 8192 ? 64 * k : 8192;
    return c < n ? c : n;
}

// Work space and tables of the full-size autoencoder (LGC_AE_CONV5; Section IV-C).
struct Ae5 {
    int64_t len[5] = {0, 0, 0, 0, 0};   // mu and the lengths after conv1..conv4
    int64_t lpad[3] = {0, 0, 0};        // positions allocated per node for the outputs of conv1..conv3 (even)
    float *act_hi[3] = {}, *act_lo[3] = {};   // [K][lpad][C] outputs of conv1..conv3, channels-last, split into two tf32 parts
    float *w_hi[3] = {}, *w_lo[3] = {};       // [C_out][3 C_in] GEMM weights of conv2..conv4, split likewise
    float *d0 = nullptr;                // [L4][4] output of deconv1
    float *dact_hi[3] = {}, *dact_lo[3] = {}; // [L3][32], [L2][64], [L1][128]: outputs of deconv2..deconv4, split likewise
    float *dw_hi[3] = {}, *dw_lo[3] = {};     // [2 C_out][2 C_in] GEMM weights of deconv3..deconv5, split likewise
    int64_t off_w[5] = {}, off_b[5] = {};     // offsets of the encoder layers' weights / biases in the parameter vector
    int64_t off_dw[6] = {}, off_db[6] = {};   // the same for the decoder's six layers
    CUtensorMap map_act_hi[3], map_act_lo[3], map_w_hi[3], map_w_lo[3];
    CUtensorMap map_dact_hi[3], map_dact_lo[3];
    // Decoders: one (ring-allreduce) or one per node (parameter server: Section IV-A), `dec_stride` parameters
    // apart; off_dw / off_db below are decoder 0's.  The parameter server's last convolution has a 33rd input,
    // the node's innovation.  dw_hi / dw_lo hold the decoders' GEMM weights back to back.
    int decoders = 1;
    int64_t dec_stride = 0;
    std::vector<CUtensorMap> map_dw_hi, map_dw_lo;   // [decoders][3]
    bool weights_ready = false;         // w_hi / w_lo match the parameter vector
    // ---- training step (lgc_ae_train_step) ----
    float *act4_hi = nullptr, *act4_lo = nullptr;    // [K][L4][64] output of conv4 (inference folds it into conv5)
    float *dact5_hi = nullptr, *dact5_lo = nullptr;  // [mu][32] output of deconv5 (inference folds it into the last conv)
    float *g_enc[4] = {};               // dLoss/d(pre-activation) of conv1..conv4.  conv4's: fp32 [K][L4][64].  conv1..conv3's:
    float *g_enc_lo[3] = {};            // two tf32 parts laid out like the layer's output, [K][lpad][C] (they feed tensor-core GEMMs)
    float *g4_hi = nullptr, *g4_lo = nullptr;   // conv4's gradient once more as two tf32 parts, [K][L4][64] (operand of its weight gradient)
    // Weight gradients of conv2..conv4 (index 0..2) on the tensor cores: maps over the gradient at the layer's output (G) and
    // over the layer's input seen as rows of a pair of positions (X: taps 0 and 1, and tap 2 one pair further), hi and lo
    // parts; positions beyond the layer's length read as zeros.  wg_splits: parts a node's rows are cut into.
    CUtensorMap map_wg_g[3][2], map_wg_x[3][2][2];
    int wg_splits[3] = {1, 1, 1}, wg_kbps[3] = {1, 1, 1};
    float *gw_hi[3] = {}, *gw_lo[3] = {};   // weights of conv2..conv4 arranged for the GEMM that makes the gradient at their input
    CUtensorMap map_g_hi[3], map_g_lo[3], map_gw_hi[3], map_gw_lo[3];
    float *g_dec[5] = {};               // the same for deconv1..deconv5: [L][C], g_dec[4] is [mu][32]
    float *dzk = nullptr;               // [K][L4][4] gradient at every node's code
    float *dzbar = nullptr;             // [L4][4]    gradient at the mean code
    float *dr = nullptr;                // [mu]       gradient at the reconstruction
    float *wt = nullptr;                // one layer's weights arranged for the backward GEMM
    float *partial = nullptr;           // per-chunk partial sums of every parameter tensor's gradient
    double *loss_part = nullptr;        // [loss_blocks]
    int loss_blocks = 0;
    struct Tensor {                     // one parameter tensor: where its partial sums live and how many chunks made them
        int64_t param_off = 0, count = 0, partial_off = 0, rows = 0, chunk = 0;
        int chunks = 0, kind = 0, cin = 0, cout = 0;
    };
    Tensor tensors[22];                 // encoder w,b x 5, decoder w,b x 6, in parameter order
};

struct Ctx {
    lgc_config cfg{};
    cudaStream_t stream = nullptr;
    int K = 0, L = 0, S = 0;       // S: index sets (1 ring-allreduce, K parameter server)
    // Per-layer treatment (Section VI-A).  A row of idx holds mu_all slots: first the mu slots of the layers
    // that go through the autoencoder (layer order), then the mu_t slots of the top-k-only layers.
    int L_ae = 0, L_sel = 0;       // layers through the autoencoder, layers that select at all
    int64_t mu_t = 0, mu_all = 0;
    bool mixed = false;            // some layer is top-k only or dense
    int64_t N = 0, mu = 0, muI = 0, L1 = 0, L2 = 0, P = 0, Penc = 0, Pdec = 0;
    int op1 = 0, op2 = 0;          // output paddings of the two transposed convolutions
    int64_t code_len = 0;          // floats per node code: c2 * L2 (identity: mu)
    std::vector<int64_t> numel, off, k_l, kslot, koff, ki_l, kioff;   // k_l, kslot per layer; koff, ki_l, kioff in slot order
    double lr = 0, beta1 = 0, beta2 = 0, eps = 0;
    int64_t adam_t = 0;
    // caller buffers
    float *u = nullptr, *v = nullptr;
    float *params = nullptr, *adam_m = nullptr, *adam_v = nullptr;
    // scratch carve-up
    int32_t *idx = nullptr;        // [S][mu_all]
    float *val = nullptr;          // [K][mu]   kept values of the autoencoder's layers
    float *val_t = nullptr;        // [K][mu_t] kept values of the top-k-only layers
    int64_t *dense_rng = nullptr;  // [num_dense] (begin, end) of the runs of dense elements inside a row
    int num_dense = 0;
    int64_t *dense_chunks = nullptr;   // [num_dense_chunks] (begin, end): the dense runs cut into pieces of kDenseChunk
    int64_t num_dense_chunks = 0;
    const float *step_grads = nullptr; // gradients of the step in flight: the dense layers are read at the scatter
    float *code = nullptr;         // [K][code_len]
    float *combined = nullptr;     // [code_len]
    float *inn = nullptr;          // [K][mu]
    int32_t *inn_pos = nullptr;    // [K][muI]
    int32_t *inn_slot_layer = nullptr; // [muI] layer of each innovation slot (parameter server)
    int32_t *kioff_dev = nullptr;  // [L + 1] first innovation slot of each layer
    int64_t *koff64_dev = nullptr; // [L] first kept slot of each layer: where a layer's innovation positions count from
    float *recon = nullptr;        // [S][mu]
    int32_t *slot_layer = nullptr; // [mu_all] layer (its number in slot order) of each kept slot
    int32_t *koff_dev = nullptr;   // [L_sel + 1] first slot of each selecting layer, slot order
    int64_t *layer_off_dev = nullptr; // [L_sel] first element of each selecting layer inside a row, slot order
    unsigned char *ic_bytes = nullptr; // [5 mu] varint form of an index list (index coding)
    int32_t *tile_lo = nullptr;    // [ceil(N / 4096) + 1] first kept slot at or after each 4096-entry tile (ring-allreduce)
    int32_t *errword = nullptr;    // device check record
    SelectTables sel_v, sel_inn;
    std::unique_ptr<Ae5> ae5;      // full-size autoencoder only
    // training work space
    float *t_h = nullptr;          // [K][c1][L1] relu(conv1)
    float *t_d = nullptr;          // [c1][L1]    relu(convT1)
    float *t_dr = nullptr;         // [mu]        d loss / d recon
    float *t_dd = nullptr;         // [c1][L1]
    float *t_dz = nullptr;         // [c2][L2]    d loss / d mean code
    float *t_dh = nullptr;         // [K][c1][L1]
    double *t_loss_part = nullptr; // [loss blocks]
    int t_loss_blocks = 0;
    // parameter-server training: the buffers above hold one slice per node ([K] in front), plus
    float *t_y = nullptr;          // [K][mu]     decoder output before the fusion with the innovation
    float *t_dy = nullptr;         // [K][mu]     d loss / d that output
    float *t_dzc = nullptr;        // [K][c2][L2] every decoder's gradient at the common code
    float *t_zsum = nullptr;       // [c2][L2]    sum over nodes of the codes
    double *t_sim_part = nullptr;  // [blocks over L2] partial sums of the similarity loss
    // step state machine
    enum Stage { kIdle, kAccumulated, kSelected, kEncoded, kCombined } stage = kIdle;
    int32_t last_leader = 0;
    int32_t epoch = 0;             // step counter (accumulations so far)
    int32_t inn_epoch = 0;         // the same counter for the innovation selection's tables
    float *cleared_update = nullptr; // buffer the last lgc_topk already cleared (its first N & ~3 floats)
    int selections = 0;            // selections run so far (saturating); the accumulation collects candidates from the
                                   // third step on, when the prediction knows how fast the threshold is growing
    int32_t fused_leader = -2;     // row whose candidates the last accumulation collected (-1: all rows, -2: none)
    bool val_valid = false;        // val holds the kept values of the current selection
    bool tile_lo_valid = false;    // tile_lo matches the current selection
    bool mean_valid = false;       // combined holds the mean code of the current selection
    // lgc_step_host: the upload runs row by row on a stream of the library's own, so that rows are
    // accumulated while later rows are still on the bus (created at the first call, released by lgc_destroy)
    // lgc_topk, many small layers (parameter server): they are selected on a side stream while the large
    // layers are finished on the context's stream (created at the first such call, released by lgc_destroy)
    cudaStream_t side_stream = nullptr;
    cudaEvent_t side_fork = nullptr, side_join = nullptr;
    cudaStream_t upload_stream = nullptr;
    std::vector<cudaEvent_t> row_uploaded;   // [K]
    cudaEvent_t tail_done = nullptr;         // the previous lgc_step_host has finished with dev_grads (before its download)
    bool tail_recorded = false;
    std::string err;
};

// A setting that belongs to a device, not to the process (a kernel's opt-in to more dynamic shared
// memory, the SM count): made once for every device ordinal that becomes current.
constexpr int kMaxDevices = 64;
struct OncePerDevice {
    std::mutex mu;
    bool done[kMaxDevices] = {};
    template <typename F>
    cudaError_t run(F &&f)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return f();          // beyond the table: every time
        std::lock_guard<std::mutex> lock(mu);
        if (done[dev]) return cudaSuccess;
        e = f();
        if (e == cudaSuccess) done[dev] = true;
        return e;
    }
};
int sm_count();                                   // of the current device

// Programmatic dependent launch: a kernel launched this way may start while its predecessor in the stream is
// still draining; it runs its own prologue (weights into shared memory) and then waits, with grid_wait(), for
// the predecessor to have completed and its memory to be visible.  Nothing it reads or writes before that wait
// may be touched by the predecessor.  Launched the ordinary way the same kernels' waits return at once.
__device__ __forceinline__ void grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... Params, typename... Args>
cudaError_t launch_dependent_smem(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}
template <typename... Params, typename... Args>
cudaError_t launch_dependent(void (*kernel)(Params...), dim3 grid, dim3 block, cudaStream_t stream, Args... args)
{
    return launch_dependent_smem(kernel, grid, block, 0, stream, args...);
}

// x = hi + lo with both parts representable in tf32 (10 explicit mantissa bits)
__device__ __forceinline__ void split_tf32(float x, float &hi, float &lo)
{
    uint32_t h;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(h) : "f"(x));
    hi = __uint_as_float(h);
    const float r = __fsub_rn(x, hi);
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(h) : "f"(r));
    lo = __uint_as_float(h);
}

extern thread_local uint64_t g_kernel_launches;   // kernels this thread has enqueued (lgc_kernel_launches)
extern thread_local std::string g_last_error;   // failures without a context (see lgc_last_error)

// ---- launchers (each enqueues on ctx stream and returns the launch status) -------------------
cudaError_t launch_zero(void *p, size_t bytes, cudaStream_t s);
cudaError_t launch_accumulate(const float *g, float *u, float *v, uint64_t count, float m, cudaStream_t s);
// rows of g are g_stride elements apart (u and v stay back to back)
// dense_rng / num_dense: runs of elements that keep no state (their u and v are left alone)
cudaError_t launch_accumulate_rows(const float *g, int64_t g_stride, float *u, float *v, int K, int64_t N, float m,
                                   const int64_t *dense_rng, int num_dense, cudaStream_t s);
cudaError_t launch_dense_mean(const float *g, int64_t g_stride, int K, int64_t n, float *update, cudaStream_t s);
// served: the accumulation of step `epoch` collected the candidates of exactly these rows.
// clear/clear_floats: optional 16-byte aligned buffer that spare CTAs of the finishing launch set to zero
// (only when the tables have large segments).
// side / fork / join (all or none): a stream and two events of the caller's; when the small segments get a launch
// of their own it runs on `side`, beside the finishing of the large ones, and `s` continues once both are done.
cudaError_t launch_select(const SelectTables &t, const float *data, int64_t row_stride, int row0,
                          int rows, int32_t *out, int64_t out_stride, bool served, int32_t epoch, float *clear,
                          int64_t clear_floats, int32_t *errword, cudaStream_t s, cudaStream_t side = nullptr,
                          cudaEvent_t fork = nullptr, cudaEvent_t join = nullptr);
// Accumulation that also collects the selection candidates of the selecting rows (sel_row0 .. +sel_rows
// of the K rows) against the predicted buckets; needs N % 4 == 0 and g_stride % 4 == 0 (rows of g are
// g_stride elements apart).
cudaError_t launch_accumulate_select(const SelectTables &t, const float *g, int64_t g_stride, float *u, float *v, int K,
                                     int64_t N, float m, int sel_row0, int sel_rows, int32_t epoch, int32_t *errword,
                                     cudaStream_t s);
cudaError_t launch_select_multipass(const SelectTables &t, const float *data, int64_t row_stride, int row0,
                                    int rows, int32_t *out, int64_t out_stride, int32_t *errword, cudaStream_t s);
cudaError_t launch_gather(Ctx &c);
cudaError_t launch_encode(Ctx &c);
cudaError_t launch_combine_mean(Ctx &c);
cudaError_t launch_combine_ps(Ctx &c, int common_node);
cudaError_t launch_decode_scatter(Ctx &c, float *update);
cudaError_t launch_topk_scatter(Ctx &c, float *update);
cudaError_t launch_train_step(Ctx &c, float *loss_out);
cudaError_t launch_encode_indices(Ctx &c, int node, unsigned char *out, int64_t capacity, unsigned long long *result);
cudaError_t launch_encode_innovation_positions(Ctx &c, int node, unsigned char *out, int64_t capacity,
                                               unsigned long long *result);
cudaError_t launch_train_step_ps(Ctx &c, int common, float lam_rec, float lam_sim, float *loss_out);
// full-size autoencoder (lgc_ae5.cu)
extern const int kAe5EncCh[5];        // channels through conv1..conv4 (conv5 maps the last to 4)
extern const int kAe5DecCh[6];        // channels through deconv1..deconv5 (the last convolution maps them to 1)
int64_t ae5_param_count(int decoders, bool innovation_channel);
bool ae5_lengths(int64_t mu, int64_t (&len)[5]);
void ae5_carve(Ae5 &a, int K, int64_t mu, bool ps, char *base, size_t *used);   // base may be null (sizes only)
cudaError_t ae5_make_maps(Ctx &c);
cudaError_t launch_ae5_encode(Ctx &c);
cudaError_t launch_ae5_decode(Ctx &c);
// training: the forward pass that keeps every layer's output (lgc_ae5.cu), then the backward pass and Adam
cudaError_t launch_ae5_train_encode(Ctx &c);           // every node's code into c.code
cudaError_t launch_ae5_train_decode(Ctx &c, int d);    // decoder d on c.combined, up to deconv5 (kept in dact5)
cudaError_t launch_ae5_train_forward(Ctx &c);          // ring-allreduce: encoder, mean, the decoder
cudaError_t launch_ae5_train_step(Ctx &c, float *loss_out);
// gradient at the input of conv2, conv3 or conv4 (layer = 1, 2, 3) from g_enc[layer] into g_enc[layer - 1], on the tensor cores
cudaError_t launch_ae5_input_gradient(Ctx &c, int layer);
// weight gradient of conv2, conv3 or conv4 (layer = 1, 2, 3) into the partial sums of tensor 2 * layer, on the tensor cores
cudaError_t launch_ae5_weight_gradient(Ctx &c, int layer);
void ae5_weight_gradient_chunks(int K, int64_t l_out, int cin, int cout, int *splits, int *kbps);   // how the rows are cut
cudaError_t launch_ae5_train_step_ps(Ctx &c, int common, float lam_rec, float lam_sim, float *loss_out);
struct AdamArgs {
    float *params, *m, *v;
    double lr, beta1, beta2, eps, corr1, corr2;
};
AdamArgs next_adam(Ctx &c);           // advances the step counter

}  // namespace lgc
