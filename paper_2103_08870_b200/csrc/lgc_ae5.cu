// The paper's full-size autoencoder (Section IV-C: encoder of five 1-D convolutions with 64, 128,
// 256, 64 and 4 filters, decoder of five transposed convolutions with 4, 32, 64, 128, 32 filters
// and a final 1x1 convolution, leaky ReLU between layers) for the ring-allreduce form of
// Section IV-B: every node's kept values are encoded, the codes averaged, one decoder
// reconstructs.
//
// Activations are kept channels-last, [node][position][channel], so that row t of the im2col
// matrix of a kernel-3 stride-2 convolution is the contiguous slice [2t C_in, (2t+3) C_in) of the
// activation: the convolutions with 64, 128 and 256 input channels are GEMMs
//     out[t][co] = sum_j A[t][j] W[co][j],   j = tau C_in + ci,
// run on the tensor cores (tcgen05.mma kind::tf32, operands staged by TMA into 128-byte-swizzled
// shared memory, accumulator in tensor memory).  fp32 accuracy is kept by splitting every
// operand into two tf32 numbers, x = hi + lo, and accumulating hi*hi + hi*lo + lo*hi.
// The first convolution (one input channel), the 1x1 convolutions and the two narrow decoder layers use the
// ordinary fp32 pipes; the decoder's three wide transposed convolutions are GEMMs of the same kernel.
// For training, the same kernel makes the gradients at the inputs of conv2..conv4 (a transposed convolution of
// the output's gradient), and ae5_wgrad_kernel their weight gradients (a GEMM that sums over rows, both operands
// read along their rows).
#include <algorithm>

#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr float kSlope = 0.01f;       // leaky-ReLU slope (the paper names the activation, not the slope)
constexpr int kTileM = 128;           // output positions per CTA of the GEMM: the M of one tcgen05.mma
constexpr int kBlockK = 32;           // fp32 per 128-byte swizzled row
constexpr int kSpinLimit = 4000000;   // mbarrier polls before a wait gives up
constexpr int kConv1Pos = 128;        // output positions per CTA of conv1
constexpr int kStagePitch = 36;       // floats per row of the epilogue's staging blocks (16-byte aligned, spreads the banks)

__device__ __forceinline__ float leaky(float x) { return x > 0.0f ? x : kSlope * x; }

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// Shared-memory matrix descriptor of a K-major tile of 128-byte rows, 128-byte swizzle: rows of
// one 8-row group are 128 bytes apart, groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);         // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset (unused with this swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                               // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}

// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x N x 8 tf32 step
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate)
{
    const uint32_t acc = accumulate ? 1u : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// Makes the mbarrier complete once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_load32(uint32_t taddr, float (&x)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(r[i]);
}

// ------------------------------------------------------------------------------------------
// conv1: gather of the kept values + Conv1d(1 -> 64, k3, s2) + leaky ReLU, written channels-last
// as (hi, lo).  Grid (ceil(L1 / 128), K), 256 threads: thread = (position of a pass of 16, four channels).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
ae5_conv1_kernel(const float *__restrict__ v, int64_t N, const int32_t *__restrict__ idx, int64_t idx_node_stride, int64_t mu,
                 int64_t L1, int64_t Lpad1, const float *__restrict__ w1, const float *__restrict__ b1, float *__restrict__ val,
                 float *__restrict__ a_hi, float *__restrict__ a_lo)
{
    __shared__ float x[2 * kConv1Pos + 2];
    __shared__ float w[64 * 3], b[64];
    grid_release_dependents();            // conv2's CTAs may set themselves up meanwhile (they wait for this launch before they load)
    const int k = blockIdx.y;
    const int64_t t0 = (int64_t)blockIdx.x * kConv1Pos;
    for (int i = threadIdx.x; i < 64 * 3; i += 256) w[i] = w1[i];
    if (threadIdx.x < 64) b[threadIdx.x] = b1[threadIdx.x];
    for (int i = threadIdx.x; i < 2 * kConv1Pos + 2; i += 256) {
        const int64_t p = 2 * t0 + i;
        float xv = 0.0f;
        if (p < mu) {
            xv = v[(int64_t)k * N + idx[(int64_t)k * idx_node_stride + p]];   // ring-allreduce: one list (stride 0)
            val[(int64_t)k * mu + p] = xv;           // the two slots shared with the next CTA are written by
        }                                            // both, with the same value
        x[i] = xv;
    }
    __syncthreads();
    // sixteen threads per position, four channels each: a warp's store is 512 consecutive bytes
    const int c4 = threadIdx.x & 15;
    float wr[4][3], br[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        br[j] = b[4 * c4 + j];
#pragma unroll
        for (int tau = 0; tau < 3; ++tau) wr[j][tau] = w[(4 * c4 + j) * 3 + tau];
    }
#pragma unroll 2
    for (int tl = threadIdx.x >> 4; tl < kConv1Pos; tl += 16) {
        const int64_t t = t0 + tl;
        if (t >= L1) break;
        const float x0 = x[2 * tl], x1 = x[2 * tl + 1], x2 = x[2 * tl + 2];
        float hi[4], lo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float acc = br[j];
            acc = __fmaf_rn(wr[j][0], x0, acc);
            acc = __fmaf_rn(wr[j][1], x1, acc);
            acc = __fmaf_rn(wr[j][2], x2, acc);
            split_tf32(leaky(acc), hi[j], lo[j]);
        }
        const int64_t at = ((int64_t)k * Lpad1 + t) * 64 + 4 * c4;
        *reinterpret_cast<float4 *>(a_hi + at) = make_float4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<float4 *>(a_lo + at) = make_float4(lo[0], lo[1], lo[2], lo[3]);
    }
}

// Weights of a kernel-3 convolution w[co][ci][tau] -> GEMM operand W[co][tau C_in + ci] as (hi, lo).
__global__ void ae5_prep_weights_kernel(const float *__restrict__ w, int cin, int cout, float *__restrict__ w_hi,
                                        float *__restrict__ w_lo)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= cout * cin * 3) return;
    const int co = i / (cin * 3), rem = i % (cin * 3), tau = rem / cin, ci = rem % cin;
    float hi, lo;
    split_tf32(w[(co * cin + ci) * 3 + tau], hi, lo);
    w_hi[i] = hi;
    w_lo[i] = lo;
}

// Weights of a kernel-3 stride-2 transposed convolution w[ci][co][tau] -> GEMM operand
// W[n][k], n in [0, 2 C_out), k in [0, 2 C_in), as (hi, lo): the first C_out rows make the even
// output position (tap 2 on the previous input position, tap 0 on the current one), the others
// the odd position (tap 1 on the current one).
__global__ void ae5_prep_deconv_weights_kernel(const float *__restrict__ w, int cin, int cout, float *__restrict__ w_hi,
                                               float *__restrict__ w_lo)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 4 * cin * cout) return;
    const int n = i / (2 * cin), k = i % (2 * cin);
    const int ci = k < cin ? k : k - cin;
    float x = 0.0f;
    if (n < cout) x = w[(ci * cout + n) * 3 + (k < cin ? 2 : 0)];
    else if (k >= cin) x = w[(ci * cout + (n - cout)) * 3 + 1];
    float hi, lo;
    split_tf32(x, hi, lo);
    w_hi[i] = hi;
    w_lo[i] = lo;
}

// ------------------------------------------------------------------------------------------
// The wide layers as GEMMs on the tensor cores.  Grid (ceil(rows / 128), nodes), 128 threads.
// Thread 0 issues the TMA loads, thread 32 the MMAs, and all four warps read the accumulator
// back (warp w owns TMEM lanes 32 w .. 32 w + 31 = rows of the tile).
//
// kConv / kConvCode: Conv1d(CIN -> COUT, k3, s2) + leaky ReLU.  Row t of the GEMM is output
//   position t; its K = 3 CIN operands are the activation floats [2t CIN, (2t + 3) CIN).  The
//   activation is addressed as rows of 2 CIN floats (a pair of positions): row t followed by the
//   first half of row t + 1.  kConvCode is conv4: its output goes straight through conv5 (1x1,
//   64 -> 4, no activation) and only the code is written.
// kDeconv / kDeconvFinal: ConvTranspose1d(CIN -> COUT, k3, s2) + leaky ReLU.  Row j of the GEMM
//   makes output positions 2j and 2j + 1 (N = 2 COUT columns: even position, then odd) from the
//   K = 2 CIN floats of input positions j - 1 and j:
//       y[2j]     = b + sum_ci w[ci][co][2] x[j-1][ci] + w[ci][co][0] x[j][ci]
//       y[2j + 1] = b + sum_ci w[ci][co][1] x[j][ci]
//   (input rows -1 and L_in read as zeros).  kDeconvFinal is deconv5: its output goes through
//   the final 1x1 convolution (32 -> 1) and only the reconstruction is written.
// Outputs that feed another GEMM are written channels-last as two tf32 parts.
// Every wait has a limit; a CTA whose wait runs out records it and leaves without touching the
// output (tensor memory is released on every path).
// ------------------------------------------------------------------------------------------
// kGradDeconv: the gradient at the input of a convolution, which is a transposed convolution of the gradient at
//   its output with the same weights (w[co][ci][tau] read as [c_in' = co][c_out' = ci][tau]).  As kDeconv, for every
//   node, but the epilogue adds no bias: it multiplies by the leaky ReLU's derivative at the convolution's input
//   (sign of the stored activation `extra`, laid out like the output) and writes the two tf32 parts.
enum GemmMode { kConv = 0, kConvCode = 1, kDeconv = 2, kDeconvFinal = 3, kGradDeconv = 4 };

template <int MODE, int CIN, int COUT>
struct GemmShape {
    static constexpr bool kIsConv = MODE == kConv || MODE == kConvCode;
    static constexpr int kK = kIsConv ? 3 * CIN : 2 * CIN;      // operands per row
    static constexpr int kN = kIsConv ? COUT : 2 * COUT;        // columns of the layer's GEMM
    static constexpr int kNT = kN > 128 ? 128 : kN;             // columns of one tile: wider layers are cut in two along N
    static constexpr int kNSplit = kN / kNT;
    static constexpr int kBlocks = kK / kBlockK;
    static constexpr int kABytes = kTileM * kBlockK * 4;        // one (hi or lo) activation tile of a k-block
    static constexpr int kBBytes = kNT * kBlockK * 4;
    static constexpr int kStageBytes = 2 * kABytes + 2 * kBBytes;
    static constexpr int kEpiBytes = 4 * 32 * kStagePitch * 4;  // one 32 x 32 staging block per epilogue warp
    // as many stages as fit beside the staging blocks (one CTA per SM)
    static constexpr int kFit = (218 * 1024 - kEpiBytes) / kStageBytes;
    static constexpr int kStages = kFit < kBlocks ? kFit : kBlocks;
    static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + 1024;   // + slack to align the tiles to 1024 bytes
    static constexpr int kTmemCols = 2 * kNT;                   // two accumulators: one is drained while the other fills
    static_assert(kNT >= 32 && kNT <= 128 && (kNT & (kNT - 1)) == 0 && kN % kNT == 0, "tile columns: a power of two in [32, 128]");
    static_assert(kStages >= 1, "a stage must fit");
};

constexpr int kGemmThreads = 192;     // warp 0: TMA loads, warp 1: tensor memory + MMA issue, warps 2..5: epilogue

// Polls the barrier; gives up when the limit is reached or another role has given up (then *failed is set).
__device__ __forceinline__ bool mbar_wait_shared(uint32_t bar, uint32_t parity, volatile int *failed)
{
    for (int i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if ((i & 255) == 255 && *failed) return false;
    }
    *failed = 1;
    return false;
}

// The kernel is persistent: a CTA takes tiles blockIdx.x, blockIdx.x + gridDim.x, ... of the layer's
// nodes x row tiles x column halves.  One thread keeps the TMA loads going through a ring of stages, one
// thread issues the MMAs of a tile into one of two accumulators in tensor memory, and four epilogue warps
// drain the other accumulator meanwhile (warp w reads the 32 lanes of tensor memory its number lets it
// reach: quarter w % 4).  Every wait is bounded; a role that gives up tells the others through `failed`,
// everybody leaves through the common exit, and tensor memory is released.
template <int MODE, int CIN, int COUT>
__global__ void __launch_bounds__(kGemmThreads)
ae5_gemm_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                const float *__restrict__ bias, int tiles_x, int nodes, int64_t L_out, int64_t Lpad_out,
                float *__restrict__ out_hi, float *__restrict__ out_lo, const float *__restrict__ w_last,
                const float *__restrict__ b_last, float *__restrict__ out_last, const float *__restrict__ extra,
                int32_t *errword, int wz0, int wz_step, int64_t param_stride)
{
    using S = GemmShape<MODE, CIN, COUT>;
    constexpr int NT = S::kNT;
    grid_release_dependents();            // the next launch may set itself up while this one runs
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[S::kStages], empty_bar[S::kStages], tfull_bar[2], tempty_bar[2];
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile int failed;
    // every epilogue warp keeps its own copy of the node's small tensors: no barrier between the warps
    __shared__ float s_bias[4][COUT];
    __shared__ float s_wl[4][MODE == kConvCode ? 4 * 64 : 32], s_bl[4][4];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const int total = tiles_x * nodes * S::kNSplit;

    if (threadIdx.x == 0) {
        failed = 0;
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tfull_bar[b]), 1);
            mbar_init(smem_u32(&tempty_bar[b]), 4);               // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                      // one warp allocates the two accumulators
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)),
                     "r"((uint32_t)S::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base_smem;
    grid_wait();                          // barriers and tensor memory are set up: now the predecessor's results are needed

    if (threadIdx.x == 0) {
        // producer: one k-block (32 floats of the operand row) of both operands, hi and lo, per stage
        int it = 0;                                               // k-blocks loaded so far, over all tiles
        for (int tile = blockIdx.x; tile < total && !failed; tile += gridDim.x) {
            const int nt = tile % S::kNSplit, tx = tile / S::kNSplit % tiles_x, node = tile / (S::kNSplit * tiles_x);
            const int t0 = tx * kTileM, wz = wz0 + node * wz_step;
            for (int kb = 0; kb < S::kBlocks; ++kb, ++it) {
                const int s = it % S::kStages;
                if (it >= S::kStages && !mbar_wait_shared(smem_u32(&empty_bar[s]), ((it / S::kStages) & 1) ^ 1, &failed)) break;
                const uint32_t bar = smem_u32(&full_bar[s]);
                const uint32_t st = tiles + (uint32_t)s * S::kStageBytes;
                mbar_expect_tx(bar, S::kStageBytes);
                const int c = kb * kBlockK;                       // column inside the operand row
                int col, row;
                if (S::kIsConv) {                                 // activation rows hold a pair of positions
                    col = c < 2 * CIN ? c : c - 2 * CIN;
                    row = c < 2 * CIN ? t0 : t0 + 1;
                } else {                                          // activation rows hold one position: j - 1, then j
                    col = c < CIN ? c : c - CIN;
                    row = c < CIN ? t0 - 1 : t0;
                }
                tma_load_3d(st, &map_a_hi, bar, col, row, node);
                tma_load_3d(st + S::kABytes, &map_a_lo, bar, col, row, node);
                tma_load_3d(st + 2 * S::kABytes, &map_b_hi, bar, c, nt * NT, wz);
                tma_load_3d(st + 2 * S::kABytes + S::kBBytes, &map_b_lo, bar, c, nt * NT, wz);
            }
        }
    } else if (threadIdx.x == 32) {
        // instruction descriptor: fp32 accumulator, tf32 x tf32, both operands K-major, NT columns, M = 128
        constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
        int it = 0, acc = 0;                                      // k-blocks consumed, tiles issued
        for (int tile = blockIdx.x; tile < total && !failed; tile += gridDim.x, ++acc) {
            const int buf = acc & 1;
            // the epilogue must have drained this accumulator's previous tile
            if (acc >= 2 && !mbar_wait_shared(smem_u32(&tempty_bar[buf]), ((acc >> 1) & 1) ^ 1, &failed)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d = tmem + (uint32_t)(buf * NT);
            bool ok = true;
            for (int kb = 0; kb < S::kBlocks; ++kb, ++it) {
                const int s = it % S::kStages;
                if (!mbar_wait_shared(smem_u32(&full_bar[s]), (it / S::kStages) & 1, &failed)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t st = tiles + (uint32_t)s * S::kStageBytes;
                const uint64_t a_hi = umma_desc(st), a_lo = umma_desc(st + S::kABytes);
                const uint64_t b_hi = umma_desc(st + 2 * S::kABytes), b_lo = umma_desc(st + 2 * S::kABytes + S::kBBytes);
#pragma unroll
                for (int ks = 0; ks < kBlockK / 8; ++ks) {        // 8 tf32 = 32 bytes per step along K
                    const uint64_t adv = (uint64_t)(ks * 32 >> 4);
                    umma_tf32(d, a_hi + adv, b_hi + adv, idesc, kb > 0 || ks > 0);
                    umma_tf32(d, a_hi + adv, b_lo + adv, idesc, true);
                    umma_tf32(d, a_lo + adv, b_hi + adv, idesc, true);
                }
                umma_commit(smem_u32(&empty_bar[s]));             // the stage may be refilled once these have run
            }
            if (!ok) break;
            umma_commit(smem_u32(&tfull_bar[buf]));               // the accumulator is complete once these have run
        }
    } else if (warp >= 2) {
        const int q = warp & 3;                                   // the quarter of tensor memory this warp reaches
        float *stage = reinterpret_cast<float *>(dyn_smem + (tiles - smem_u32(dyn_smem)) + S::kStages * S::kStageBytes) +
                       q * (32 * kStagePitch);
        int acc = 0, cur_node = -1;
        for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++acc) {
            const int nt = tile % S::kNSplit, tx = tile / S::kNSplit % tiles_x, node = tile / (S::kNSplit * tiles_x);
            const int t0 = tx * kTileM, buf = acc & 1;
            if (node != cur_node) {                               // this node's (decoder's) small tensors
                __syncwarp();
                const float *nb = bias + (int64_t)node * param_stride;
                if (MODE != kGradDeconv)
                    for (int i = lane; i < COUT; i += 32) s_bias[q][i] = nb[i];
                if (MODE == kConvCode) {
                    for (int i = lane; i < 4 * 64; i += 32) s_wl[q][i] = w_last[(int64_t)node * param_stride + i];
                    if (lane < 4) s_bl[q][lane] = b_last[(int64_t)node * param_stride + lane];
                }
                if (MODE == kDeconvFinal) {
                    s_wl[q][lane] = w_last[(int64_t)node * param_stride + lane];
                    if (lane == 0) {
                        s_bl[q][0] = b_last[(int64_t)node * param_stride];
                        s_bl[q][1] = extra ? w_last[(int64_t)node * param_stride + 32] : 0.0f;   // parameter server: the tap on the innovation
                    }
                }
                __syncwarp();
                cur_node = node;
            }
            int have = 0;
            if (lane == 0) have = mbar_wait_shared(smem_u32(&tfull_bar[buf]), (acc >> 1) & 1, &failed) ? 1 : 0;
            have = __shfl_sync(0xffffffffu, have, 0);
            if (!have) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int64_t t = (int64_t)t0 + q * 32 + lane;          // this thread's row
            const uint32_t trow = tmem + (uint32_t)(buf * NT) + ((uint32_t)(q * 32) << 16);
            float last[4] = {0.f, 0.f, 0.f, 0.f};                   // kConvCode: the 4 code channels; kDeconvFinal: 2 positions
#pragma unroll 1
            for (int cl = 0; cl < NT; cl += 32) {
                float x[32];
                tmem_load32(trow + (uint32_t)cl, x);
                const int c0 = nt * NT + cl;                        // column of the layer's GEMM
                const int cb = S::kIsConv ? c0 : c0 % COUT;         // channel of column c0
                if (MODE == kGradDeconv) {
                    const int64_t pos = 2 * t + (c0 >= COUT ? 1 : 0);
                    if (pos < L_out) {
                        const float4 *m4 = reinterpret_cast<const float4 *>(extra + ((int64_t)node * Lpad_out + pos) * COUT + cb);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float4 m = m4[v];
                            x[4 * v] = m.x > 0.0f ? x[4 * v] : __fmul_rn(kSlope, x[4 * v]);
                            x[4 * v + 1] = m.y > 0.0f ? x[4 * v + 1] : __fmul_rn(kSlope, x[4 * v + 1]);
                            x[4 * v + 2] = m.z > 0.0f ? x[4 * v + 2] : __fmul_rn(kSlope, x[4 * v + 2]);
                            x[4 * v + 3] = m.w > 0.0f ? x[4 * v + 3] : __fmul_rn(kSlope, x[4 * v + 3]);
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) x[j] = leaky(__fadd_rn(x[j], s_bias[q][cb + j]));
                }
                if (MODE == kConvCode) {
#pragma unroll
                    for (int o = 0; o < 4; ++o)
#pragma unroll
                        for (int j = 0; j < 32; ++j) last[o] = __fmaf_rn(s_wl[q][o * 64 + c0 + j], x[j], last[o]);
                } else if (MODE == kDeconvFinal) {                   // COUT = 32: columns 0..31 position 2t, 32..63 position 2t + 1
                    float a = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) a = __fmaf_rn(s_wl[q][j], x[j], a);
                    last[c0 / 32] = a;
                } else {
                    // The 32 x 32 block of this warp (row = lane) goes through shared memory, first its hi parts, then
                    // its lo parts, so that the global stores are whole 128-byte rows.
#pragma unroll 1
                    for (int part = 0; part < 2; ++part) {
                        __syncwarp();                                // the previous block has been read out
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            float hi[4], lo[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) split_tf32(x[4 * v + j], hi[j], lo[j]);
                            *reinterpret_cast<float4 *>(stage + lane * kStagePitch + 4 * v) =
                                part == 0 ? make_float4(hi[0], hi[1], hi[2], hi[3]) : make_float4(lo[0], lo[1], lo[2], lo[3]);
                        }
                        __syncwarp();
                        float *out = part == 0 ? out_hi : out_lo;
#pragma unroll
                        for (int itr = 0; itr < 8; ++itr) {
                            const int rr = itr * 4 + (lane >> 3), cq = lane & 7;      // four rows per pass, eight lanes per row
                            const int64_t tr = (int64_t)t0 + q * 32 + rr;
                            // conv: row tr is position tr; deconv: columns below COUT are position 2 tr, the others 2 tr + 1
                            const int64_t pos = S::kIsConv ? tr : 2 * tr + (c0 >= COUT ? 1 : 0);
                            if (pos < L_out) {
                                const int64_t at = (S::kIsConv ? ((int64_t)node * Lpad_out + tr) * COUT
                                                               : ((int64_t)node * Lpad_out + 2 * tr) * COUT) + c0 + 4 * cq;
                                *reinterpret_cast<float4 *>(out + at) = *reinterpret_cast<const float4 *>(stage + rr * kStagePitch + 4 * cq);
                            }
                        }
                    }
                }
            }
            if (MODE == kConvCode && t < L_out)
                reinterpret_cast<float4 *>(out_last)[(int64_t)node * L_out + t] =
                    make_float4(__fadd_rn(last[0], s_bl[q][0]), __fadd_rn(last[1], s_bl[q][1]), __fadd_rn(last[2], s_bl[q][2]),
                                __fadd_rn(last[3], s_bl[q][3]));
            if (MODE == kDeconvFinal) {
                const int64_t row0 = (int64_t)node * L_out;              // decoder `node` reconstructs row `node`
                if (2 * t < L_out) {
                    const float y = __fadd_rn(last[0], s_bl[q][0]);
                    out_last[row0 + 2 * t] = extra ? __fmaf_rn(s_bl[q][1], extra[row0 + 2 * t], y) : y;
                }
                if (2 * t + 1 < L_out) {
                    const float y = __fadd_rn(last[1], s_bl[q][0]);
                    out_last[row0 + 2 * t + 1] = extra ? __fmaf_rn(s_bl[q][1], extra[row0 + 2 * t + 1], y) : y;
                }
            }
            // the accumulator may be overwritten
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&tempty_bar[buf])) : "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && failed) atomicExch(errword, 0x5EA5);          // a wait ran out
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::kTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------
// Weight gradients of the wide convolutions as GEMMs that sum over rows (the backward pass's
//     dW[co][tau C_in + ci] = sum over (node, t) of G[t][co] X[2t + tau][ci]):
// the reduction runs along the ROWS of both operands, so both are read "MN-major": a k-block is 32 rows
// (positions t) of 128-byte pieces of the operand's columns, and one tcgen05.mma consumes 8 rows.
// Shared-memory layout of an operand tile of C columns: C / 32 pieces, each 32 rows x 128 bytes as the TMA
// writes a box of 32 floats x 32 rows with the 128-byte swizzle of 32-byte atoms (the one layout the tensor
// cores read 32-bit operands from in this orientation); the matrix descriptor's leading offset is the
// piece (4096 bytes), its stride offset the group of 4 rows (512 bytes), and the instruction descriptor marks
// both operands as transposed.  The M operand is 128 columns of one matrix, the N operand NT columns of the
// other; each is either the gradient G (one map) or the input slices X (two maps: columns below `split` are
// taps 0 and 1 of pair-row t, the others tap 2 = the first C_in floats of pair-row t + 1).  Rows beyond the
// layer's length are outside the maps and arrive as zeros.
// One CTA = (M tile, N tile, node, part of the node's rows); its 128 x NT sums go to partial[chunk], chunk =
// node * splits + part, as [M][N] or (TRANS) as [N][M]; the kernel that applies Adam adds the chunks up.
// Same roles and bounded waits as ae5_gemm_kernel: TMA thread, MMA thread, four warps that read the accumulator.
// ------------------------------------------------------------------------------------------
struct alignas(64) WgradMaps {
    CUtensorMap m[2][2], n[2][2];      // [hi, lo][columns below the split, columns from the split on]
};

template <int NT>
struct WgradShape {
    static constexpr int kABytes = 128 * kBlockK * 4;          // one part (hi or lo) of the M operand's k-block
    static constexpr int kBBytes = NT * kBlockK * 4;
    static constexpr int kStageBytes = 2 * kABytes + 2 * kBBytes;
    static constexpr int kFit = 218 * 1024 / kStageBytes;
    static constexpr int kStages = kFit < 4 ? kFit : 4;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024;
    static constexpr int kTmemCols = NT <= 32 ? 32 : NT <= 64 ? 64 : NT <= 128 ? 128 : 256;
    static_assert(NT % 32 == 0 && NT >= 32 && NT <= 256, "N tile: whole 128-byte pieces, one accumulator");
    static_assert(kStages >= 2, "two stages must fit");
};

// Matrix descriptor of an MN-major operand tile as laid out above.  32-bit operands read along their rows have
// one layout: the 128-byte swizzle in units of 32 bytes, whose pattern repeats every 4 rows (512 bytes).
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);         // start address, 16-byte units
    d |= (uint64_t)(4096 >> 4) << 16;                     // leading byte offset: from one 128-byte piece of columns to the next
    d |= (uint64_t)(512 >> 4) << 32;                      // stride byte offset: from one group of 4 rows to the next
    d |= (uint64_t)1 << 46;                               // descriptor version of this architecture
    d |= (uint64_t)1 << 61;                               // 128-byte swizzle with 32-byte atoms
    return d;
}

template <int NT, bool TRANS>
__global__ void __launch_bounds__(kGemmThreads)
ae5_wgrad_kernel(const __grid_constant__ WgradMaps maps, int m_split, int n_split, int tiles_m, int tiles_n, int splits,
                 int kb_per_node, int kbps, int m_total, int n_total, float *__restrict__ partial, int64_t pstride,
                 int32_t *errword)
{
    using S = WgradShape<NT>;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t full_bar[S::kStages], empty_bar[S::kStages], tfull_bar;
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile int failed;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    // this CTA's work
    int w = blockIdx.x;
    const int tm = w % tiles_m; w /= tiles_m;
    const int tn = w % tiles_n; w /= tiles_n;
    const int part = w % splits, node = w / splits;
    const int kb0 = part * kbps, kb1 = kb0 + kbps < kb_per_node ? kb0 + kbps : kb_per_node;   // (never empty: see the host)
    const int m0 = tm * 128, n0 = tn * NT;

    if (threadIdx.x == 0) {
        failed = 0;
        for (int s = 0; s < S::kStages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        mbar_init(smem_u32(&tfull_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)),
                     "r"((uint32_t)S::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base_smem;

    if (threadIdx.x == 0) {
        for (int kb = kb0, it = 0; kb < kb1; ++kb, ++it) {
            const int s = it % S::kStages;
            if (it >= S::kStages && !mbar_wait_shared(smem_u32(&empty_bar[s]), ((it / S::kStages) & 1) ^ 1, &failed)) break;
            const uint32_t bar = smem_u32(&full_bar[s]);
            const uint32_t st = tiles + (uint32_t)s * S::kStageBytes;
            mbar_expect_tx(bar, S::kStageBytes);
            const int row = kb * kBlockK;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {                 // the M operand: four pieces of 32 columns
                    const int col = m0 + 32 * j;
                    const uint32_t dst = st + (uint32_t)(h * S::kABytes + j * 4096);
                    if (col < m_split) tma_load_3d(dst, &maps.m[h][0], bar, col, row, node);
                    else tma_load_3d(dst, &maps.m[h][1], bar, col - m_split, row + 1, node);
                }
#pragma unroll
                for (int j = 0; j < NT / 32; ++j) {
                    const int col = n0 + 32 * j;
                    const uint32_t dst = st + (uint32_t)(2 * S::kABytes + h * S::kBBytes + j * 4096);
                    if (col < n_split) tma_load_3d(dst, &maps.n[h][0], bar, col, row, node);
                    else tma_load_3d(dst, &maps.n[h][1], bar, col - n_split, row + 1, node);
                }
            }
        }
    } else if (threadIdx.x == 32) {
        // instruction descriptor: fp32 accumulator, tf32 x tf32, both operands MN-major (bits 15 and 16), N = NT, M = 128
        constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(NT >> 3) << 17) |
                                   ((uint32_t)(128 >> 4) << 24);
        bool ok = true;
        for (int kb = kb0, it = 0; kb < kb1; ++kb, ++it) {
            const int s = it % S::kStages;
            if (!mbar_wait_shared(smem_u32(&full_bar[s]), (it / S::kStages) & 1, &failed)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t st = tiles + (uint32_t)s * S::kStageBytes;
#pragma unroll
            for (int ks = 0; ks < kBlockK / 8; ++ks) {            // 8 rows per step: two groups of the layout
                const uint64_t a_hi = umma_desc_mn(st + ks * 1024), a_lo = umma_desc_mn(st + S::kABytes + ks * 1024);
                const uint64_t b_hi = umma_desc_mn(st + 2 * S::kABytes + ks * 1024);
                const uint64_t b_lo = umma_desc_mn(st + 2 * S::kABytes + S::kBBytes + ks * 1024);
                umma_tf32(tmem, a_hi, b_hi, idesc, it > 0 || ks > 0);
                umma_tf32(tmem, a_hi, b_lo, idesc, true);
                umma_tf32(tmem, a_lo, b_hi, idesc, true);
            }
            umma_commit(smem_u32(&empty_bar[s]));
        }
        if (ok) umma_commit(smem_u32(&tfull_bar));
    } else if (warp >= 2) {
        const int q = warp & 3;
        int have = 0;
        if (lane == 0) have = mbar_wait_shared(smem_u32(&tfull_bar), 0, &failed) ? 1 : 0;
        have = __shfl_sync(0xffffffffu, have, 0);
        if (have) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float *out = partial + (int64_t)(node * splits + part) * pstride;
            const int m = m0 + q * 32 + lane;                     // this thread's row of the accumulator
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int cl = 0; cl < NT; cl += 32) {
                float x[32];
                tmem_load32(trow + (uint32_t)cl, x);
                if (TRANS) {                                      // out[n][m]: a warp writes 32 consecutive floats per column
#pragma unroll
                    for (int j = 0; j < 32; ++j) out[(int64_t)(n0 + cl + j) * m_total + m] = x[j];
                } else {                                          // out[m][n]: 128 bytes per thread
                    float4 *o4 = reinterpret_cast<float4 *>(out + (int64_t)m * n_total + n0 + cl);
#pragma unroll
                    for (int v = 0; v < 8; ++v) o4[v] = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && failed) atomicExch(errword, 0x5EA6);          // a wait ran out
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::kTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------
// Decoder (one pass, fp32 pipes), channels-last.
// ------------------------------------------------------------------------------------------
// deconv1: ConvTranspose1d(4 -> 4, k3, stride 1, padding 1) + leaky ReLU on the mean code.
// blockIdx.y: the decoder (its parameters lie param_stride floats after the previous one's, its output L4 rows on).
__global__ void ae5_deconv1_kernel(const float *__restrict__ z, int64_t L4, const float *__restrict__ w,
                                   const float *__restrict__ b, float *__restrict__ out, int64_t param_stride)
{
    grid_release_dependents();
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= L4) return;
    w += (int64_t)blockIdx.y * param_stride;
    b += (int64_t)blockIdx.y * param_stride;
    out += (int64_t)blockIdx.y * L4 * 4;
    float acc[4] = {b[0], b[1], b[2], b[3]};
    grid_wait();                          // the code comes from the launch in front
#pragma unroll
    for (int tau = 0; tau < 3; ++tau) {
        const int64_t j = s + 1 - tau;                            // y[s] += w[ci][co][tau] x[ci][j], s = j + tau - 1
        if (j < 0 || j >= L4) continue;
        const float4 x = reinterpret_cast<const float4 *>(z)[j];
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int ci = 0; ci < 4; ++ci)
#pragma unroll
            for (int co = 0; co < 4; ++co) acc[co] = __fmaf_rn(w[(ci * 4 + co) * 3 + tau], xs[ci], acc[co]);
    }
    reinterpret_cast<float4 *>(out)[s] = make_float4(leaky(acc[0]), leaky(acc[1]), leaky(acc[2]), leaky(acc[3]));
}

// ConvTranspose1d(CIN -> COUT, k3, s2, output padding) + leaky ReLU on the fp32 pipes (deconv2, 4 -> 32):
//   y[2j]     = b + sum_ci w[ci][co][0] x[j][ci] + w[ci][co][2] x[j-1][ci]
//   y[2j + 1] = b + sum_ci w[ci][co][1] x[j][ci]
// CTA: TP input positions j0 .. j0 + TP - 1 -> outputs 2 j0 .. 2 j0 + 2 TP - 1; thread = (output
// channel, slice of positions); weights and the input rows sit in shared memory.
template <int CIN, int COUT, int TP>
__global__ void __launch_bounds__(256)
ae5_deconv_kernel(const float *__restrict__ x, int64_t L_in, int64_t L_out, const float *__restrict__ w,
                  const float *__restrict__ b, float *__restrict__ y, float *__restrict__ y_lo, int64_t param_stride)
{
    extern __shared__ float dsm[];
    grid_release_dependents();
    x += (int64_t)blockIdx.y * L_in * CIN;                  // blockIdx.y: the decoder
    w += (int64_t)blockIdx.y * param_stride;
    b += (int64_t)blockIdx.y * param_stride;
    y += (int64_t)blockIdx.y * L_out * COUT;
    y_lo += (int64_t)blockIdx.y * L_out * COUT;
    float *sw = dsm;                          // [tau][ci][co]
    float *sx = dsm + 3 * CIN * COUT;         // [TP + 1][CIN]: rows j0 - 1 .. j0 + TP - 1
    const int64_t j0 = (int64_t)blockIdx.x * TP;
    for (int i = threadIdx.x; i < 3 * CIN * COUT; i += 256) {
        const int tau = i / (CIN * COUT), rem = i % (CIN * COUT), ci = rem / COUT, co = rem % COUT;
        sw[i] = w[(ci * COUT + co) * 3 + tau];
    }
    grid_wait();                          // the weights are in place: now the input rows of the launch in front
    for (int i = threadIdx.x; i < (TP + 1) * CIN; i += 256) {
        const int64_t j = j0 - 1 + i / CIN;
        sx[i] = j >= 0 && j < L_in ? x[j * CIN + i % CIN] : 0.0f;
    }
    __syncthreads();
    constexpr int kSlices = 256 / COUT;       // threads along positions
    const int co = threadIdx.x % COUT, sl = threadIdx.x / COUT;
    const float bias = b[co];
    for (int jl = sl; jl < TP; jl += kSlices) {
        const int64_t j = j0 + jl;
        if (2 * j >= L_out) break;
        float even = bias, odd = bias;
        const float *xj = sx + (jl + 1) * CIN, *xp = sx + jl * CIN;
#pragma unroll 8
        for (int ci = 0; ci < CIN; ++ci) {
            const float a = xj[ci], p = xp[ci];
            even = __fmaf_rn(sw[(0 * CIN + ci) * COUT + co], a, even);
            even = __fmaf_rn(sw[(2 * CIN + ci) * COUT + co], p, even);
            odd = __fmaf_rn(sw[(1 * CIN + ci) * COUT + co], a, odd);
        }
        float hi, lo;                                          // the output feeds a GEMM: two tf32 parts
        split_tf32(leaky(even), hi, lo);
        y[(2 * j) * COUT + co] = hi;
        y_lo[(2 * j) * COUT + co] = lo;
        if (2 * j + 1 < L_out) {
            split_tf32(leaky(odd), hi, lo);
            y[(2 * j + 1) * COUT + co] = hi;
            y_lo[(2 * j + 1) * COUT + co] = lo;
        }
    }
}

inline unsigned blocks(int64_t n, int per) { return (unsigned)((n + per - 1) / per); }

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link the driver
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t encode_fn(EncodeTiledFn *out)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    *out = reinterpret_cast<EncodeTiledFn>(fn);
    return cudaSuccess;
}

// Activation [K][Lpad][C] (Lpad even) seen as [K][Lpad / 2][2 C]; box: 32 floats x 128 rows.
bool make_act_map(EncodeTiledFn enc, CUtensorMap *m, float *base, int C, int64_t Lpad, int K)
{
    const cuuint64_t dims[3] = {(cuuint64_t)(2 * C), (cuuint64_t)(Lpad / 2), (cuuint64_t)K};
    const cuuint64_t strides[2] = {(cuuint64_t)(2 * C) * 4, (cuuint64_t)Lpad * C * 4};
    const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Decoder activations [decoders][L][C]; box: 32 floats x 128 rows of one decoder.
bool make_dact_map(EncodeTiledFn enc, CUtensorMap *m, float *base, int C, int64_t L, int decoders)
{
    const cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)L, (cuuint64_t)decoders};
    const cuuint64_t strides[2] = {(cuuint64_t)C * 4, (cuuint64_t)L * C * 4};
    const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// GEMM weights [count][rows][k] (count sets of weights back to back); box: 32 floats x all rows of one set.
bool make_matrix_map(EncodeTiledFn enc, CUtensorMap *m, float *base, int k, int rows, int count = 1)
{
    const cuuint64_t dims[3] = {(cuuint64_t)k, (cuuint64_t)rows, (cuuint64_t)count};
    const cuuint64_t strides[2] = {(cuuint64_t)k * 4, (cuuint64_t)k * rows * 4};
    const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)(rows > 128 ? 128 : rows), 1};   // the columns of one tile
    const cuuint32_t es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MODE, int CIN, int COUT>
cudaError_t launch_gemm(Ctx &c, const CUtensorMap &a_hi, const CUtensorMap &a_lo, const CUtensorMap &b_hi,
                        const CUtensorMap &b_lo, const float *bias, int64_t rows, int nodes, int64_t L_out, int64_t Lpad_out,
                        float *out_hi, float *out_lo, const float *w_last, const float *b_last, float *out_last,
                        const float *extra = nullptr, int wz0 = 0, int wz_step = 0, int64_t param_stride = 0)
{
    using S = GemmShape<MODE, CIN, COUT>;
    auto kern = ae5_gemm_kernel<MODE, CIN, COUT>;
    static OncePerDevice configured;            // one per instantiation of this template
    {
        const cudaError_t e = configured.run(
            [&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kSmemBytes); });
        if (e != cudaSuccess) return e;
    }
    const int tiles_x = (int)blocks(rows, kTileM);
    const int64_t total = (int64_t)tiles_x * nodes * S::kNSplit;
    const unsigned grid = (unsigned)(total < sm_count() ? total : sm_count());     // persistent: one CTA per SM at most
    const cudaError_t e = launch_dependent_smem(kern, dim3(grid), dim3(kGemmThreads), S::kSmemBytes, c.stream, a_hi, a_lo, b_hi, b_lo, bias,
                                                tiles_x, nodes, L_out, Lpad_out, out_hi, out_lo, w_last, b_last, out_last, extra,
                                                c.errword, wz0, wz_step, param_stride);
    if (e != cudaSuccess) return e;
    ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace

const int kAe5EncCh[5] = {1, 64, 128, 256, 64};
const int kAe5DecCh[6] = {4, 4, 32, 64, 128, 32};

static int64_t ae5_decoder_params(bool innovation_channel)
{
    int64_t n = 0;
    for (int i = 0; i < 5; ++i) n += (int64_t)kAe5DecCh[i] * kAe5DecCh[i + 1] * 3 + kAe5DecCh[i + 1];
    return n + 32 + 1 + (innovation_channel ? 1 : 0);
}

int64_t ae5_param_count(int decoders, bool innovation_channel)
{
    int64_t n = 0;
    for (int i = 0; i < 4; ++i) n += (int64_t)kAe5EncCh[i + 1] * kAe5EncCh[i] * 3 + kAe5EncCh[i + 1];
    n += 4 * 64 + 4;
    return n + decoders * ae5_decoder_params(innovation_channel);
}

// Lengths after conv1..conv4; false when the input is too short.
bool ae5_lengths(int64_t mu, int64_t (&len)[5])
{
    len[0] = mu;
    for (int i = 0; i < 4; ++i) {
        if (len[i] < 3) return false;
        len[i + 1] = (len[i] - 3) / 2 + 1;
    }
    return true;
}

// How the rows of a wide convolution's weight gradient are cut: every node's l_out rows (k-blocks of 32) into
// `splits` parts of `kbps` k-blocks, so that tiles x nodes x parts comes to at most two CTAs per SM (two rounds
// of one CTA per SM), a part has at least four k-blocks where the layer is long enough, and none is empty.
void ae5_weight_gradient_chunks(int K, int64_t l_out, int cin, int cout, int *splits, int *kbps)
{
    const int kb = (int)((l_out + kBlockK - 1) / kBlockK);
    // tiles of the launch (launch_ae5_weight_gradient): 128 output channels x 192 or 128 slice columns; 64 channels: 128 slice columns x 64
    const int tiles = cout >= 128 ? (cout / 128) * (3 * cin % 128 == 0 ? 3 * cin / 128 : 1) : 3 * cin / 128;
    int want = 2 * 148 / (tiles * K);                 // (a tuning figure: the SM count of the B200; any device computes the same sums)
    want = std::max(1, std::min(want, std::max(1, kb / 4)));
    *kbps = (kb + want - 1) / want;
    *splits = (kb + *kbps - 1) / *kbps;
}

void ae5_carve(Ae5 &a, int K, int64_t mu, bool ps, char *base, size_t *used)
{
    ae5_lengths(mu, a.len);
    a.decoders = ps ? K : 1;
    a.dec_stride = ae5_decoder_params(ps);
    size_t at = *used;
    auto take = [&](size_t floats) {
        at = (at + 1023) / 1024 * 1024;                     // TMA sources: generously aligned
        float *p = base ? reinterpret_cast<float *>(base + at) : nullptr;
        at += floats * sizeof(float);
        return p;
    };
    for (int l = 0; l < 3; ++l) {                           // outputs of conv1..conv3
        a.lpad[l] = (a.len[l + 1] + 1) / 2 * 2;
        const size_t n = (size_t)K * a.lpad[l] * kAe5EncCh[l + 1];
        a.act_hi[l] = take(n);
        a.act_lo[l] = take(n);
    }
    for (int l = 0; l < 3; ++l) {                           // GEMM weights of conv2..conv4
        const size_t n = (size_t)kAe5EncCh[l + 2] * kAe5EncCh[l + 1] * 3;
        a.w_hi[l] = take(n);
        a.w_lo[l] = take(n);
    }
    a.d0 = take((size_t)a.decoders * a.len[4] * 4);
    for (int l = 0; l < 3; ++l) {                           // outputs of deconv2..deconv4 of every decoder: lengths L3, L2, L1
        const size_t n = (size_t)a.decoders * a.len[3 - l] * kAe5DecCh[l + 2];
        a.dact_hi[l] = take(n);
        a.dact_lo[l] = take(n);
    }
    for (int l = 0; l < 3; ++l) {                           // GEMM weights of deconv3..deconv5, every decoder's
        const size_t n = (size_t)a.decoders * 4 * kAe5DecCh[l + 2] * kAe5DecCh[l + 3];
        a.dw_hi[l] = take(n);
        a.dw_lo[l] = take(n);
    }
    {
        // training: the two outputs inference never stores, the gradients at every layer's pre-activation,
        // the products of the backward GEMMs and the per-chunk partial sums of the parameter gradients
        a.act4_hi = take((size_t)K * a.len[4] * 64);
        a.act4_lo = take((size_t)K * a.len[4] * 64);
        a.dact5_hi = take((size_t)mu * 32);
        a.dact5_lo = take((size_t)mu * 32);
        for (int l = 0; l < 3; ++l) {                       // laid out like the outputs of conv1..conv3
            a.g_enc[l] = take((size_t)K * a.lpad[l] * kAe5EncCh[l + 1]);
            a.g_enc_lo[l] = take((size_t)K * a.lpad[l] * kAe5EncCh[l + 1]);
        }
        a.g_enc[3] = take((size_t)K * a.len[4] * 64);
        a.g4_hi = take((size_t)K * a.len[4] * 64);
        a.g4_lo = take((size_t)K * a.len[4] * 64);
        for (int j = 0; j < 3; ++j) {
            a.gw_hi[j] = take((size_t)4 * kAe5EncCh[j + 1] * kAe5EncCh[j + 2]);
            a.gw_lo[j] = take((size_t)4 * kAe5EncCh[j + 1] * kAe5EncCh[j + 2]);
        }
        a.g_dec[0] = take((size_t)a.len[4] * 4);
        for (int l = 1; l < 5; ++l) a.g_dec[l] = take((size_t)a.len[4 - l] * kAe5DecCh[l + 1]);
        a.dzk = take((size_t)K * a.len[4] * 4);
        a.dzbar = take((size_t)a.len[4] * 4);
        a.dr = take((size_t)mu);
        a.wt = take((size_t)256 * 384);
        a.loss_blocks = (int)((mu + 255) / 256);
        // partial sums of the loss: per decoder the reconstruction term's, then the similarity term's (parameter server)
        a.loss_part = reinterpret_cast<double *>(take((size_t)(a.decoders + 1) * a.loss_blocks * 2));
    }
    *used = at;
    // offsets of the layers' parameters inside the flat vector (encoder, then decoder)
    int64_t pos = 0;
    for (int i = 0; i < 4; ++i) {
        a.off_w[i] = pos; pos += (int64_t)kAe5EncCh[i + 1] * kAe5EncCh[i] * 3;
        a.off_b[i] = pos; pos += kAe5EncCh[i + 1];
    }
    a.off_w[4] = pos; pos += 4 * 64;
    a.off_b[4] = pos; pos += 4;
    for (int i = 0; i < 5; ++i) {
        a.off_dw[i] = pos; pos += (int64_t)kAe5DecCh[i] * kAe5DecCh[i + 1] * 3;
        a.off_db[i] = pos; pos += kAe5DecCh[i + 1];
    }
    a.off_dw[5] = pos; pos += ps ? 33 : 32;      // parameter server: one more tap, on the innovation channel
    a.off_db[5] = pos;
    // parameter tensors in order, with the rows their gradient sums run over and the chunks these are cut into
    int64_t part = 0;
    auto tensor = [&](int i, int64_t off, int64_t count, int64_t rows, int kind, int cin, int cout) {
        Ae5::Tensor &t = a.tensors[i];
        t.param_off = off; t.count = count; t.rows = rows; t.kind = kind; t.cin = cin; t.cout = cout;
        // up to 192 chunks: the decoder's weight gradients (64 x 64 tiles of a few thousand rows of ONE node) are a
        // handful of tiles, and a CTA's walk over its rows is a chain of load-multiply trips; biases, conv1 and the 1x1
        // convolutions are summed by few CTAs per chunk
        t.chunk = count > 256 ? std::max<int64_t>(64, (rows + 191) / 192) : std::max<int64_t>(128, (rows + 191) / 192);
        t.chunks = kind == 3 ? 1 : (int)((rows + t.chunk - 1) / t.chunk);
        if (kind == 1 && cin >= 64) {        // conv2..conv4: summed on the tensor cores, node by node
            const int l = i / 2;
            ae5_weight_gradient_chunks(K, a.len[l + 1], cin, cout, &a.wg_splits[l - 1], &a.wg_kbps[l - 1]);
            t.chunks = K * a.wg_splits[l - 1];
        }
        t.partial_off = part;
        part += t.chunks * ((count + 3) / 4 * 4);
    };
    for (int i = 0; i < 4; ++i) {            // conv1..conv4: sums over K L_out rows
        tensor(2 * i, a.off_w[i], (int64_t)kAe5EncCh[i + 1] * kAe5EncCh[i] * 3, (int64_t)K * a.len[i + 1], 1, kAe5EncCh[i], kAe5EncCh[i + 1]);
        tensor(2 * i + 1, a.off_b[i], kAe5EncCh[i + 1], (int64_t)K * a.len[i + 1], 0, 0, 0);
    }
    tensor(8, a.off_w[4], 4 * 64, (int64_t)K * a.len[4], 0, 0, 0);
    tensor(9, a.off_b[4], 4, (int64_t)K * a.len[4], 0, 0, 0);
    tensor(10, a.off_dw[0], 48, a.len[4], 3, 0, 0);       // deconv1: reduced by a kernel of its own
    tensor(11, a.off_db[0], 4, a.len[4], 3, 0, 0);
    for (int i = 1; i < 5; ++i) {            // deconv2..deconv5: weights sum over L_in rows, biases over L_out rows
        tensor(10 + 2 * i, a.off_dw[i], (int64_t)kAe5DecCh[i] * kAe5DecCh[i + 1] * 3, a.len[5 - i], 2, kAe5DecCh[i], kAe5DecCh[i + 1]);
        tensor(11 + 2 * i, a.off_db[i], kAe5DecCh[i + 1], a.len[4 - i], 0, 0, 0);
    }
    tensor(20, a.off_dw[5], ps ? 33 : 32, mu, 0, 0, 0);
    tensor(21, a.off_db[5], 1, mu, 0, 0, 0);
    if (base) a.partial = reinterpret_cast<float *>(base + (*used + 1023) / 1024 * 1024);
    *used = (*used + 1023) / 1024 * 1024 + (size_t)part * sizeof(float);
}

cudaError_t ae5_make_maps(Ctx &c)
{
    Ae5 &a = *c.ae5;
    EncodeTiledFn enc = nullptr;
    const cudaError_t e = encode_fn(&enc);
    if (e != cudaSuccess) return e;
    bool ok = true;
    for (int l = 0; l < 3; ++l) {
        const int cin = kAe5EncCh[l + 1], cout = kAe5EncCh[l + 2];
        ok = ok && make_act_map(enc, &a.map_act_hi[l], a.act_hi[l], cin, a.lpad[l], c.K);
        ok = ok && make_act_map(enc, &a.map_act_lo[l], a.act_lo[l], cin, a.lpad[l], c.K);
        ok = ok && make_matrix_map(enc, &a.map_w_hi[l], a.w_hi[l], 3 * cin, cout);
        ok = ok && make_matrix_map(enc, &a.map_w_lo[l], a.w_lo[l], 3 * cin, cout);
        const int dcin = kAe5DecCh[l + 2];
        ok = ok && make_dact_map(enc, &a.map_dact_hi[l], a.dact_hi[l], dcin, a.len[3 - l], a.decoders);
        ok = ok && make_dact_map(enc, &a.map_dact_lo[l], a.dact_lo[l], dcin, a.len[3 - l], a.decoders);
    }
    for (int j = 0; j < 3; ++j) {            // input-gradient GEMMs of conv2..conv4: A = the gradient at the layer's output
        const int C = kAe5EncCh[j + 2], cin = kAe5EncCh[j + 1];
        const cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)a.len[j + 2], (cuuint64_t)c.K};
        const cuuint64_t strides[2] = {(cuuint64_t)C * 4, (cuuint64_t)(j == 2 ? a.len[4] : a.lpad[j + 1]) * C * 4};
        const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        for (int h = 0; h < 2; ++h) {
            float *g = j == 2 ? (h ? a.g4_lo : a.g4_hi) : (h ? a.g_enc_lo[j + 1] : a.g_enc[j + 1]);
            ok = ok && enc(h ? &a.map_g_lo[j] : &a.map_g_hi[j], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, g, dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        }
        ok = ok && make_matrix_map(enc, &a.map_gw_hi[j], a.gw_hi[j], 2 * C, 2 * cin);
        ok = ok && make_matrix_map(enc, &a.map_gw_lo[j], a.gw_lo[j], 2 * C, 2 * cin);
    }
    for (int l = 1; l <= 3; ++l) {           // weight gradients of conv2..conv4: boxes of 32 floats x 32 rows, zeros beyond the length
        const int cin = kAe5EncCh[l], cout = kAe5EncCh[l + 1];
        const int64_t lout = a.len[l + 1];
        const cuuint32_t box[3] = {32, 32, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        for (int h = 0; h < 2; ++h) {
            float *g = l == 3 ? (h ? a.g4_lo : a.g4_hi) : (h ? a.g_enc_lo[l] : a.g_enc[l]);
            const cuuint64_t gdims[3] = {(cuuint64_t)cout, (cuuint64_t)lout, (cuuint64_t)c.K};
            const cuuint64_t gstr[2] = {(cuuint64_t)cout * 4, (cuuint64_t)(l == 3 ? lout : a.lpad[l]) * cout * 4};
            ok = ok && enc(&a.map_wg_g[l - 1][h], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, g, gdims, gstr, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            float *x = h ? a.act_lo[l - 1] : a.act_hi[l - 1];
            const cuuint64_t xstr[2] = {(cuuint64_t)(2 * cin) * 4, (cuuint64_t)a.lpad[l - 1] * cin * 4};
            // taps 0 and 1: pair-rows 0 .. lout - 1 in full; tap 2: the first half of pair-rows 1 .. lout
            const cuuint64_t xdims0[3] = {(cuuint64_t)(2 * cin), (cuuint64_t)lout, (cuuint64_t)c.K};
            const cuuint64_t xdims1[3] = {(cuuint64_t)cin, (cuuint64_t)(lout + 1), (cuuint64_t)c.K};
            ok = ok && enc(&a.map_wg_x[l - 1][h][0], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, x, xdims0, xstr, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            ok = ok && enc(&a.map_wg_x[l - 1][h][1], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, x, xdims1, xstr, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        }
    }
    a.map_dw_hi.resize(3);                   // one map per layer: slice d holds decoder d's weights
    a.map_dw_lo.resize(3);
    for (int l = 0; l < 3; ++l) {
        const int dcin = kAe5DecCh[l + 2], dcout = kAe5DecCh[l + 3];
        ok = ok && make_matrix_map(enc, &a.map_dw_hi[l], a.dw_hi[l], 2 * dcin, 2 * dcout, a.decoders);
        ok = ok && make_matrix_map(enc, &a.map_dw_lo[l], a.dw_lo[l], 2 * dcin, 2 * dcout, a.decoders);
    }
    return ok ? cudaSuccess : cudaErrorInvalidValue;
}

// The GEMM forms of the weights follow the parameter vector; redone after lgc_set_ae_params.
static void prepare_weights(Ctx &c)
{
    Ae5 &a = *c.ae5;
    if (a.weights_ready) return;
    const float *P = c.params;
    for (int l = 0; l < 3; ++l) {
        const int cin = kAe5EncCh[l + 1], cout = kAe5EncCh[l + 2];
        ae5_prep_weights_kernel<<<blocks((int64_t)cin * cout * 3, 256), 256, 0, c.stream>>>(P + a.off_w[l + 1], cin, cout, a.w_hi[l],
                                                                                           a.w_lo[l]),
            ++g_kernel_launches;
        const int dcin = kAe5DecCh[l + 2], dcout = kAe5DecCh[l + 3];
        for (int d = 0; d < a.decoders; ++d) {
            const size_t at = (size_t)d * 4 * dcin * dcout;
            ae5_prep_deconv_weights_kernel<<<blocks((int64_t)4 * dcin * dcout, 256), 256, 0, c.stream>>>(
                P + a.off_dw[l + 2] + d * a.dec_stride, dcin, dcout, a.dw_hi[l] + at, a.dw_lo[l] + at),
                ++g_kernel_launches;
        }
    }
    a.weights_ready = true;
}

// Stage 4 for the full-size autoencoder: gather, conv1..conv5 for every node; the codes are
// [K][L4][4] (position-major).
cudaError_t launch_ae5_encode(Ctx &c)
{
    Ae5 &a = *c.ae5;
    const float *P = c.params;
    prepare_weights(c);
    ae5_conv1_kernel<<<dim3(blocks(a.len[1], kConv1Pos), c.K), 256, 0, c.stream>>>(c.v, c.N, c.idx, c.S == 1 ? 0 : c.mu_all, c.mu, a.len[1], a.lpad[0],
                                                                            P + a.off_w[0], P + a.off_b[0], c.val, a.act_hi[0],
                                                                            a.act_lo[0]),
        ++g_kernel_launches;
    c.val_valid = true;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess)
        e = launch_gemm<kConv, 64, 128>(c, a.map_act_hi[0], a.map_act_lo[0], a.map_w_hi[0], a.map_w_lo[0], P + a.off_b[1],
                                        a.len[2], c.K, a.len[2], a.lpad[1], a.act_hi[1], a.act_lo[1], nullptr, nullptr, nullptr);
    if (e == cudaSuccess)
        e = launch_gemm<kConv, 128, 256>(c, a.map_act_hi[1], a.map_act_lo[1], a.map_w_hi[1], a.map_w_lo[1], P + a.off_b[2],
                                         a.len[3], c.K, a.len[3], a.lpad[2], a.act_hi[2], a.act_lo[2], nullptr, nullptr, nullptr);
    if (e == cudaSuccess)
        e = launch_gemm<kConvCode, 256, 64>(c, a.map_act_hi[2], a.map_act_lo[2], a.map_w_hi[2], a.map_w_lo[2], P + a.off_b[3],
                                            a.len[4], c.K, a.len[4], 0, nullptr, nullptr, P + a.off_w[4], P + a.off_b[4], c.code);
    return e;
}

// conv5 (1x1, 64 -> 4, no activation) on the stored output of conv4: thread per (node, position).
__global__ void ae5_conv5_kernel(const float *__restrict__ a_hi, const float *__restrict__ a_lo, int64_t rows,
                                 const float *__restrict__ w5, const float *__restrict__ b5, float *__restrict__ code)
{
    __shared__ float w[4 * 64], b[4];
    for (int i = threadIdx.x; i < 4 * 64; i += blockDim.x) w[i] = w5[i];
    if (threadIdx.x < 4) b[threadIdx.x] = b5[threadIdx.x];
    __syncthreads();
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int q = 0; q < 16; ++q) {
        const float4 h = reinterpret_cast<const float4 *>(a_hi + r * 64)[q], l = reinterpret_cast<const float4 *>(a_lo + r * 64)[q];
        const float x[4] = {__fadd_rn(h.x, l.x), __fadd_rn(h.y, l.y), __fadd_rn(h.z, l.z), __fadd_rn(h.w, l.w)};
#pragma unroll
        for (int o = 0; o < 4; ++o)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[o] = __fmaf_rn(w[o * 64 + 4 * q + j], x[j], acc[o]);
    }
    reinterpret_cast<float4 *>(code)[r] = make_float4(__fadd_rn(acc[0], b[0]), __fadd_rn(acc[1], b[1]), __fadd_rn(acc[2], b[2]),
                                                      __fadd_rn(acc[3], b[3]));
}

// Forward pass of a training step: the same kernels as inference, but conv4 and deconv5 store
// their outputs (the backward pass needs them) and conv5, the combination of the codes and the last
// convolution run as launches of their own.
// Encoder: leaves every node's code in c.code (and the kept values in c.val).
cudaError_t launch_ae5_train_encode(Ctx &c)
{
    Ae5 &a = *c.ae5;
    const float *P = c.params;
    prepare_weights(c);
    ae5_conv1_kernel<<<dim3(blocks(a.len[1], kConv1Pos), c.K), 256, 0, c.stream>>>(c.v, c.N, c.idx, c.S == 1 ? 0 : c.mu_all, c.mu, a.len[1], a.lpad[0],
                                                                            P + a.off_w[0], P + a.off_b[0], c.val, a.act_hi[0],
                                                                            a.act_lo[0]),
        ++g_kernel_launches;
    c.val_valid = true;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess)
        e = launch_gemm<kConv, 64, 128>(c, a.map_act_hi[0], a.map_act_lo[0], a.map_w_hi[0], a.map_w_lo[0], P + a.off_b[1],
                                        a.len[2], c.K, a.len[2], a.lpad[1], a.act_hi[1], a.act_lo[1], nullptr, nullptr, nullptr);
    if (e == cudaSuccess)
        e = launch_gemm<kConv, 128, 256>(c, a.map_act_hi[1], a.map_act_lo[1], a.map_w_hi[1], a.map_w_lo[1], P + a.off_b[2],
                                         a.len[3], c.K, a.len[3], a.lpad[2], a.act_hi[2], a.act_lo[2], nullptr, nullptr, nullptr);
    if (e == cudaSuccess)
        e = launch_gemm<kConv, 256, 64>(c, a.map_act_hi[2], a.map_act_lo[2], a.map_w_hi[2], a.map_w_lo[2], P + a.off_b[3],
                                        a.len[4], c.K, a.len[4], a.len[4], a.act4_hi, a.act4_lo, nullptr, nullptr, nullptr);
    if (e != cudaSuccess) return e;
    const int64_t rows = (int64_t)c.K * a.len[4];
    ae5_conv5_kernel<<<blocks(rows, 128), 128, 0, c.stream>>>(a.act4_hi, a.act4_lo, rows, P + a.off_w[4], P + a.off_b[4], c.code),
        ++g_kernel_launches;
    return cudaGetLastError();
}

// Decoder d on the code in c.combined, up to deconv5, whose output stays in dact5.
cudaError_t launch_ae5_train_decode(Ctx &c, int d)
{
    Ae5 &a = *c.ae5;
    const float *P = c.params + d * a.dec_stride;
    ae5_deconv1_kernel<<<blocks(a.len[4], 128), 128, 0, c.stream>>>(c.combined, a.len[4], P + a.off_dw[0], P + a.off_db[0], a.d0, 0),
        ++g_kernel_launches;
    constexpr int kTp = 64, kSmem2 = (3 * 4 * 32 + (kTp + 1) * 4) * 4;
    ae5_deconv_kernel<4, 32, kTp><<<blocks(a.len[4] + 1, kTp), 256, kSmem2, c.stream>>>(a.d0, a.len[4], a.len[3], P + a.off_dw[1],
                                                                                        P + a.off_db[1], a.dact_hi[0], a.dact_lo[0], 0),
        ++g_kernel_launches;
    cudaError_t e = cudaGetLastError();
    // the first slice of the activation buffers, slice d of the weights
    if (e == cudaSuccess)
        e = launch_gemm<kDeconv, 32, 64>(c, a.map_dact_hi[0], a.map_dact_lo[0], a.map_dw_hi[0], a.map_dw_lo[0], P + a.off_db[2],
                                         a.len[3] + 1, 1, a.len[2], 0, a.dact_hi[1], a.dact_lo[1], nullptr, nullptr, nullptr, nullptr, d);
    if (e == cudaSuccess)
        e = launch_gemm<kDeconv, 64, 128>(c, a.map_dact_hi[1], a.map_dact_lo[1], a.map_dw_hi[1], a.map_dw_lo[1], P + a.off_db[3],
                                          a.len[2] + 1, 1, a.len[1], 0, a.dact_hi[2], a.dact_lo[2], nullptr, nullptr, nullptr, nullptr, d);
    if (e == cudaSuccess)
        e = launch_gemm<kDeconv, 128, 32>(c, a.map_dact_hi[2], a.map_dact_lo[2], a.map_dw_hi[2], a.map_dw_lo[2], P + a.off_db[4],
                                          a.len[1] + 1, 1, a.len[0], 0, a.dact5_hi, a.dact5_lo, nullptr, nullptr, nullptr, nullptr, d);
    return e;
}

// Ring-allreduce: encoder, mean of the codes, the one decoder.
cudaError_t launch_ae5_train_forward(Ctx &c)
{
    cudaError_t e = launch_ae5_train_encode(c);
    if (e != cudaSuccess) return e;
    c.mean_valid = false;
    e = launch_combine_mean(c);
    return e != cudaSuccess ? e : launch_ae5_train_decode(c, 0);
}

cudaError_t launch_ae5_input_gradient(Ctx &c, int layer)
{
    Ae5 &a = *c.ae5;
    const int j = layer - 1;                                   // 0: conv2, 1: conv3
    const int cin = kAe5EncCh[layer], cout = kAe5EncCh[layer + 1];
    // the convolution's weights w[co][ci][tau] are a transposed convolution's with c_in' = co, c_out' = ci
    ae5_prep_deconv_weights_kernel<<<blocks((int64_t)4 * cin * cout, 256), 256, 0, c.stream>>>(c.params + a.off_w[layer], cout, cin,
                                                                                             a.gw_hi[j], a.gw_lo[j]),
        ++g_kernel_launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t rows = a.len[layer + 1] + 1;                 // one more than the output positions: the last makes the tail
    if (layer == 1)
        return launch_gemm<kGradDeconv, 128, 64>(c, a.map_g_hi[0], a.map_g_lo[0], a.map_gw_hi[0], a.map_gw_lo[0], nullptr, rows, c.K,
                                                 a.len[1], a.lpad[0], a.g_enc[0], a.g_enc_lo[0], nullptr, nullptr, nullptr, a.act_hi[0]);
    if (layer == 2)
        return launch_gemm<kGradDeconv, 256, 128>(c, a.map_g_hi[1], a.map_g_lo[1], a.map_gw_hi[1], a.map_gw_lo[1], nullptr, rows, c.K,
                                                  a.len[2], a.lpad[1], a.g_enc[1], a.g_enc_lo[1], nullptr, nullptr, nullptr, a.act_hi[1]);
    // conv4: 64 channels in, 2 x 256 columns out, cut into four column tiles
    return launch_gemm<kGradDeconv, 64, 256>(c, a.map_g_hi[2], a.map_g_lo[2], a.map_gw_hi[2], a.map_gw_lo[2], nullptr, rows, c.K,
                                             a.len[3], a.lpad[2], a.g_enc[2], a.g_enc_lo[2], nullptr, nullptr, nullptr, a.act_hi[2]);
}

template <int NT, bool TRANS>
static cudaError_t launch_wgrad(Ctx &c, const WgradMaps &maps, int m_split, int n_split, int m_total, int n_total, int layer)
{
    using S = WgradShape<NT>;
    Ae5 &a = *c.ae5;
    auto kern = ae5_wgrad_kernel<NT, TRANS>;
    static OncePerDevice configured;
    {
        const cudaError_t e = configured.run(
            [&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kSmemBytes); });
        if (e != cudaSuccess) return e;
    }
    const Ae5::Tensor &T = a.tensors[2 * layer];
    const int splits = a.wg_splits[layer - 1], kbps = a.wg_kbps[layer - 1];
    const int kb_per_node = (int)((a.len[layer + 1] + kBlockK - 1) / kBlockK);
    const int tiles_m = m_total / 128, tiles_n = n_total / NT;
    const unsigned grid = (unsigned)(tiles_m * tiles_n * splits * c.K);
    kern<<<grid, kGemmThreads, S::kSmemBytes, c.stream>>>(maps, m_split, n_split, tiles_m, tiles_n, splits, kb_per_node, kbps, m_total,
                                                          n_total, a.partial + T.partial_off, (T.count + 3) / 4 * 4, c.errword),
        ++g_kernel_launches;
    return cudaGetLastError();
}

cudaError_t launch_ae5_weight_gradient(Ctx &c, int layer)
{
    Ae5 &a = *c.ae5;
    const int cin = kAe5EncCh[layer], cout = kAe5EncCh[layer + 1];
    const int l = layer - 1;
    constexpr int kNoSplit = 1 << 30;
    WgradMaps maps;
    if (layer == 3) {                         // 64 output channels: the slices make the rows of the accumulator, dW comes out transposed
        for (int h = 0; h < 2; ++h) {
            maps.m[h][0] = a.map_wg_x[l][h][0]; maps.m[h][1] = a.map_wg_x[l][h][1];
            maps.n[h][0] = a.map_wg_g[l][h];    maps.n[h][1] = a.map_wg_g[l][h];
        }
        return launch_wgrad<64, true>(c, maps, 2 * cin, kNoSplit, 3 * cin, cout, layer);
    }
    for (int h = 0; h < 2; ++h) {
        maps.m[h][0] = a.map_wg_g[l][h];    maps.m[h][1] = a.map_wg_g[l][h];
        maps.n[h][0] = a.map_wg_x[l][h][0]; maps.n[h][1] = a.map_wg_x[l][h][1];
    }
    if (layer == 1) return launch_wgrad<192, false>(c, maps, kNoSplit, 2 * cin, cout, 3 * cin, layer);
    return launch_wgrad<128, false>(c, maps, kNoSplit, 2 * cin, cout, 3 * cin, layer);
}

// Stage 5 up to the reconstruction.  Ring-allreduce: the decoder on the mean code; c.recon gets the mu
// values.  Parameter server (Section IV-A): node k's decoder on the common code, its innovation as the 33rd
// input of the last convolution; c.recon gets [K][mu].  Every layer is ONE launch over all decoders
// (blockIdx.y = decoder: its own weights, its own slice of the activation buffers), so that the K decoders'
// tiles fill the device together.
cudaError_t launch_ae5_decode(Ctx &c)
{
    Ae5 &a = *c.ae5;
    prepare_weights(c);
    const bool ps = c.cfg.variant == LGC_VARIANT_PS;
    const float *P = c.params;                                 // decoder d's tensors: dec_stride floats per decoder further on
    const int D = a.decoders;
    const int64_t ps_stride = a.dec_stride;
    cudaError_t e = launch_dependent(ae5_deconv1_kernel, dim3(blocks(a.len[4], 128), D), dim3(128), c.stream, c.combined, a.len[4],
                                     P + a.off_dw[0], P + a.off_db[0], a.d0, ps_stride);
    if (e != cudaSuccess) return e;
    ++g_kernel_launches;
    // deconv2 (4 -> 32): too narrow for the tensor cores
    constexpr int kTp = 64, kSmem2 = (3 * 4 * 32 + (kTp + 1) * 4) * 4;
    e = launch_dependent_smem(ae5_deconv_kernel<4, 32, kTp>, dim3(blocks(a.len[4] + 1, kTp), D), dim3(256), kSmem2, c.stream, a.d0,
                              a.len[4], a.len[3], P + a.off_dw[1], P + a.off_db[1], a.dact_hi[0], a.dact_lo[0], ps_stride);
    if (e != cudaSuccess) return e;
    ++g_kernel_launches;
    e = cudaGetLastError();
    // deconv3..5: rows j = 0 .. L_in (one more than the input positions: the last makes the tail)
    if (e == cudaSuccess)
        e = launch_gemm<kDeconv, 32, 64>(c, a.map_dact_hi[0], a.map_dact_lo[0], a.map_dw_hi[0], a.map_dw_lo[0], P + a.off_db[2],
                                         a.len[3] + 1, D, a.len[2], a.len[2], a.dact_hi[1], a.dact_lo[1], nullptr, nullptr, nullptr,
                                         nullptr, 0, 1, ps_stride);
    if (e == cudaSuccess)
        e = launch_gemm<kDeconv, 64, 128>(c, a.map_dact_hi[1], a.map_dact_lo[1], a.map_dw_hi[1], a.map_dw_lo[1], P + a.off_db[3],
                                          a.len[2] + 1, D, a.len[1], a.len[1], a.dact_hi[2], a.dact_lo[2], nullptr, nullptr, nullptr,
                                          nullptr, 0, 1, ps_stride);
    if (e == cudaSuccess)
        e = launch_gemm<kDeconvFinal, 128, 32>(c, a.map_dact_hi[2], a.map_dact_lo[2], a.map_dw_hi[2], a.map_dw_lo[2], P + a.off_db[4],
                                               a.len[1] + 1, D, a.len[0], 0, nullptr, nullptr, P + a.off_dw[5], P + a.off_db[5],
                                               c.recon, ps ? c.inn : nullptr, 0, 1, ps_stride);
    return e;
}

}  // namespace lgc
