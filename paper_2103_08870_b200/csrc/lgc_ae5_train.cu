// Training step of the paper's full-size autoencoder (Section IV-C) for the ring-allreduce form:
// loss of Section IV-B on the kept values of the last selection (Section V-B, second phase),
//     loss = (1/mu) || D_c((1/K) sum_k E_c(g~_k)) - (1/K) sum_k g~_k ||^2,
// backward pass through every layer, Adam.
//
// The forward pass is the inference path's (tensor cores; lgc_ae5.cu) with every layer's output
// kept.  The backward pass works on channels-last fp32 buffers.  With G the gradient at a
// layer's pre-activation output and X its (post-activation) input:
//   convolution  y[t][co] = b + sum w[co][ci][tau] x[2t+tau][ci]
//     dW[co][tau C_in + ci] = sum_t G[t][co] X[2t+tau][ci]      (rows of X seen as slices of 3 C_in floats)
//     dX                    = fold(G W), W[co][tau C_in + ci]    (products first, then summed onto 2t+tau)
//   transposed convolution  y[2j+tau][co] += w[ci][co][tau] x[j][ci]
//     dW[ci][tau C_out + co] = sum_j X[j][ci] G[2j+tau][co]      (rows of G seen as slices of 3 C_out floats)
//     dX[j][ci]              = sum G[2j+tau][co] w[ci][co][tau]
// so every layer is one GEMM over rows (dX) and one GEMM that sums over rows (dW): for the encoder's wide
// convolutions both run on the tensor cores (lgc_ae5.cu), for the decoder (one pass, not one per node) and the
// narrow layers on the fp32 pipes here; the sums over rows are cut into chunks whose partial results are added
// up in fp64, in chunk order, by the kernel that applies Adam.  Leaky-ReLU derivatives are taken from the sign of
// the stored outputs (the slope is positive, so output and pre-activation have the same sign).
#include <algorithm>

#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr float kSlope = 0.01f;       // leaky-ReLU slope of the full-size autoencoder
constexpr int kTile = 64;             // GEMM tile: 64 x 64 outputs per CTA of 256 threads (4 x 4 per thread)
constexpr int kStep = 16;             // rows (TN) or inner entries (NN) staged per trip
constexpr int kPitch = kTile + 4;

// M rows of `len` floats, row m = (node, t): value hi[...] (+ lo[...] when the buffer is kept as two tf32 parts).
struct Rows {
    const float *hi, *lo;
    int64_t node_stride, row_stride, rows_per_node;
    int len;
    int vec;                          // rows start 16-byte aligned and len % 4 == 0
    __device__ __forceinline__ int64_t at(int64_t m) const
    {
        const int64_t k = m / rows_per_node, t = m - k * rows_per_node;
        return k * node_stride + t * row_stride;
    }
};

// Walks the rows m, m + step, m + 2 step, ... of a Rows without a division per row.
struct RowCursor {
    int64_t k, t;
    __device__ __forceinline__ RowCursor(const Rows &r, int64_t m) : k(m / r.rows_per_node), t(m - (m / r.rows_per_node) * r.rows_per_node) {}
    __device__ __forceinline__ int64_t at(const Rows &r) const { return k * r.node_stride + t * r.row_stride; }
    __device__ __forceinline__ void advance(const Rows &r, int step)
    {
        t += step;
        while (t >= r.rows_per_node) {
            t -= r.rows_per_node;
            ++k;
        }
    }
};

Rows rows_of(const float *hi, const float *lo, int64_t node_stride, int64_t row_stride, int64_t rows_per_node, int len)
{
    Rows r;
    r.hi = hi; r.lo = lo; r.node_stride = node_stride; r.row_stride = row_stride; r.rows_per_node = rows_per_node; r.len = len;
    r.vec = len % 4 == 0 && node_stride % 4 == 0 && row_stride % 4 == 0 && (reinterpret_cast<uintptr_t>(hi) & 15) == 0 &&
            (lo == nullptr || (reinterpret_cast<uintptr_t>(lo) & 15) == 0);
    return r;
}

// four consecutive entries of a row from column c on (zeros beyond the row's length)
__device__ __forceinline__ float4 load4(const Rows &r, int64_t base, int c)
{
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r.vec) {
        if (c < r.len) {
            x = *reinterpret_cast<const float4 *>(r.hi + base + c);
            if (r.lo) {
                const float4 l = *reinterpret_cast<const float4 *>(r.lo + base + c);
                x.x = __fadd_rn(x.x, l.x); x.y = __fadd_rn(x.y, l.y); x.z = __fadd_rn(x.z, l.z); x.w = __fadd_rn(x.w, l.w);
            }
        }
        return x;
    }
    float *e = &x.x;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (c + j < r.len) e[j] = r.lo ? __fadd_rn(r.hi[base + c + j], r.lo[base + c + j]) : r.hi[base + c + j];
    return x;
}

// C[m][n] = sum_kd A(m, kd) B[kd][n] for m < M, n < N; B dense [Kd][N], Kd a multiple of 16, N of 4.
// MASK: the result is the gradient at the output of a leaky ReLU whose stored output is X(m, n):
// it is multiplied by 1 or by the slope.  Grid (ceil(N / 64), ceil(M / 64)), 256 threads.
template <bool MASK>
__global__ void __launch_bounds__(256)
nn_gemm_kernel(Rows A, int64_t M, const float *__restrict__ B, int N, float *__restrict__ C, int64_t ldc, Rows X)
{
    __shared__ __align__(16) float As[kStep][kPitch], Bs[kStep][kPitch];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * kTile;
    const int n0 = blockIdx.x * kTile;
    float2 acc[4][2] = {};
    const int ar = threadIdx.x >> 2, akq = threadIdx.x & 3;          // A tile: 64 rows x 16 entries, a float4 per thread
    const int64_t am = m0 + ar;
    const int64_t abase = am < M ? A.at(am) : 0;
    const int bk = threadIdx.x >> 4, bnq = threadIdx.x & 15;         // B tile: 16 rows x 64 columns
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool bcol = n0 + 4 * bnq < N;
    float4 a = am < M ? load4(A, abase, 4 * akq) : zero;
    float4 b = bcol ? *reinterpret_cast<const float4 *>(B + (int64_t)bk * N + n0 + 4 * bnq) : zero;
    for (int k0 = 0; k0 < A.len; k0 += kStep) {
        As[4 * akq + 0][ar] = a.x; As[4 * akq + 1][ar] = a.y; As[4 * akq + 2][ar] = a.z; As[4 * akq + 3][ar] = a.w;
        *reinterpret_cast<float4 *>(&Bs[bk][4 * bnq]) = b;
        __syncthreads();
        if (k0 + kStep < A.len) {               // the next entries travel while these are multiplied
            a = am < M ? load4(A, abase, k0 + kStep + 4 * akq) : zero;
            b = bcol ? *reinterpret_cast<const float4 *>(B + (int64_t)(k0 + kStep + bk) * N + n0 + 4 * bnq) : zero;
        }
#pragma unroll
        for (int k = 0; k < kStep; ++k) {
            const float4 av = *reinterpret_cast<const float4 *>(&As[k][4 * ty]);
            const float4 bv = *reinterpret_cast<const float4 *>(&Bs[k][4 * tx]);
            // packed fp32 FMAs (two per instruction on this architecture), each lane rounded like __fmaf_rn
            const float aa[4] = {av.x, av.y, av.z, av.w};
            const float2 b01 = make_float2(bv.x, bv.y), b23 = make_float2(bv.z, bv.w);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 a2 = make_float2(aa[i], aa[i]);
                acc[i][0] = __ffma2_rn(a2, b01, acc[i][0]);
                acc[i][1] = __ffma2_rn(a2, b23, acc[i][1]);
            }
        }
        __syncthreads();
    }
    const int n = n0 + 4 * tx;
    if (n >= N) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + 4 * ty + i;
        if (m >= M) break;
        float4 out = make_float4(acc[i][0].x, acc[i][0].y, acc[i][1].x, acc[i][1].y);
        if (MASK) {
            const int64_t xb = X.at(m);
            const float4 x = *reinterpret_cast<const float4 *>(X.hi + xb + n);   // the sign of the leading part is the value's
            out.x = x.x > 0.f ? out.x : __fmul_rn(kSlope, out.x);
            out.y = x.y > 0.f ? out.y : __fmul_rn(kSlope, out.y);
            out.z = x.z > 0.f ? out.z : __fmul_rn(kSlope, out.z);
            out.w = x.w > 0.f ? out.w : __fmul_rn(kSlope, out.w);
        }
        *reinterpret_cast<float4 *>(C + m * ldc + n) = out;
    }
}

// partial[s][p][q] = sum over the rows m of chunk s of A(m, p) B(m, q).  Grid (ceil(Q / 64), ceil(P / 64), chunks).
__global__ void __launch_bounds__(256)
tn_gemm_kernel(Rows A, Rows B, int64_t M, int64_t chunk, float *__restrict__ partial, int64_t pstride)
{
    __shared__ __align__(16) float As[kStep][kPitch], Bs[kStep][kPitch];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int p0 = blockIdx.y * kTile, q0 = blockIdx.x * kTile;
    const int64_t first = (int64_t)blockIdx.z * chunk;
    const int64_t last = first + chunk < M ? first + chunk : M;
    float2 acc[4][2] = {};
    const int lr = threadIdx.x >> 4, lc = threadIdx.x & 15;          // 16 rows x 64 columns of each operand per trip
    RowCursor ca(A, first + lr), cb(B, first + lr);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 a = zero, b = zero;
    if (first + lr < last) {
        a = load4(A, ca.at(A), p0 + 4 * lc);
        b = load4(B, cb.at(B), q0 + 4 * lc);
    }
    for (int64_t r0 = first; r0 < last; r0 += kStep) {
        *reinterpret_cast<float4 *>(&As[lr][4 * lc]) = a;
        *reinterpret_cast<float4 *>(&Bs[lr][4 * lc]) = b;
        __syncthreads();
        // the next trip's rows travel while this one is multiplied
        ca.advance(A, kStep);
        cb.advance(B, kStep);
        a = b = zero;
        if (r0 + kStep + lr < last) {
            a = load4(A, ca.at(A), p0 + 4 * lc);
            b = load4(B, cb.at(B), q0 + 4 * lc);
        }
#pragma unroll
        for (int k = 0; k < kStep; ++k) {
            const float4 av = *reinterpret_cast<const float4 *>(&As[k][4 * ty]);
            const float4 bv = *reinterpret_cast<const float4 *>(&Bs[k][4 * tx]);
            // packed fp32 FMAs (two per instruction on this architecture), each lane rounded like __fmaf_rn
            const float aa[4] = {av.x, av.y, av.z, av.w};
            const float2 b01 = make_float2(bv.x, bv.y), b23 = make_float2(bv.z, bv.w);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 a2 = make_float2(aa[i], aa[i]);
                acc[i][0] = __ffma2_rn(a2, b01, acc[i][0]);
                acc[i][1] = __ffma2_rn(a2, b23, acc[i][1]);
            }
        }
        __syncthreads();
    }
    float *out = partial + (int64_t)blockIdx.z * pstride;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = p0 + 4 * ty + i;
        if (p >= A.len) break;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int q = q0 + 4 * tx + j;
            if (q < B.len) out[(int64_t)p * B.len + q] = j & 1 ? acc[i][j >> 1].y : acc[i][j >> 1].x;
        }
    }
}

// Column sums of a wide A (a bias gradient) in one streaming pass:  psum[s][p] = sum over the rows m of chunk s of
// A(m, p), and with Q > 0 also the sums weighted by the Q entries of B's row (conv1's weight gradient, whose rows are the
// three kept values a position reads):  pw[s][p][q] = sum_m A(m, p) B(m, q).
// A.len is 4 times a power of two, at most 1024, rows 16-byte aligned.  A thread holds four columns; 256 / (A.len / 4) rows
// are in flight per pass and four passes per trip, so that a CTA keeps 32 KB (64 KB with two tf32 parts) in flight;
// the rows' sums are then added across the threads of a column in thread order.  Grid: the chunks.
template <int Q>
__global__ void __launch_bounds__(256)
colsum_kernel(Rows A, Rows B, int64_t M, int64_t chunk, float *__restrict__ psum, int64_t psum_stride, float *__restrict__ pw,
              int64_t pw_stride)
{
    __shared__ float4 red[1 + Q][256];
    const int tpr = A.len >> 2, rpp = 256 / tpr;             // threads per row, rows per pass
    const int c4 = threadIdx.x % tpr, rr = threadIdx.x / tpr;
    const int64_t first = (int64_t)blockIdx.x * chunk;
    const int64_t last = first + chunk < M ? first + chunk : M;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), accw[Q > 0 ? Q : 1];
#pragma unroll
    for (int q = 0; q < Q; ++q) accw[q] = acc;
    RowCursor ca(A, first + rr), cb(B, first + rr);
    int64_t m = first + rr;
    // whole trips of four rows: the eight loads are issued back to back, without a branch between them (a thread that
    // waits for each load before the next keeps a quarter of the bytes in flight)
    for (; m + 3 * (int64_t)rpp < last; m += 4 * rpp) {
        float4 a[4], l[4];
        float b[4][Q > 0 ? Q : 1];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int64_t ab = ca.at(A) + 4 * c4;
            a[r] = *reinterpret_cast<const float4 *>(A.hi + ab);
            l[r] = A.lo ? *reinterpret_cast<const float4 *>(A.lo + ab) : make_float4(0.f, 0.f, 0.f, 0.f);
            if (Q > 0) {
                const int64_t bb = cb.at(B);
#pragma unroll
                for (int q = 0; q < Q; ++q) b[r][q] = B.hi[bb + q];
                cb.advance(B, rpp);
            }
            ca.advance(A, rpp);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (A.lo) {
                a[r].x = __fadd_rn(a[r].x, l[r].x); a[r].y = __fadd_rn(a[r].y, l[r].y);
                a[r].z = __fadd_rn(a[r].z, l[r].z); a[r].w = __fadd_rn(a[r].w, l[r].w);
            }
            acc.x = __fadd_rn(acc.x, a[r].x); acc.y = __fadd_rn(acc.y, a[r].y);
            acc.z = __fadd_rn(acc.z, a[r].z); acc.w = __fadd_rn(acc.w, a[r].w);
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                accw[q].x = __fmaf_rn(a[r].x, b[r][q], accw[q].x); accw[q].y = __fmaf_rn(a[r].y, b[r][q], accw[q].y);
                accw[q].z = __fmaf_rn(a[r].z, b[r][q], accw[q].z); accw[q].w = __fmaf_rn(a[r].w, b[r][q], accw[q].w);
            }
        }
    }
    for (; m < last; m += rpp) {                              // the rows that are left, one at a time
        float4 x = load4(A, ca.at(A), 4 * c4);
        acc.x = __fadd_rn(acc.x, x.x); acc.y = __fadd_rn(acc.y, x.y);
        acc.z = __fadd_rn(acc.z, x.z); acc.w = __fadd_rn(acc.w, x.w);
        if (Q > 0) {
            const int64_t bb = cb.at(B);
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const float bq = B.hi[bb + q];
                accw[q].x = __fmaf_rn(x.x, bq, accw[q].x); accw[q].y = __fmaf_rn(x.y, bq, accw[q].y);
                accw[q].z = __fmaf_rn(x.z, bq, accw[q].z); accw[q].w = __fmaf_rn(x.w, bq, accw[q].w);
            }
            cb.advance(B, rpp);
        }
        ca.advance(A, rpp);
    }
    red[0][threadIdx.x] = acc;
#pragma unroll
    for (int q = 0; q < Q; ++q) red[1 + q][threadIdx.x] = accw[q];
    __syncthreads();
    if (rr != 0) return;
    for (int j = 0; j <= Q; ++j) {
        float4 tot = red[j][c4];
        for (int g = 1; g < rpp; ++g) {
            const float4 x = red[j][g * tpr + c4];
            tot.x = __fadd_rn(tot.x, x.x); tot.y = __fadd_rn(tot.y, x.y); tot.z = __fadd_rn(tot.z, x.z); tot.w = __fadd_rn(tot.w, x.w);
        }
        if (j == 0) {
            *reinterpret_cast<float4 *>(psum + (int64_t)blockIdx.x * psum_stride + 4 * c4) = tot;
        } else {
            float *o = pw + (int64_t)blockIdx.x * pw_stride + (int64_t)(4 * c4) * Q + (j - 1);
            o[0] = tot.x; o[Q] = tot.y; o[2 * Q] = tot.z; o[3 * Q] = tot.w;
        }
    }
}

// The same for a narrow right-hand side (at most four columns; B.hi == nullptr: one column of ones,
// which makes the column sums of A, i.e. a bias gradient): partial[s][p][q] = sum_m A(m, p) B(m, q).
// Grid (chunks, ceil(P / 32)), 256 threads: lane = column p, the eight warps stride over the rows and are
// added up in warp order.
__global__ void __launch_bounds__(256)
tn_narrow_kernel(Rows A, Rows B, int Q, int64_t M, int64_t chunk, float *__restrict__ partial, int64_t pstride)
{
    __shared__ float part[8][32][4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t first = (int64_t)blockIdx.x * chunk;
    const int64_t last = first + chunk < M ? first + chunk : M;
    const int p = blockIdx.y * 32 + lane;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    RowCursor ca(A, first + warp), cb(B, first + warp);
    // four of the warp's rows per trip: their loads are in flight together, the sums are added in row order
    for (int64_t m = first + warp; m < last; m += 32) {
        float a[4], b[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            a[r] = 0.f;
            b[r][0] = 1.f; b[r][1] = b[r][2] = b[r][3] = 0.f;
            if (m + 8 * r < last) {
                if (B.hi) {
                    const int64_t bb = cb.at(B);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (q < Q) b[r][q] = B.lo ? __fadd_rn(B.hi[bb + q], B.lo[bb + q]) : B.hi[bb + q];
                }
                if (p < A.len) {
                    const int64_t ab = ca.at(A) + p;
                    a[r] = A.lo ? __fadd_rn(A.hi[ab], A.lo[ab]) : A.hi[ab];
                }
            }
            ca.advance(A, 8);
            cb.advance(B, 8);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = __fmaf_rn(a[r], b[r][q], acc[q]);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) part[warp][lane][q] = acc[q];
    __syncthreads();
    if (warp == 0 && p < A.len) {
        for (int q = 0; q < Q; ++q) {
            float tot = 0.f;
            for (int w = 0; w < 8; ++w) tot = __fadd_rn(tot, part[w][lane][q]);
            partial[(int64_t)blockIdx.x * pstride + (int64_t)p * Q + q] = tot;
        }
    }
}

// One layer's weights arranged as the dense [Kd][N] operand of nn_gemm_kernel.
//   mode 0, convolution w[co][ci][tau]            -> W[co][tau C_in + ci]   (Kd = C_out, N = 3 C_in)
//   mode 1, transposed convolution w[ci][co][tau] -> W[tau C_out + co][ci]  (Kd = 3 C_out, N = C_in)
__global__ void arrange_weights_kernel(const float *__restrict__ w, int cin, int cout, int mode, float *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 3 * cin * cout) return;
    if (mode == 0) {
        const int co = i / (3 * cin), tau = i % (3 * cin) / cin, ci = i % cin;
        out[i] = w[(co * cin + ci) * 3 + tau];
    } else {
        const int tau = i / (cout * cin), co = i / cin % cout, ci = i % cin;
        out[i] = w[(ci * cout + co) * 3 + tau];
    }
}

__device__ __forceinline__ double block_sum256(double x, double *warp_part)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_down_sync(0xffffffffu, x, d);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = x;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < 8; ++w) tot += warp_part[w];
    return tot;                                                   // valid in thread 0
}

// The last convolution (1x1) on deconv5's stored output, the loss, and the way back through it:
// recon[p] = b6 + sum_c w6[c] d5[p][c] (+ w6[32] extra[p]: the parameter server's innovation channel),
// dr[p] = scale * 2 (recon[p] - target[p]) / mu with target = (1/Kt) sum_k rows_k[p] (node order; the
// parameter server compares with the node's own vector: Kt = 1), this CTA's part of
// sum (recon - target)^2, and g5[p][c] = dr[p] w6[c] leaky'(d5[p][c]).
__global__ void __launch_bounds__(256)
final_loss_kernel(const float *__restrict__ d5_hi, const float *__restrict__ d5_lo, const float *__restrict__ rows, int Kt,
                  int64_t mu, const float *__restrict__ w6, const float *__restrict__ b6, const float *__restrict__ extra,
                  float scale, float *__restrict__ recon, float *__restrict__ dr, float *__restrict__ g5,
                  double *__restrict__ loss_part)
{
    __shared__ float w[33];
    __shared__ double warp_part[8];
    if (threadIdx.x < 32) w[threadIdx.x] = w6[threadIdx.x];
    if (threadIdx.x == 32) w[32] = extra ? w6[32] : 0.0f;
    __syncthreads();
    const int64_t p = (int64_t)blockIdx.x * 256 + threadIdx.x;
    double sq = 0.0;
    if (p < mu) {
        float hi[32];
        float r = b6[0];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 h = reinterpret_cast<const float4 *>(d5_hi + p * 32)[q], l = reinterpret_cast<const float4 *>(d5_lo + p * 32)[q];
            hi[4 * q] = h.x; hi[4 * q + 1] = h.y; hi[4 * q + 2] = h.z; hi[4 * q + 3] = h.w;
            r = __fmaf_rn(w[4 * q], __fadd_rn(h.x, l.x), r);
            r = __fmaf_rn(w[4 * q + 1], __fadd_rn(h.y, l.y), r);
            r = __fmaf_rn(w[4 * q + 2], __fadd_rn(h.z, l.z), r);
            r = __fmaf_rn(w[4 * q + 3], __fadd_rn(h.w, l.w), r);
        }
        if (extra) r = __fmaf_rn(w[32], extra[p], r);
        float target = 0.f;
        for (int k = 0; k < Kt; ++k) target = __fadd_rn(target, rows[(int64_t)k * mu + p]);
        target = __fdiv_rn(target, (float)Kt);
        const double diff = (double)r - (double)target;
        sq = diff * diff;
        const float g = (float)((double)scale * 2.0 * diff / (double)mu);
        recon[p] = r;
        dr[p] = g;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float4 o;
            o.x = __fmul_rn(g, w[4 * q]);     o.x = hi[4 * q] > 0.f ? o.x : __fmul_rn(kSlope, o.x);
            o.y = __fmul_rn(g, w[4 * q + 1]); o.y = hi[4 * q + 1] > 0.f ? o.y : __fmul_rn(kSlope, o.y);
            o.z = __fmul_rn(g, w[4 * q + 2]); o.z = hi[4 * q + 2] > 0.f ? o.z : __fmul_rn(kSlope, o.z);
            o.w = __fmul_rn(g, w[4 * q + 3]); o.w = hi[4 * q + 3] > 0.f ? o.w : __fmul_rn(kSlope, o.w);
            reinterpret_cast<float4 *>(g5 + p * 32)[q] = o;
        }
    }
    const double tot = block_sum256(sq, warp_part);
    if (threadIdx.x == 0) loss_part[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(256)
loss_sum_kernel(const double *__restrict__ part, int n, int64_t mu, float *__restrict__ out)
{
    __shared__ double warp_part[8];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) acc += part[i];
    const double tot = block_sum256(acc, warp_part);
    if (threadIdx.x == 0) *out = (float)(tot / (double)mu);
}

// deconv1 (4 -> 4, stride 1, padding 1), y[s][co] = b + sum w[ci][co][tau] zbar[s + 1 - tau][ci]:
// gradient at the mean code, dzbar[j][ci] = sum over (tau, co) of w[ci][co][tau] g1[j + tau - 1][co].
__global__ void dec1_bwd_kernel(const float *__restrict__ g1, int64_t L4, const float *__restrict__ w, float *__restrict__ dzbar)
{
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L4) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int tau = 0; tau < 3; ++tau) {
        const int64_t s = j + tau - 1;
        if (s < 0 || s >= L4) continue;
        const float4 g = reinterpret_cast<const float4 *>(g1)[s];
        const float gs[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
        for (int ci = 0; ci < 4; ++ci)
#pragma unroll
            for (int co = 0; co < 4; ++co) acc[ci] = __fmaf_rn(w[(ci * 4 + co) * 3 + tau], gs[co], acc[ci]);
    }
    reinterpret_cast<float4 *>(dzbar)[j] = make_float4(acc[0], acc[1], acc[2], acc[3]);
}

// deconv1's 48 weight and 4 bias gradients: one CTA each, summed in fp64.
__global__ void __launch_bounds__(256)
dec1_grad_kernel(const float *__restrict__ zbar, const float *__restrict__ g1, int64_t L4, float *__restrict__ gw,
                 float *__restrict__ gb)
{
    __shared__ double warp_part[8];
    const int id = blockIdx.x;
    double acc = 0.0;
    if (id < 48) {
        const int ci = id / 12, co = id / 3 % 4, tau = id % 3;
        for (int64_t j = threadIdx.x; j < L4; j += 256) {
            const int64_t s = j + tau - 1;
            if (s >= 0 && s < L4) acc += (double)zbar[j * 4 + ci] * (double)g1[s * 4 + co];
        }
    } else {
        for (int64_t s = threadIdx.x; s < L4; s += 256) acc += (double)g1[s * 4 + (id - 48)];
    }
    const double tot = block_sum256(acc, warp_part);
    if (threadIdx.x == 0) (id < 48 ? gw[id] : gb[id - 48]) = (float)tot;
}

// Way back through conv5 (1x1, 64 -> 4):  g4[k][t][c] = leaky'(a4[k][t][c]) * sum_o w5[o][c] dzk[k][t][o].
// Ring-allreduce (dzbar given): every node's code gets dzbar / K (the mean), written to dzk.
// Parameter server (dzbar == nullptr): dzk already holds every node's own gradient.  Thread per (node, position).
__global__ void code_bwd_kernel(const float *__restrict__ dzbar, int K, int64_t L4, const float *__restrict__ w5,
                                const float *__restrict__ a4_hi, float *__restrict__ dzk, float *__restrict__ g4,
                                float *__restrict__ g4_hi, float *__restrict__ g4_lo)
{
    __shared__ float w[4 * 64];
    for (int i = threadIdx.x; i < 4 * 64; i += blockDim.x) w[i] = w5[i];
    __syncthreads();
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= (int64_t)K * L4) return;
    float dz[4];
    if (dzbar) {
        const float4 z = reinterpret_cast<const float4 *>(dzbar)[r % L4];
        const float fk = (float)K;
        dz[0] = __fdiv_rn(z.x, fk); dz[1] = __fdiv_rn(z.y, fk); dz[2] = __fdiv_rn(z.z, fk); dz[3] = __fdiv_rn(z.w, fk);
        reinterpret_cast<float4 *>(dzk)[r] = make_float4(dz[0], dz[1], dz[2], dz[3]);
    } else {
        const float4 z = reinterpret_cast<const float4 *>(dzk)[r];
        dz[0] = z.x; dz[1] = z.y; dz[2] = z.z; dz[3] = z.w;
    }
    for (int q = 0; q < 16; ++q) {
        const float4 a = reinterpret_cast<const float4 *>(a4_hi + r * 64)[q];
        const float as[4] = {a.x, a.y, a.z, a.w};
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float acc = 0.f;
#pragma unroll
            for (int oo = 0; oo < 4; ++oo) acc = __fmaf_rn(w[oo * 64 + 4 * q + j], dz[oo], acc);
            o[j] = as[j] > 0.f ? acc : __fmul_rn(kSlope, acc);
        }
        reinterpret_cast<float4 *>(g4 + r * 64)[q] = make_float4(o[0], o[1], o[2], o[3]);
        float hi[4], lo[4];                       // and as two tf32 parts, for the weight gradient on the tensor cores
#pragma unroll
        for (int j = 0; j < 4; ++j) split_tf32(o[j], hi[j], lo[j]);
        reinterpret_cast<float4 *>(g4_hi + r * 64)[q] = make_float4(hi[0], hi[1], hi[2], hi[3]);
        reinterpret_cast<float4 *>(g4_lo + r * 64)[q] = make_float4(lo[0], lo[1], lo[2], lo[3]);
    }
}

// Parameter server, similarity loss of Section IV-A over the codes z[K][n]: for every entry e this thread's
// part of sum over ordered pairs k != m of (z_k[e] - z_m[e])^2 = 2 K sum_k z_k^2 - 2 (sum_k z_k)^2, and the
// gradient it sends to every node's code, dzk[k][e] = lam_sim * 4 (K z_k[e] - sum_m z_m[e]) / n.
__global__ void __launch_bounds__(256)
ps_code_grad_kernel(const float *__restrict__ z, int K, int64_t n, float lam_sim, float *__restrict__ dzk,
                    double *__restrict__ sim_part)
{
    __shared__ double warp_part[8];
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    double part = 0.0;
    if (e < n) {
        double sum = 0.0, sq = 0.0;
        for (int k = 0; k < K; ++k) {
            const double x = (double)z[(int64_t)k * n + e];
            sum += x;
            sq += x * x;
        }
        part = 2.0 * (double)K * sq - 2.0 * sum * sum;
        for (int k = 0; k < K; ++k)
            dzk[(int64_t)k * n + e] = (float)((double)lam_sim * 4.0 * ((double)K * (double)z[(int64_t)k * n + e] - sum) / (double)n);
    }
    const double tot = block_sum256(part, warp_part);
    if (threadIdx.x == 0) sim_part[blockIdx.x] = tot;
}

__global__ void add_kernel(float *__restrict__ dst, const float *__restrict__ src, int64_t n)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __fadd_rn(dst[i], src[i]);
}

// loss = lam_rec * (sum of the decoders' squared errors) / mu + lam_sim * (pair sum) / n
__global__ void __launch_bounds__(256)
ps_loss_sum_kernel(const double *__restrict__ rec_part, int n_rec, const double *__restrict__ sim_part, int n_sim, int64_t mu,
                   int64_t n, float lam_rec, float lam_sim, float *__restrict__ out)
{
    __shared__ double warp_part[8];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n_rec; i += 256) acc += rec_part[i];
    const double rec = block_sum256(acc, warp_part);
    __syncthreads();
    acc = 0.0;
    for (int i = threadIdx.x; i < n_sim; i += 256) acc += sim_part[i];
    const double sim = block_sum256(acc, warp_part);
    if (threadIdx.x == 0) *out = (float)((double)lam_rec * rec / (double)mu + (double)lam_sim * sim / (double)n);
}

// Gradient of every parameter from its tensor's per-chunk partial sums (fp64, chunk order), then Adam.
//   kind 0 / 3: entry e of the tensor is parameter e;  kind 1: e = (co, tau, ci) -> w[co][ci][tau];
//   kind 2: e = (ci, tau, co) -> w[ci][co][tau].   Thread per parameter; `first` lists the tensors' first threads.
struct TensorTable {
    int64_t first[23], param_off[22], partial_off[22], pstride[22];
    int chunks[22], kind[22], cin[22], cout[22];
};
__global__ void reduce_adam_kernel(const float *__restrict__ partial, TensorTable tt, AdamArgs ad)
{
    const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= tt.first[22]) return;
    int t = 0;
    while (id >= tt.first[t + 1]) ++t;
    const int64_t e = id - tt.first[t];
    const float *part = partial + tt.partial_off[t];
    double g = 0.0;
    for (int s = 0; s < tt.chunks[t]; ++s) g += (double)part[(int64_t)s * tt.pstride[t] + e];
    int64_t i = e;
    const int cin = tt.cin[t], cout = tt.cout[t];
    if (tt.kind[t] == 1) {
        const int64_t co = e / (3 * cin), tau = e % (3 * cin) / cin, ci = e % cin;
        i = (co * cin + ci) * 3 + tau;
    } else if (tt.kind[t] == 2) {
        const int64_t ci = e / (3 * cout), tau = e % (3 * cout) / cout, co = e % cout;
        i = (ci * cout + co) * 3 + tau;
    }
    i += tt.param_off[t];
    const double m = ad.beta1 * (double)ad.m[i] + (1.0 - ad.beta1) * g;
    const double v = ad.beta2 * (double)ad.v[i] + (1.0 - ad.beta2) * g * g;
    ad.m[i] = (float)m;
    ad.v[i] = (float)v;
    ad.params[i] = (float)((double)ad.params[i] - ad.lr * (m / ad.corr1) / (sqrt(v / ad.corr2) + ad.eps));
}

inline unsigned blocks(int64_t n, int per) { return (unsigned)((n + per - 1) / per); }

struct Launcher {
    Ctx &c;
    Ae5 &a;
    cudaError_t err = cudaSuccess;
    bool ok() { if (err == cudaSuccess) err = cudaGetLastError(); return err == cudaSuccess; }

    float *partial_of(int t) { return a.partial + a.tensors[t].partial_off; }
    int64_t pstride_of(int t) { return (a.tensors[t].count + 3) / 4 * 4; }

    void nn(const Rows &A, int64_t M, const float *B, int N, float *C, const Rows *mask)
    {
        if (!ok()) return;
        const dim3 grid(blocks(N, kTile), blocks(M, kTile));
        if (mask) nn_gemm_kernel<true><<<grid, 256, 0, c.stream>>>(A, M, B, N, C, N, *mask);
        else nn_gemm_kernel<false><<<grid, 256, 0, c.stream>>>(A, M, B, N, C, N, A);
        ++g_kernel_launches;
    }
    // weight gradient of tensor t: sum over rows of A(m, .)^T B(m, .)
    void tn(int t, const Rows &A, const Rows &B)
    {
        if (!ok()) return;
        const Ae5::Tensor &T = a.tensors[t];
        const dim3 grid(blocks(B.len, kTile), blocks(A.len, kTile), T.chunks);
        tn_gemm_kernel<<<grid, 256, 0, c.stream>>>(A, B, T.rows, T.chunk, partial_of(t), pstride_of(t));
        ++g_kernel_launches;
    }
    // the same with at most four columns on the right (B.hi == nullptr: column sums of A, a bias gradient)
    void tn_narrow(int t, const Rows &A, const Rows &B, int Q)
    {
        if (!ok()) return;
        const Ae5::Tensor &T = a.tensors[t];
        tn_narrow_kernel<<<dim3(T.chunks, blocks(A.len, 32)), 256, 0, c.stream>>>(A, B, Q, T.rows, T.chunk, partial_of(t),
                                                                                  pstride_of(t));
        ++g_kernel_launches;
    }
    static bool streams(const Rows &A) { return A.vec && A.len >= 4 && A.len <= 1024 && (A.len & (A.len - 1)) == 0; }
    void colsum(int t, const Rows &A)
    {
        if (!streams(A)) return tn_narrow(t, A, rows_of(nullptr, nullptr, 0, 0, 1, 1), 1);
        if (!ok()) return;
        const Ae5::Tensor &T = a.tensors[t];
        colsum_kernel<0><<<T.chunks, 256, 0, c.stream>>>(A, A, T.rows, T.chunk, partial_of(t), pstride_of(t), nullptr, 0);
        ++g_kernel_launches;
    }
    // conv1: the bias gradient (tensor tb, column sums of A) and the weight gradient (tensor tw, A^T B with B's three columns)
    // from one pass over A
    void colsum_and_narrow3(int tb, int tw, const Rows &A, const Rows &B)
    {
        const Ae5::Tensor &Tb = a.tensors[tb], &Tw = a.tensors[tw];
        if (!streams(A) || Tb.chunks != Tw.chunks || Tb.chunk != Tw.chunk || B.lo) {
            colsum(tb, A);
            return tn_narrow(tw, A, B, 3);
        }
        if (!ok()) return;
        colsum_kernel<3><<<Tb.chunks, 256, 0, c.stream>>>(A, B, Tb.rows, Tb.chunk, partial_of(tb), pstride_of(tb), partial_of(tw),
                                                          pstride_of(tw));
        ++g_kernel_launches;
    }
    void arrange(const float *w, int cin, int cout, int mode)
    {
        if (!ok()) return;
        arrange_weights_kernel<<<blocks(3 * cin * cout, 256), 256, 0, c.stream>>>(w, cin, cout, mode, a.wt);
        ++g_kernel_launches;
    }
};

}  // namespace

namespace {

// Backward pass of decoder d from g_dec[4] (gradient at deconv5's pre-activation) and dr (gradient at the
// reconstruction) down to the code it read from c.combined: fills the partial sums of tensors 10..21 and
// leaves the gradient at that code in dzbar.  `extra`: the innovation row of the parameter server's decoder.
void decoder_backward(Launcher &L, int d, const float *extra)
{
    Ctx &c = L.c;
    Ae5 &a = L.a;
    const float *P = c.params + d * a.dec_stride;
    const int64_t *len = a.len, mu = c.mu;
    const Rows dr_rows = rows_of(a.dr, nullptr, 0, 1, mu, 1);
    L.tn_narrow(20, rows_of(a.dact5_hi, a.dact5_lo, 0, 32, mu, 32), dr_rows, 1);     // dW6[c] = sum_p d5[p][c] dr[p]
    if (extra && L.ok()) {                                                           // dW6[32] = sum_p innovation[p] dr[p]
        const Ae5::Tensor &T = a.tensors[20];
        tn_narrow_kernel<<<dim3(T.chunks, 1), 256, 0, c.stream>>>(rows_of(extra, nullptr, 0, 1, mu, 1), dr_rows, 1, T.rows, T.chunk,
                                                                  L.partial_of(20) + 32, L.pstride_of(20));
        ++g_kernel_launches;
    }
    L.colsum(21, dr_rows);
    // inputs: deconv5 <- dact[2] [L1][128], deconv4 <- dact[1] [L2][64], deconv3 <- dact[0] [L3][32], deconv2 <- d0 [L4][4]
    for (int i = 4; i >= 1; --i) {
        const int cin = kAe5DecCh[i], cout = kAe5DecCh[i + 1];
        const int64_t lin = len[5 - i], lout = len[4 - i];
        const float *g_out = a.g_dec[i];                                    // [lout][cout]
        const float *x_hi = i == 1 ? a.d0 : a.dact_hi[i - 2], *x_lo = i == 1 ? nullptr : a.dact_lo[i - 2];
        const Rows x = rows_of(x_hi, x_lo, 0, cin, lin, cin);
        const Rows g_slices = rows_of(g_out, nullptr, 0, 2 * cout, lin, 3 * cout);   // row j: positions 2j .. 2j + 2
        L.colsum(11 + 2 * i, rows_of(g_out, nullptr, 0, cout, lout, cout));
        L.tn(10 + 2 * i, x, g_slices);
        L.arrange(P + a.off_dw[i], cin, cout, 1);
        L.nn(g_slices, lin, a.wt, cin, a.g_dec[i - 1], &x);
    }
    if (L.ok()) {
        dec1_grad_kernel<<<52, 256, 0, c.stream>>>(c.combined, a.g_dec[0], len[4], L.partial_of(10), L.partial_of(11)), ++g_kernel_launches;
        dec1_bwd_kernel<<<blocks(len[4], 128), 128, 0, c.stream>>>(a.g_dec[0], len[4], P + a.off_dw[0], a.dzbar), ++g_kernel_launches;
    }
}

// Backward pass of the encoder from the gradients at the codes.  dzbar != nullptr: every node's code gets
// dzbar / K (ring-allreduce); nullptr: dzk holds them already.  Fills the partial sums of tensors 0..9.
void encoder_backward(Launcher &L, const float *dzbar)
{
    Ctx &c = L.c;
    Ae5 &a = L.a;
    const float *P = c.params;
    const int K = c.K;
    const int64_t *len = a.len, mu = c.mu;
    if (L.ok()) {
        code_bwd_kernel<<<blocks((int64_t)K * len[4], 128), 128, 0, c.stream>>>(dzbar, K, len[4], P + a.off_w[4], a.act4_hi, a.dzk,
                                                                              a.g_enc[3], a.g4_hi, a.g4_lo),
            ++g_kernel_launches;
    }
    const Rows dzk_rows = rows_of(a.dzk, nullptr, len[4] * 4, 4, len[4], 4);
    L.tn(8, dzk_rows, rows_of(a.act4_hi, a.act4_lo, len[4] * 64, 64, len[4], 64));
    L.colsum(9, dzk_rows);
    for (int i = 3; i >= 0; --i) {
        const int cout = kAe5EncCh[i + 1];
        const int64_t lout = len[i + 1];
        // gradient at conv(i+1)'s output: conv4's is fp32, the others are two tf32 parts laid out like the output
        const Rows g = i == 3 ? rows_of(a.g_enc[3], nullptr, lout * cout, cout, lout, cout)
                              : rows_of(a.g_enc[i], a.g_enc_lo[i], a.lpad[i] * cout, cout, lout, cout);
        if (i == 0) {        // conv1 reads the kept values themselves: rows of three floats, two apart
            L.colsum_and_narrow3(1, 0, g, rows_of(c.val, nullptr, mu, 2, lout, 3));
            break;
        }
        L.colsum(2 * i + 1, g);
        if (L.ok()) L.err = launch_ae5_weight_gradient(c, i);       // dW = sum over rows of G^T X, on the tensor cores
        // the gradient at the layer's input: a transposed convolution of g with the same weights, on the tensor cores
        if (L.ok()) L.err = launch_ae5_input_gradient(c, i);
    }
}

// Adam on the tensors t0 .. t1 - 1, whose parameters sit `shift` floats behind their place in decoder 0's layout.
void adam_on(Launcher &L, const AdamArgs &ad, int t0, int t1, int64_t shift)
{
    if (!L.ok()) return;
    TensorTable tt;
    tt.first[0] = 0;
    for (int t = 0; t < 22; ++t) {
        const Ae5::Tensor &T = L.a.tensors[t];
        tt.first[t + 1] = tt.first[t] + (t >= t0 && t < t1 ? T.count : 0);
        tt.param_off[t] = T.param_off + shift; tt.partial_off[t] = T.partial_off; tt.pstride[t] = L.pstride_of(t);
        tt.chunks[t] = T.chunks; tt.kind[t] = T.kind; tt.cin[t] = T.cin; tt.cout[t] = T.cout;
    }
    reduce_adam_kernel<<<blocks(tt.first[22], 256), 256, 0, L.c.stream>>>(L.a.partial, tt, ad), ++g_kernel_launches;
}

}  // namespace

cudaError_t launch_ae5_train_step(Ctx &c, float *loss_out)
{
    Ae5 &a = *c.ae5;
    const float *P = c.params;
    cudaError_t e = launch_ae5_train_forward(c);
    if (e != cudaSuccess) return e;
    Launcher L{c, a};
    cudaStream_t s = c.stream;
    // the last convolution and the loss against the mean of the nodes' vectors
    final_loss_kernel<<<a.loss_blocks, 256, 0, s>>>(a.dact5_hi, a.dact5_lo, c.val, c.K, c.mu, P + a.off_dw[5], P + a.off_db[5], nullptr,
                                                    1.0f, c.recon, a.dr, a.g_dec[4], a.loss_part),
        ++g_kernel_launches;
    if (loss_out) loss_sum_kernel<<<1, 256, 0, s>>>(a.loss_part, a.loss_blocks, c.mu, loss_out), ++g_kernel_launches;
    decoder_backward(L, 0, nullptr);
    encoder_backward(L, a.dzbar);
    if (!L.ok()) return L.err;
    adam_on(L, next_adam(c), 0, 22, 0);
    a.weights_ready = false;                       // the GEMM forms of the weights follow the new parameters
    return cudaGetLastError();
}

// Parameter server (Section IV-A): every node's vector is encoded; the similarity term couples the codes;
// the common node's code goes through every node's decoder (one after the other, each followed by its
// backward pass and its Adam update, since they share the activation buffers); the gradients the decoders
// send back add up, in node order, at the common node's code; then the encoder's backward pass.
cudaError_t launch_ae5_train_step_ps(Ctx &c, int common, float lam_rec, float lam_sim, float *loss_out)
{
    Ae5 &a = *c.ae5;
    cudaStream_t s = c.stream;
    const int64_t n = 4 * a.len[4];                                   // entries of one code
    cudaError_t e = launch_ae5_train_encode(c);
    if (e == cudaSuccess) e = launch_combine_ps(c, common);           // the common code and every node's innovation
    if (e != cudaSuccess) return e;
    Launcher L{c, a};
    const AdamArgs ad = next_adam(c);
    double *sim_part = a.loss_part + (size_t)a.decoders * a.loss_blocks;
    const int sim_blocks = (int)blocks(n, 256);
    ps_code_grad_kernel<<<sim_blocks, 256, 0, s>>>(c.code, c.K, n, lam_sim, a.dzk, sim_part), ++g_kernel_launches;
    for (int d = 0; d < a.decoders && L.ok(); ++d) {
        const float *P = c.params + d * a.dec_stride;
        L.err = launch_ae5_train_decode(c, d);
        if (!L.ok()) break;
        const float *inn = c.inn + (int64_t)d * c.mu;
        final_loss_kernel<<<a.loss_blocks, 256, 0, s>>>(a.dact5_hi, a.dact5_lo, c.val + (int64_t)d * c.mu, 1, c.mu, P + a.off_dw[5],
                                                        P + a.off_db[5], inn, lam_rec, c.recon + (int64_t)d * c.mu, a.dr, a.g_dec[4],
                                                        a.loss_part + (size_t)d * a.loss_blocks),
            ++g_kernel_launches;
        decoder_backward(L, d, inn);
        if (L.ok()) add_kernel<<<blocks(n, 256), 256, 0, s>>>(a.dzk + (int64_t)common * n, a.dzbar, n), ++g_kernel_launches;
        adam_on(L, ad, 10, 22, d * a.dec_stride);
    }
    if (loss_out && L.ok())
        ps_loss_sum_kernel<<<1, 256, 0, s>>>(a.loss_part, a.decoders * a.loss_blocks, sim_part, sim_blocks, c.mu, n, lam_rec, lam_sim,
                                             loss_out),
            ++g_kernel_launches;
    encoder_backward(L, nullptr);
    if (!L.ok()) return L.err;
    adam_on(L, ad, 0, 10, 0);
    a.weights_ready = false;
    return cudaGetLastError();
}

}  // namespace lgc
