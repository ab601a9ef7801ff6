// Stages 3-5 of the LGC step: gather of the kept values, the lightweight autoencoder (Section IV
// of the paper, two strided 1-D convolutions each way), the across-node combination of the codes
// (ring-allreduce: mean, Section IV-B; parameter server: common code + innovation, Algorithm 1),
// decoding, and the scatter into the dense update with the removal of sent entries from u and v.
//
// Everything here works on mu ~ N/1000 values: the kernels are latency bound, so each fuses what
// it can (both convolutions of a side in one kernel, decode + scatter + clearing in one kernel)
// and keeps the handful of weights in shared memory.  fp32 FMA arithmetic, no tensor cores: the
// largest contraction is a 48-term dot product.
#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr int kAeThreads = 128;

// Kept values of every node: slots below mu (the autoencoder's layers) go to val, the others (top-k-only
// layers) to val_t.  A row of idx holds mu_all slots.
__global__ void gather_kernel(const float *__restrict__ v, int64_t N, const int32_t *__restrict__ idx,
                              int S, int64_t mu, int64_t mu_all, float *__restrict__ val, float *__restrict__ val_t)
{
    const int k = blockIdx.y;
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= mu_all) return;
    const int32_t i = idx[(S == 1 ? 0 : (int64_t)k * mu_all) + p];
    const float x = v[(int64_t)k * N + i];
    if (p < mu) val[(int64_t)k * mu + p] = x;
    else val_t[(int64_t)k * (mu_all - mu) + (p - mu)] = x;
}

// Layers sent as they are (Section VI-A: the first layer): update[j] = (((g_0[j] + g_1[j]) + ...) + g_{K-1}[j]) / K
// for the elements of one piece [begin, end) of a dense run; pieces hold at most kDenseChunk elements.
__device__ __forceinline__ void dense_piece(const int64_t *__restrict__ pieces, int64_t piece, const float *__restrict__ g,
                                            int64_t g_stride, int K, float *__restrict__ update)
{
    const int64_t a = pieces[2 * piece], b = pieces[2 * piece + 1];
    const float fk = (float)K;
    for (int64_t j = a + threadIdx.x; j < b; j += blockDim.x) {
        float acc = __ldcs(g + j);
        for (int k = 1; k < K; ++k) acc = __fadd_rn(acc, __ldcs(g + (int64_t)k * g_stride + j));
        update[j] = __fdiv_rn(acc, fk);
    }
}

__global__ void dense_pieces_kernel(const int64_t *__restrict__ pieces, const float *__restrict__ g, int64_t g_stride, int K,
                                    float *__restrict__ update)
{
    dense_piece(pieces, blockIdx.x, g, g_stride, K, update);
}

// code[k][co][t] = b2[co] + sum_{ci,tau} w2[co][ci][tau] * relu(b1[ci] + sum_tau' w1[ci][tau'] x[2(2t+tau)+tau'])
template <int C1, int C2>
__global__ void __launch_bounds__(kAeThreads)
encode_kernel(const float *__restrict__ val, int64_t mu, int64_t L2, const float *__restrict__ params,
              float *__restrict__ code)
{
    constexpr int kEnc = C1 * 3 + C1 + C2 * C1 * 3 + C2;
    __shared__ float w[kEnc];
    for (int i = threadIdx.x; i < kEnc; i += kAeThreads) w[i] = params[i];
    __syncthreads();
    const float *w1 = w, *b1 = w + C1 * 3, *w2 = b1 + C1, *b2 = w2 + C2 * C1 * 3;
    const int k = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kAeThreads + threadIdx.x;
    if (t >= L2) return;
    const float *x = val + (int64_t)k * mu + 4 * t;
    float xin[7];
#pragma unroll
    for (int i = 0; i < 7; ++i) xin[i] = x[i];
    float h[3][C1];
#pragma unroll
    for (int ci = 0; ci < C1; ++ci)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            float a = b1[ci];
#pragma unroll
            for (int tau = 0; tau < 3; ++tau) a = __fmaf_rn(w1[ci * 3 + tau], xin[2 * j + tau], a);
            h[j][ci] = fmaxf(a, 0.0f);
        }
#pragma unroll
    for (int co = 0; co < C2; ++co) {
        float a = b2[co];
#pragma unroll
        for (int ci = 0; ci < C1; ++ci)
#pragma unroll
            for (int tau = 0; tau < 3; ++tau) a = __fmaf_rn(w2[(co * C1 + ci) * 3 + tau], h[tau][ci], a);
        code[((int64_t)k * C2 + co) * L2 + t] = a;
    }
}

// tile_lo[q] = first kept slot p whose index lies in or after tile q of the dense update
// (tiles of kDenseTile entries; q = 0 .. ceil(N / kDenseTile)).  The thread that owns slot p
// writes the entries of the tiles that begin between idx[p-1] and idx[p].
constexpr int kDenseTile = 4096;
__device__ __forceinline__ void write_tile_lo(const int32_t *__restrict__ idx, int64_t p, int64_t mu, int64_t N,
                                              int32_t *__restrict__ tile_lo)
{
    const int64_t prev = p == 0 ? -1 : idx[p - 1] / kDenseTile;
    const int64_t mine = idx[p] / kDenseTile;
    for (int64_t q = prev + 1; q <= mine; ++q) tile_lo[q] = (int32_t)p;
    if (p == mu - 1) {
        const int64_t tiles = (N + kDenseTile - 1) / kDenseTile;
        for (int64_t q = mine + 1; q <= tiles; ++q) tile_lo[q] = (int32_t)mu;
    }
}

__global__ void tile_lo_kernel(const int32_t *__restrict__ idx, int64_t mu, int64_t N, int32_t *__restrict__ tile_lo)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < mu) write_tile_lo(idx, p, mu, N, tile_lo);
}

// Ring-allreduce fast path: gather, both encoder convolutions and the node-ordered mean of the
// codes in one kernel.  A CTA covers TT code positions for all K nodes (thread = (node, position)):
// each thread reads the seven kept values v[k][idx[4t .. 4t+6]] of its node, stores the first four
// as val (the last position also stores the tail), computes the node's code, and the K codes of
// a position meet in shared memory where the node-0 thread sums them in node order.
template <int C1, int C2>
__global__ void __launch_bounds__(256)
gather_encode_mean_kernel(const float *__restrict__ v, int64_t N, const int32_t *__restrict__ idx, int K, int TT,
                          int64_t mu, int64_t L2, const float *__restrict__ params, float *__restrict__ val,
                          float *__restrict__ code, float *__restrict__ combined, int32_t *__restrict__ tile_lo)
{
    constexpr int kEnc = C1 * 3 + C1 + C2 * C1 * 3 + C2;
    __shared__ float w[kEnc];
    __shared__ float zs[256 * C2];          // [node][channel][position in CTA]
    grid_release_dependents();              // a single wave: the next kernel's CTAs may come in beside this one's
    for (int i = threadIdx.x; i < kEnc; i += blockDim.x) w[i] = params[i];
    __syncthreads();
    grid_wait();                            // the selection's indices are complete from here on
    const float *w1 = w, *b1 = w + C1 * 3, *w2 = b1 + C1, *b2 = w2 + C2 * C1 * 3;
    const int k = threadIdx.x / TT, tt = threadIdx.x % TT;
    const int64_t t = (int64_t)blockIdx.x * TT + tt;
    if (t < L2) {
        const float *vk = v + (int64_t)k * N;
        int32_t at[7];
#pragma unroll
        for (int i = 0; i < 7; ++i) at[i] = idx[4 * t + i];
        float xin[7];
#pragma unroll
        for (int i = 0; i < 7; ++i) xin[i] = vk[at[i]];
        float *vo = val + (int64_t)k * mu + 4 * t;
#pragma unroll
        for (int i = 0; i < 4; ++i) vo[i] = xin[i];
        const bool last = t == L2 - 1;
        if (last) {
#pragma unroll
            for (int i = 4; i < 7; ++i) vo[i] = xin[i];
            for (int64_t p = 4 * t + 7; p < mu; ++p) val[(int64_t)k * mu + p] = vk[idx[p]];
        }
        if (k == 0 && tile_lo) {
            for (int64_t p = 4 * t; p < (last ? mu : 4 * t + 4); ++p) write_tile_lo(idx, p, mu, N, tile_lo);
        }
        float h[3][C1];
#pragma unroll
        for (int ci = 0; ci < C1; ++ci)
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                float a = b1[ci];
#pragma unroll
                for (int tau = 0; tau < 3; ++tau) a = __fmaf_rn(w1[ci * 3 + tau], xin[2 * j + tau], a);
                h[j][ci] = fmaxf(a, 0.0f);
            }
#pragma unroll
        for (int co = 0; co < C2; ++co) {
            float a = b2[co];
#pragma unroll
            for (int ci = 0; ci < C1; ++ci)
#pragma unroll
                for (int tau = 0; tau < 3; ++tau) a = __fmaf_rn(w2[(co * C1 + ci) * 3 + tau], h[tau][ci], a);
            code[((int64_t)k * C2 + co) * L2 + t] = a;
            zs[(k * C2 + co) * TT + tt] = a;
        }
    }
    __syncthreads();
    if (k == 0 && t < L2) {
#pragma unroll
        for (int co = 0; co < C2; ++co) {
            float a = zs[co * TT + tt];
            for (int kk = 1; kk < K; ++kk) a = __fadd_rn(a, zs[(kk * C2 + co) * TT + tt]);
            combined[(int64_t)co * L2 + t] = __fdiv_rn(a, (float)K);
        }
    }
}

// out[i] = (rows[0][i] + rows[1][i] + ... + rows[K-1][i]) / K, summed in node order
__global__ void mean_rows_kernel(const float *__restrict__ rows, int K, int64_t len, float *__restrict__ out)
{
    grid_release_dependents();
    grid_wait();                          // (launched as a dependent of the kernel that writes the rows)
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len) return;
    float a = rows[i];
    for (int k = 1; k < K; ++k) a = __fadd_rn(a, rows[(int64_t)k * len + i]);
    out[i] = __fdiv_rn(a, (float)K);
}

__global__ void copy_kernel(const float *__restrict__ src, int64_t len, float *__restrict__ dst)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < len) dst[i] = src[i];
}

// inn[k][pos] = val[k][pos] at the selected positions (inn was zeroed before)
__global__ void innovation_fill_kernel(const float *__restrict__ val, const int32_t *__restrict__ pos,
                                       int64_t mu, int64_t muI, float *__restrict__ inn)
{
    const int k = blockIdx.y;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= muI) return;
    const int32_t p = pos[(int64_t)k * muI + q];
    inn[(int64_t)k * mu + p] = val[(int64_t)k * mu + p];
}

// Decoder output at position p for the code z[C2][L2]:
//   d[ci][i] = relu(b1[ci] + sum_{c2, (j,tau'): 2j+tau' = i} w1[c2][ci][tau'] z[c2][j]),   i < L1
//   y[p]     = b2 + sum_{ci, (i,tau): 2i+tau = p} w2[ci][tau] d[ci][i]
template <int C1, int C2>
__device__ __forceinline__ float decode_at(int64_t p, const float *__restrict__ z, int64_t L1, int64_t L2,
                                           const float *w1, const float *b1, const float *w2, float b2)
{
    float y = b2;
    for (int tau = (int)(p & 1); tau < 3; tau += 2) {
        const int64_t i = (p - tau) >> 1;
        if (p < tau || i >= L1) continue;
        float d[C1];
#pragma unroll
        for (int ci = 0; ci < C1; ++ci) d[ci] = b1[ci];
        for (int tq = (int)(i & 1); tq < 3; tq += 2) {
            const int64_t j = (i - tq) >> 1;
            if (i < tq || j >= L2) continue;
#pragma unroll
            for (int c2 = 0; c2 < C2; ++c2) {
                const float zz = z[(int64_t)c2 * L2 + j];
#pragma unroll
                for (int ci = 0; ci < C1; ++ci) d[ci] = __fmaf_rn(w1[(c2 * C1 + ci) * 3 + tq], zz, d[ci]);
            }
        }
#pragma unroll
        for (int ci = 0; ci < C1; ++ci) y = __fmaf_rn(w2[ci * 3 + tau], fmaxf(d[ci], 0.0f), y);
    }
    return y;
}

// One row of reconstructions per decoder: ring-allreduce has one decoder and no innovation;
// the parameter server has one decoder per node and fuses the innovation with (w0, w1, b).
template <int C1, int C2, bool PS>
__global__ void __launch_bounds__(kAeThreads)
decode_kernel(const float *__restrict__ z, int64_t mu, int64_t L1, int64_t L2,
              const float *__restrict__ dec_params, int dec_stride, const float *__restrict__ inn,
              float *__restrict__ recon)
{
    constexpr int kDec = C2 * C1 * 3 + C1 + C1 * 3 + 1 + (PS ? 3 : 0);
    __shared__ float w[kDec];
    const int s = blockIdx.y;
    for (int i = threadIdx.x; i < kDec; i += kAeThreads) w[i] = dec_params[(int64_t)s * dec_stride + i];
    __syncthreads();
    const float *w1 = w, *b1 = w + C2 * C1 * 3, *w2 = b1 + C1;
    const int64_t p = (int64_t)blockIdx.x * kAeThreads + threadIdx.x;
    if (p >= mu) return;
    float y = decode_at<C1, C2>(p, z, L1, L2, w1, b1, w2, w2[C1 * 3]);
    if (PS) {
        const float *f = w2 + C1 * 3 + 1;
        y = __fmaf_rn(f[1], inn[(int64_t)s * mu + p], __fmaf_rn(f[0], y, f[2]));
    }
    recon[(int64_t)s * mu + p] = y;
}

// The same reconstructions, organised by the first transposed convolution's output positions: a thread
// computes the activations d[.][i] of ONE position i once (decode_kernel recomputes them for each of the
// two or three outputs they feed) and from them the three sums e_tau = sum_ci w2[ci][tau] d[ci][i] that
// position i adds to outputs 2i, 2i + 1 and 2i + 2.  Thread i then writes
//     y[2i] = b2 + e_0(i) + e_2(i - 1),    y[2i + 1] = b2 + e_1(i)
// with e_2(i - 1) handed over through shared memory (the CTA's first slot is the halo i0 - 1 and writes
// nothing).  Slot i = L1 (no activations) finishes the tail: y[2 L1] = b2 + e_2(L1 - 1), y[2 L1 + 1] = b2.
// Even and odd positions use different taps of the first layer, so the CTA's first half takes the even
// slots and the second half the odd ones: warps do not diverge.  Weights sit in shared memory with the
// hidden channel innermost (16-byte reads).  Grid (ceil((L1 + 1) / 255), decoders), 256 threads.
template <int C1, int C2, bool PS>
__global__ void __launch_bounds__(256)
decode_rows_kernel(const float *__restrict__ z, int64_t mu, int64_t L1, int64_t L2, const float *__restrict__ dec_params,
                   int dec_stride, const float *__restrict__ inn, float *__restrict__ recon)
{
    static_assert(C1 % 4 == 0, "hidden channels are read four at a time");
    __shared__ __align__(16) float w1s[3][C2][C1];      // [tap][code channel][hidden channel]
    __shared__ __align__(16) float b1s[C1];
    __shared__ float w2s[3][C1], e2s[256], tail[4];     // tail: b2, then the fusion scalars w0, w1, b
    const int s = blockIdx.y;
    const float *P = dec_params + (int64_t)s * dec_stride;
    for (int i = threadIdx.x; i < C2 * C1 * 3; i += 256) {
        const int c2 = i / (C1 * 3), ci = i / 3 % C1, tq = i % 3;
        w1s[tq][c2][ci] = P[i];
    }
    if (threadIdx.x < C1) b1s[threadIdx.x] = P[C2 * C1 * 3 + threadIdx.x];
    for (int i = threadIdx.x; i < C1 * 3; i += 256) w2s[i % 3][i / 3] = P[C2 * C1 * 3 + C1 + i];
    if (threadIdx.x < (PS ? 4 : 1)) tail[threadIdx.x] = P[C2 * C1 * 3 + C1 + C1 * 3 + threadIdx.x];
    __syncthreads();
    const int slot = threadIdx.x < 128 ? 2 * (int)threadIdx.x : 2 * ((int)threadIdx.x - 128) + 1;
    const int64_t i = (int64_t)blockIdx.x * 255 - 1 + slot;
    float e0 = 0.f, e1 = 0.f, e2 = 0.f;
    if (i >= 0 && i < L1) {
        float d[C1];
#pragma unroll
        for (int ci = 0; ci < C1; ++ci) d[ci] = b1s[ci];
        for (int tq = (int)(i & 1); tq < 3; tq += 2) {           // the taps that reach position i: i = 2j + tq
            const int64_t j = (i - tq) >> 1;
            if (i < tq || j >= L2) continue;
#pragma unroll
            for (int c2 = 0; c2 < C2; ++c2) {
                const float zz = z[(int64_t)c2 * L2 + j];
#pragma unroll
                for (int q = 0; q < C1 / 4; ++q) {
                    const float4 w = *reinterpret_cast<const float4 *>(&w1s[tq][c2][4 * q]);
                    d[4 * q] = __fmaf_rn(w.x, zz, d[4 * q]);
                    d[4 * q + 1] = __fmaf_rn(w.y, zz, d[4 * q + 1]);
                    d[4 * q + 2] = __fmaf_rn(w.z, zz, d[4 * q + 2]);
                    d[4 * q + 3] = __fmaf_rn(w.w, zz, d[4 * q + 3]);
                }
            }
        }
#pragma unroll
        for (int ci = 0; ci < C1; ++ci) {
            const float r = fmaxf(d[ci], 0.0f);
            e0 = __fmaf_rn(w2s[0][ci], r, e0);
            e1 = __fmaf_rn(w2s[1][ci], r, e1);
            e2 = __fmaf_rn(w2s[2][ci], r, e2);
        }
    }
    e2s[slot] = e2;
    __syncthreads();
    if (slot == 0 || i > L1) return;
    const float b2 = tail[0];
    float y[2] = {__fadd_rn(b2, __fadd_rn(e0, e2s[slot - 1])), __fadd_rn(b2, e1)};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int64_t p = 2 * i + h;
        if (p >= mu) break;
        float out = y[h];
        if (PS) out = __fmaf_rn(tail[2], inn[(int64_t)s * mu + p], __fmaf_rn(tail[1], out, tail[3]));
        recon[(int64_t)s * mu + p] = out;
    }
}

// identity autoencoder, parameter server: recon_k = code + innovation_k
__global__ void identity_ps_kernel(const float *__restrict__ z, const float *__restrict__ inn, int64_t mu,
                                   float *__restrict__ recon)
{
    const int k = blockIdx.y;
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < mu) recon[(int64_t)k * mu + p] = __fadd_rn(z[p], inn[(int64_t)k * mu + p]);
}

// Ring-allreduce scatter: one index set for all nodes; the sent entries leave every node's u, v.
__global__ void scatter_shared_kernel(const float *__restrict__ values, const int32_t *__restrict__ idx,
                                      int64_t mu, int K, int64_t N, float *__restrict__ update,
                                      float *__restrict__ u, float *__restrict__ v)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= mu) return;
    const int32_t i = idx[p];
    update[i] = values[p];
    for (int k = 0; k < K; ++k) {
        u[(int64_t)k * N + i] = 0.0f;
        v[(int64_t)k * N + i] = 0.0f;
    }
}

constexpr int kDenseThreads = 256;

// Ring-allreduce fast path for stage 5: one pass writes the whole dense update.  A CTA owns 4096
// consecutive entries: it clears a shared-memory tile, decodes the few reconstruction values
// whose index falls into its range (the range of kept slots of a tile comes from tile_lo),
// places them in the tile, removes those entries from every node's u and v, and streams the
// tile out: every entry of the update is written exactly once and no store waits for another.
// MODE 0: the values are the decoder's output already in recon; 1: identity (the mean code is
// the value); 2: mean over nodes of the kept values.
template <int C1, int C2, int MODE>
__global__ void __launch_bounds__(kDenseThreads)
dense_scatter_kernel(const float *__restrict__ z, const float *__restrict__ val, const int32_t *__restrict__ idx,
                     const int32_t *__restrict__ tile_lo, int64_t mu, int64_t L1, int64_t L2,
                     const float *__restrict__ dec, int K, int64_t N, float *__restrict__ recon,
                     float *__restrict__ update, float *__restrict__ u, float *__restrict__ v)
{
    __shared__ __align__(16) float tile[kDenseTile];
    const int64_t base = (int64_t)blockIdx.x * kDenseTile;
    const int64_t end = base + kDenseTile < N ? base + kDenseTile : N;
    const int64_t lo = tile_lo[blockIdx.x], hi = tile_lo[blockIdx.x + 1];
#pragma unroll
    for (int i = threadIdx.x; i < kDenseTile / 4; i += kDenseThreads)
        reinterpret_cast<float4 *>(tile)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    for (int64_t p = lo + threadIdx.x; p < hi; p += kDenseThreads) {
        float y;
        if (MODE == 0) {
            y = recon[p];                 // decoded by decode_kernel just before
        } else if (MODE == 1) {
            y = z[p];
        } else {
            y = val[p];
            for (int k = 1; k < K; ++k) y = __fadd_rn(y, val[(int64_t)k * mu + p]);
            y = __fdiv_rn(y, (float)K);
        }
        tile[idx[p] - base] = y;
        if (MODE != 0) recon[p] = y;
    }
    __syncthreads();
    float *dst = update + base;
    if (end - base == kDenseTile) {
#pragma unroll
        for (int i = threadIdx.x; i < kDenseTile / 4; i += kDenseThreads)
            __stcs(reinterpret_cast<float4 *>(dst) + i, reinterpret_cast<const float4 *>(tile)[i]);
    } else {
        for (int i = threadIdx.x; i < (int)(end - base); i += kDenseThreads) dst[i] = tile[i];
    }
    // the sent entries leave every node's u and v; these scattered stores come last so that no
    // thread reaches the barrier late because of them
    for (int64_t p = lo + threadIdx.x; p < hi; p += kDenseThreads) {
        const int32_t i = idx[p];
        for (int k = 0; k < K; ++k) {
            u[(int64_t)k * N + i] = 0.0f;
            v[(int64_t)k * N + i] = 0.0f;
        }
    }
}

// Ring-allreduce stage 5 when the update buffer has been cleared already: decode (MODE 0), take the
// mean code (1) or average the kept values (2) for slot p, write it at its index, and remove the
// entry from every node's u and v.  One thread per kept slot.  Slots from mu on belong to top-k-only
// layers (Section VI-A: the last layer): their value is the mean over the nodes of the kept entries
// themselves, read from v.  CTAs beyond the slots average the pieces of the dense layers.
template <int C1, int C2, int MODE>
__global__ void __launch_bounds__(kAeThreads)
sparse_scatter_kernel(const float *__restrict__ z, const float *__restrict__ val, const int32_t *__restrict__ idx,
                      int64_t mu, int64_t mu_all, int64_t L1, int64_t L2, const float *__restrict__ dec, int K, int64_t N,
                      float *__restrict__ recon, float *__restrict__ update, float *__restrict__ u,
                      float *__restrict__ v, unsigned slot_ctas, const int64_t *__restrict__ pieces,
                      const float *__restrict__ g, int64_t g_stride)
{
    constexpr int kDec = C2 * C1 * 3 + C1 + C1 * 3 + 1;
    __shared__ float w[kDec];
    grid_release_dependents();
    if (blockIdx.x >= slot_ctas) {
        grid_wait();                                // the update buffer has been cleared by then
        dense_piece(pieces, blockIdx.x - slot_ctas, g, g_stride, K, update);
        return;
    }
    if (MODE == 0) {
        for (int i = threadIdx.x; i < kDec; i += kAeThreads) w[i] = dec[i];
        __syncthreads();
    }
    grid_wait();                                    // codes, indices and the cleared update are complete from here on
    const int64_t p = (int64_t)blockIdx.x * kAeThreads + threadIdx.x;
    if (p >= mu_all) return;
    const int32_t i = idx[p];
    float y;
    if (p >= mu) {
        y = v[i];
        for (int k = 1; k < K; ++k) y = __fadd_rn(y, v[(int64_t)k * N + i]);
        y = __fdiv_rn(y, (float)K);
    } else if (MODE == 0) {
        const float *w1 = w, *b1 = w + C2 * C1 * 3, *w2 = b1 + C1;
        y = decode_at<C1, C2>(p, z, L1, L2, w1, b1, w2, w2[C1 * 3]);
    } else if (MODE == 1) {
        y = z[p];
    } else {
        y = val[p];
        for (int k = 1; k < K; ++k) y = __fadd_rn(y, val[(int64_t)k * mu + p]);
        y = __fdiv_rn(y, (float)K);
    }
    update[i] = y;
    if (p < mu) recon[p] = y;
    for (int k = 0; k < K; ++k) {
        u[(int64_t)k * N + i] = 0.0f;
        v[(int64_t)k * N + i] = 0.0f;
    }
}

// Parameter-server scatter: update[i] = sum over nodes k (ascending) that kept i of values_k / K.
// The lowest node holding an index sums for all of them, so the order of additions is fixed and
// no atomics are needed.  Each node's own sent entries leave its u and v.
// The index is looked up in the other nodes' lists of the same layer eight nodes at a time: the
// searches halve the same range in lock step, so their loads are in flight together.
constexpr int kOwnBatch = 8;
// Serves the slots [slot0, slot0 + nslots) of every node's index row (rows are idx_stride apart); the
// values of node k's slot p are values[k * val_stride + (p - slot0)].
__global__ void scatter_own_kernel(const float *__restrict__ values, int64_t val_stride, const int32_t *__restrict__ idx,
                                   int64_t idx_stride, int64_t slot0, int64_t nslots,
                                   const int32_t *__restrict__ slot_layer, const int32_t *__restrict__ koff,
                                   int K, int64_t N, float *__restrict__ update,
                                   float *__restrict__ u, float *__restrict__ v)
{
    const int k = blockIdx.y;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= nslots) return;
    const int64_t p = slot0 + q;
    const int32_t i = idx[(int64_t)k * idx_stride + p];
    u[(int64_t)k * N + i] = 0.0f;
    v[(int64_t)k * N + i] = 0.0f;
    const int l = slot_layer[p];
    const int lo = koff[l], len = koff[l + 1] - lo;            // at least one kept entry per layer
    const float fk = (float)K;
    float acc = 0.0f;
    bool own_added = false;
    for (int k0 = 0; k0 < K; k0 += kOwnBatch) {
        // lower bound of i in the layer's slice of nodes k0 .. k0 + 7 (the own node and nodes >= K idle)
        const int32_t *base[kOwnBatch];
#pragma unroll
        for (int j = 0; j < kOwnBatch; ++j) base[j] = idx + (int64_t)(k0 + j < K ? k0 + j : k) * idx_stride + lo;
        for (int n = len; n > 1;) {
            const int half = n >> 1;
            int32_t probe[kOwnBatch];
#pragma unroll
            for (int j = 0; j < kOwnBatch; ++j) probe[j] = __ldg(base[j] + half - 1);
#pragma unroll
            for (int j = 0; j < kOwnBatch; ++j)
                if (probe[j] < i) base[j] += half;
            n -= half;
        }
        // the lower bound is base[j], or the slot after it when that entry is still below i
        int32_t at[kOwnBatch];
#pragma unroll
        for (int j = 0; j < kOwnBatch; ++j) at[j] = __ldg(base[j]);
#pragma unroll
        for (int j = 0; j < kOwnBatch; ++j) {
            const int kk = k0 + j;
            if (kk >= K) break;
            if (kk == k) {
                acc = __fadd_rn(acc, __fdiv_rn(values[(int64_t)k * val_stride + q], fk));
                own_added = true;
                continue;
            }
            const int32_t *row = idx + (int64_t)kk * idx_stride;
            const int32_t *hit = nullptr;
            if (at[j] == i) hit = base[j];
            else if (at[j] < i && base[j] + 1 < row + lo + len && __ldg(base[j] + 1) == i) hit = base[j] + 1;
            if (!hit) continue;
            if (!own_added) return;                               // a lower node owns this index
            acc = __fadd_rn(acc, __fdiv_rn(values[(int64_t)kk * val_stride + ((hit - row) - slot0)], fk));
        }
    }
    update[i] = acc;
}

inline unsigned blocks_for(int64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

#define LGC_DISPATCH_AE(c1, c2, CALL)                                   \
    if ((c1) == 8 && (c2) == 4) { CALL(8, 4), ++g_kernel_launches; }                         \
    else if ((c1) == 16 && (c2) == 8) { CALL(16, 8), ++g_kernel_launches; }                  \
    else if ((c1) == 4 && (c2) == 2) { CALL(4, 2), ++g_kernel_launches; }                    \
    else if ((c1) == 3 && (c2) == 2) { CALL(3, 2), ++g_kernel_launches; }                    \
    else return cudaErrorInvalidValue;

}  // namespace

cudaError_t launch_gather(Ctx &c)
{
    if (c.val_valid) return cudaSuccess;
    gather_kernel<<<dim3(blocks_for(c.mu_all, 256), c.K), 256, 0, c.stream>>>(c.v, c.N, c.idx, c.S, c.mu, c.mu_all, c.val, c.val_t),
        ++g_kernel_launches;
    c.val_valid = true;
    return cudaGetLastError();
}

cudaError_t launch_encode(Ctx &c)
{
    if (c.cfg.ae_kind == LGC_AE_IDENTITY) return cudaSuccess;   // the code is the kept values themselves
    if (c.cfg.ae_kind == LGC_AE_CONV5) return launch_ae5_encode(c);
    if (c.S == 1 && c.K <= 256) {   // ring-allreduce: gather + encode + mean in one launch
        int tt = 256 / c.K;
        if (tt > 64) tt = 64;
        const unsigned grid = blocks_for(c.L2, tt);
        cudaError_t le = cudaSuccess;
#define CALL(A, B) le = launch_dependent(gather_encode_mean_kernel<A, B>, dim3(grid), dim3(tt * c.K), c.stream,        \
        c.v, c.N, c.idx, c.K, tt, c.mu, c.L2, c.params, c.val, c.code, c.combined, c.mixed ? nullptr : c.tile_lo)
        LGC_DISPATCH_AE(c.cfg.ae_c1, c.cfg.ae_c2, CALL)
#undef CALL
        if (le != cudaSuccess) return le;
        c.val_valid = c.mu_t == 0;              // the values of top-k-only layers are not gathered here
        c.mean_valid = true;
        c.tile_lo_valid = !c.mixed;
        return cudaGetLastError();
    }
    if (c.S == 1) {
        const cudaError_t e = launch_gather(c);
        if (e != cudaSuccess) return e;
    }
    const dim3 grid(blocks_for(c.L2, kAeThreads), c.K);
#define CALL(A, B) encode_kernel<A, B><<<grid, kAeThreads, 0, c.stream>>>(c.val, c.mu, c.L2, c.params, c.code)
    LGC_DISPATCH_AE(c.cfg.ae_c1, c.cfg.ae_c2, CALL)
#undef CALL
    return cudaGetLastError();
}

cudaError_t launch_combine_mean(Ctx &c)
{
    if (c.mean_valid) return cudaSuccess;   // the encoder launch already averaged the codes
    const cudaError_t e = launch_dependent(mean_rows_kernel, dim3(blocks_for(c.code_len, 256)), dim3(256), c.stream, c.code, c.K,
                                           c.code_len, c.combined);
    if (e != cudaSuccess) return e;
    ++g_kernel_launches;
    return cudaGetLastError();
}

cudaError_t launch_combine_ps(Ctx &c, int common_node)
{
    copy_kernel<<<blocks_for(c.code_len, 256), 256, 0, c.stream>>>(c.code + (int64_t)common_node * c.code_len,
                                                                   c.code_len, c.combined), ++g_kernel_launches;
    cudaError_t e = launch_zero(c.inn, (size_t)c.K * c.mu * sizeof(float), c.stream);
    if (e != cudaSuccess) return e;
    e = launch_select(c.sel_inn, c.val, c.mu, 0, c.K, c.inn_pos, c.muI, false, ++c.inn_epoch, nullptr, 0, c.errword,
                      c.stream);
    if (e != cudaSuccess) return e;
    innovation_fill_kernel<<<dim3(blocks_for(c.muI, 256), c.K), 256, 0, c.stream>>>(c.val, c.inn_pos, c.mu, c.muI, c.inn), ++g_kernel_launches;
    return cudaGetLastError();
}

// Averages the dense layers of the step's gradient into their places of the update (a launch of its own).
static cudaError_t launch_dense_layers(Ctx &c, float *update)
{
    if (!c.num_dense_chunks) return cudaSuccess;
    const int64_t gs = c.cfg.grad_row_stride ? c.cfg.grad_row_stride : c.N;
    dense_pieces_kernel<<<(unsigned)c.num_dense_chunks, kAeThreads, 0, c.stream>>>(c.dense_chunks, c.step_grads, gs, c.K, update),
        ++g_kernel_launches;
    return cudaGetLastError();
}

// values: [S][mu] of the autoencoder layers' slots; the top-k-only layers' slots send their kept values.
static cudaError_t launch_scatter(Ctx &c, const float *values, float *update)
{
    if (update != c.cleared_update) {       // otherwise lgc_topk's finishing launch has cleared it already
        const cudaError_t e = launch_zero(update, (size_t)c.N * sizeof(float), c.stream);
        if (e != cudaSuccess) return e;
    }
    if (c.S == 1 && !c.mixed) {
        scatter_shared_kernel<<<blocks_for(c.mu, 256), 256, 0, c.stream>>>(values, c.idx, c.mu, c.K, c.N, update, c.u, c.v), ++g_kernel_launches;
    } else {
        scatter_own_kernel<<<dim3(blocks_for(c.mu, 128), c.K), 128, 0, c.stream>>>(
            values, c.mu, c.idx, c.mu_all, 0, c.mu, c.slot_layer, c.koff_dev, c.K, c.N, update, c.u, c.v), ++g_kernel_launches;
        if (c.mu_t)
            scatter_own_kernel<<<dim3(blocks_for(c.mu_t, 128), c.K), 128, 0, c.stream>>>(
                c.val_t, c.mu_t, c.idx, c.mu_all, c.mu, c.mu_t, c.slot_layer, c.koff_dev, c.K, c.N, update, c.u, c.v), ++g_kernel_launches;
    }
    const cudaError_t e = cudaGetLastError();
    return e != cudaSuccess ? e : launch_dense_layers(c, update);
}

// Ring-allreduce: the whole of stage 5 (or the phase-two sparse mean) in one pass over the update.
// mode 0: decode the mean code; 1: the values are in `src` (default: the mean code of the identity
// autoencoder); 2: mean over nodes of the kept values.
static cudaError_t launch_dense_scatter(Ctx &c, int mode, float *update, const float *src = nullptr)
{
    const float *dec = c.params + c.Penc;
    const float *z1 = src ? src : c.combined;
    if (c.mixed && update != c.cleared_update) {
        // per-layer modes are served by the slot-wise kernel only: clear the buffer here
        const cudaError_t e = launch_zero(update, (size_t)c.N * sizeof(float), c.stream);
        if (e != cudaSuccess) return e;
        c.cleared_update = update;
    }
    if (update == c.cleared_update) {
        // the buffer has been cleared (by lgc_topk's finishing launch, as a rule): only the kept entries and
        // the dense layers are written
        const unsigned slots = blocks_for(c.mu_all, kAeThreads), sgrid = slots + (unsigned)c.num_dense_chunks;
        const int64_t gs = c.cfg.grad_row_stride ? c.cfg.grad_row_stride : c.N;
#define SCATTER_ARGS(Z) Z, c.val, c.idx, c.mu, c.mu_all, c.L1, c.L2, dec, c.K, c.N, c.recon, update, c.u, c.v, slots, c.dense_chunks, \
                        c.step_grads, gs
        if (mode == 1) {
            sparse_scatter_kernel<3, 2, 1><<<sgrid, kAeThreads, 0, c.stream>>>(SCATTER_ARGS(z1)), ++g_kernel_launches;
        } else if (mode == 2) {
            sparse_scatter_kernel<3, 2, 2><<<sgrid, kAeThreads, 0, c.stream>>>(SCATTER_ARGS(c.combined)), ++g_kernel_launches;
        } else {
            cudaError_t le = cudaSuccess;
#define CALL(A, B) le = launch_dependent(sparse_scatter_kernel<A, B, 0>, dim3(sgrid), dim3(kAeThreads), c.stream, SCATTER_ARGS(c.combined))
            LGC_DISPATCH_AE(c.cfg.ae_c1, c.cfg.ae_c2, CALL)
#undef CALL
            if (le != cudaSuccess) return le;
        }
#undef SCATTER_ARGS
        return cudaGetLastError();
    }
    if (!c.tile_lo_valid) {
        tile_lo_kernel<<<blocks_for(c.mu, 256), 256, 0, c.stream>>>(c.idx, c.mu, c.N, c.tile_lo), ++g_kernel_launches;
        c.tile_lo_valid = true;
    }
    const unsigned grid = blocks_for(c.N, kDenseTile);
    if (mode == 1) {
        dense_scatter_kernel<3, 2, 1><<<grid, kDenseThreads, 0, c.stream>>>(
            z1, c.val, c.idx, c.tile_lo, c.mu, c.L1, c.L2, dec, c.K, c.N, c.recon, update, c.u, c.v), ++g_kernel_launches;
    } else if (mode == 2) {
        dense_scatter_kernel<3, 2, 2><<<grid, kDenseThreads, 0, c.stream>>>(
            c.combined, c.val, c.idx, c.tile_lo, c.mu, c.L1, c.L2, dec, c.K, c.N, c.recon, update, c.u, c.v), ++g_kernel_launches;
    } else {
        // the decoder runs as its own short, fully parallel launch: inside the dense pass its serial
        // chain would hold every CTA's barrier for several microseconds
        const dim3 dgrid(blocks_for(c.mu, kAeThreads), 1);
#define CALL(A, B) decode_kernel<A, B, false><<<dgrid, kAeThreads, 0, c.stream>>>(c.combined, c.mu, c.L1, c.L2, dec,    \
                                                                                 (int)c.Pdec, nullptr, c.recon)
        LGC_DISPATCH_AE(c.cfg.ae_c1, c.cfg.ae_c2, CALL)
#undef CALL
        dense_scatter_kernel<3, 2, 0><<<grid, kDenseThreads, 0, c.stream>>>(
            c.combined, c.val, c.idx, c.tile_lo, c.mu, c.L1, c.L2, dec, c.K, c.N, c.recon, update, c.u, c.v), ++g_kernel_launches;
    }
    return cudaGetLastError();
}

cudaError_t launch_decode_scatter(Ctx &c, float *update)
{
    const bool ps = c.cfg.variant == LGC_VARIANT_PS;
    if (!ps && c.cfg.ae_kind == LGC_AE_CONV5) {
        const cudaError_t e = launch_ae5_decode(c);
        return e != cudaSuccess ? e : launch_dense_scatter(c, 1, update, c.recon);
    }
    if (!ps) return launch_dense_scatter(c, c.cfg.ae_kind == LGC_AE_IDENTITY ? 1 : 0, update);
    if (c.cfg.ae_kind == LGC_AE_CONV5) {                 // K full-size decoders, each with its node's innovation
        const cudaError_t e = launch_ae5_decode(c);
        return e != cudaSuccess ? e : launch_scatter(c, c.recon, update);
    }
    if (c.cfg.ae_kind == LGC_AE_IDENTITY) {
        identity_ps_kernel<<<dim3(blocks_for(c.mu, 256), c.K), 256, 0, c.stream>>>(c.combined, c.inn, c.mu, c.recon), ++g_kernel_launches;
    } else {
        const float *dec = c.params + c.Penc;
        if (c.cfg.ae_c1 % 4 == 0) {        // one thread per position of the hidden layer
            const dim3 grid(blocks_for(c.L1 + 1, 255), c.S);
            if (c.cfg.ae_c1 == 8 && c.cfg.ae_c2 == 4)
                decode_rows_kernel<8, 4, true><<<grid, 256, 0, c.stream>>>(c.combined, c.mu, c.L1, c.L2, dec, (int)c.Pdec, c.inn, c.recon);
            else if (c.cfg.ae_c1 == 16 && c.cfg.ae_c2 == 8)
                decode_rows_kernel<16, 8, true><<<grid, 256, 0, c.stream>>>(c.combined, c.mu, c.L1, c.L2, dec, (int)c.Pdec, c.inn, c.recon);
            else if (c.cfg.ae_c1 == 4 && c.cfg.ae_c2 == 2)
                decode_rows_kernel<4, 2, true><<<grid, 256, 0, c.stream>>>(c.combined, c.mu, c.L1, c.L2, dec, (int)c.Pdec, c.inn, c.recon);
            else
                return cudaErrorInvalidValue;
            ++g_kernel_launches;
        } else {
            const dim3 grid(blocks_for(c.mu, kAeThreads), c.S);
#define CALL(A, B) decode_kernel<A, B, true><<<grid, kAeThreads, 0, c.stream>>>(c.combined, c.mu, c.L1, c.L2, dec,     \
                                                                               (int)c.Pdec, c.inn, c.recon)
            LGC_DISPATCH_AE(c.cfg.ae_c1, c.cfg.ae_c2, CALL)
#undef CALL
        }
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_scatter(c, c.recon, update);
}

cudaError_t launch_topk_scatter(Ctx &c, float *update)
{
    cudaError_t e = launch_gather(c);
    if (e != cudaSuccess) return e;
    if (c.S == 1) return launch_dense_scatter(c, 2, update);
    return launch_scatter(c, c.val, update);
}

}  // namespace lgc
