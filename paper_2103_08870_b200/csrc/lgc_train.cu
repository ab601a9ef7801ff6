// Training steps of the two-layer autoencoders.  Ring-allreduce (Section IV-B of the paper): the nodes'
// kept-value vectors are encoded one after the other, the codes are averaged, the decoder
// reconstructs, and the loss compares the reconstruction with the mean of the vectors:
//     loss = (1/mu) || D_c((1/K) sum_k E_c(g~_k)) - (1/K) sum_k g~_k ||^2
// followed by the analytic backward pass and one Adam step.
//
// Activations and data gradients are fp32 and elementwise; every reduction over positions (the
// loss and each parameter's gradient) is accumulated in fp64 by a single CTA in a fixed order,
// so a step is deterministic.  One CTA per parameter: it reduces that parameter's gradient and
// applies its Adam update; the kernel reads no parameter, so there is no hazard.
#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr int kTrThreads = 128;
constexpr int kRedThreads = 256;

template <int C1>
__global__ void __launch_bounds__(kTrThreads)
fwd_enc1_kernel(const float *__restrict__ val, int64_t mu, int64_t L1, const float *__restrict__ params,
                float *__restrict__ h)
{
    __shared__ float w[C1 * 4];
    for (int i = threadIdx.x; i < C1 * 4; i += kTrThreads) w[i] = params[i];
    __syncthreads();
    const int k = blockIdx.y;
    const int64_t t = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (t >= L1) return;
    const float *x = val + (int64_t)k * mu + 2 * t;
    const float x0 = x[0], x1 = x[1], x2 = x[2];
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) {
        float a = w[C1 * 3 + ci];
        a = __fmaf_rn(w[ci * 3 + 0], x0, a);
        a = __fmaf_rn(w[ci * 3 + 1], x1, a);
        a = __fmaf_rn(w[ci * 3 + 2], x2, a);
        h[((int64_t)k * C1 + ci) * L1 + t] = fmaxf(a, 0.0f);
    }
}

template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
fwd_enc2_mean_kernel(const float *__restrict__ h, int K, int64_t L1, int64_t L2,
                     const float *__restrict__ params, float *__restrict__ zbar)
{
    constexpr int kW = C2 * C1 * 3 + C2;
    __shared__ float w[kW];
    for (int i = threadIdx.x; i < kW; i += kTrThreads) w[i] = params[C1 * 4 + i];
    __syncthreads();
    const int64_t t = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (t >= L2) return;
    float sum[C2];
    for (int k = 0; k < K; ++k) {
        float z[C2];
#pragma unroll
        for (int co = 0; co < C2; ++co) z[co] = w[C2 * C1 * 3 + co];
#pragma unroll
        for (int ci = 0; ci < C1; ++ci) {
            const float *hp = h + ((int64_t)k * C1 + ci) * L1 + 2 * t;
            const float h0 = hp[0], h1 = hp[1], h2 = hp[2];
#pragma unroll
            for (int co = 0; co < C2; ++co) {
                z[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 0], h0, z[co]);
                z[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 1], h1, z[co]);
                z[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 2], h2, z[co]);
            }
        }
#pragma unroll
        for (int co = 0; co < C2; ++co) sum[co] = k == 0 ? z[co] : __fadd_rn(sum[co], z[co]);
    }
#pragma unroll
    for (int co = 0; co < C2; ++co) zbar[(int64_t)co * L2 + t] = __fdiv_rn(sum[co], (float)K);
}

template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
fwd_dec1_kernel(const float *__restrict__ zbar, int64_t L1, int64_t L2, const float *__restrict__ dec,
                int64_t dec_stride, float *__restrict__ d)
{
    // blockIdx.y: decoder (parameter server: one per node, dec_stride floats apart; its output follows suit)
    constexpr int kW = C2 * C1 * 3 + C1;
    __shared__ float w[kW];
    dec += (int64_t)blockIdx.y * dec_stride;
    d += (int64_t)blockIdx.y * C1 * L1;
    for (int i = threadIdx.x; i < kW; i += kTrThreads) w[i] = dec[i];
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (i >= L1) return;
    float a[C1];
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) a[ci] = w[C2 * C1 * 3 + ci];
    for (int tq = (int)(i & 1); tq < 3; tq += 2) {
        const int64_t j = (i - tq) >> 1;
        if (i < tq || j >= L2) continue;
#pragma unroll
        for (int c2 = 0; c2 < C2; ++c2) {
            const float zz = zbar[(int64_t)c2 * L2 + j];
#pragma unroll
            for (int ci = 0; ci < C1; ++ci) a[ci] = __fmaf_rn(w[(c2 * C1 + ci) * 3 + tq], zz, a[ci]);
        }
    }
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) d[(int64_t)ci * L1 + i] = fmaxf(a[ci], 0.0f);
}

__device__ __forceinline__ double block_sum(double x, double *warp_part)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) warp_part[warp] = x;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0)
        for (int wdx = 0; wdx < (int)(blockDim.x >> 5); ++wdx) tot += warp_part[wdx];
    return tot;   // valid in thread 0
}

template <int C1>
__global__ void __launch_bounds__(kTrThreads)
fwd_dec2_loss_kernel(const float *__restrict__ d, const float *__restrict__ val, int K, int64_t mu, int64_t L1,
                     const float *__restrict__ dec_w2, float *__restrict__ recon, float *__restrict__ dr,
                     double *__restrict__ loss_part)
{
    __shared__ float w[C1 * 3 + 1];
    __shared__ double warp_part[kTrThreads / 32];
    for (int i = threadIdx.x; i < C1 * 3 + 1; i += kTrThreads) w[i] = dec_w2[i];
    __syncthreads();
    const int64_t p = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    double sq = 0.0;
    if (p < mu) {
        float y = w[C1 * 3];
        for (int tau = (int)(p & 1); tau < 3; tau += 2) {
            const int64_t i = (p - tau) >> 1;
            if (p < tau || i >= L1) continue;
#pragma unroll
            for (int ci = 0; ci < C1; ++ci) y = __fmaf_rn(w[ci * 3 + tau], d[(int64_t)ci * L1 + i], y);
        }
        float target = val[p];
        for (int k = 1; k < K; ++k) target = __fadd_rn(target, val[(int64_t)k * mu + p]);
        target = __fdiv_rn(target, (float)K);
        const float diff = __fsub_rn(y, target);
        recon[p] = y;
        dr[p] = __fdiv_rn(__fmul_rn(2.0f, diff), (float)mu);
        sq = (double)diff * (double)diff;
    }
    const double tot = block_sum(sq, warp_part);
    if (threadIdx.x == 0) loss_part[blockIdx.x] = tot;
}

template <int C1>
__global__ void __launch_bounds__(kTrThreads)
bwd_dec2_kernel(const float *__restrict__ dr, int64_t mu, const float *__restrict__ d, int64_t L1,
                const float *__restrict__ dec_w2, int64_t dec_stride, float *__restrict__ dd)
{
    // blockIdx.y: decoder (see fwd_dec1_kernel); dr: the gradient at that decoder's output, mu floats per decoder
    __shared__ float w[C1 * 3];
    dec_w2 += (int64_t)blockIdx.y * dec_stride;
    dr += (int64_t)blockIdx.y * mu;
    d += (int64_t)blockIdx.y * C1 * L1;
    dd += (int64_t)blockIdx.y * C1 * L1;
    for (int i = threadIdx.x; i < C1 * 3; i += kTrThreads) w[i] = dec_w2[i];
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (i >= L1) return;
    const float r0 = dr[2 * i], r1 = dr[2 * i + 1], r2 = dr[2 * i + 2];
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) {
        float a = __fmul_rn(w[ci * 3 + 0], r0);
        a = __fmaf_rn(w[ci * 3 + 1], r1, a);
        a = __fmaf_rn(w[ci * 3 + 2], r2, a);
        dd[(int64_t)ci * L1 + i] = d[(int64_t)ci * L1 + i] > 0.0f ? a : 0.0f;
    }
}

// dz[c2][j] = (1/K) sum_{ci,tau} w1[c2][ci][tau] dd[ci][2j+tau]   (the gradient every node's code gets)
template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
bwd_dec1_kernel(const float *__restrict__ dd, float div, int64_t L1, int64_t L2, const float *__restrict__ dec,
                int64_t dec_stride, float *__restrict__ dz)
{
    // blockIdx.y: decoder (see fwd_dec1_kernel); div: K for the ring-allreduce mean, 1 for the parameter server
    __shared__ float w[C2 * C1 * 3];
    dec += (int64_t)blockIdx.y * dec_stride;
    dd += (int64_t)blockIdx.y * C1 * L1;
    dz += (int64_t)blockIdx.y * C2 * L2;
    for (int i = threadIdx.x; i < C2 * C1 * 3; i += kTrThreads) w[i] = dec[i];
    __syncthreads();
    const int64_t j = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (j >= L2) return;
    float a[C2];
#pragma unroll
    for (int c2 = 0; c2 < C2; ++c2) a[c2] = 0.0f;
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) {
        const float *q = dd + (int64_t)ci * L1 + 2 * j;
        const float q0 = q[0], q1 = q[1], q2 = q[2];
#pragma unroll
        for (int c2 = 0; c2 < C2; ++c2) {
            a[c2] = __fmaf_rn(w[(c2 * C1 + ci) * 3 + 0], q0, a[c2]);
            a[c2] = __fmaf_rn(w[(c2 * C1 + ci) * 3 + 1], q1, a[c2]);
            a[c2] = __fmaf_rn(w[(c2 * C1 + ci) * 3 + 2], q2, a[c2]);
        }
    }
#pragma unroll
    for (int c2 = 0; c2 < C2; ++c2) dz[(int64_t)c2 * L2 + j] = __fdiv_rn(a[c2], div);
}

// dh_k[ci][i] = [h_k[ci][i] > 0] sum_{co, (t,tau): 2t+tau = i} w2[co][ci][tau] dz[co][t]
template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
bwd_enc2_kernel(const float *__restrict__ dz, int64_t dz_stride, const float *__restrict__ h, int64_t L1, int64_t L2,
                const float *__restrict__ params, float *__restrict__ dh)
{
    // dz_stride: 0 when every node's code gets the same gradient (ring-allreduce), else C2 * L2
    __shared__ float w[C2 * C1 * 3];
    for (int i = threadIdx.x; i < C2 * C1 * 3; i += kTrThreads) w[i] = params[C1 * 4 + i];
    __syncthreads();
    const int k = blockIdx.y;
    dz += (int64_t)k * dz_stride;
    const int64_t i = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (i >= L1) return;
    float a[C1];
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) a[ci] = 0.0f;
    for (int tau = (int)(i & 1); tau < 3; tau += 2) {
        const int64_t t = (i - tau) >> 1;
        if (i < tau || t >= L2) continue;
#pragma unroll
        for (int co = 0; co < C2; ++co) {
            const float g = dz[(int64_t)co * L2 + t];
#pragma unroll
            for (int ci = 0; ci < C1; ++ci) a[ci] = __fmaf_rn(w[(co * C1 + ci) * 3 + tau], g, a[ci]);
        }
    }
#pragma unroll
    for (int ci = 0; ci < C1; ++ci) {
        const int64_t o = ((int64_t)k * C1 + ci) * L1 + i;
        dh[o] = h[o] > 0.0f ? a[ci] : 0.0f;
    }
}

// One CTA per parameter: reduce its gradient in fp64, then apply Adam to it.
template <int C1, int C2>
__global__ void __launch_bounds__(kRedThreads)
param_grad_adam_kernel(const float *__restrict__ val, const float *__restrict__ h, const float *__restrict__ zbar,
                       const float *__restrict__ d, const float *__restrict__ dr, const float *__restrict__ dd,
                       const float *__restrict__ dz, const float *__restrict__ dh, int K, int64_t mu,
                       int64_t L1, int64_t L2, AdamArgs ad)
{
    constexpr int nE1w = C1 * 3, nE1b = C1, nE2w = C2 * C1 * 3, nE2b = C2;
    constexpr int nD1w = C2 * C1 * 3, nD1b = C1, nD2w = C1 * 3;
    __shared__ double warp_part[kRedThreads / 32];
    int pid = blockIdx.x;
    double acc = 0.0;
    if (pid < nE1w) {                               // enc.w1[ci][0][tau]
        const int ci = pid / 3, tau = pid % 3;
        for (int64_t q = threadIdx.x; q < (int64_t)K * L1; q += kRedThreads) {
            const int64_t k = q / L1, t = q % L1;
            acc += (double)val[k * mu + 2 * t + tau] * (double)dh[(k * C1 + ci) * L1 + t];
        }
    } else if ((pid -= nE1w) < nE1b) {              // enc.b1[ci]
        for (int64_t q = threadIdx.x; q < (int64_t)K * L1; q += kRedThreads) {
            const int64_t k = q / L1, t = q % L1;
            acc += (double)dh[(k * C1 + pid) * L1 + t];
        }
    } else if ((pid -= nE1b) < nE2w) {              // enc.w2[co][ci][tau]
        const int co = pid / (C1 * 3), ci = (pid / 3) % C1, tau = pid % 3;
        for (int64_t q = threadIdx.x; q < (int64_t)K * L2; q += kRedThreads) {
            const int64_t k = q / L2, t = q % L2;
            acc += (double)h[(k * C1 + ci) * L1 + 2 * t + tau] * (double)dz[(int64_t)co * L2 + t];
        }
    } else if ((pid -= nE2w) < nE2b) {              // enc.b2[co]
        for (int64_t q = threadIdx.x; q < (int64_t)K * L2; q += kRedThreads)
            acc += (double)dz[(int64_t)pid * L2 + q % L2];
    } else if ((pid -= nE2b) < nD1w) {              // dec.w1[c2][ci][tau]
        const int c2 = pid / (C1 * 3), ci = (pid / 3) % C1, tau = pid % 3;
        for (int64_t j = threadIdx.x; j < L2; j += kRedThreads)
            acc += (double)zbar[(int64_t)c2 * L2 + j] * (double)dd[(int64_t)ci * L1 + 2 * j + tau];
    } else if ((pid -= nD1w) < nD1b) {              // dec.b1[ci]
        for (int64_t i = threadIdx.x; i < L1; i += kRedThreads) acc += (double)dd[(int64_t)pid * L1 + i];
    } else if ((pid -= nD1b) < nD2w) {              // dec.w2[ci][0][tau]
        const int ci = pid / 3, tau = pid % 3;
        for (int64_t i = threadIdx.x; i < L1; i += kRedThreads)
            acc += (double)d[(int64_t)ci * L1 + i] * (double)dr[2 * i + tau];
    } else {                                        // dec.b2
        for (int64_t p = threadIdx.x; p < mu; p += kRedThreads) acc += (double)dr[p];
    }
    const double g = block_sum(acc, warp_part);
    if (threadIdx.x == 0) {
        const int i = blockIdx.x;
        const double m = ad.beta1 * (double)ad.m[i] + (1.0 - ad.beta1) * g;
        const double v = ad.beta2 * (double)ad.v[i] + (1.0 - ad.beta2) * g * g;
        ad.m[i] = (float)m;
        ad.v[i] = (float)v;
        ad.params[i] = (float)((double)ad.params[i] - ad.lr * (m / ad.corr1) / (sqrt(v / ad.corr2) + ad.eps));
    }
}

__global__ void loss_finalize_kernel(const double *__restrict__ part, int n, int64_t mu, float *__restrict__ out)
{
    __shared__ double warp_part[kRedThreads / 32];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += kRedThreads) acc += part[i];
    const double tot = block_sum(acc, warp_part);
    if (threadIdx.x == 0) *out = (float)(tot / (double)mu);
}

inline unsigned blocks_for(int64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

template <int C1, int C2>
cudaError_t train_step(Ctx &c, float *loss_out, const AdamArgs &ad)
{
    cudaStream_t s = c.stream;
    const float *enc = c.params, *dec = c.params + c.Penc;
    const float *dec_w2 = dec + C2 * C1 * 3 + C1;
    fwd_enc1_kernel<C1><<<dim3(blocks_for(c.L1, kTrThreads), c.K), kTrThreads, 0, s>>>(c.val, c.mu, c.L1, enc, c.t_h), ++g_kernel_launches;
    fwd_enc2_mean_kernel<C1, C2><<<blocks_for(c.L2, kTrThreads), kTrThreads, 0, s>>>(c.t_h, c.K, c.L1, c.L2, enc, c.combined), ++g_kernel_launches;
    fwd_dec1_kernel<C1, C2><<<blocks_for(c.L1, kTrThreads), kTrThreads, 0, s>>>(c.combined, c.L1, c.L2, dec, 0, c.t_d), ++g_kernel_launches;
    fwd_dec2_loss_kernel<C1><<<c.t_loss_blocks, kTrThreads, 0, s>>>(c.t_d, c.val, c.K, c.mu, c.L1, dec_w2, c.recon,
                                                                     c.t_dr, c.t_loss_part), ++g_kernel_launches;
    bwd_dec2_kernel<C1><<<blocks_for(c.L1, kTrThreads), kTrThreads, 0, s>>>(c.t_dr, c.mu, c.t_d, c.L1, dec_w2, 0, c.t_dd), ++g_kernel_launches;
    bwd_dec1_kernel<C1, C2><<<blocks_for(c.L2, kTrThreads), kTrThreads, 0, s>>>(c.t_dd, (float)c.K, c.L1, c.L2, dec, 0, c.t_dz), ++g_kernel_launches;
    bwd_enc2_kernel<C1, C2><<<dim3(blocks_for(c.L1, kTrThreads), c.K), kTrThreads, 0, s>>>(c.t_dz, 0, c.t_h, c.L1, c.L2, enc, c.t_dh), ++g_kernel_launches;
    param_grad_adam_kernel<C1, C2><<<(unsigned)c.P, kRedThreads, 0, s>>>(c.val, c.t_h, c.combined, c.t_d, c.t_dr, c.t_dd,
                                                                        c.t_dz, c.t_dh, c.K, c.mu, c.L1, c.L2, ad), ++g_kernel_launches;
    if (loss_out) loss_finalize_kernel<<<1, kRedThreads, 0, s>>>(c.t_loss_part, c.t_loss_blocks, c.mu, loss_out), ++g_kernel_launches;
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Parameter server (Section IV-A): L = lam_rec L_rec + lam_sim L_sim.  All nodes' vectors are
// encoded; L_sim = sum over ordered pairs k != m of ||z_k - z_m||^2 / (C2 L2); the code of the
// common node goes through every node's decoder together with that node's innovation and
// L_rec = sum_k ||g~_k - g~^rec_k||^2 / mu.
// ------------------------------------------------------------------------------------------
// z_k for every node, their node-ordered sum, and this CTA's part of the pair sum.
template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
ps_fwd_enc2_kernel(const float *__restrict__ h, int K, int64_t L1, int64_t L2, const float *__restrict__ params,
                   float *__restrict__ z, float *__restrict__ zsum, double *__restrict__ sim_part)
{
    constexpr int kW = C2 * C1 * 3 + C2;
    __shared__ float w[kW];
    __shared__ double warp_part[kTrThreads / 32];
    for (int i = threadIdx.x; i < kW; i += kTrThreads) w[i] = params[C1 * 4 + i];
    __syncthreads();
    const int64_t t = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    double pairs = 0.0;
    if (t < L2) {
        float sum[C2];
        for (int k = 0; k < K; ++k) {
            float zk[C2];
#pragma unroll
            for (int co = 0; co < C2; ++co) zk[co] = w[C2 * C1 * 3 + co];
#pragma unroll
            for (int ci = 0; ci < C1; ++ci) {
                const float *hp = h + ((int64_t)k * C1 + ci) * L1 + 2 * t;
                const float h0 = hp[0], h1 = hp[1], h2 = hp[2];
#pragma unroll
                for (int co = 0; co < C2; ++co) {
                    zk[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 0], h0, zk[co]);
                    zk[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 1], h1, zk[co]);
                    zk[co] = __fmaf_rn(w[(co * C1 + ci) * 3 + 2], h2, zk[co]);
                }
            }
#pragma unroll
            for (int co = 0; co < C2; ++co) {
                z[((int64_t)k * C2 + co) * L2 + t] = zk[co];
                sum[co] = k == 0 ? zk[co] : __fadd_rn(sum[co], zk[co]);
                // the pairs (k, m) and (m, k) for every earlier node m: this thread wrote z_m itself
                for (int m = 0; m < k; ++m) {
                    const double df = (double)zk[co] - (double)z[((int64_t)m * C2 + co) * L2 + t];
                    pairs += 2.0 * df * df;
                }
            }
        }
#pragma unroll
        for (int co = 0; co < C2; ++co) zsum[(int64_t)co * L2 + t] = sum[co];
    }
    const double tot = block_sum(pairs, warp_part);
    if (threadIdx.x == 0) sim_part[blockIdx.x] = tot;
}

// Offsets inside one node's decoder parameters: w1[c2][c1][3], b1[c1], w2[c1][1][3], b2, (w0, w1, b).
template <int C1, int C2>
struct PsDec {
    static constexpr int kW2 = C2 * C1 * 3 + C1, kB2 = kW2 + C1 * 3, kFuse = kB2 + 1, kSize = kFuse + 3;
};

// Second decoder layer, fusion with the innovation, reconstruction error of every node.
// Grid (blocks over mu, K).  dy = w0 * dr is the gradient at the decoder stack's output.
template <int C1, int C2>
__global__ void __launch_bounds__(kTrThreads)
ps_fwd_dec2_loss_kernel(const float *__restrict__ d, const float *__restrict__ val, const float *__restrict__ inn,
                        int64_t mu, int64_t L1, const float *__restrict__ dec, float lam_rec, float *__restrict__ y_out,
                        float *__restrict__ recon, float *__restrict__ dr, float *__restrict__ dy,
                        double *__restrict__ rec_part)
{
    using D = PsDec<C1, C2>;
    __shared__ float w[C1 * 3 + 4];
    __shared__ double warp_part[kTrThreads / 32];
    const int k = blockIdx.y;
    dec += (int64_t)k * D::kSize;
    for (int i = threadIdx.x; i < C1 * 3 + 4; i += kTrThreads) w[i] = dec[D::kW2 + i];   // w2, b2, w0, w1, b
    __syncthreads();
    d += (int64_t)k * C1 * L1;
    const int64_t p = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    double sq = 0.0;
    if (p < mu) {
        float y = w[C1 * 3];
        for (int tau = (int)(p & 1); tau < 3; tau += 2) {
            const int64_t i = (p - tau) >> 1;
            if (p < tau || i >= L1) continue;
#pragma unroll
            for (int ci = 0; ci < C1; ++ci) y = __fmaf_rn(w[ci * 3 + tau], d[(int64_t)ci * L1 + i], y);
        }
        const float w0 = w[C1 * 3 + 1], w1 = w[C1 * 3 + 2], b = w[C1 * 3 + 3];
        const int64_t o = (int64_t)k * mu + p;
        const float r = __fmaf_rn(w1, inn[o], __fmaf_rn(w0, y, b));
        const float diff = __fsub_rn(r, val[o]);
        const float g = __fmul_rn(lam_rec, __fdiv_rn(__fmul_rn(2.0f, diff), (float)mu));
        y_out[o] = y;
        recon[o] = r;
        dr[o] = g;
        dy[o] = __fmul_rn(w0, g);
        sq = (double)diff * (double)diff;
    }
    const double tot = block_sum(sq, warp_part);
    if (threadIdx.x == 0) rec_part[(int64_t)k * gridDim.x + blockIdx.x] = tot;
}

// dz_k = lam_sim * 4 (K z_k - sum_m z_m) / (C2 L2), plus, for the common node, the decoders'
// gradients at the code, added in node order.  Grid (blocks over C2 L2, K).
__global__ void __launch_bounds__(kTrThreads)
ps_dz_kernel(const float *__restrict__ z, const float *__restrict__ zsum, const float *__restrict__ dzc, int K,
             int64_t nz, int common, float lam_sim, float *__restrict__ dz)
{
    const int k = blockIdx.y;
    const int64_t e = (int64_t)blockIdx.x * kTrThreads + threadIdx.x;
    if (e >= nz) return;
    const float pull = __fsub_rn(__fmul_rn((float)K, z[(int64_t)k * nz + e]), zsum[e]);
    float g = __fmul_rn(lam_sim, __fdiv_rn(__fmul_rn(4.0f, pull), (float)nz));
    if (k == common) {
        float acc = dzc[e];
        for (int j = 1; j < K; ++j) acc = __fadd_rn(acc, dzc[(int64_t)j * nz + e]);
        g = __fadd_rn(g, acc);
    }
    dz[(int64_t)k * nz + e] = g;
}

// One CTA per parameter (encoder first, then node 0's decoder, node 1's, ...): reduce its
// gradient in fp64 in a fixed order, then apply Adam to it.  Reads no parameter.
template <int C1, int C2>
__global__ void __launch_bounds__(kRedThreads)
ps_param_grad_adam_kernel(const float *__restrict__ val, const float *__restrict__ h, const float *__restrict__ zc,
                          const float *__restrict__ d, const float *__restrict__ y, const float *__restrict__ inn,
                          const float *__restrict__ dr, const float *__restrict__ dy, const float *__restrict__ dd,
                          const float *__restrict__ dz, const float *__restrict__ dh, int K, int64_t mu, int64_t L1,
                          int64_t L2, AdamArgs ad)
{
    using D = PsDec<C1, C2>;
    constexpr int nE1w = C1 * 3, nE1b = C1, nE2w = C2 * C1 * 3, nE2b = C2, nEnc = nE1w + nE1b + nE2w + nE2b;
    __shared__ double warp_part[kRedThreads / 32];
    int pid = blockIdx.x;
    double acc = 0.0;
    if (pid < nE1w) {                               // enc.w1[ci][0][tau]
        const int ci = pid / 3, tau = pid % 3;
        for (int64_t q = threadIdx.x; q < (int64_t)K * L1; q += kRedThreads) {
            const int64_t k = q / L1, t = q % L1;
            acc += (double)val[k * mu + 2 * t + tau] * (double)dh[(k * C1 + ci) * L1 + t];
        }
    } else if ((pid -= nE1w) < nE1b) {              // enc.b1[ci]
        for (int64_t q = threadIdx.x; q < (int64_t)K * L1; q += kRedThreads) {
            const int64_t k = q / L1, t = q % L1;
            acc += (double)dh[(k * C1 + pid) * L1 + t];
        }
    } else if ((pid -= nE1b) < nE2w) {              // enc.w2[co][ci][tau]
        const int co = pid / (C1 * 3), ci = (pid / 3) % C1, tau = pid % 3;
        for (int64_t q = threadIdx.x; q < (int64_t)K * L2; q += kRedThreads) {
            const int64_t k = q / L2, t = q % L2;
            acc += (double)h[(k * C1 + ci) * L1 + 2 * t + tau] * (double)dz[(k * C2 + co) * L2 + t];
        }
    } else if ((pid -= nE2w) < nE2b) {              // enc.b2[co]
        for (int64_t q = threadIdx.x; q < (int64_t)K * L2; q += kRedThreads) {
            const int64_t k = q / L2, t = q % L2;
            acc += (double)dz[(k * C2 + pid) * L2 + t];
        }
    } else {
        pid -= nE2b;
        const int k = pid / D::kSize;               // this node's decoder
        pid %= D::kSize;
        const float *ddk = dd + (int64_t)k * C1 * L1, *dk = d + (int64_t)k * C1 * L1;
        const float *drk = dr + (int64_t)k * mu, *dyk = dy + (int64_t)k * mu;
        if (pid < C2 * C1 * 3) {                    // dec_k.w1[c2][ci][tau]
            const int c2 = pid / (C1 * 3), ci = (pid / 3) % C1, tau = pid % 3;
            for (int64_t j = threadIdx.x; j < L2; j += kRedThreads)
                acc += (double)zc[(int64_t)c2 * L2 + j] * (double)ddk[(int64_t)ci * L1 + 2 * j + tau];
        } else if (pid < D::kW2) {                  // dec_k.b1[ci]
            const int ci = pid - C2 * C1 * 3;
            for (int64_t i = threadIdx.x; i < L1; i += kRedThreads) acc += (double)ddk[(int64_t)ci * L1 + i];
        } else if (pid < D::kB2) {                  // dec_k.w2[ci][0][tau]
            const int ci = (pid - D::kW2) / 3, tau = (pid - D::kW2) % 3;
            for (int64_t i = threadIdx.x; i < L1; i += kRedThreads)
                acc += (double)dk[(int64_t)ci * L1 + i] * (double)dyk[2 * i + tau];
        } else if (pid == D::kB2) {                 // dec_k.b2
            for (int64_t p = threadIdx.x; p < mu; p += kRedThreads) acc += (double)dyk[p];
        } else if (pid == D::kFuse) {               // w0_k: weight of the decoder stack's output
            for (int64_t p = threadIdx.x; p < mu; p += kRedThreads) acc += (double)drk[p] * (double)y[(int64_t)k * mu + p];
        } else if (pid == D::kFuse + 1) {           // w1_k: weight of the innovation
            for (int64_t p = threadIdx.x; p < mu; p += kRedThreads) acc += (double)drk[p] * (double)inn[(int64_t)k * mu + p];
        } else {                                    // b_k
            for (int64_t p = threadIdx.x; p < mu; p += kRedThreads) acc += (double)drk[p];
        }
    }
    (void)nEnc;
    const double g = block_sum(acc, warp_part);
    if (threadIdx.x == 0) {
        const int i = blockIdx.x;
        const double m = ad.beta1 * (double)ad.m[i] + (1.0 - ad.beta1) * g;
        const double v = ad.beta2 * (double)ad.v[i] + (1.0 - ad.beta2) * g * g;
        ad.m[i] = (float)m;
        ad.v[i] = (float)v;
        ad.params[i] = (float)((double)ad.params[i] - ad.lr * (m / ad.corr1) / (sqrt(v / ad.corr2) + ad.eps));
    }
}

__global__ void ps_loss_finalize_kernel(const double *__restrict__ rec_part, int n_rec, const double *__restrict__ sim_part,
                                        int n_sim, int64_t mu, int64_t nz, float lam_rec, float lam_sim,
                                        float *__restrict__ out)
{
    __shared__ double warp_part[kRedThreads / 32];
    double a = 0.0, b = 0.0;
    for (int i = threadIdx.x; i < n_rec; i += kRedThreads) a += rec_part[i];
    for (int i = threadIdx.x; i < n_sim; i += kRedThreads) b += sim_part[i];
    const double rec = block_sum(a, warp_part);
    __syncthreads();
    const double sim = block_sum(b, warp_part);
    if (threadIdx.x == 0) *out = (float)((double)lam_rec * rec / (double)mu + (double)lam_sim * sim / (double)nz);
}

template <int C1, int C2>
cudaError_t train_step_ps(Ctx &c, int common, float lam_rec, float lam_sim, float *loss_out, const AdamArgs &ad)
{
    using D = PsDec<C1, C2>;
    cudaStream_t s = c.stream;
    const float *enc = c.params, *dec = c.params + c.Penc;
    const int64_t nz = (int64_t)C2 * c.L2;
    const unsigned b1 = blocks_for(c.L1, kTrThreads), b2 = blocks_for(c.L2, kTrThreads), bmu = blocks_for(c.mu, kTrThreads);
    fwd_enc1_kernel<C1><<<dim3(b1, c.K), kTrThreads, 0, s>>>(c.val, c.mu, c.L1, enc, c.t_h), ++g_kernel_launches;
    ps_fwd_enc2_kernel<C1, C2><<<b2, kTrThreads, 0, s>>>(c.t_h, c.K, c.L1, c.L2, enc, c.code, c.t_zsum, c.t_sim_part), ++g_kernel_launches;
    cudaError_t e = launch_combine_ps(c, common);     // the common code and every node's innovation
    if (e != cudaSuccess) return e;
    fwd_dec1_kernel<C1, C2><<<dim3(b1, c.K), kTrThreads, 0, s>>>(c.combined, c.L1, c.L2, dec, D::kSize, c.t_d), ++g_kernel_launches;
    ps_fwd_dec2_loss_kernel<C1, C2><<<dim3(bmu, c.K), kTrThreads, 0, s>>>(c.t_d, c.val, c.inn, c.mu, c.L1, dec, lam_rec, c.t_y,
                                                                         c.recon, c.t_dr, c.t_dy, c.t_loss_part), ++g_kernel_launches;
    bwd_dec2_kernel<C1><<<dim3(b1, c.K), kTrThreads, 0, s>>>(c.t_dy, c.mu, c.t_d, c.L1, dec + D::kW2, D::kSize, c.t_dd), ++g_kernel_launches;
    bwd_dec1_kernel<C1, C2><<<dim3(b2, c.K), kTrThreads, 0, s>>>(c.t_dd, 1.0f, c.L1, c.L2, dec, D::kSize, c.t_dzc), ++g_kernel_launches;
    ps_dz_kernel<<<dim3(blocks_for(nz, kTrThreads), c.K), kTrThreads, 0, s>>>(c.code, c.t_zsum, c.t_dzc, c.K, nz, common, lam_sim,
                                                                              c.t_dz), ++g_kernel_launches;
    bwd_enc2_kernel<C1, C2><<<dim3(b1, c.K), kTrThreads, 0, s>>>(c.t_dz, nz, c.t_h, c.L1, c.L2, enc, c.t_dh), ++g_kernel_launches;
    ps_param_grad_adam_kernel<C1, C2><<<(unsigned)c.P, kRedThreads, 0, s>>>(c.val, c.t_h, c.combined, c.t_d, c.t_y, c.inn, c.t_dr,
                                                                           c.t_dy, c.t_dd, c.t_dz, c.t_dh, c.K, c.mu, c.L1, c.L2, ad),
        ++g_kernel_launches;
    if (loss_out)
        ps_loss_finalize_kernel<<<1, kRedThreads, 0, s>>>(c.t_loss_part, (int)(bmu * c.K), c.t_sim_part, (int)b2, c.mu, nz, lam_rec,
                                                          lam_sim, loss_out), ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace

AdamArgs next_adam(Ctx &c)
{
    c.adam_t += 1;
    AdamArgs ad;
    ad.params = c.params; ad.m = c.adam_m; ad.v = c.adam_v;
    ad.lr = c.lr; ad.beta1 = c.beta1; ad.beta2 = c.beta2; ad.eps = c.eps;
    ad.corr1 = 1.0 - pow(c.beta1, (double)c.adam_t);
    ad.corr2 = 1.0 - pow(c.beta2, (double)c.adam_t);
    return ad;
}

cudaError_t launch_train_step_ps(Ctx &c, int common, float lam_rec, float lam_sim, float *loss_out)
{
    const AdamArgs ad = next_adam(c);
    const int c1 = c.cfg.ae_c1, c2 = c.cfg.ae_c2;
    if (c1 == 8 && c2 == 4) return train_step_ps<8, 4>(c, common, lam_rec, lam_sim, loss_out, ad);
    if (c1 == 16 && c2 == 8) return train_step_ps<16, 8>(c, common, lam_rec, lam_sim, loss_out, ad);
    if (c1 == 4 && c2 == 2) return train_step_ps<4, 2>(c, common, lam_rec, lam_sim, loss_out, ad);
    if (c1 == 3 && c2 == 2) return train_step_ps<3, 2>(c, common, lam_rec, lam_sim, loss_out, ad);
    return cudaErrorInvalidValue;
}

cudaError_t launch_train_step(Ctx &c, float *loss_out)
{
    const AdamArgs ad = next_adam(c);
    const int c1 = c.cfg.ae_c1, c2 = c.cfg.ae_c2;
    if (c1 == 8 && c2 == 4) return train_step<8, 4>(c, loss_out, ad);
    if (c1 == 16 && c2 == 8) return train_step<16, 8>(c, loss_out, ad);
    if (c1 == 4 && c2 == 2) return train_step<4, 2>(c, loss_out, ad);
    if (c1 == 3 && c2 == 2) return train_step<3, 2>(c, loss_out, ad);
    return cudaErrorInvalidValue;
}

}  // namespace lgc
