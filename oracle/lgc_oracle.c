/*
 * CPU oracle for the Learned Gradient Compression (LGC) per-step path.
 *
 * TEST INFRASTRUCTURE ONLY.  A plain, slow, single-threaded restatement of what the path
 * computes, written from the paper (arXiv 2103.08870) so that a reader can check each function
 * against the cited passage by eye.  It shares no code with the CUDA library and is never on a
 * product path: only tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Precision.  The residual/velocity buffers and every decision taken on them (which entries are
 * selected) are fp32, because those buffers ARE the method's fp32 state and are compared bit for
 * bit.  Everything downstream of the gather (autoencoder, combine, losses, optimiser) is
 * evaluated in fp64 on the fp32 inputs.
 *
 * Pins (tests/test_oracle_*.py): brute-force sort for the selection, closed forms and the
 * "sent + kept == accumulated" identity for the accumulation, torch's CPU conv1d /
 * conv_transpose1d and autograd for the convolutions and their gradients, adjointness,
 * finite differences for the training step, special weights for the parameter-server decoder.
 * PARITY UNPINNED: where the innovation joins a TWO-layer parameter-server decoder is a reading of
 * Section IV-C / Fig. 3(a), which define it for the six-layer decoder only.  What the reading
 * states -- decoder output and innovation concatenated, then a one-tap Conv1d(2 -> 1) -- is pinned:
 * lgc_oracle_ps_fuse against torch.cat + torch's conv1d with random per-node weights, and the
 * special weights that reduce it to either channel.  The reading itself no test can pin.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Section V-A: number of entries kept in a layer, mu_l = (alpha/100) n_l.
 * alpha is given in parts per million of n_l; rounded half up, at least 1, at most n_l.
 * ---------------------------------------------------------------------------------------- */
int64_t lgc_oracle_keep_count(int64_t n, uint32_t density_ppm)
{
    int64_t k = (n * (int64_t)density_ppm + 500000) / 1000000;
    if (k < 1) k = 1;
    if (k > n) k = n;
    return k;
}

/* Innovation count inside a layer's kept values: Algorithm 1 keeps their top tenth. */
int64_t lgc_oracle_innovation_count(int64_t k_l, uint32_t permille)
{
    int64_t ki = (k_l * (int64_t)permille + 500) / 1000;
    if (ki < 1) ki = 1;
    if (ki > k_l) ki = k_l;
    return ki;
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1 / Algorithm 2, local accumulation (the fresh gradient is added to what the node
 * still holds back), with the momentum correction that Section V-A borrows from Deep Gradient
 * Compression:
 *     u <- m u + g            (velocity)
 *     v <- v + u              (v: the accumulated gradient the selection then looks at)
 * fp32, the product-sum fused with one rounding.  m = 0 gives Algorithm 2 verbatim.
 * ---------------------------------------------------------------------------------------- */
void lgc_oracle_accumulate(float *u, float *v, const float *g, int64_t n, float m)
{
    for (int64_t j = 0; j < n; ++j) {
        u[j] = fmaf(m, u[j], g[j]);
        v[j] = v[j] + u[j];
    }
}

/* Magnitude key: the IEEE-754 bit pattern with the sign cleared.  For finite values the
 * integer order of keys is the order of |x|. */
static inline uint32_t mag_key(float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    return b & 0x7fffffffu;
}

typedef struct { uint32_t key; int32_t idx; } key_idx;

static int cmp_key_desc_idx_asc(const void *pa, const void *pb)
{
    const key_idx *a = (const key_idx *)pa, *b = (const key_idx *)pb;
    if (a->key != b->key) return a->key > b->key ? -1 : 1;
    if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
    return 0;
}

static int cmp_i32_asc(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1 / 2, magnitude threshold and mask of a layer (Section V-A: the alpha% entries of
 * highest magnitude), made exact: the k entries of largest magnitude, equal magnitudes resolved in favour of the
 * lower index, reported in ascending index order (plus `base`).
 * This is the definition written out: sort all (key, index) pairs, take the first k.
 * Returns 0, or -1 if memory ran out.
 * ---------------------------------------------------------------------------------------- */
int lgc_oracle_topk_sort(const float *v, int64_t n, int64_t k, int32_t base, int32_t *idx_out)
{
    key_idx *p = (key_idx *)malloc((size_t)n * sizeof *p);
    if (!p) return -1;
    for (int64_t j = 0; j < n; ++j) { p[j].key = mag_key(v[j]); p[j].idx = (int32_t)j; }
    qsort(p, (size_t)n, sizeof *p, cmp_key_desc_idx_asc);
    for (int64_t i = 0; i < k; ++i) idx_out[i] = base + p[i].idx;
    qsort(idx_out, (size_t)k, sizeof *idx_out, cmp_i32_asc);
    free(p);
    return 0;
}

/* k-th largest element of a[0..n) (k >= 1) by three-way-partition quickselect; a is permuted. */
static uint32_t kth_largest(uint32_t *a, int64_t n, int64_t k)
{
    int64_t lo = 0, hi = n - 1;          /* answer lies in a[lo..hi] */
    int64_t want = k - 1;                /* position in descending order */
    uint64_t rng = 0x2545F4914F6CDD1Dull;
    for (;;) {
        if (lo == hi) return a[lo];
        rng ^= rng << 13; rng ^= rng >> 7; rng ^= rng << 17;
        uint32_t pivot = a[lo + (int64_t)(rng % (uint64_t)(hi - lo + 1))];
        /* partition a[lo..hi] into  > pivot | == pivot | < pivot  */
        int64_t gt = lo, i = lo, lt = hi;
        while (i <= lt) {
            if (a[i] > pivot) { uint32_t t = a[i]; a[i] = a[gt]; a[gt] = t; ++gt; ++i; }
            else if (a[i] < pivot) { uint32_t t = a[i]; a[i] = a[lt]; a[lt] = t; --lt; }
            else ++i;
        }
        if (want < gt) hi = gt - 1;
        else if (want > lt) lo = lt + 1;
        else return pivot;
    }
}

/* ------------------------------------------------------------------------------------------
 * The same selection in linear time for large layers: find the k-th largest key T, keep every
 * entry with key > T, then the lowest-index entries with key == T until k are kept.
 * Pinned against lgc_oracle_topk_sort.
 * ---------------------------------------------------------------------------------------- */
int lgc_oracle_topk_select(const float *v, int64_t n, int64_t k, int32_t base, int32_t *idx_out)
{
    uint32_t *keys = (uint32_t *)malloc((size_t)n * sizeof *keys);
    if (!keys) return -1;
    for (int64_t j = 0; j < n; ++j) keys[j] = mag_key(v[j]);
    uint32_t T = kth_largest(keys, n, k);
    free(keys);
    int64_t above = 0;
    for (int64_t j = 0; j < n; ++j) above += mag_key(v[j]) > T;
    int64_t ties_wanted = k - above, out = 0;
    for (int64_t j = 0; j < n; ++j) {
        uint32_t key = mag_key(v[j]);
        if (key > T) idx_out[out++] = base + (int32_t)j;
        else if (key == T && ties_wanted > 0) { idx_out[out++] = base + (int32_t)j; --ties_wanted; }
    }
    return out == k ? 0 : -2;
}

/* Algorithm 1 / 2, masked gradient followed by the concatenation over layers: the kept values,
 * in index order, of one node. */
void lgc_oracle_gather(const float *v, const int32_t *idx, int64_t count, float *val)
{
    for (int64_t p = 0; p < count; ++p) val[p] = v[idx[p]];
}

/* Algorithm 1 / 2, residual update: only what the mask left out stays accumulated, so the sent
 * entries are zeroed; with momentum correction the velocity is masked the same way. */
void lgc_oracle_clear(float *u, float *v, const int32_t *idx, int64_t count)
{
    for (int64_t p = 0; p < count; ++p) { u[idx[p]] = 0.0f; v[idx[p]] = 0.0f; }
}

/* Algorithm 1, innovation: inside one layer's kept values val[0..k_l), keep the ki entries of
 * largest magnitude (ties: lower position), zero elsewhere. */
int lgc_oracle_innovation(const float *val, int64_t k_l, int64_t ki, float *inn)
{
    int32_t *pos = (int32_t *)malloc((size_t)ki * sizeof *pos);
    if (!pos) return -1;
    int rc = lgc_oracle_topk_sort(val, k_l, ki, 0, pos);
    for (int64_t p = 0; p < k_l; ++p) inn[p] = 0.0f;
    if (rc == 0) for (int64_t i = 0; i < ki; ++i) inn[pos[i]] = val[pos[i]];
    free(pos);
    return rc;
}

/* ==========================================================================================
 * Autoencoder (Section IV; the two-layer "lightweight" instance): 1-D convolutions with three
 * taps and stride two, no padding.  fp64.  Tensors are row-major [channel][position].
 * ======================================================================================== */

int64_t lgc_oracle_conv_len(int64_t lin) { return lin >= 3 ? (lin - 3) / 2 + 1 : 0; }
int64_t lgc_oracle_convt_len(int64_t lin, int out_pad) { return 2 * (lin - 1) + 3 + out_pad; }

/* y[co][t] = b[co] + sum_ci sum_tau w[co][ci][tau] x[ci][2t + tau],  t < (lin-3)/2 + 1 */
void lgc_oracle_conv1d(const double *x, int cin, int64_t lin, const double *w, const double *b,
                       int cout, double *y)
{
    int64_t lout = lgc_oracle_conv_len(lin);
    for (int co = 0; co < cout; ++co)
        for (int64_t t = 0; t < lout; ++t) {
            double acc = b[co];
            for (int ci = 0; ci < cin; ++ci)
                for (int tau = 0; tau < 3; ++tau)
                    acc += w[(co * cin + ci) * 3 + tau] * x[ci * lin + 2 * t + tau];
            y[co * lout + t] = acc;
        }
}

/* Gradients of the convolution above for an upstream gradient dy[cout][lout]:
 * dx[ci][2t+tau] += w[co][ci][tau] dy[co][t];  dw[co][ci][tau] += x[ci][2t+tau] dy[co][t];
 * db[co] += dy[co][t].  dx is overwritten; dw and db are ADDED to (pass NULL to skip). */
void lgc_oracle_conv1d_bwd(const double *x, int cin, int64_t lin, const double *w, int cout,
                           const double *dy, double *dx, double *dw, double *db)
{
    int64_t lout = lgc_oracle_conv_len(lin);
    if (dx) for (int64_t i = 0; i < (int64_t)cin * lin; ++i) dx[i] = 0.0;
    for (int co = 0; co < cout; ++co)
        for (int64_t t = 0; t < lout; ++t) {
            double d = dy[co * lout + t];
            if (db) db[co] += d;
            for (int ci = 0; ci < cin; ++ci)
                for (int tau = 0; tau < 3; ++tau) {
                    if (dx) dx[ci * lin + 2 * t + tau] += w[(co * cin + ci) * 3 + tau] * d;
                    if (dw) dw[(co * cin + ci) * 3 + tau] += x[ci * lin + 2 * t + tau] * d;
                }
        }
}

/* Transposed convolution (the decoder's "deconvolution"), weight w[ci][co][tau]:
 * y[co][s] = b[co] + sum_ci sum_{i, tau : 2i + tau = s} w[ci][co][tau] x[ci][i],
 * s < 2(lin-1) + 3 + out_pad.  Written as the scatter it is defined by. */
void lgc_oracle_convt1d(const double *x, int cin, int64_t lin, const double *w, const double *b,
                        int cout, int out_pad, double *y)
{
    int64_t lout = lgc_oracle_convt_len(lin, out_pad);
    for (int co = 0; co < cout; ++co)
        for (int64_t s = 0; s < lout; ++s) y[co * lout + s] = b[co];
    for (int ci = 0; ci < cin; ++ci)
        for (int64_t i = 0; i < lin; ++i)
            for (int co = 0; co < cout; ++co)
                for (int tau = 0; tau < 3; ++tau)
                    y[co * lout + 2 * i + tau] += w[(ci * cout + co) * 3 + tau] * x[ci * lin + i];
}

/* Gradients of the transposed convolution: dx[ci][i] = sum w[ci][co][tau] dy[co][2i+tau];
 * dw[ci][co][tau] += x[ci][i] dy[co][2i+tau];  db[co] += dy[co][s] (all s). */
void lgc_oracle_convt1d_bwd(const double *x, int cin, int64_t lin, const double *w, int cout,
                            int out_pad, const double *dy, double *dx, double *dw, double *db)
{
    int64_t lout = lgc_oracle_convt_len(lin, out_pad);
    if (db) for (int co = 0; co < cout; ++co)
        for (int64_t s = 0; s < lout; ++s) db[co] += dy[co * lout + s];
    for (int ci = 0; ci < cin; ++ci)
        for (int64_t i = 0; i < lin; ++i) {
            double acc = 0.0;
            for (int co = 0; co < cout; ++co)
                for (int tau = 0; tau < 3; ++tau) {
                    double d = dy[co * lout + 2 * i + tau];
                    acc += w[(ci * cout + co) * 3 + tau] * d;
                    if (dw) dw[(ci * cout + co) * 3 + tau] += x[ci * lin + i] * d;
                }
            if (dx) dx[ci * lin + i] = acc;
        }
}

void lgc_oracle_relu(double *x, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) if (!(x[i] > 0.0)) x[i] = 0.0;
}

/* d <- d where the forward output y was positive, else 0 */
void lgc_oracle_relu_bwd(const double *y, double *d, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) if (!(y[i] > 0.0)) d[i] = 0.0;
}

/* Section IV-C / Fig. 3(a): the decoder output and the innovation are concatenated (2 channels)
 * and a 1x1 convolution with weights (w0, w1) and bias b maps them to the reconstruction. */
void lgc_oracle_ps_fuse(const double *y, const float *inn, int64_t n, double w0, double w1,
                        double b, double *r)
{
    for (int64_t p = 0; p < n; ++p) r[p] = w0 * y[p] + w1 * (double)inn[p] + b;
}

/* Adam (Kingma & Ba) with bias correction, step counter t >= 1, no weight decay. */
void lgc_oracle_adam(double *p, double *m, double *v, const double *g, int64_t n, int64_t t,
                     double lr, double beta1, double beta2, double eps)
{
    double c1 = 1.0 - pow(beta1, (double)t), c2 = 1.0 - pow(beta2, (double)t);
    for (int64_t i = 0; i < n; ++i) {
        m[i] = beta1 * m[i] + (1.0 - beta1) * g[i];
        v[i] = beta2 * v[i] + (1.0 - beta2) * g[i] * g[i];
        double mhat = m[i] / c1, vhat = v[i] / c2;
        p[i] -= lr * mhat / (sqrt(vhat) + eps);
    }
}
