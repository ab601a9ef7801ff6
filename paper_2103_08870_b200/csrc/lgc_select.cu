// Stage 2 of the LGC step: exact per-layer top-k by magnitude (Section V-A; the threshold and
// mask of Algorithm 1/2 made exact: exactly k_l entries, equal magnitudes go to the lower index),
// reported in ascending index order so that the concatenated vector g~ has a fixed order.
//
// Keys are the fp32 bit patterns with the sign cleared (integer order == order of |x|).
// For every (row, segment) the k-th largest key T and the number r of entries equal to T that
// still belong to the selection are found by a most-significant-digit radix search; entries are
// then emitted in index order by counting: an entry is selected iff key > T, or key == T and
// fewer than r equal keys precede it.  No sorting, no order-dependent atomics: the result is a
// pure function of the data.
//
// This file: launch_select_multipass, the selection from chunked passes over the data alone
// (histogram/scan x3 -> count -> chunk scan -> emit) with minimal work space; segments of at
// most kSelChunk elements are done by one CTA each (keys live in registers).  The path the
// step uses (fewer reads, candidates, fusion with the accumulation) is in lgc_select_fast.cu.
#include "lgc_select_common.cuh"

namespace lgc {

namespace {

using namespace sel;

__global__ void __launch_bounds__(kSelThreads)
select_small_kernel(const float *__restrict__ data, int64_t row_stride, int row0,
                    const int64_t *__restrict__ seg_off, const int32_t *__restrict__ seg_len,
                    const int32_t *__restrict__ seg_k, const int32_t *__restrict__ seg_out,
                    const int32_t *__restrict__ small_ids, int32_t *__restrict__ out,
                    int64_t out_stride, int32_t *errword)
{
    __shared__ SmallShared sh;
    select_small_body(data, row_stride, row0, seg_off, seg_len, seg_k, seg_out, small_ids[blockIdx.x], blockIdx.y,
                      out, out_stride, errword, sh);
}

// ------------------------------------------------------------------------------------------
// large segments
// ------------------------------------------------------------------------------------------
struct LargeArgs {
    const float *data;
    int64_t row_stride;
    int row0;
    const int64_t *seg_off;
    const int32_t *seg_len;
    const int32_t *seg_k;
    const int32_t *seg_out;
    const int32_t *large_ids;
    const int32_t *large_chunk0;
    const int32_t *chunk_large;
    int num_large;
    int num_chunks;
    uint32_t *hist;
    uint32_t *prefix;
    int32_t *k_rem;
    int2 *chunk_cnt;
    int32_t *out;
    int64_t out_stride;
    int32_t *errword;
};

__device__ __forceinline__ int chunk_keys(const LargeArgs &a, int chunk, int row, int &li, int &s,
                                          int &start, uint32_t (&key)[kSelPerThread])
{
    li = a.chunk_large[chunk];
    s = a.large_ids[li];
    start = (chunk - a.large_chunk0[li]) * kSelChunk;
    const float *seg = a.data + (int64_t)(a.row0 + row) * a.row_stride + a.seg_off[s];
    return load_keys16(seg, start, a.seg_len[s], key);
}

// PASS 0: digit = key bits 30..20; PASS 1: bits 19..10 of keys matching the 11-bit prefix;
// PASS 2: bits 9..0 of keys matching the 21-bit prefix.
template <int PASS>
__global__ void __launch_bounds__(kSelThreads) hist_kernel(LargeArgs a)
{
    __shared__ unsigned h[PASS == 0 ? kHistBins : 1];
    const int row = blockIdx.y;
    int li, s, start;
    uint32_t key[kSelPerThread];
    if (PASS == 0) {
        for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0;
        __syncthreads();
    }
    const int valid = chunk_keys(a, blockIdx.x, row, li, s, start, key);
    uint32_t *gh = a.hist + ((int64_t)row * a.num_large + li) * kHistBins;
    if (PASS == 0) {
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i)
            if (i < valid) atomicAdd(&h[key[i] >> 20], 1u);
        __syncthreads();
        for (int b = threadIdx.x; b < kHistBins; b += kSelThreads)
            if (h[b]) atomicAdd(gh + b, h[b]);
    } else {
        const uint32_t prefix = a.prefix[(int64_t)row * a.num_large + li];
        const int pshift = PASS == 1 ? 20 : 10;
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i)
            if (i < valid && (key[i] >> pshift) == prefix) atomicAdd(gh + ((key[i] >> (pshift - 10)) & 1023u), 1u);
    }
}

// One CTA per (large segment, row): finds the digit holding the k_rem-th largest key, extends
// the prefix, and leaves the histogram zeroed for the next pass / the next call.
template <int PASS>
__global__ void __launch_bounds__(kSelThreads) scan_kernel(LargeArgs a)
{
    constexpr int kBins = PASS == 0 ? kHistBins : 1024;
    constexpr int kPer = kBins / kSelThreads;
    __shared__ int warp_tot[kWarps];
    const int li = blockIdx.x, row = blockIdx.y;
    const int64_t slot = (int64_t)row * a.num_large + li;
    uint32_t *gh = a.hist + slot * kHistBins;
    const int k_rem = PASS == 0 ? a.seg_k[a.large_ids[li]] : a.k_rem[slot];
    const uint32_t prefix = PASS == 0 ? 0u : a.prefix[slot];
    int h[kPer], part = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) { h[i] = (int)gh[threadIdx.x * kPer + i]; part += h[i]; }
#pragma unroll
    for (int i = 0; i < kPer; ++i) gh[threadIdx.x * kPer + i] = 0u;
    const int incl = block_suffix_incl(part, warp_tot);
    if (incl >= k_rem && incl - part < k_rem) {
        int above = incl - part;
#pragma unroll
        for (int i = kPer - 1; i >= 0; --i) {
            if (above + h[i] >= k_rem) {
                a.prefix[slot] = (prefix << (PASS == 0 ? 0 : 10)) | (uint32_t)(threadIdx.x * kPer + i);
                a.k_rem[slot] = k_rem - above;
                break;
            }
            above += h[i];
        }
    }
    if (threadIdx.x == 0 && incl < k_rem) atomicExch(a.errword, 0x5E20 + PASS);   // histogram lost entries
}

__global__ void __launch_bounds__(kSelThreads) count_kernel(LargeArgs a)
{
    __shared__ unsigned warp_tot[kWarps];
    const int row = blockIdx.y;
    int li, s, start;
    uint32_t key[kSelPerThread];
    const int valid = chunk_keys(a, blockIdx.x, row, li, s, start, key);
    const uint32_t T = a.prefix[(int64_t)row * a.num_large + li];
    unsigned gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if (i < valid) { gt += key[i] > T; eq += key[i] == T; }
    unsigned total;
    block_prefix_excl<unsigned>(gt | (eq << 16), warp_tot, &total);
    if (threadIdx.x == 0)
        a.chunk_cnt[(int64_t)row * a.num_chunks + blockIdx.x] = make_int2((int)(total & 0xffff), (int)(total >> 16));
}

// One CTA per (large segment, row): exclusive prefix over the segment's chunk counts, in place.
__global__ void __launch_bounds__(kSelThreads) chunk_scan_kernel(LargeArgs a)
{
    __shared__ unsigned long long warp_tot[kWarps];
    const int li = blockIdx.x, row = blockIdx.y;
    const int c0 = a.large_chunk0[li], c1 = a.large_chunk0[li + 1];
    int2 *cnt = a.chunk_cnt + (int64_t)row * a.num_chunks;
    unsigned long long carry = 0;
    for (int base = c0; base < c1; base += kSelThreads) {
        const int c = base + threadIdx.x;
        int2 mine = make_int2(0, 0);
        if (c < c1) mine = cnt[c];
        unsigned long long total;
        const unsigned long long x = (unsigned long long)(unsigned)mine.x | ((unsigned long long)(unsigned)mine.y << 32);
        const unsigned long long before = carry + block_prefix_excl<unsigned long long>(x, warp_tot, &total);
        if (c < c1) cnt[c] = make_int2((int)(before & 0xffffffffu), (int)(before >> 32));
        carry += total;
    }
    if (threadIdx.x == 0) {
        const int64_t slot = (int64_t)row * a.num_large + li;
        const long long gt = (long long)(carry & 0xffffffffu), eq = (long long)(carry >> 32);
        const int r = a.k_rem[slot], k = a.seg_k[a.large_ids[li]];
        if (gt + r != k || eq < r) atomicExch(a.errword, 0x5E30);
    }
}

__global__ void __launch_bounds__(kSelThreads) emit_kernel(LargeArgs a)
{
    __shared__ unsigned warp_tot[kWarps];
    const int row = blockIdx.y;
    int li, s, start;
    uint32_t key[kSelPerThread];
    const int valid = chunk_keys(a, blockIdx.x, row, li, s, start, key);
    const int64_t slot = (int64_t)row * a.num_large + li;
    const uint32_t T = a.prefix[slot];
    const int r = a.k_rem[slot];
    const int2 chunk_before = a.chunk_cnt[(int64_t)row * a.num_chunks + blockIdx.x];
    unsigned gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if (i < valid) { gt += key[i] > T; eq += key[i] == T; }
    unsigned total;
    const unsigned before = block_prefix_excl<unsigned>(gt | (eq << 16), warp_tot, &total);
    if ((total & 0xffff) == 0 && chunk_before.y >= r) return;   // nothing of this chunk is selected
    emit16(key, valid, T, r, chunk_before.x + (int)(before & 0xffff), chunk_before.y + (int)(before >> 16),
           a.seg_off[s] + start + (int64_t)threadIdx.x * kSelPerThread,
           a.out + (int64_t)row * a.out_stride + a.seg_out[s], a.seg_k[s], a.errword);
}

}  // namespace

// Selection by full passes over the data only: small scratch (tables, one histogram per large
// segment, per-chunk counts), five reads of every large segment.
cudaError_t launch_select_multipass(const SelectTables &t, const float *data, int64_t row_stride, int row0,
                                    int rows, int32_t *out, int64_t out_stride, int32_t *errword, cudaStream_t st)
{
    if (rows <= 0 || t.num_segments == 0) return cudaSuccess;
    if (t.num_small) {
        select_small_kernel<<<dim3(t.num_small, rows), kSelThreads, 0, st>>>(
            data, row_stride, row0, t.seg_off, t.seg_len, t.seg_k, t.seg_out, t.small_ids, out, out_stride, errword), ++g_kernel_launches;
    }
    if (t.num_large) {
        LargeArgs a;
        a.data = data; a.row_stride = row_stride; a.row0 = row0;
        a.seg_off = t.seg_off; a.seg_len = t.seg_len; a.seg_k = t.seg_k; a.seg_out = t.seg_out;
        a.large_ids = t.large_ids; a.large_chunk0 = t.large_chunk0; a.chunk_large = t.chunk_large;
        a.num_large = t.num_large; a.num_chunks = t.num_chunks;
        a.hist = t.hist; a.prefix = t.prefix; a.k_rem = t.k_rem; a.chunk_cnt = t.chunk_cnt;
        a.out = out; a.out_stride = out_stride; a.errword = errword;
        const dim3 gc(t.num_chunks, rows), gl(t.num_large, rows);
        hist_kernel<0><<<gc, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        scan_kernel<0><<<gl, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        hist_kernel<1><<<gc, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        scan_kernel<1><<<gl, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        hist_kernel<2><<<gc, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        scan_kernel<2><<<gl, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        count_kernel<<<gc, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        chunk_scan_kernel<<<gl, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
        emit_kernel<<<gc, kSelThreads, 0, st>>>(a), ++g_kernel_launches;
    }
    return cudaGetLastError();
}


}  // namespace lgc
