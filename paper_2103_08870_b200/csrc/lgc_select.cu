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
//  - segments of at most kSelChunk elements: one CTA does everything (keys live in registers);
//  - larger segments (launch_select): two reads of the data -- leading-digit histogram, then the
//    candidates at or above the k-th key's bucket -- and one finishing CTA per segment;
//  - launch_select_multipass: the same result from chunked passes over the data alone
//    (histogram/scan x3 -> count -> chunk scan -> emit), for callers with minimal work space.
#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kWarps = kSelThreads / 32;

__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// Thread t of a CTA takes elements [start + 16 t, start + 16 t + 16) of a segment of `len`
// elements; returns how many of them exist.  128-bit loads when the address allows.
__device__ __forceinline__ int load_keys16(const float *__restrict__ seg, int start, int len,
                                           uint32_t (&key)[kSelPerThread])
{
    const int j0 = start + (int)threadIdx.x * kSelPerThread;
    int valid = len - j0;
    valid = valid < 0 ? 0 : (valid > kSelPerThread ? kSelPerThread : valid);
    const float *p = seg + j0;
    if (valid == kSelPerThread && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
        const float4 *p4 = reinterpret_cast<const float4 *>(p);
#pragma unroll
        for (int q = 0; q < kSelPerThread / 4; ++q) {
            const float4 x = __ldg(p4 + q);
            key[4 * q + 0] = mag_key(x.x);
            key[4 * q + 1] = mag_key(x.y);
            key[4 * q + 2] = mag_key(x.z);
            key[4 * q + 3] = mag_key(x.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i) key[i] = i < valid ? mag_key(__ldg(p + i)) : 0u;
    }
    return valid;
}

// Sum of x over threads with index >= own (inclusive suffix sum) in the CTA; warp_tot: one slot per warp.
__device__ __forceinline__ int block_suffix_incl(int x, int *warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_down_sync(kFull, x, d);
        if (lane + d < 32) x += y;
    }
    if (lane == 0) warp_tot[warp] = x;
    __syncthreads();
    int add = 0;
    for (int w = warp + 1; w < (int)(blockDim.x >> 5); ++w) add += warp_tot[w];
    __syncthreads();
    return x + add;
}

// Sum of x over threads with index < own (exclusive prefix sum); *total gets the CTA sum.
template <typename T>
__device__ __forceinline__ T block_prefix_excl(T x, T *warp_tot, T *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T y = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    T add = 0, tot = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
        const T t = warp_tot[w];
        if (w < warp) add += t;
        tot += t;
    }
    __syncthreads();
    if (total) *total = tot;
    return add + incl - x;
}

// Ordered emission of one thread's selected entries.  gt_before / eq_before: entries of the
// segment before this thread's first element with key > T / key == T.
__device__ __forceinline__ void emit16(const uint32_t (&key)[kSelPerThread], int valid, uint32_t T,
                                       int r, int gt_before, int eq_before, int64_t first_index,
                                       int32_t *__restrict__ out, int k, int32_t *errword)
{
    int gt = gt_before, eq = eq_before;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i) {
        if (i < valid) {
            const uint32_t x = key[i];
            int pos = -1;
            if (x > T) {
                pos = gt + (eq < r ? eq : r);
                ++gt;
            } else if (x == T) {
                if (eq < r) pos = gt + eq;
                ++eq;
            }
            if (pos >= 0) {
                if (pos < k) out[pos] = (int32_t)(first_index + i);
                else atomicExch(errword, 0x5E10);   // would write past the segment's slots
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// small segments: one CTA per (segment, row)
// ------------------------------------------------------------------------------------------
struct alignas(16) SmallShared {
    int hist[256];
    int warp_tot[kWarps];
    unsigned scan_tot[kWarps];
    int found[2];
};

// Whole selection of segment `s` of row `row` by one CTA of kSelThreads threads.
__device__ __forceinline__ void
select_small_body(const float *__restrict__ data, int64_t row_stride, int row0,
                  const int64_t *__restrict__ seg_off, const int32_t *__restrict__ seg_len,
                  const int32_t *__restrict__ seg_k, const int32_t *__restrict__ seg_out, int s, int row,
                  int32_t *__restrict__ out, int64_t out_stride, int32_t *errword, SmallShared &sh)
{
    int (&hist)[256] = sh.hist;
    int (&warp_tot)[kWarps] = sh.warp_tot;
    int (&found)[2] = sh.found;
    const int64_t off = seg_off[s];
    const int len = seg_len[s], k = seg_k[s];
    const float *seg = data + (int64_t)(row0 + row) * row_stride + off;
    uint32_t key[kSelPerThread];
    const int valid = load_keys16(seg, 0, len, key);

    uint32_t prefix = 0, decided = 0;
    int k_rem = k;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        hist[threadIdx.x] = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i)
            if (i < valid && (key[i] & decided) == prefix) atomicAdd(&hist[(key[i] >> shift) & 0xff], 1);
        __syncthreads();
        const int mine = hist[threadIdx.x];
        const int incl = block_suffix_incl(mine, warp_tot);
        if (incl >= k_rem && incl - mine < k_rem) { found[0] = threadIdx.x; found[1] = k_rem - (incl - mine); }
        __syncthreads();
        prefix |= (uint32_t)found[0] << shift;
        decided |= 0xffu << shift;
        k_rem = found[1];
        __syncthreads();
    }
    const uint32_t T = prefix;
    const int r = k_rem;
    int gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if (i < valid) { gt += key[i] > T; eq += key[i] == T; }
    unsigned total;
    const unsigned before = block_prefix_excl<unsigned>((unsigned)gt | ((unsigned)eq << 16), sh.scan_tot, &total);
    emit16(key, valid, T, r, (int)(before & 0xffff), (int)(before >> 16),
           off + (int64_t)threadIdx.x * kSelPerThread, out + (int64_t)row * out_stride + seg_out[s], k, errword);
}

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

// ------------------------------------------------------------------------------------------
// large segments, two reads of the data:  histogram of the leading digit -> bucket of the k-th
// key -> every entry at or above that bucket becomes a candidate (positions kept per chunk, so
// index order survives) -> one CTA per segment compacts the candidates, finishes the radix
// search on them and emits.  Segments whose bucket holds too many entries (ties, e.g. a layer
// of zeros) are finished by the same CTA streaming over the data instead.
// ------------------------------------------------------------------------------------------
struct FastArgs {
    LargeArgs a;
    int32_t *cand_cnt;
    uint16_t *cand_pos;
    int32_t *seg_m;
    int32_t *seg_ticket;
    const int64_t *comp_off;
    int64_t comp_total;
    uint32_t *comp_key;
    int32_t *comp_idx;
};

constexpr int kFinThreads = 1024;
constexpr int kFinWarps = kFinThreads / 32;
constexpr int kFinSmemCap = 8192;     // candidates a finishing CTA keeps in shared memory
constexpr int kFinPerThread = 4;      // consecutive entries per thread in the ordered passes

// Keys of one chunk in striped order: key[4 q + j] is element 1024 q + 4 t + j of the chunk
// (thread t), so a warp reads 512 consecutive bytes per request.  Returns a 16-bit validity mask.
__device__ __forceinline__ unsigned load_keys_striped(const float *__restrict__ seg, int start, int len,
                                                      uint32_t (&key)[kSelPerThread])
{
    const float *p = seg + start;
    const bool vec = (reinterpret_cast<uintptr_t>(p) & 15) == 0;
    unsigned valid = 0;
#pragma unroll
    for (int q = 0; q < kSelPerThread / 4; ++q) {
        const int e = q * (kSelThreads * 4) + (int)threadIdx.x * 4;
        if (vec && start + e + 4 <= len) {
            const float4 x = __ldg(reinterpret_cast<const float4 *>(p + e));
            key[4 * q + 0] = mag_key(x.x);
            key[4 * q + 1] = mag_key(x.y);
            key[4 * q + 2] = mag_key(x.z);
            key[4 * q + 3] = mag_key(x.w);
            valid |= 0xfu << (4 * q);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = start + e + j < len;
                key[4 * q + j] = in ? mag_key(__ldg(p + e + j)) : 0u;
                valid |= (in ? 1u : 0u) << (4 * q + j);
            }
        }
    }
    return valid;
}

// Leading-digit histogram of one chunk, added to its segment's histogram.  The CTA that
// completes a segment (a ticket counter tells; nobody waits) finds the bucket d0 of the k-th key,
// the rank k_rem still to find inside it and the number m of entries at or above the bucket, and
// leaves histogram and ticket zeroed for the next call.
__global__ void __launch_bounds__(kSelThreads) hist0_fast_kernel(FastArgs f)
{
    const LargeArgs &a = f.a;
    constexpr int kPer = kHistBins / kSelThreads;
    __shared__ unsigned h[kHistBins];
    __shared__ int warp_tot[kWarps];
    __shared__ int is_last;
    const int row = blockIdx.y;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0;
    __syncthreads();
    const int li = a.chunk_large[blockIdx.x];
    const int s = a.large_ids[li];
    const int start = (blockIdx.x - a.large_chunk0[li]) * kSelChunk;
    const float *seg = a.data + (int64_t)(a.row0 + row) * a.row_stride + a.seg_off[s];
    uint32_t key[kSelPerThread];
    const unsigned valid = load_keys_striped(seg, start, a.seg_len[s], key);
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if (valid >> i & 1u) atomicAdd(&h[key[i] >> 20], 1u);
    __syncthreads();
    const int64_t slot = (int64_t)row * a.num_large + li;
    uint32_t *gh = a.hist + slot * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads)
        if (h[b]) atomicAdd(gh + b, h[b]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int chunks = a.large_chunk0[li + 1] - a.large_chunk0[li];
        is_last = atomicAdd(&f.seg_ticket[slot], 1) == chunks - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int k_rem = a.seg_k[s];
    int hh[kPer], part = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        hh[i] = (int)__ldcg(gh + threadIdx.x * kPer + i);
        part += hh[i];
    }
#pragma unroll
    for (int i = 0; i < kPer; ++i) gh[threadIdx.x * kPer + i] = 0u;
    if (threadIdx.x == 0) f.seg_ticket[slot] = 0;
    const int incl = block_suffix_incl(part, warp_tot);
    if (incl >= k_rem && incl - part < k_rem) {
        int above = incl - part;
#pragma unroll
        for (int i = kPer - 1; i >= 0; --i) {
            if (above + hh[i] >= k_rem) {
                a.prefix[slot] = (uint32_t)(threadIdx.x * kPer + i);
                a.k_rem[slot] = k_rem - above;
                f.seg_m[slot] = above + hh[i];
                break;
            }
            above += hh[i];
        }
    }
    if (threadIdx.x == 0 && incl < k_rem) atomicExch(a.errword, 0x5E40);
}

// Candidates of one chunk: positions (ascending) of the entries whose leading digit is at least
// the bucket's; skipped for segments that will be finished from the data.  The first num_small
// CTAs each select one small segment completely.
__global__ void __launch_bounds__(kSelThreads) collect_small_kernel(FastArgs f, const int32_t *__restrict__ small_ids, int num_small)
{
    const LargeArgs &a = f.a;
    __shared__ SmallShared small_sh;
    const int row = blockIdx.y;
    if ((int)blockIdx.x < num_small) {          // the longer-running CTAs go first
        select_small_body(a.data, a.row_stride, a.row0, a.seg_off, a.seg_len, a.seg_k, a.seg_out,
                          small_ids[blockIdx.x], row, a.out, a.out_stride, a.errword, small_sh);
        return;
    }
    const int chunk = (int)blockIdx.x - num_small;
    unsigned long long *warp_tot = reinterpret_cast<unsigned long long *>(small_sh.hist);
    const int li = a.chunk_large[chunk];
    const int64_t slot = (int64_t)row * a.num_large + li;
    if ((int64_t)f.seg_m[slot] > f.comp_off[li + 1] - f.comp_off[li]) return;
    const int s = a.large_ids[li];
    const int start = (chunk - a.large_chunk0[li]) * kSelChunk;
    const float *seg = a.data + (int64_t)(a.row0 + row) * a.row_stride + a.seg_off[s];
    uint32_t key[kSelPerThread];
    const unsigned valid = load_keys_striped(seg, start, a.seg_len[s], key);
    const uint32_t d0 = a.prefix[slot];
    unsigned flags = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if ((valid >> i & 1u) && (key[i] >> 20) >= d0) flags |= 1u << i;
    // per-stripe counts packed into four 16-bit fields, one CTA-wide scan for all four
    unsigned long long mine = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) mine |= (unsigned long long)__popc(flags >> (4 * q) & 0xfu) << (16 * q);
    unsigned long long total;
    const unsigned long long before = block_prefix_excl<unsigned long long>(mine, warp_tot, &total);
    const int64_t c = (int64_t)row * a.num_chunks + chunk;
    if (threadIdx.x == 0)
        f.cand_cnt[c] = (int)((total & 0xffff) + (total >> 16 & 0xffff) + (total >> 32 & 0xffff) + (total >> 48));
    if (flags) {
        uint16_t *dst = f.cand_pos + c * kSelChunk;
        unsigned stripe_base = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            unsigned at = stripe_base + (unsigned)(before >> (16 * q) & 0xffff);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (flags >> (4 * q + j) & 1u) dst[at++] = (uint16_t)(q * (kSelThreads * 4) + threadIdx.x * 4 + j);
            stripe_base += (unsigned)(total >> (16 * q) & 0xffff);
        }
    }
}

// Where a finishing CTA reads its entries from: the compacted candidates or the segment itself.
struct CompactSource {
    const uint32_t *key;
    const int32_t *idx;
    int n;
    __device__ __forceinline__ uint32_t key_at(int i) const { return key[i]; }
    __device__ __forceinline__ int32_t idx_at(int i) const { return idx[i]; }
};
struct DataSource {
    const float *seg;
    int64_t off;
    int n;
    __device__ __forceinline__ uint32_t key_at(int i) const { return mag_key(__ldg(seg + i)); }
    __device__ __forceinline__ int32_t idx_at(int i) const { return (int32_t)(off + i); }
};

struct FinishShared {
    int hist[256];
    int warp_i[kFinWarps];
    unsigned warp_u[kFinWarps];
    int found[2];
};

// Completes the radix search below the 11-bit bucket d0 (k_rem entries still to find inside it)
// and emits the k selected offsets in order.  Entries below the bucket, if the source has any,
// are ignored.
template <typename Source>
__device__ void finish_from(const Source &src, uint32_t d0, int k_rem, int k, int32_t *__restrict__ out,
                            FinishShared &sh, int32_t *errword)
{
    uint32_t prefix = d0 << 20, decided = 0x7ff00000u;
    const int shifts[3] = {12, 4, 0};
    const uint32_t masks[3] = {0xffu, 0xffu, 0xfu};
#pragma unroll 1
    for (int p = 0; p < 3; ++p) {
        if (threadIdx.x < 256) sh.hist[threadIdx.x] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < src.n; i += kFinThreads) {
            const uint32_t x = src.key_at(i);
            if ((x & decided) == prefix) atomicAdd(&sh.hist[(x >> shifts[p]) & masks[p]], 1);
        }
        __syncthreads();
        const int mine = threadIdx.x < 256 ? sh.hist[threadIdx.x] : 0;
        const int incl = block_suffix_incl(mine, sh.warp_i);
        if (threadIdx.x < 256 && incl >= k_rem && incl - mine < k_rem) {
            sh.found[0] = threadIdx.x;
            sh.found[1] = k_rem - (incl - mine);
        }
        if (threadIdx.x == 0 && incl < k_rem) atomicExch(errword, 0x5E50 + p);
        __syncthreads();
        prefix |= (uint32_t)sh.found[0] << shifts[p];
        decided |= masks[p] << shifts[p];
        k_rem = sh.found[1];
        __syncthreads();
    }
    const uint32_t T = prefix;
    const int r = k_rem;
    int gt_done = 0, eq_done = 0;            // entries before the current tile
    const int tile = kFinThreads * kFinPerThread;
    for (int base = 0; base < src.n; base += tile) {
        uint32_t key[kFinPerThread];
        const int first = base + (int)threadIdx.x * kFinPerThread;
        unsigned gt = 0, eq = 0;
#pragma unroll
        for (int i = 0; i < kFinPerThread; ++i) {
            key[i] = first + i < src.n ? src.key_at(first + i) : 0u;
            if (first + i < src.n) { gt += key[i] > T; eq += key[i] == T; }
        }
        unsigned total;
        const unsigned before = block_prefix_excl<unsigned>(gt | (eq << 16), sh.warp_u, &total);
        int g = gt_done + (int)(before & 0xffff), e = eq_done + (int)(before >> 16);
#pragma unroll
        for (int i = 0; i < kFinPerThread; ++i) {
            if (first + i < src.n) {
                int pos = -1;
                if (key[i] > T) { pos = g + (e < r ? e : r); ++g; }
                else if (key[i] == T) { if (e < r) pos = g + e; ++e; }
                if (pos >= 0) {
                    if (pos < k) out[pos] = src.idx_at(first + i);
                    else atomicExch(errword, 0x5E60);
                }
            }
        }
        gt_done += (int)(total & 0xffff);
        eq_done += (int)(total >> 16);
        if (gt_done + (eq_done < r ? eq_done : r) >= k) break;     // everything is emitted
    }
}

__global__ void __launch_bounds__(kFinThreads) finish_kernel(FastArgs f)
{
    const LargeArgs &a = f.a;
    __shared__ FinishShared sh;
    extern __shared__ __align__(16) uint32_t fin_dyn[];     // kFinSmemCap keys, then kFinSmemCap offsets
    uint32_t *s_key = fin_dyn;
    int32_t *s_idx = reinterpret_cast<int32_t *>(fin_dyn + kFinSmemCap);
    const int li = blockIdx.x, row = blockIdx.y;
    const int64_t slot = (int64_t)row * a.num_large + li;
    const int s = a.large_ids[li];
    const int64_t off = a.seg_off[s];
    const int len = a.seg_len[s], k = a.seg_k[s];
    const float *seg = a.data + (int64_t)(a.row0 + row) * a.row_stride + off;
    int32_t *out = a.out + (int64_t)row * a.out_stride + a.seg_out[s];
    const uint32_t d0 = a.prefix[slot];
    const int k_rem = a.k_rem[slot];
    const int m = f.seg_m[slot];
    const int64_t cap = f.comp_off[li + 1] - f.comp_off[li];
    if ((int64_t)m > cap) {                   // too many entries share the bucket: work on the data
        DataSource src{seg, off, len};
        finish_from(src, d0, k_rem, k, out, sh, a.errword);
        return;
    }
    // compact the candidates, chunk after chunk (thread t owns chunk t of a group of 1024 chunks)
    const bool in_smem = m <= kFinSmemCap;
    uint32_t *ckey = in_smem ? s_key : f.comp_key + (int64_t)row * f.comp_total + f.comp_off[li];
    int32_t *cidx = in_smem ? s_idx : f.comp_idx + (int64_t)row * f.comp_total + f.comp_off[li];
    const int c0 = a.large_chunk0[li], c1 = a.large_chunk0[li + 1];
    const int32_t *cnt = f.cand_cnt + (int64_t)row * a.num_chunks;
    int done = 0;
    for (int base = c0; base < c1; base += kFinThreads) {
        const int c = base + (int)threadIdx.x;
        const unsigned n = c < c1 ? (unsigned)cnt[c] : 0u;
        unsigned total;
        unsigned at = (unsigned)done + block_prefix_excl<unsigned>(n, sh.warp_u, &total);
        if (n) {
            // eight positions per 128-bit load, then eight independent gathers
            const uint4 *pos8 = reinterpret_cast<const uint4 *>(f.cand_pos + ((int64_t)row * a.num_chunks + c) * kSelChunk);
            const int chunk_start = (c - c0) * kSelChunk;
            for (unsigned q0 = 0; q0 < n; q0 += 8) {
                const uint4 pv = pos8[q0 >> 3];
                const unsigned w[4] = {pv.x, pv.y, pv.z, pv.w};
                uint32_t kk[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int j = chunk_start + (int)(w[q >> 1] >> (16 * (q & 1)) & 0xffffu);
                    kk[q] = q0 + q < n ? mag_key(__ldg(seg + j)) : 0u;
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q0 + q < n && at + q < (unsigned)m) {
                        ckey[at + q] = kk[q];
                        cidx[at + q] = (int32_t)(off + chunk_start + (int)(w[q >> 1] >> (16 * (q & 1)) & 0xffffu));
                    }
                }
                at += 8;
            }
        }
        done += (int)total;
    }
    if (threadIdx.x == 0 && done != m) atomicExch(a.errword, 0x5E70);
    __syncthreads();
    CompactSource src{ckey, cidx, m};
    finish_from(src, d0, k_rem, k, out, sh, a.errword);
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


cudaError_t launch_select(const SelectTables &t, const float *data, int64_t row_stride, int row0,
                          int rows, int32_t *out, int64_t out_stride, int32_t *errword, cudaStream_t st)
{
    if (rows <= 0 || t.num_segments == 0) return cudaSuccess;
    if (!t.cand_cnt && t.num_large)   // tables without the two-pass work space
        return launch_select_multipass(t, data, row_stride, row0, rows, out, out_stride, errword, st);
    if (!t.num_large) {
        select_small_kernel<<<dim3(t.num_small, rows), kSelThreads, 0, st>>>(
            data, row_stride, row0, t.seg_off, t.seg_len, t.seg_k, t.seg_out, t.small_ids, out, out_stride, errword), ++g_kernel_launches;
    } else {
        constexpr int kFinDyn = 2 * kFinSmemCap * (int)sizeof(uint32_t);
        static bool configured = false;
        if (!configured) {
            const cudaError_t e = cudaFuncSetAttribute(finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinDyn);
            if (e != cudaSuccess) return e;
            configured = true;
        }
        FastArgs f;
        LargeArgs &a = f.a;
        a.data = data; a.row_stride = row_stride; a.row0 = row0;
        a.seg_off = t.seg_off; a.seg_len = t.seg_len; a.seg_k = t.seg_k; a.seg_out = t.seg_out;
        a.large_ids = t.large_ids; a.large_chunk0 = t.large_chunk0; a.chunk_large = t.chunk_large;
        a.num_large = t.num_large; a.num_chunks = t.num_chunks;
        a.hist = t.hist; a.prefix = t.prefix; a.k_rem = t.k_rem; a.chunk_cnt = t.chunk_cnt;
        a.out = out; a.out_stride = out_stride; a.errword = errword;
        f.cand_cnt = t.cand_cnt; f.cand_pos = t.cand_pos; f.seg_m = t.seg_m; f.seg_ticket = t.seg_ticket;
        f.comp_off = t.comp_off;
        f.comp_total = t.comp_total; f.comp_key = t.comp_key; f.comp_idx = t.comp_idx;
        const dim3 gc(t.num_chunks, rows), gl(t.num_large, rows);
        hist0_fast_kernel<<<gc, kSelThreads, 0, st>>>(f), ++g_kernel_launches;
        collect_small_kernel<<<dim3(t.num_chunks + t.num_small, rows), kSelThreads, 0, st>>>(f, t.small_ids, t.num_small), ++g_kernel_launches;
        finish_kernel<<<gl, kFinThreads, kFinDyn, st>>>(f), ++g_kernel_launches;
    }
    return cudaGetLastError();
}

}  // namespace lgc
