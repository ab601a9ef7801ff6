// Device helpers shared by the selection kernels: magnitude keys, CTA-wide scans, the ordered
// emission rule, and the complete selection of one small segment by one CTA.
#pragma once

#include "lgc_internal.cuh"

namespace lgc {
namespace sel {

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

// Sum of x over threads with index < own (exclusive prefix sum); *total gets the CTA sum.  warp_tot: one slot per
// warp.  Every warp scans the warps' totals itself with shuffles: with each thread adding the totals up one by one
// (32 of them in a CTA of 1024 threads) this function was most of what a finishing CTA executed per tile of data.
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
    const T t = lane < (int)(blockDim.x >> 5) ? warp_tot[lane] : T(0);
    T s = t;                                      // inclusive scan of the warps' totals; lanes beyond them keep the CTA's sum
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T y = __shfl_up_sync(kFull, s, d);
        if (lane >= d) s += y;
    }
    const T before = __shfl_sync(kFull, s - t, warp);
    const T tot = __shfl_sync(kFull, s, 31);
    __syncthreads();                              // warp_tot may be written again
    if (total) *total = tot;
    return before + incl - x;
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
    int warp_tot[32];
    unsigned scan_tot[32];
    int found[2];
};

// Whole selection of segment `s` of row `row` by one CTA of at least kSelThreads threads (the
// first kSelThreads hold the keys; any further threads only take part in the barriers).
__device__ __forceinline__ void
select_small_body(const float *__restrict__ data, int64_t row_stride, int row0,
                  const int64_t *__restrict__ seg_off, const int32_t *__restrict__ seg_len,
                  const int32_t *__restrict__ seg_k, const int32_t *__restrict__ seg_out, int s, int row,
                  int32_t *__restrict__ out, int64_t out_stride, int32_t *errword, SmallShared &sh)
{
    int (&hist)[256] = sh.hist;
    int (&warp_tot)[32] = sh.warp_tot;
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
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i)
            if (i < valid && (key[i] & decided) == prefix) atomicAdd(&hist[(key[i] >> shift) & 0xff], 1);
        __syncthreads();
        const int mine = threadIdx.x < 256 ? hist[threadIdx.x] : 0;
        const int incl = block_suffix_incl(mine, warp_tot);
        if (threadIdx.x < 256 && incl >= k_rem && incl - mine < k_rem) {
            found[0] = threadIdx.x;
            found[1] = k_rem - (incl - mine);
        }
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

}  // namespace sel
}  // namespace lgc
