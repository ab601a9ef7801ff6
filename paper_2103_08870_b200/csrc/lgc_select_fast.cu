// The selection path the LGC step uses (Section V-A of the paper: per layer, the alpha% entries
// of largest magnitude), built to touch the residual v as little as possible.
//
// A large segment (layer) of a row is cut where the row's 4096-element tiles cut it.  For every
// such chunk the positions of its CANDIDATES are kept, ascending: the entries whose leading key
// digit (11 bits: exponent + 3 mantissa bits) is at least a lower bucket.  One CTA per segment
// then compacts the candidates in index order, finishes the radix search on them and emits the
// k selected offsets by counting -- exact, ties to the lower index, no sorting.
//
// Where the candidates come from:
//  (a) fused: the accumulation kernel (accumulate_select_kernel, below) tests the freshly written
//      v of the selecting rows against a key PREDICTED from the previous step (a few per cent
//      below that step's k-th key) and histograms and lists the entries that pass.  The finishing
//      CTA checks that at least k entries passed; then v is not read again except at the candidates.
//  (b) without a usable prediction (first step, leader not announced, rows not 16-byte aligned):
//      hist0_fast_kernel histograms the segment, the CTA that completes it (a ticket counter
//      tells; nobody waits) finds the bucket of the k-th key, and collect_kernel lists the
//      entries from that bucket upwards: two reads of v.
// If a prediction turns out too high, or a segment's candidates exceed its compact capacity
// (ties, e.g. a layer of zeros), the finishing CTA works on the data itself.  The result is
// exact in every case.
#include "lgc_select_common.cuh"

namespace lgc {

namespace {

using namespace sel;

struct FastArgs {
    const float *data;
    int64_t row_stride;
    int row0;
    int num_large, num_small, num_tchunks;
    int fin_small;                 // small segments served by CTAs of finish_kernel (0 or num_small)
    int smem_keys;                 // candidate keys a finishing CTA can keep in its dynamic shared memory
    const int32_t *large_order;    // large segments, longest first: the order the finishing CTAs take them in
    const int2 *group_job;         // (large segment, first chunk) of every group that the wide kernels serve
    int num_group_jobs;
    int2 *job_range;               // [rows][groups] (candidates of the segment before the group, candidates of the group)
    int2 *job_cnt;                 // [rows][groups] (entries above the k-th key, entries equal to it)
    int32_t *seg_wide;             // [rows][num_large] 1: the wide kernels serve the segment in this step
    uint4 *zero_ptr;               // buffer the spare CTAs of the finishing launch clear (row 0 only), or nullptr
    uint64_t zero_vecs;            // its length in whole 16-byte units
    int zero_tail;                 // floats beyond them (0..3)
    int zero_ctas, zero_threads;   // spare CTAs that share the clearing, and how many of their threads store
    int32_t epoch;                 // step whose fused accumulation may have filled the lists (-1: none)
    const int64_t *seg_off;
    const int32_t *seg_len, *seg_k, *seg_out, *small_ids, *large_ids, *seg_large, *large_q0, *tchunk0, *tchunk_large;
    const int4 *tile_desc;
    const int64_t *dense_rng;      // (begin, end) of the runs of dense elements inside a row (layers kept out of u and v)
    int num_dense;
    uint32_t *hist, *prefix, *lbkey, *last_key;
    float2 *key_trend;
    int32_t *k_rem, *cand_cnt, *seg_m, *seg_ticket, *seg_epoch, *seg_path;
    uint2 *cand;                   // [rows][num_tchunks][kCandCap] candidates of a chunk: (key, position in tile), ascending position
    const int64_t *comp_off;
    int64_t comp_total;
    uint32_t *comp_key;
    int32_t *comp_idx;
    int32_t *out;
    int64_t out_stride;
    int32_t *errword;
};

// A finishing CTA has 512 threads and keeps up to 20480 candidate keys in shared memory (80 KB: two CTAs per SM).
// Two other shapes of the same kernel serve the extremes: when every segment can have an SM of its own (one
// selecting row of a ResNet: 53 segments), 1024 threads halve everything that is done per candidate; when there
// are many times more segments than SMs (every row selecting: 16 x 104), 256 threads and 6144 keys let four
// CTAs share an SM, and these latency-bound CTAs overlap twice as well.
constexpr int kFinThreads = 512;      // also the CTA size of the kernels that serve segments of several groups
constexpr int kFinWarps = kFinThreads / 32;
constexpr int kFinSmemCap = 20480;    // candidate keys in shared memory, 512- and 1024-thread shapes
constexpr int kFinSmemCapSmall = 6144;   // 256-thread shape
constexpr int kFinGroup = kSelGroup;  // chunks whose candidate counts are scanned together during the compaction
constexpr int kFinPerThread = 16;     // consecutive entries per thread in the ordered passes
constexpr int kCandCap = kSelCandCap;  // entries a chunk's list can hold; a chunk with more sends its segment to the data
// Spare CTAs that clear the update: at least about one per SM, each thread up to kZeroPerThread stores.  Up to
// kZeroGentleBytes only a quarter of a CTA's threads store: CTAs of 512 storing threads on every SM made the selecting
// CTAs beside them wait on the load/store path (their shared-memory searches took ~100 cycles a read), and a buffer of
// that size is cleared long before the selection is done anyway.  Larger buffers need every thread to reach the
// memory's write rate.
constexpr int kZeroCtasMin = 148;
constexpr int kZeroPerThread = 512;     // stores per thread, gentle form
constexpr int kZeroPerThreadFast = 8;   // large buffers: many short CTAs of 512 storing threads (4 GiB in 0.66 ms)
constexpr int kZeroGentleThreads = 128;
constexpr uint64_t kZeroGentleBytes = 512ull << 20;
constexpr int kAccThreads = 1024;     // accumulation: one 128-bit g/u/v triple per thread, 4096 elements per CTA

// The key from which the next step collects candidates, given this step's k-th key T.  Error
// feedback piles entries up just below the threshold (each 3 % below T holds about k more).  In
// steady state T itself moves by a per cent or two per step, but the rows differ: a row that led
// recently has had its own largest entries removed and sits a few per cent lower than one that
// has not.  6 % (10 % for k < 64, whose k-th key is noisier) below T keeps the candidates at
// 4-6 k and makes a prediction that is too high rare; when it happens only the fallback is paid.
// While the residual is still filling up (the first tens of steps of a run) T grows from step to
// step, by a factor r that itself shrinks towards 1 (about 1.8, 1.45, 1.35, ... 1.1 after a
// dozen steps on the synthetic gradients); the prediction follows with 60 % of the last growth
// beyond 10 %, which stays below the growth actually seen next.  Growth of less than 10 % is
// not followed: in steady state that is the difference between rows (leaders alternate), and
// chasing it put the prediction above the next key for most layers of a step every ~15 steps.
// Tprev = 0: no earlier key known.
__device__ __forceinline__ uint32_t predict_lbkey(uint32_t T, uint32_t Tprev, int k)
{
    float t = __uint_as_float(T);
    if (Tprev != 0 && T > Tprev) {
        float r = t / __uint_as_float(Tprev);
        r = r < 2.0f ? r : 2.0f;
        if (r > 1.1f) t *= 1.0f + 0.6f * (r - 1.1f);
    }
    t *= k >= 64 ? 0.94f : 0.90f;
    return __float_as_uint(t) & 0x7fffffffu;     // 0 (no prediction) when T is 0 or the product underflows
}

// After a selection: stores the k-th key T and the key from which the next accumulation collects candidates.
// Two rules, the higher key wins.  predict_lbkey above holds whatever the history.  The second rule trusts
// the key's own trend when that has been smooth: with every row selecting on its own residual (parameter
// server) the k-th key climbs by a ratio that shrinks slowly towards 1 (1.016 per step after 60 steps,
// 1.002 after 200 on the synthetic gradients) and never jumps, while a margin of 6 % below it ends up
// holding tens of times k entries (error feedback piles entries up just below the threshold: in steady
// state every per cent below T holds about 10 k of them).  So the next key is taken as T r^0.8 (r: the last
// ratio; a falling key is followed in full) and the margin as half the last move plus twice the largest
// recent jump of ln r (a maximum that decays by 15 % per step) plus 0.2 % (2 % for k < 64).  Where ratios
// jump by several per cent from step to step (ring-allreduce with alternating leaders) this margin comes
// out wider than the first rule's, which then decides.  failed: this step's prediction was too high.
__device__ __forceinline__ void store_prediction(const FastArgs &f, int64_t slot, uint32_t T, int k, bool failed)
{
    const uint32_t Tprev = f.last_key[slot];
    uint32_t lb = predict_lbkey(T, Tprev, k);
    float2 trend = f.key_trend[slot];
    if (Tprev != 0 && T != 0) {
        const float t = __uint_as_float(T);
        const float lnr = __logf(t / __uint_as_float(Tprev));
        trend.y = fmaxf(fabsf(lnr - trend.x), 0.85f * trend.y);
        if (failed) trend.y = fmaxf(trend.y, 0.05f);
        trend.x = lnr;
        const float margin = 0.5f * fabsf(lnr) + 2.0f * trend.y + (k >= 64 ? 0.002f : 0.02f);
        const float next = t * __expf((lnr > 0.0f ? 0.8f * lnr : lnr) - margin);
        const uint32_t lb2 = __float_as_uint(next) & 0x7fffffffu;
        if (next > 0.0f && lb2 > lb) lb = lb2;           // (may lie above T: the key is climbing)
    } else {
        trend = make_float2(0.0f, 1.0f);                  // no ratio yet: nothing to trust
    }
    f.key_trend[slot] = trend;
    f.lbkey[slot] = lb;
    f.last_key[slot] = T;
}

// Geometry of tile-chunk c: the part [lo, hi) of tile q (positions inside the tile) that belongs
// to large segment li.
struct ChunkGeom {
    int li, s, q, lo, hi;
};
__device__ __forceinline__ ChunkGeom chunk_geom(const FastArgs &f, int c)
{
    ChunkGeom g;
    g.li = f.tchunk_large[c];
    g.s = f.large_ids[g.li];
    g.q = f.large_q0[g.li] + (c - f.tchunk0[g.li]);
    const int64_t tile_base = (int64_t)g.q * kSelChunk, off = f.seg_off[g.s], end = off + f.seg_len[g.s];
    g.lo = off > tile_base ? (int)(off - tile_base) : 0;
    g.hi = end - tile_base < kSelChunk ? (int)(end - tile_base) : kSelChunk;
    return g;
}

// Keys of the tile at `tile` in striped order: key[4 r + j] is position 1024 r + 4 t + j (thread
// t of 256), so a warp reads 512 consecutive bytes per request.  Only positions in [lo, hi) are
// loaded; returns their 16-bit validity mask.
__device__ __forceinline__ unsigned load_keys_tile(const float *__restrict__ tile, int lo, int hi,
                                                   uint32_t (&key)[kSelPerThread])
{
    const bool vec = (reinterpret_cast<uintptr_t>(tile) & 15) == 0;
    unsigned valid = 0;
#pragma unroll
    for (int r = 0; r < kSelPerThread / 4; ++r) {
        const int e = r * (kSelThreads * 4) + (int)threadIdx.x * 4;
        if (vec && e >= lo && e + 4 <= hi) {
            const float4 x = __ldg(reinterpret_cast<const float4 *>(tile + e));
            key[4 * r + 0] = mag_key(x.x);
            key[4 * r + 1] = mag_key(x.y);
            key[4 * r + 2] = mag_key(x.z);
            key[4 * r + 3] = mag_key(x.w);
            valid |= 0xfu << (4 * r);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = e + j >= lo && e + j < hi;
                key[4 * r + j] = in ? mag_key(__ldg(tile + e + j)) : 0u;
                valid |= (in ? 1u : 0u) << (4 * r + j);
            }
        }
    }
    return valid;
}

// Run by every thread of the CTA that completed a segment's leading-digit histogram: finds the
// bucket d0 of the k-th largest key, stores d0, the rank still to find inside d0 and the number
// of entries from d0 upwards (the candidates), and leaves histogram and ticket zeroed.  Returns
// false if the histogram holds fewer than k entries.
template <int THREADS>
__device__ __forceinline__ bool bucket_scan(const FastArgs &f, int64_t slot, int k, int *warp_tot, int *flag)
{
    constexpr int kPer = kHistBins / THREADS;
    uint32_t *gh = f.hist + slot * kHistBins;
    int hh[kPer], part = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        hh[i] = (int)__ldcg(gh + threadIdx.x * kPer + i);
        part += hh[i];
    }
#pragma unroll
    for (int i = 0; i < kPer; ++i) gh[threadIdx.x * kPer + i] = 0u;
    if (threadIdx.x == 0) {
        f.seg_ticket[slot] = 0;
        *flag = 0;
    }
    const int incl = block_suffix_incl(part, warp_tot);      // two barriers inside: *flag = 0 is visible
    if (incl >= k && incl - part < k) {
        int above = incl - part;
#pragma unroll
        for (int i = kPer - 1; i >= 0; --i) {
            if (above + hh[i] >= k) {
                f.prefix[slot] = (uint32_t)(threadIdx.x * kPer + i);
                f.k_rem[slot] = k - above;
                f.seg_m[slot] = above + hh[i];
                *flag = 1;
                break;
            }
            above += hh[i];
        }
    }
    __syncthreads();
    return *flag != 0;
}

// (b) Leading-digit histogram of one tile-chunk; the CTA that completes a segment settles it.
__global__ void __launch_bounds__(kSelThreads) hist0_fast_kernel(FastArgs f)
{
    __shared__ unsigned h[kHistBins];
    __shared__ int warp_tot[kWarps];
    __shared__ int is_last, scan_flag;
    const int row = blockIdx.y;
    const ChunkGeom g = chunk_geom(f, blockIdx.x);
    const int64_t slot = (int64_t)row * f.num_large + g.li;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads) h[b] = 0;
    __syncthreads();
    const float *tile = f.data + (int64_t)(f.row0 + row) * f.row_stride + (int64_t)g.q * kSelChunk;
    uint32_t key[kSelPerThread];
    const unsigned valid = load_keys_tile(tile, g.lo, g.hi, key);
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if (valid >> i & 1u) atomicAdd(&h[key[i] >> 20], 1u);
    __syncthreads();
    uint32_t *gh = f.hist + slot * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kSelThreads)
        if (h[b]) atomicAdd(gh + b, h[b]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int chunks = f.tchunk0[g.li + 1] - f.tchunk0[g.li];
        is_last = atomicAdd(&f.seg_ticket[slot], 1) == chunks - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const bool ok = bucket_scan<kSelThreads>(f, slot, f.seg_k[g.s], warp_tot, &scan_flag);
    if (threadIdx.x == 0) {
        if (ok) f.seg_epoch[slot] = f.epoch;                   // settled for this step
        else atomicExch(f.errword, 0x5E40);                    // a complete histogram always holds k entries
    }
}

// (b) Candidates of one tile-chunk: positions (ascending) of the entries at or above the bucket
// of the k-th key; skipped for segments that will be finished from the data.
__global__ void __launch_bounds__(kSelThreads) collect_kernel(FastArgs f)
{
    __shared__ unsigned long long warp_tot[kWarps];
    const int row = blockIdx.y, chunk = blockIdx.x;
    const ChunkGeom g = chunk_geom(f, chunk);
    const int64_t slot = (int64_t)row * f.num_large + g.li;
    if ((int64_t)f.seg_m[slot] > f.comp_off[g.li + 1] - f.comp_off[g.li]) return;
    const float *tile = f.data + (int64_t)(f.row0 + row) * f.row_stride + (int64_t)g.q * kSelChunk;
    uint32_t key[kSelPerThread];
    const unsigned valid = load_keys_tile(tile, g.lo, g.hi, key);
    const uint32_t d0 = f.prefix[slot];
    unsigned flags = 0;
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i)
        if ((valid >> i & 1u) && (key[i] >> 20) >= d0) flags |= 1u << i;
    // per-stripe counts packed into four 16-bit fields, one CTA-wide scan for all four
    unsigned long long mine = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) mine |= (unsigned long long)__popc(flags >> (4 * r) & 0xfu) << (16 * r);
    unsigned long long total;
    const unsigned long long before = block_prefix_excl<unsigned long long>(mine, warp_tot, &total);
    const int64_t c = (int64_t)row * f.num_tchunks + chunk;
    if (threadIdx.x == 0)
        f.cand_cnt[c] = (int)((total & 0xffff) + (total >> 16 & 0xffff) + (total >> 32 & 0xffff) + (total >> 48));
    if (flags) {
        uint2 *dst = f.cand + c * kCandCap;
        unsigned stripe_base = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            unsigned at = stripe_base + (unsigned)(before >> (16 * r) & 0xffff);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (flags >> (4 * r + j) & 1u) {
                    if (at < (unsigned)kCandCap)
                        dst[at] = make_uint2(key[4 * r + j], (unsigned)(r * (kSelThreads * 4) + threadIdx.x * 4 + j));
                    ++at;
                }
            stripe_base += (unsigned)(total >> (16 * r) & 0xffff);
        }
    }
}

// Where a finishing CTA reads its entries from: the compacted candidates or the segment itself.
struct CompactSource {
    static constexpr bool kIndirect = true;       // offsets come from an array in global memory
    const uint32_t *key;
    const int32_t *idx;
    int n;
    __device__ __forceinline__ uint32_t key_at(int i) const { return key[i]; }
    __device__ __forceinline__ int32_t idx_at(int i) const { return idx[i]; }
};
struct DataSource {
    static constexpr bool kIndirect = false;
    const float *seg;
    int64_t off;
    int n;
    __device__ __forceinline__ uint32_t key_at(int i) const { return mag_key(__ldg(seg + i)); }
    __device__ __forceinline__ int32_t idx_at(int i) const { return (int32_t)(off + i); }
};

struct FinishShared {
    int hist[1024];
    int warp_i[32];
    unsigned warp_u[32];
    int found[2];
};

// Ordered emission by counting: an entry of `src` is selected iff its key is above T, or equals T
// and fewer than r equal keys precede it in the whole segment; its output slot is the number of
// selected entries before it.  gt_done / eq_done: entries with key > T / == T that precede src.
// A warp takes 32 * kFinPerThread consecutive entries, 32 consecutive ones per round (lane = entry:
// shared-memory reads without bank conflicts, coalesced global ones); inside a round the entries before a
// lane's own are counted with ballots.
// TRANSLATE (the CTA emits all k entries of the segment, and the source's offsets sit in global memory): the
// rounds write an entry's NUMBER into its slot and a last pass replaces the numbers by the offsets, k
// independent loads at once; fetched inside the rounds, every round waited for its winners' offsets.
template <int THREADS, bool TRANSLATE, typename Source>
__device__ void emit_ordered(const Source &src, uint32_t T, int r, int gt_done, int eq_done, int k,
                             int32_t *__restrict__ out, FinishShared &sh, int32_t *errword)
{
    const int tile = THREADS * kFinPerThread;
    const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5;
    const unsigned below = (1u << lane) - 1u;
    for (int base = 0; base < src.n; base += tile) {
        uint32_t key[kFinPerThread];
        const int first = base + warp * (32 * kFinPerThread) + lane;
        unsigned gt = 0, eq = 0;
#pragma unroll
        for (int i = 0; i < kFinPerThread; ++i) {
            const int at = first + 32 * i;
            key[i] = at < src.n ? src.key_at(at) : 0u;
            if (at < src.n) { gt += key[i] > T; eq += key[i] == T; }
        }
        unsigned total;
        unsigned before = block_prefix_excl<unsigned>(gt | (eq << 16), sh.warp_u, &total);
        before = __shfl_sync(kFull, before, 0);                   // what the warps in front of this one hold
        int g = gt_done + (int)(before & 0xffff), e = eq_done + (int)(before >> 16);
#pragma unroll
        for (int i = 0; i < kFinPerThread; ++i) {
            const int at = first + 32 * i;
            const bool is_gt = at < src.n && key[i] > T, is_eq = at < src.n && key[i] == T;
            const unsigned G = __ballot_sync(kFull, is_gt), E = __ballot_sync(kFull, is_eq);
            if (G | E) {
                const int gi = g + __popc(G & below), ei = e + __popc(E & below);
                int pos = -1;
                if (is_gt) pos = gi + (ei < r ? ei : r);
                else if (is_eq && ei < r) pos = gi + ei;
                if (pos >= 0) {
                    if (pos < k) out[pos] = TRANSLATE ? at : src.idx_at(at);
                    else atomicExch(errword, 0x5E60);
                }
                g += __popc(G);
                e += __popc(E);
            }
        }
        gt_done += (int)(total & 0xffff);
        eq_done += (int)(total >> 16);
        if (gt_done + (eq_done < r ? eq_done : r) >= k) break;     // everything is emitted
    }
    if (TRANSLATE) {
        __syncthreads();                                           // the CTA's own stores to out are visible to it
        for (int j = threadIdx.x; j < k; j += THREADS) {
            const int at = out[j];
            if (at >= 0 && at < src.n) out[j] = src.idx_at(at);
        }
    }
}

// Completes the radix search below the 11-bit bucket d0 (k_rem entries still to find inside it)
// and emits the k selected offsets in order; returns the k-th key.  Entries below the bucket, if
// the source has any, are ignored.
template <int THREADS, typename Source>
__device__ uint32_t finish_from(const Source &src, uint32_t d0, int k_rem, int k, int32_t *__restrict__ out,
                                FinishShared &sh, int32_t *errword)
{
    // the 20 bits below the bucket, ten at a time
    uint32_t prefix = d0 << 20, decided = 0x7ff00000u;
    constexpr int kBinsPer = 1024 / THREADS;
#pragma unroll 1
    for (int shift = 10; shift >= 0; shift -= 10) {
        for (int b = threadIdx.x; b < 1024; b += THREADS) sh.hist[b] = 0;
        __syncthreads();
        for (int base = 0; base < src.n; base += THREADS * 8) {      // eight independent loads per thread
            uint32_t x[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = base + j * THREADS + (int)threadIdx.x;
                x[j] = i < src.n ? src.key_at(i) : 0xffffffffu;          // never matches the prefix
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if ((x[j] & decided) == prefix) atomicAdd(&sh.hist[(x[j] >> shift) & 1023u], 1);
        }
        __syncthreads();
        int mine = 0;
#pragma unroll
        for (int j = 0; j < kBinsPer; ++j) mine += sh.hist[threadIdx.x * kBinsPer + j];
        const int incl = block_suffix_incl(mine, sh.warp_i);
        if (incl >= k_rem && incl - mine < k_rem) {
            int above = incl - mine;
            for (int j = kBinsPer - 1; j >= 0; --j) {
                const int h = sh.hist[threadIdx.x * kBinsPer + j];
                if (above + h >= k_rem) {
                    sh.found[0] = threadIdx.x * kBinsPer + j;
                    sh.found[1] = k_rem - above;
                    break;
                }
                above += h;
            }
        }
        if (threadIdx.x == 0 && incl < k_rem) atomicExch(errword, 0x5E50 + shift);
        __syncthreads();
        prefix |= (uint32_t)sh.found[0] << shift;
        decided |= 1023u << shift;
        k_rem = sh.found[1];
        __syncthreads();
    }
    emit_ordered<THREADS, Source::kIndirect>(src, prefix, k_rem, 0, 0, k, out, sh, errword);
    const uint32_t T = prefix;
    return T;
}

// Bucket of the k-th largest key from a complete leading-digit histogram in shared memory (which
// holds at least k entries): leaves the bucket in sh.found[0] and the rank still to find inside
// it in sh.found[1].  Run by every thread of the CTA; ends with a barrier.
template <int THREADS>
__device__ __forceinline__ void digit_scan(const unsigned *hist, int k, FinishShared &sh)
{
    constexpr int kPer = kHistBins / THREADS;
    int part = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) part += (int)hist[threadIdx.x * kPer + i];
    const int incl = block_suffix_incl(part, sh.warp_i);
    if (incl >= k && incl - part < k) {
        int above = incl - part;
        for (int i = kPer - 1; i >= 0; --i) {
            const int h = (int)hist[threadIdx.x * kPer + i];
            if (above + h >= k) {
                sh.found[0] = threadIdx.x * kPer + i;
                sh.found[1] = k - above;
                break;
            }
            above += h;
        }
    }
    __syncthreads();
}

// Whether the candidate lists of large segment li of `row` can serve this step's selection, and
// how many candidates they hold.  They cannot if they are not from this step, a chunk's list
// overflowed, the candidates exceed the segment's compact capacity, or fewer than k entries
// passed a predicted key.  `upto`: a chunk of the segment; *before gets the candidates of the
// chunks in front of it.  Every thread of the CTA calls this and gets the same answer; it is a
// pure function of what earlier launches left, so separate launches agree on it.
struct ListVerdict {
    bool settled;    // the two-pass path found the bucket of the k-th key in this step
    bool lists;
    bool too_high;   // the lists are complete but hold fewer than k entries: the predicted key was too high
    int m;           // candidates of the segment (valid when lists)
};
__device__ __forceinline__ ListVerdict list_verdict(const FastArgs &f, int row, int li, int upto, unsigned *before,
                                                    unsigned *warp_u)
{
    const int64_t slot = (int64_t)row * f.num_large + li;
    const int k = f.seg_k[f.large_ids[li]];
    const int64_t cap = f.comp_off[li + 1] - f.comp_off[li];
    const int c0 = f.tchunk0[li], c1 = f.tchunk0[li + 1];
    const int32_t *cnt = f.cand_cnt + (int64_t)row * f.num_tchunks;
    ListVerdict v;
    v.settled = f.seg_epoch[slot] == f.epoch;
    v.lists = v.settled ? (int64_t)f.seg_m[slot] <= cap : f.lbkey[slot] != 0;
    v.too_high = false;
    v.m = 0;
    if (before) *before = 0;
    if (!v.lists) return v;
    unsigned sum = 0, front = 0, over = 0;
    for (int c = c0 + (int)threadIdx.x; c < c1; c += (int)blockDim.x) {
        const unsigned n = (unsigned)cnt[c];
        sum += n;
        if (c < upto) front += n;
        over |= n > (unsigned)kCandCap;
    }
    unsigned total, total_front;
    block_prefix_excl<unsigned>(sum, warp_u, &total);            // per-segment totals stay below 2^31
    if (before) {
        block_prefix_excl<unsigned>(front, warp_u, &total_front);
        *before = total_front;
    }
    const int64_t m64 = total;
    if (__syncthreads_or((int)over) || m64 > cap) v.lists = false;
    else if (!v.settled && m64 < k) v.lists = false, v.too_high = true;
    v.m = (int)m64;
    return v;
}

// Compacts the candidates of the gn chunks from chunk gb on (large segment li of `row`) in index
// order into ckey/cidx, which already hold `done` entries; returns how many it added.
// group_off: kFinGroup + 1 ints of shared memory.  All THREADS threads of the CTA take part.
// A warp copies a chunk's list at a time (its records lie side by side: one coalesced read of up to 32 records,
// further reads for longer lists), four chunks in flight; where a chunk's records go follows from the prefix
// of the counts.  (One candidate per thread with a binary search for its chunk spent more issue slots on the
// searches than the copies take: 12 k cycles per 8192 candidates with 1024 threads.)
template <int THREADS>
__device__ __forceinline__ int compact_group(const FastArgs &f, int row, int li, int gb, int gn, int done,
                                             uint32_t *ckey, int32_t *cidx, int *group_off, unsigned *warp_u)
{
    constexpr int kPerT = kFinGroup / THREADS;
    constexpr int kWarps = THREADS / 32, kTrip = 4;
    const int c0 = f.tchunk0[li], q0 = f.large_q0[li];
    const int32_t *cnt = f.cand_cnt + (int64_t)row * f.num_tchunks;
    // exclusive prefix of the chunk counts of this group, in shared memory
    int mine[kPerT];
    unsigned sum = 0;
#pragma unroll
    for (int j = 0; j < kPerT; ++j) {
        const int e = (int)threadIdx.x * kPerT + j;
        mine[j] = e < gn ? cnt[gb + e] : 0;
        sum += (unsigned)mine[j];
    }
    unsigned total;
    unsigned at = block_prefix_excl<unsigned>(sum, warp_u, &total);
#pragma unroll
    for (int j = 0; j < kPerT; ++j) {
        group_off[threadIdx.x * kPerT + j] = (int)at;
        at += (unsigned)mine[j];
    }
    if (threadIdx.x == THREADS - 1) group_off[kFinGroup] = (int)total;
    __syncthreads();
    const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5;
    const uint2 *lists = f.cand + ((int64_t)row * f.num_tchunks + gb) * kCandCap;
    for (int base = warp * kTrip; base < gn; base += kWarps * kTrip) {
        int first[kTrip], n[kTrip];
        uint2 kp[kTrip];
#pragma unroll
        for (int t = 0; t < kTrip; ++t) {
            const int ch = base + t;
            first[t] = n[t] = 0;
            if (ch < gn) {
                first[t] = group_off[ch];
                n[t] = group_off[ch + 1] - first[t];
            }
            kp[t] = lane < n[t] ? __ldg(lists + (int64_t)ch * kCandCap + lane) : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int t = 0; t < kTrip; ++t) {
            const int ch = base + t;
            const int tile0 = (q0 + (gb + ch - c0)) * kSelChunk;               // N < 2^31
            if (lane < n[t]) {
                ckey[done + first[t] + lane] = kp[t].x;
                cidx[done + first[t] + lane] = tile0 + (int)kp[t].y;
            }
            for (int j = lane + 32; j < n[t]; j += 32) {                       // a list of more than 32 records
                const uint2 more = __ldg(lists + (int64_t)ch * kCandCap + j);
                ckey[done + first[t] + j] = more.x;
                cidx[done + first[t] + j] = tile0 + (int)more.y;
            }
        }
    }
    __syncthreads();                                       // group_off may be rewritten by the caller's next group
    return (int)total;
}

// ------------------------------------------------------------------------------------------
// Segments of more than kFinGroup chunks (tens of millions of entries) are not left to one CTA:
// every step of the finishing is spread over the groups of chunks, one CTA per group and launch,
// grid (groups, rows).  compact_groups_kernel compacts each group's candidates into the
// segment's global compact arrays and finds the bucket of the k-th key; wide_digit_kernel<10>
// and <0> settle the remaining 20 bits of the key; wide_count_kernel counts, per group, the
// entries above and at the key; wide_emit_kernel writes each group's selected offsets behind
// those of the groups before it.  Where CTAs of a launch contribute to one result, the CTA that
// arrives last (a ticket counter tells; nobody waits) completes it.  If the lists cannot serve
// the step, all five return at once and the finishing CTA of finish_kernel works on the data.
// ------------------------------------------------------------------------------------------
struct JobGeom {
    int li, gb, job, njobs;      // large segment, first chunk of the group, its number inside the segment, groups of the segment
    int64_t slot, rec;           // (row, segment) and (row, group) record
};
__device__ __forceinline__ JobGeom job_geom(const FastArgs &f, int row)
{
    JobGeom g;
    const int2 j = f.group_job[blockIdx.x];
    g.li = j.x;
    g.gb = j.y;
    const int c0 = f.tchunk0[g.li], c1 = f.tchunk0[g.li + 1];
    g.job = (g.gb - c0) / kFinGroup;
    g.njobs = (c1 - c0 + kFinGroup - 1) / kFinGroup;
    g.slot = (int64_t)row * f.num_large + g.li;
    g.rec = (int64_t)row * f.num_group_jobs + blockIdx.x;
    return g;
}

// True in the CTA that is the last of n to arrive at the ticket; its later reads see what the
// others wrote before they arrived.  Every thread of the CTA calls this.
__device__ __forceinline__ bool arrives_last(int32_t *ticket, int n, int *flag)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *flag = atomicAdd(ticket, 1) == n - 1;
    __syncthreads();
    const bool last = *flag != 0;
    if (last) __threadfence();
    return last;
}

__global__ void __launch_bounds__(kFinThreads) compact_groups_kernel(FastArgs f)
{
    __shared__ unsigned h[kHistBins];
    __shared__ int group_off[kFinGroup + 1];
    __shared__ unsigned warp_u[kFinWarps];
    __shared__ int warp_i[kFinWarps];
    __shared__ int is_last, scan_flag;
    const int row = blockIdx.y;
    const JobGeom g = job_geom(f, row);
    unsigned before;
    const ListVerdict v = list_verdict(f, row, g.li, g.gb, &before, warp_u);
    if (g.job == 0 && threadIdx.x == 0) f.seg_wide[g.slot] = v.lists ? 1 : 0;
    if (!v.lists) return;
    const int c1 = f.tchunk0[g.li + 1];
    const int gn = c1 - g.gb < kFinGroup ? c1 - g.gb : kFinGroup;
    uint32_t *ckey = f.comp_key + (int64_t)row * f.comp_total + f.comp_off[g.li];
    int32_t *cidx = f.comp_idx + (int64_t)row * f.comp_total + f.comp_off[g.li];
    const int added = compact_group<kFinThreads>(f, row, g.li, g.gb, gn, (int)before, ckey, cidx, group_off, warp_u);
    if (threadIdx.x == 0) {
        f.job_range[g.rec] = make_int2((int)before, added);
        if ((int64_t)before + added > (int64_t)v.m) atomicExch(f.errword, 0x5E71);
    }
    if (v.settled) return;                                   // the two-pass path found the bucket already
    // leading digits of this group's candidates (every entry at or above the predicted key is a
    // candidate and there are at least k, so the bucket of the k-th key is among them)
    for (int b = threadIdx.x; b < kHistBins; b += kFinThreads) h[b] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < added; i += kFinThreads) atomicAdd(&h[ckey[before + i] >> 20], 1u);
    __syncthreads();
    uint32_t *gh = f.hist + g.slot * kHistBins;
    for (int b = threadIdx.x; b < kHistBins; b += kFinThreads)
        if (h[b]) atomicAdd(gh + b, h[b]);
    if (!arrives_last(&f.seg_ticket[g.slot], g.njobs, &is_last)) return;
    const bool ok = bucket_scan<kFinThreads>(f, g.slot, f.seg_k[f.large_ids[g.li]], warp_i, &scan_flag);
    if (threadIdx.x == 0 && !ok) atomicExch(f.errword, 0x5E41);
}

// Ten more bits of the k-th key: histogram of that digit over the candidates that match the bits
// found so far; SHIFT 10 follows the bucket (prefix holds the 11-bit bucket), SHIFT 0 follows
// that (prefix holds the key so far).  Leaves the key so far in prefix and the rank inside it in k_rem.
template <int SHIFT>
__global__ void __launch_bounds__(kFinThreads) wide_digit_kernel(FastArgs f)
{
    __shared__ int h[1024];
    __shared__ int warp_i[kFinWarps];
    __shared__ int is_last;
    const int row = blockIdx.y;
    const JobGeom g = job_geom(f, row);
    if (!f.seg_wide[g.slot]) return;
    const int2 range = f.job_range[g.rec];
    const uint32_t prefix = SHIFT == 10 ? f.prefix[g.slot] << 20 : f.prefix[g.slot];
    const uint32_t decided = SHIFT == 10 ? 0x7ff00000u : 0x7ffffc00u;
    for (int b = threadIdx.x; b < 1024; b += kFinThreads) h[b] = 0;
    __syncthreads();
    const uint32_t *key = f.comp_key + (int64_t)row * f.comp_total + f.comp_off[g.li] + range.x;
    for (int base = 0; base < range.y; base += kFinThreads * 8) {        // eight independent loads per thread
        uint32_t x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = base + j * kFinThreads + (int)threadIdx.x;
            x[j] = i < range.y ? key[i] : 0xffffffffu;                   // never matches the prefix
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if ((x[j] & decided) == prefix) atomicAdd(&h[(x[j] >> SHIFT) & 1023u], 1);
    }
    __syncthreads();
    uint32_t *gh = f.hist + g.slot * kHistBins;
    for (int b = threadIdx.x; b < 1024; b += kFinThreads)
        if (h[b]) atomicAdd(gh + b, (unsigned)h[b]);
    if (!arrives_last(&f.seg_ticket[g.slot], g.njobs, &is_last)) return;
    constexpr int kPer = 1024 / kFinThreads;
    const int k_rem = f.k_rem[g.slot];
    int hh[kPer], part = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        hh[i] = (int)__ldcg(gh + threadIdx.x * kPer + i);
        part += hh[i];
        gh[threadIdx.x * kPer + i] = 0u;
    }
    if (threadIdx.x == 0) f.seg_ticket[g.slot] = 0;
    const int incl = block_suffix_incl(part, warp_i);
    if (incl >= k_rem && incl - part < k_rem) {
        int above = incl - part;
#pragma unroll
        for (int i = kPer - 1; i >= 0; --i) {
            if (above + hh[i] >= k_rem) {
                f.prefix[g.slot] = prefix | (uint32_t)(threadIdx.x * kPer + i) << SHIFT;
                f.k_rem[g.slot] = k_rem - above;
                break;
            }
            above += hh[i];
        }
    }
    if (threadIdx.x == 0 && incl < k_rem) atomicExch(f.errword, 0x5E51 + SHIFT);
}

// Entries of each group above and at the k-th key.
__global__ void __launch_bounds__(kFinThreads) wide_count_kernel(FastArgs f)
{
    __shared__ unsigned long long warp_l[kFinWarps];
    const int row = blockIdx.y;
    const JobGeom g = job_geom(f, row);
    if (!f.seg_wide[g.slot]) return;
    const int2 range = f.job_range[g.rec];
    const uint32_t T = f.prefix[g.slot];
    const uint32_t *key = f.comp_key + (int64_t)row * f.comp_total + f.comp_off[g.li] + range.x;
    unsigned long long mine = 0;
    for (int i = threadIdx.x; i < range.y; i += kFinThreads) {
        const uint32_t x = key[i];
        mine += (unsigned long long)(x > T) | (unsigned long long)(x == T) << 32;
    }
    unsigned long long total;
    block_prefix_excl<unsigned long long>(mine, warp_l, &total);
    if (threadIdx.x == 0) f.job_cnt[g.rec] = make_int2((int)(total & 0xffffffffu), (int)(total >> 32));
}

// Selected offsets of each group, behind those of the groups before it; the first group's CTA
// also stores the key from which the next step collects candidates.
__global__ void __launch_bounds__(kFinThreads) wide_emit_kernel(FastArgs f)
{
    __shared__ FinishShared sh;
    __shared__ unsigned long long warp_l[kFinWarps];
    const int row = blockIdx.y;
    const JobGeom g = job_geom(f, row);
    if (!f.seg_wide[g.slot]) return;
    const int2 range = f.job_range[g.rec];
    const uint32_t T = f.prefix[g.slot];
    const int r = f.k_rem[g.slot];
    const int s = f.large_ids[g.li];
    const int k = f.seg_k[s];
    unsigned long long mine = 0;
    unsigned cands = 0;
    for (int j = threadIdx.x; j < g.njobs; j += kFinThreads) {
        const int64_t rec = g.rec - g.job + j;
        cands += (unsigned)f.job_range[rec].y;
        if (j < g.job) {
            const int2 c = f.job_cnt[rec];
            mine += (unsigned long long)(unsigned)c.x | (unsigned long long)(unsigned)c.y << 32;
        }
    }
    unsigned long long total;
    block_prefix_excl<unsigned long long>(mine, warp_l, &total);
    unsigned m;
    block_prefix_excl<unsigned>(cands, sh.warp_u, &m);
    const int gt0 = (int)(total & 0xffffffffu), eq0 = (int)(total >> 32);
    if (gt0 + (eq0 < r ? eq0 : r) < k) {
        const int64_t base = (int64_t)row * f.comp_total + f.comp_off[g.li] + range.x;
        CompactSource src{f.comp_key + base, f.comp_idx + base, range.y};
        emit_ordered<kFinThreads, false>(src, T, r, gt0, eq0, k, f.out + (int64_t)row * f.out_stride + f.seg_out[s], sh, f.errword);
    }
    if (g.job == 0 && threadIdx.x == 0) {
        f.seg_m[g.slot] = (int)m;
        store_prediction(f, g.slot, T, k, false);
        f.seg_path[g.slot] = f.seg_epoch[g.slot] == f.epoch ? 1 : 0;
    }
}

// One read of a segment (len entries at seg, offset `off` in the row): the entries whose key is at least
// `from`, compacted in index order into ckey/cidx, of which only the first `cap` are stored; returns how many
// there are.  All THREADS threads of the CTA take part; ends with a barrier.  The next tile's loads are issued
// before this tile's scan (two barriers) so that they overlap it.
template <int THREADS>
__device__ __forceinline__ int collect_from_data(const float *__restrict__ seg, int64_t off, int len, uint32_t from,
                                                 int64_t cap, uint32_t *ckey, int32_t *cidx, unsigned *warp_u)
{
    constexpr int kTile = THREADS * kSelPerThread;
    int done = 0;                                  // (a segment has fewer than 2^31 entries)
    uint32_t next[kSelPerThread];
    int next_valid = load_keys16(seg, 0, len, next);
    for (int base = 0; base < len; base += kTile) {
        uint32_t key[kSelPerThread];
        const int valid = next_valid;
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i) key[i] = next[i];
        if (base + kTile < len) next_valid = load_keys16(seg, base + kTile, len, next);
        unsigned flags = 0;
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i)
            if (i < valid && key[i] >= from) flags |= 1u << i;
        unsigned total;
        int at = done + (int)block_prefix_excl<unsigned>((unsigned)__popc(flags), warp_u, &total);
        // a thread holds a candidate in one tile of three: a loop over the set bits instead of sixteen predicated stores
        // (the read is bound by the instructions a lone CTA can issue, not by memory)
        const int32_t first = (int32_t)off + base + (int)threadIdx.x * kSelPerThread;
        while (flags) {
            const int i = __ffs((int)flags) - 1;
            flags &= flags - 1u;
            if (at < cap) {           // (the key once more from the line this thread has just read: registers cannot be indexed)
                ckey[at] = mag_key(__ldg(seg + base + (int)threadIdx.x * kSelPerThread + i));
                cidx[at] = first + i;
            }
            ++at;
        }
        done += (int)total;
    }
    __syncthreads();
    return done;
}

// The selection of one (segment, row) is completed by one CTA.  The first num_small CTAs of a
// row each do one small segment outright.  For a large segment the CTA
//  1. settles the bucket of the k-th key from the histogram the accumulation left, unless path
//     (b) already did; if fewer than k entries had passed the predicted key it counts the
//     leading digits of the whole segment itself;
//  2. compacts the candidates in index order (each thread takes candidate ranks and finds their
//     chunk by binary search; a segment of more than kFinGroup chunks arrives compacted) and
//     finishes on them -- or on the data when there are no valid lists or too many entries;
//  3. stores the key from which the next step should collect candidates.
// CTA order: large segments longest first, then the small ones, then spare CTAs that clear the
// dense update buffer (if the caller announced it) while the rest of the launch is busy.
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) finish_kernel(FastArgs f)
{
    __shared__ FinishShared sh;
    __shared__ SmallShared small_sh;
    __shared__ unsigned full_hist[kHistBins];
    __shared__ int group_off[kFinGroup + 1];
    extern __shared__ __align__(16) uint32_t fin_dyn[];     // f.smem_keys candidate keys
    const int row = blockIdx.y;
    if ((int)blockIdx.x >= f.num_large + f.fin_small) {      // spare CTAs: clear the dense update meanwhile
        if (row != 0) return;
        if ((int)threadIdx.x >= f.zero_threads) return;
        const uint64_t stride = (uint64_t)f.zero_ctas * f.zero_threads;
        for (uint64_t e = (uint64_t)(blockIdx.x - f.num_large - f.fin_small) * f.zero_threads + threadIdx.x; e <= f.zero_vecs; e += stride) {
            if (e < f.zero_vecs) __stcs(f.zero_ptr + e, make_uint4(0u, 0u, 0u, 0u));
            else
                for (int j = 0; j < f.zero_tail; ++j) reinterpret_cast<float *>(f.zero_ptr + e)[j] = 0.0f;
        }
        return;
    }
    if ((int)blockIdx.x >= f.num_large) {
        select_small_body(f.data, f.row_stride, f.row0, f.seg_off, f.seg_len, f.seg_k, f.seg_out,
                          f.small_ids[blockIdx.x - f.num_large], row, f.out, f.out_stride, f.errword, small_sh);
        return;
    }
    uint32_t *s_key = fin_dyn;
    const int li = f.large_order[blockIdx.x];
    const int64_t slot = (int64_t)row * f.num_large + li;
    const int s = f.large_ids[li];
    const int64_t off = f.seg_off[s];
    const int len = f.seg_len[s], k = f.seg_k[s];
    const float *rowp = f.data + (int64_t)(f.row0 + row) * f.row_stride;
    int32_t *out = f.out + (int64_t)row * f.out_stride + f.seg_out[s];
    const int64_t cap = f.comp_off[li + 1] - f.comp_off[li];
    const int c0 = f.tchunk0[li], c1 = f.tchunk0[li + 1];
    // 1. are there lists for this step, and how many candidates do they hold?  A segment of more than
    // one group of chunks has been served by the wide kernels, or is left to the data.
    const bool grouped = c1 - c0 > kFinGroup;
    if (grouped && f.seg_wide[slot]) return;
    ListVerdict verdict;
    if (grouped) {
        verdict.settled = f.seg_epoch[slot] == f.epoch;
        verdict.lists = false;
        verdict.too_high = false;
        verdict.m = 0;
    } else {
        verdict = list_verdict(f, row, li, c0, nullptr, sh.warp_u);
    }
    const bool settled = verdict.settled, lists = verdict.lists;
    const int m = verdict.m;
    int path, retried = 0;
    uint32_t d0 = 0, T;
    int k_rem = 0;
    if (lists) {
        path = settled ? 1 : 0;
        // 2. compaction.  Keys stay in shared memory when they fit; offsets are needed only for the winners.
        uint32_t *ckey = m <= f.smem_keys ? s_key : f.comp_key + (int64_t)row * f.comp_total + f.comp_off[li];
        int32_t *cidx = f.comp_idx + (int64_t)row * f.comp_total + f.comp_off[li];
        const int done = compact_group<THREADS>(f, row, li, c0, c1 - c0, 0, ckey, cidx, group_off, sh.warp_u);
        if (threadIdx.x == 0 && done != m) atomicExch(f.errword, 0x5E70);
        // 3. the bucket of the k-th key: from path (b), or from the candidates' own leading digits
        // (every entry at or above the predicted key is a candidate, and there are at least k)
        if (settled) {
            d0 = f.prefix[slot];
            k_rem = f.k_rem[slot];
        } else {
            for (int b = threadIdx.x; b < kHistBins; b += THREADS) full_hist[b] = 0;
            __syncthreads();
            for (int i = threadIdx.x; i < m; i += THREADS) atomicAdd(&full_hist[ckey[i] >> 20], 1u);
            __syncthreads();
            digit_scan<THREADS>(full_hist, k, sh);
            d0 = (uint32_t)sh.found[0];
            k_rem = sh.found[1];
        }
        __syncthreads();
        CompactSource src{ckey, cidx, m};
        T = finish_from<THREADS>(src, d0, k_rem, k, out, sh, f.errword);
    } else {
        // no lists for this step, a chunk list overflowed, too many candidates, or a prediction
        // that turned out too high: work on the data
        if (settled) {
            path = 3;
            d0 = f.prefix[slot];
            k_rem = f.k_rem[slot];
        } else {
            if (verdict.too_high) {
                // The predicted key was a little too high (the usual miss is a few per cent): one read of the
                // segment with the key lowered by 12 % (a quarter lower already collects more than the compact
                // arrays hold, so thickly do the residuals lie below the k-th key), then on as with lists.  Only
                // if that still brings fewer than k entries, or more than the arrays hold, the full search below runs.
                const uint32_t from = __float_as_uint(__uint_as_float(f.lbkey[slot]) * 0.88f);
                uint32_t *ckey = f.comp_key + (int64_t)row * f.comp_total + f.comp_off[li];
                int32_t *cidx = f.comp_idx + (int64_t)row * f.comp_total + f.comp_off[li];
                const int got = collect_from_data<THREADS>(rowp + off, off, len, from, cap, ckey, cidx, sh.warp_u);
                if (got >= k && got <= cap) {
                    path = 4;
                    retried = got;
                    for (int b = threadIdx.x; b < kHistBins; b += THREADS) full_hist[b] = 0;
                    __syncthreads();
                    for (int i = threadIdx.x; i < retried; i += THREADS) atomicAdd(&full_hist[ckey[i] >> 20], 1u);
                    __syncthreads();
                    digit_scan<THREADS>(full_hist, k, sh);
                    d0 = (uint32_t)sh.found[0];
                    k_rem = sh.found[1];
                    __syncthreads();
                    CompactSource src{ckey, cidx, retried};
                    T = finish_from<THREADS>(src, d0, k_rem, k, out, sh, f.errword);
                    goto finished;
                }
            }
            path = 2;
            // first read of the segment: its complete leading-digit histogram
            for (int b = threadIdx.x; b < kHistBins; b += THREADS) full_hist[b] = 0;
            __syncthreads();
            constexpr int kTile = THREADS * kSelPerThread;
            for (int base = 0; base < len; base += kTile) {
                uint32_t key[kSelPerThread];
                const int valid = load_keys16(rowp + off, base, len, key);
#pragma unroll
                for (int i = 0; i < kSelPerThread; ++i)
                    if (i < valid) atomicAdd(&full_hist[key[i] >> 20], 1u);
            }
            __syncthreads();
            digit_scan<THREADS>(full_hist, k, sh);
            d0 = (uint32_t)sh.found[0];
            k_rem = sh.found[1];
            const int64_t at_or_above = (int64_t)(k - k_rem) + (int64_t)full_hist[d0];
            __syncthreads();
            if (at_or_above <= cap) {
                // second read: the entries from the bucket upwards, compacted in index order
                const int mm = (int)at_or_above;
                uint32_t *ckey = mm <= f.smem_keys ? s_key : f.comp_key + (int64_t)row * f.comp_total + f.comp_off[li];
                int32_t *cidx = f.comp_idx + (int64_t)row * f.comp_total + f.comp_off[li];
                const int done = collect_from_data<THREADS>(rowp + off, off, len, d0 << 20, cap, ckey, cidx, sh.warp_u);
                if (threadIdx.x == 0 && done != mm) atomicExch(f.errword, 0x5E80);
                CompactSource src{ckey, cidx, mm};
                T = finish_from<THREADS>(src, d0, k_rem, k, out, sh, f.errword);
                goto finished;
            }
        }
        {
            DataSource src{rowp + off, off, len};
            T = finish_from<THREADS>(src, d0, k_rem, k, out, sh, f.errword);
        }
    }
finished:
    if (threadIdx.x == 0) f.seg_m[slot] = lists ? m : path == 4 ? retried : len;
    if (threadIdx.x == 0) {
        store_prediction(f, slot, T, k, (path == 2 || path == 4) && f.lbkey[slot] != 0);
        f.seg_path[slot] = path;
    }
}

// ------------------------------------------------------------------------------------------
// (a) Stage 1 fused with candidate collection.  Grid (tiles per row, K); a CTA streams one tile
// of one row exactly as accumulate_kernel does (u <- m u + g fused, v <- v + u; Algorithm 1/2 and
// Section V-A).  A CTA of a selecting row then looks at its fresh v: for every large segment the
// tile overlaps and that has a predicted key, the entries at or above that key are listed, in
// position order, with their keys.
// ------------------------------------------------------------------------------------------
// The part [lo, hi) of a tile, held four consecutive entries per thread (positions p0 .. p0+3):
// the entries whose key reaches lbkey are written, ascending, to the chunk's candidate list.
__device__ __forceinline__ void collect_tile(const FastArgs &f, int64_t chunk, const uint32_t (&key)[4], uint32_t lbkey,
                                             bool live, int p0, int lo, int hi, unsigned *warp_u)
{
    unsigned flags = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (live && p0 + i >= lo && p0 + i < hi && key[i] >= lbkey) flags |= 1u << i;
    // Candidates are rare (a handful per tile): most warps have none and skip the scan; one barrier,
    // and only the threads that hold a candidate add up the warps before theirs.
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const unsigned cnt = (unsigned)__popc(flags);
    unsigned incl = cnt;
    if (__ballot_sync(kFull, cnt != 0)) {
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned y = __shfl_up_sync(kFull, incl, d);
            if (lane >= (unsigned)d) incl += y;
        }
    }
    if (lane == 31) warp_u[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const unsigned total = __reduce_add_sync(kFull, warp_u[lane]);
        if (lane == 0) f.cand_cnt[chunk] = (int)total;
    }
    if (flags) {
        unsigned at = incl - cnt;
        for (unsigned w = 0; w < warp; ++w) at += warp_u[w];
        uint2 *dst = f.cand + chunk * kCandCap;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (flags >> i & 1u) {
                if (at < (unsigned)kCandCap) dst[at] = make_uint2(key[i], (unsigned)(p0 + i));
                ++at;
            }
    }
}

__device__ __forceinline__ void acc4(float4 &u, float4 &v, const float4 &g, float m)
{
    u.x = __fmaf_rn(m, u.x, g.x); v.x = __fadd_rn(v.x, u.x);
    u.y = __fmaf_rn(m, u.y, g.y); v.y = __fadd_rn(v.y, u.y);
    u.z = __fmaf_rn(m, u.z, g.z); v.z = __fadd_rn(v.z, u.z);
    u.w = __fmaf_rn(m, u.w, g.w); v.w = __fadd_rn(v.w, u.w);
}

// DENSE: the model has layers that are sent as they are (Section VI-A) and keep no state; the instantiation
// without them is the plain kernel, free of every test this needs.
template <bool DENSE>
__global__ void __launch_bounds__(kAccThreads, 2)
accumulate_select_kernel(FastArgs f, const float *__restrict__ g, int64_t g_stride, float *__restrict__ u,
                         float *__restrict__ v, int64_t N, float m, int sel_row0, int sel_rows)
{
    __shared__ unsigned warp_u[kAccThreads / 32];
    const int row = blockIdx.y, q = blockIdx.x;
    const int64_t tile_base = (int64_t)q * kSelChunk;
    const int in_tile = N - tile_base < kSelChunk ? (int)(N - tile_base) : kSelChunk;    // a multiple of 4
    const int p0 = (int)threadIdx.x * 4;
    const bool live = p0 < in_tile;
    // a selecting row fetches its tile's description and predicted key before the stream, so that
    // they are at hand when the stores have been issued; so does every row of a model with dense layers
    const int sel = row - sel_row0;
    const bool selecting = sel >= 0 && sel < sel_rows;
    int4 desc = make_int4(0, -2, 0, 0);         // x: first segment, y: the one large segment covering the tile
                                                // (-1: several segments, -2: no large segment), z: its chunk,
                                                // w: 0 no dense element, > 0 one dense run (packed), < 0 several
    uint32_t lbkey1 = 0;
    if (selecting || DENSE) desc = __ldg(f.tile_desc + q);      // consumed after the stream's loads are on their way
    float4 vv = make_float4(0.f, 0.f, 0.f, 0.f), gg = vv, uu = vv;
    const int64_t e = ((int64_t)row * N + tile_base + p0) >> 2;
    if (live) {
        gg = __ldcs(reinterpret_cast<const float4 *>(g) + (((int64_t)row * g_stride + tile_base + p0) >> 2));
        uu = __ldcs(reinterpret_cast<float4 *>(u) + e);
        vv = __ldcs(reinterpret_cast<float4 *>(v) + e);
    }
    // (only now the description is looked at: the predicted key's address depends on it, and a warp that waits for the
    // description before it has issued its three loads starts its stream a memory latency late)
    if (selecting && desc.y >= 0) lbkey1 = f.lbkey[(int64_t)sel * f.num_large + desc.y];
    if (live) {
        // Dense elements among these four take no gradient: their u and v are zero from lgc_init on and stay
        // exactly zero (m * 0 + 0 = 0, 0 + 0 = 0), which is "no state" for the layers sent as they are.
        if (DENSE && desc.w > 0) {                  // one dense run [lo, hi) inside the tile
            const int lo = (desc.w - 1) & 8191, hi = (desc.w - 1) >> 13;
            if (p0 >= lo && p0 < hi) gg.x = 0.0f;
            if (p0 + 1 >= lo && p0 + 1 < hi) gg.y = 0.0f;
            if (p0 + 2 >= lo && p0 + 2 < hi) gg.z = 0.0f;
            if (p0 + 3 >= lo && p0 + 3 < hi) gg.w = 0.0f;
        } else if (DENSE && desc.w < 0) {           // several runs (tiny dense layers side by side)
            const int64_t pos = tile_base + p0, tile_end = tile_base + in_tile;
            for (int r = -desc.w - 1; r < f.num_dense && f.dense_rng[2 * r] < tile_end; ++r) {
                const int64_t a = f.dense_rng[2 * r], b = f.dense_rng[2 * r + 1];
                if (pos >= a && pos < b) gg.x = 0.0f;
                if (pos + 1 >= a && pos + 1 < b) gg.y = 0.0f;
                if (pos + 2 >= a && pos + 2 < b) gg.z = 0.0f;
                if (pos + 3 >= a && pos + 3 < b) gg.w = 0.0f;
            }
        }
        acc4(uu, vv, gg, m);
        __stcs(reinterpret_cast<float4 *>(u) + e, uu);
        __stcs(reinterpret_cast<float4 *>(v) + e, vv);
    }
    if (!selecting || desc.y == -2) return;
    const uint32_t key[4] = {mag_key(vv.x), mag_key(vv.y), mag_key(vv.z), mag_key(vv.w)};
    if (desc.y >= 0) {
        if (lbkey1 == 0) return;                                 // no prediction: the finishing CTA counts itself
        collect_tile(f, (int64_t)sel * f.num_tchunks + desc.z, key, lbkey1, live, p0, 0, in_tile, warp_u);
        return;
    }
    const int64_t tile_end = tile_base + in_tile;
    for (int s = desc.x; s < f.num_large + f.num_small && f.seg_off[s] < tile_end; ++s) {
        const int li = f.seg_large[s];
        if (li < 0) continue;
        const int64_t slot = (int64_t)sel * f.num_large + li;
        const uint32_t lbkey = f.lbkey[slot];
        if (lbkey == 0) continue;
        const int64_t off = f.seg_off[s], end = off + f.seg_len[s];
        const int lo = off > tile_base ? (int)(off - tile_base) : 0;
        const int hi = end < tile_end ? (int)(end - tile_base) : in_tile;
        collect_tile(f, (int64_t)sel * f.num_tchunks + f.tchunk0[li] + (q - f.large_q0[li]), key, lbkey, live, p0, lo,
                     hi, warp_u);
        __syncthreads();                                         // warp_u is reused by the next segment
    }
}

void fill_args(FastArgs &f, const SelectTables &t, const float *data, int64_t row_stride, int row0, int32_t *out,
               int64_t out_stride, int32_t epoch, int32_t *errword)
{
    f.data = data; f.row_stride = row_stride; f.row0 = row0;
    f.num_large = t.num_large; f.num_small = t.num_small; f.num_tchunks = t.num_tchunks; f.epoch = epoch;
    f.fin_small = 0;
    f.smem_keys = 0;
    f.large_order = t.large_order; f.group_job = t.group_job; f.num_group_jobs = t.num_group_jobs;
    f.job_range = t.job_range; f.job_cnt = t.job_cnt; f.seg_wide = t.seg_wide; f.zero_ptr = nullptr; f.zero_vecs = 0; f.zero_tail = 0; f.zero_ctas = 0; f.zero_threads = 0;
    f.seg_off = t.seg_off; f.seg_len = t.seg_len; f.seg_k = t.seg_k; f.seg_out = t.seg_out;
    f.small_ids = t.small_ids; f.large_ids = t.large_ids; f.seg_large = t.seg_large; f.large_q0 = t.large_q0;
    f.tchunk0 = t.tchunk0; f.tchunk_large = t.tchunk_large; f.tile_desc = t.tile_desc;
    f.dense_rng = t.dense_rng; f.num_dense = t.num_dense;
    f.hist = t.hist; f.prefix = t.prefix; f.k_rem = t.k_rem; f.cand_cnt = t.cand_cnt; f.seg_m = t.seg_m;
    f.seg_ticket = t.seg_ticket; f.seg_epoch = t.seg_epoch; f.seg_path = t.seg_path; f.lbkey = t.lbkey; f.last_key = t.last_key; f.key_trend = t.key_trend; f.cand = t.cand;
    f.comp_off = t.comp_off; f.comp_total = t.comp_total; f.comp_key = t.comp_key; f.comp_idx = t.comp_idx;
    f.out = out; f.out_stride = out_stride; f.errword = errword;
}

__global__ void __launch_bounds__(kSelThreads) select_small_only_kernel(FastArgs f)
{
    __shared__ SmallShared sh;
    select_small_body(f.data, f.row_stride, f.row0, f.seg_off, f.seg_len, f.seg_k, f.seg_out, f.small_ids[blockIdx.x],
                      blockIdx.y, f.out, f.out_stride, f.errword, sh);
}

}  // namespace

// `served`: the accumulation of this step collected the candidates of exactly these rows (path a);
// otherwise the two passes of path (b) run first.  `clear` (may be null): a buffer of `clear_floats`
// floats that spare CTAs of the finishing launch set to zero; used only when there are large segments.
cudaError_t launch_select(const SelectTables &t, const float *data, int64_t row_stride, int row0, int rows,
                          int32_t *out, int64_t out_stride, bool served, int32_t epoch, float *clear, int64_t clear_floats,
                          int32_t *errword, cudaStream_t st, cudaStream_t side, cudaEvent_t fork, cudaEvent_t join)
{
    if (rows <= 0 || t.num_segments == 0) return cudaSuccess;
    FastArgs f;
    fill_args(f, t, data, row_stride, row0, out, out_stride, epoch, errword);
    // the finishing launch's shape (see kFinThreads above)
    const int64_t large_jobs = (int64_t)rows * t.num_large;
    const int fin_threads = large_jobs <= sm_count() ? 1024 : large_jobs > 4 * (int64_t)sm_count() ? 256 : kFinThreads;
    f.smem_keys = fin_threads == 256 ? kFinSmemCapSmall : kFinSmemCap;
    const int fin_dyn = f.smem_keys * (int)sizeof(uint32_t);
    static OncePerDevice configured;
    {
        const cudaError_t e = configured.run([] {
            cudaError_t x = cudaFuncSetAttribute(finish_kernel<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinSmemCap * 4);
            if (x == cudaSuccess) x = cudaFuncSetAttribute(finish_kernel<kFinThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinSmemCap * 4);
            if (x == cudaSuccess) x = cudaFuncSetAttribute(finish_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFinSmemCapSmall * 4);
            return x;
        });
        if (e != cudaSuccess) return e;
    }
    if (t.num_large && !served) {
        hist0_fast_kernel<<<dim3(t.num_tchunks, rows), kSelThreads, 0, st>>>(f), ++g_kernel_launches;
        collect_kernel<<<dim3(t.num_tchunks, rows), kSelThreads, 0, st>>>(f), ++g_kernel_launches;
    }
    // a few small segments ride along in the finishing launch; many get CTAs of their own size
    f.fin_small = (int64_t)rows * t.num_small <= 512 && t.num_large ? t.num_small : 0;
    bool forked = false;
    if (t.num_small && !f.fin_small) {
        // both launches are latency bound and write disjoint slots: side by side when the caller lent a stream
        forked = side && fork && join && t.num_large;
        cudaStream_t where = st;
        if (forked) {
            cudaError_t e = cudaEventRecord(fork, st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(side, fork, 0);
            if (e != cudaSuccess) return e;
            where = side;
        }
        select_small_only_kernel<<<dim3(t.num_small, rows), kSelThreads, 0, where>>>(f), ++g_kernel_launches;
        if (forked) {
            const cudaError_t e = cudaEventRecord(join, side);
            if (e != cudaSuccess) return e;
        }
    }
    if (t.num_group_jobs) {
        const dim3 grid(t.num_group_jobs, rows);
        compact_groups_kernel<<<grid, kFinThreads, 0, st>>>(f), ++g_kernel_launches;
        wide_digit_kernel<10><<<grid, kFinThreads, 0, st>>>(f), ++g_kernel_launches;
        wide_digit_kernel<0><<<grid, kFinThreads, 0, st>>>(f), ++g_kernel_launches;
        wide_count_kernel<<<grid, kFinThreads, 0, st>>>(f), ++g_kernel_launches;
        wide_emit_kernel<<<grid, kFinThreads, 0, st>>>(f), ++g_kernel_launches;
    }
    unsigned spare = 0;
    if (clear && clear_floats > 0 && t.num_large) {
        f.zero_ptr = reinterpret_cast<uint4 *>(clear);
        f.zero_vecs = (uint64_t)clear_floats >> 2;
        f.zero_tail = (int)(clear_floats & 3);
        // (a 1024-thread finishing CTA has its SM to itself, registers and all: the clearing CTAs run on other SMs
        // and need not be gentle)
        const bool gentle = f.zero_vecs * 16 <= kZeroGentleBytes && fin_threads != 1024;
        f.zero_threads = gentle ? kZeroGentleThreads : fin_threads;
        const uint64_t per_cta = (uint64_t)f.zero_threads * (gentle ? kZeroPerThread : kZeroPerThreadFast);
        uint64_t ctas = (f.zero_vecs + 1 + per_cta - 1) / per_cta;
        if (ctas < (uint64_t)kZeroCtasMin) ctas = (f.zero_vecs + 1 + f.zero_threads - 1) / f.zero_threads < (uint64_t)kZeroCtasMin
                                                      ? (f.zero_vecs + 1 + f.zero_threads - 1) / f.zero_threads : (uint64_t)kZeroCtasMin;
        spare = (unsigned)ctas;
        f.zero_ctas = (int)spare;
    }
    if (t.num_large + f.fin_small) {
        const dim3 grid(t.num_large + f.fin_small + spare, rows);
        if (fin_threads == 1024) finish_kernel<1024><<<grid, 1024, fin_dyn, st>>>(f);
        else if (fin_threads == 256) finish_kernel<256><<<grid, 256, fin_dyn, st>>>(f);
        else finish_kernel<kFinThreads><<<grid, kFinThreads, fin_dyn, st>>>(f);
        ++g_kernel_launches;
    }
    if (forked) {
        const cudaError_t e = cudaStreamWaitEvent(st, join, 0);
        if (e != cudaSuccess) return e;
    }
    return cudaGetLastError();
}

cudaError_t launch_accumulate_select(const SelectTables &t, const float *g, int64_t g_stride, float *u, float *v, int K,
                                     int64_t N, float m, int sel_row0, int sel_rows, int32_t epoch, int32_t *errword,
                                     cudaStream_t st)
{
    FastArgs f;
    fill_args(f, t, v, N, 0, nullptr, 0, epoch, errword);
    if (t.num_dense)
        accumulate_select_kernel<true><<<dim3(t.tiles_per_row, K), kAccThreads, 0, st>>>(f, g, g_stride, u, v, N, m, sel_row0, sel_rows);
    else
        accumulate_select_kernel<false><<<dim3(t.tiles_per_row, K), kAccThreads, 0, st>>>(f, g, g_stride, u, v, N, m, sel_row0, sel_rows);
    ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace lgc
