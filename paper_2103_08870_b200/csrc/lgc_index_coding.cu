// Entropy coding of a node's index list (Section V-A of the paper: the transferred indices are
// coded with DEFLATE and their rate counts in the compression ratio).
//
// The list is first turned into bytes: per layer the ascending offsets become gaps (the first one
// counted from the layer's start, the others from the previous offset + 1), each written as a
// little-endian base-128 varint (7 bits per byte, top bit = "more follows").  The bytes are then
// written as ONE DEFLATE block (RFC 1951) with dynamic Huffman codes and literals only: gaps of
// a top-k selection hardly repeat, so the stream's gain is the entropy coding, which is kept, and
// not the string matching, which is left out.  Any inflate implementation decodes the stream.
//
// One CTA does all of it (a list is some tens of kilobytes): varint lengths and a scan, the byte
// histogram, the two length-limited Huffman codes (built by one thread with the two-queue
// method on symbols ranked in parallel), the block header, and the bit-parallel payload (every
// thread packs a contiguous run of bytes and merges its boundary words with atomicOr).
#include "lgc_internal.cuh"

namespace lgc {

namespace {

constexpr int kIcThreads = 1024;
constexpr int kLit = 257;            // literals 0..255 and the end-of-block symbol 256
constexpr int kMaxSyms = 288;

struct HuffWork {
    unsigned freq[kMaxSyms];         // symbol frequencies (halved until the code fits the length limit)
    unsigned node_freq[2 * kMaxSyms];
    short parent[2 * kMaxSyms];
    short order[kMaxSyms];           // symbols with a non-zero frequency, ascending frequency
    unsigned char len[kMaxSyms];
    unsigned short code[kMaxSyms];   // bit-reversed canonical codes: ready for the LSB-first stream
    int used;
};

// rank of every used symbol by (frequency, symbol), computed by all threads; order[] filled
__device__ void rank_symbols(HuffWork &h, int n)
{
    __syncthreads();
    if (threadIdx.x == 0) h.used = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += kIcThreads) {
        const unsigned f = h.freq[i];
        if (f == 0) continue;
        int r = 0;
        for (int j = 0; j < n; ++j) {
            const unsigned g = h.freq[j];
            r += g != 0 && (g < f || (g == f && j < i));
        }
        h.order[r] = (short)i;
        atomicAdd(&h.used, 1);
    }
    __syncthreads();
}

// Huffman code lengths of the n symbols of h.freq, none longer than `limit` bits (frequencies are
// halved, never to zero, and the tree rebuilt until it fits), then the canonical codes of
// RFC 1951 section 3.2.2, stored bit-reversed.  Called by every thread of the CTA.
__device__ void build_code(HuffWork &h, int n, int limit)
{
    __shared__ int too_long;
    for (int i = threadIdx.x; i < n; i += kIcThreads) h.len[i] = 0;
    for (;;) {
        rank_symbols(h, n);
        if (threadIdx.x == 0) {
            const int m = h.used;
            too_long = 0;
            if (m == 1) {
                h.len[h.order[0]] = 1;                    // a lone symbol still needs one bit
            } else if (m > 1) {
                // two queues: the sorted leaves 0 .. m-1 and the internal nodes m .. 2m-2 in creation order
                for (int i = 0; i < m; ++i) h.node_freq[i] = h.freq[h.order[i]];
                int leaf = 0, inner = m, next = m;
                for (; next < 2 * m - 1; ++next) {
                    int pick[2];
                    for (int q = 0; q < 2; ++q) {
                        if (leaf < m && (inner >= next || h.node_freq[leaf] <= h.node_freq[inner])) pick[q] = leaf++;
                        else pick[q] = inner++;
                    }
                    h.node_freq[next] = h.node_freq[pick[0]] + h.node_freq[pick[1]];
                    h.parent[pick[0]] = (short)next;
                    h.parent[pick[1]] = (short)next;
                }
                // depths from the root down: a parent is always created after its children
                unsigned char *depth = reinterpret_cast<unsigned char *>(h.node_freq);   // frequencies are done with
                depth[2 * m - 2] = 0;
                int deepest = 0;
                for (int i = 2 * m - 3; i >= 0; --i) {
                    const int d = depth[h.parent[i]] + 1;
                    depth[i] = (unsigned char)(d > 255 ? 255 : d);
                    if (i < m && d > deepest) deepest = d;
                }
                if (deepest > limit) {
                    too_long = 1;
                    for (int i = 0; i < n; ++i)
                        if (h.freq[i]) h.freq[i] = (h.freq[i] + 1) >> 1;
                } else {
                    for (int i = 0; i < m; ++i) h.len[h.order[i]] = depth[i];
                }
            }
        }
        __syncthreads();
        if (!too_long) break;
    }
    if (threadIdx.x == 0) {
        unsigned count[16] = {0}, next_code[16];
        for (int i = 0; i < n; ++i) count[h.len[i]]++;
        count[0] = 0;
        unsigned c = 0;
        for (int b = 1; b < 16; ++b) {
            c = (c + count[b - 1]) << 1;
            next_code[b] = c;
        }
        for (int i = 0; i < n; ++i) {
            const int l = h.len[i];
            if (!l) continue;
            const unsigned v = next_code[l]++;
            h.code[i] = (unsigned short)(__brev(v) >> (32 - l));
        }
    }
    __syncthreads();
}

// LSB-first bit writer of one thread
struct BitWriter {
    uint32_t *words;
    unsigned long long acc;
    int fill;                        // bits held in acc
    int64_t word;                    // next word to write
    bool shared_first;               // the first word is shared with the previous writer
    __device__ void put(unsigned v, int nbits)
    {
        acc |= (unsigned long long)v << fill;
        fill += nbits;
        if (fill >= 32) flush_word();
    }
    __device__ void flush_word()
    {
        const uint32_t w = (uint32_t)acc;
        if (shared_first) { atomicOr(&words[word], w); shared_first = false; }
        else words[word] = w;
        ++word;
        acc >>= 32;
        fill -= 32;
    }
    __device__ void finish()         // the last, partial word is shared with the next writer
    {
        if ((uint32_t)acc) atomicOr(&words[word], (uint32_t)acc);
    }
};

__device__ __forceinline__ int varint_len(uint32_t g) { return g < (1u << 7) ? 1 : g < (1u << 14) ? 2 : g < (1u << 21) ? 3 : g < (1u << 28) ? 4 : 5; }

__device__ __forceinline__ uint32_t gap_of(const int32_t *__restrict__ idx, const int32_t *__restrict__ slot_layer,
                                           const int32_t *__restrict__ koff, const int64_t *__restrict__ layer_off, int64_t p)
{
    const int l = slot_layer[p];
    return p == koff[l] ? (uint32_t)(idx[p] - (int32_t)layer_off[l]) : (uint32_t)(idx[p] - idx[p - 1] - 1);
}

// out: capacity bytes (a multiple of 4, 4-byte aligned); bytes: work space of 5 mu bytes;
// result[0] = bytes of the stream (if larger than the capacity nothing valid was written),
// result[1] = bytes of the varint form.
__global__ void __launch_bounds__(kIcThreads)
deflate_indices_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ slot_layer,
                       const int32_t *__restrict__ koff, const int64_t *__restrict__ layer_off, int64_t mu,
                       unsigned char *__restrict__ bytes, uint32_t *__restrict__ out, int64_t capacity,
                       unsigned long long *__restrict__ result)
{
    __shared__ HuffWork lit, cl;
    __shared__ unsigned long long scan[kIcThreads];
    __shared__ unsigned long long header_bits_s, total_bytes_s;
    const int tid = threadIdx.x;
    for (int64_t i = tid; i < capacity / 4; i += kIcThreads) out[i] = 0u;
    for (int i = tid; i < kMaxSyms; i += kIcThreads) { lit.freq[i] = 0; cl.freq[i] = 0; }
    __syncthreads();
    // 1. varint bytes: thread t owns slots [p0, p1)
    const int64_t per = (mu + kIcThreads - 1) / kIcThreads;
    const int64_t p0 = per * tid < mu ? per * tid : mu, p1 = p0 + per < mu ? p0 + per : mu;
    unsigned long long mine = 0;
    for (int64_t p = p0; p < p1; ++p) mine += varint_len(gap_of(idx, slot_layer, koff, layer_off, p));
    scan[tid] = mine;
    __syncthreads();
    if (tid == 0) {
        unsigned long long run = 0;
        for (int i = 0; i < kIcThreads; ++i) { const unsigned long long v = scan[i]; scan[i] = run; run += v; }
        total_bytes_s = run;
    }
    __syncthreads();
    {
        unsigned long long at = scan[tid];
        for (int64_t p = p0; p < p1; ++p) {
            uint32_t g = gap_of(idx, slot_layer, koff, layer_off, p);
            do {
                const unsigned char b = (unsigned char)((g & 0x7fu) | (g >= 0x80u ? 0x80u : 0u));
                bytes[at++] = b;
                atomicAdd(&lit.freq[b], 1u);
                g >>= 7;
            } while (g);
        }
    }
    if (tid == 0) lit.freq[256] = 1;                       // one end-of-block symbol
    __syncthreads();
    const unsigned long long total_bytes = total_bytes_s;
    // 2. the literal code (at most 15 bits), and the code for its 258 lengths (at most 7 bits): 257
    //    literal/length code lengths followed by the single, unused distance code of length 0
    build_code(lit, kLit, 15);
    for (int i = tid; i < kLit; i += kIcThreads) atomicAdd(&cl.freq[lit.len[i]], 1u);
    if (tid == 0) atomicAdd(&cl.freq[0], 1u);
    __syncthreads();
    build_code(cl, 19, 7);
    // 3. the header, by one thread
    if (tid == 0) {
        BitWriter w{out, 0ull, 0, 0, false};
        const int perm[19] = {16, 17, 18, 0, 8, 7, 9, 6, 10, 5, 11, 4, 12, 3, 13, 2, 14, 1, 15};
        int hclen = 19;
        while (hclen > 4 && cl.len[perm[hclen - 1]] == 0) --hclen;
        w.put(1, 1);                 // last block
        w.put(2, 2);                 // dynamic Huffman codes
        w.put(kLit - 257, 5);        // HLIT
        w.put(0, 5);                 // HDIST: one distance code
        w.put(hclen - 4, 4);         // HCLEN
        for (int i = 0; i < hclen; ++i) w.put(cl.len[perm[i]], 3);
        for (int i = 0; i < kLit; ++i) w.put(cl.code[lit.len[i]], cl.len[lit.len[i]]);
        w.put(cl.code[0], cl.len[0]);                      // the distance code's length: 0 = no distances used
        header_bits_s = (unsigned long long)w.word * 32 + w.fill;
        if (w.fill > 0) out[w.word] = (uint32_t)w.acc;     // nobody else has written yet
    }
    __syncthreads();
    // 4. the payload: thread t owns bytes [b0, b1)
    const unsigned long long bper = (total_bytes + kIcThreads - 1) / kIcThreads;
    const unsigned long long b0 = bper * tid < total_bytes ? bper * tid : total_bytes;
    const unsigned long long b1 = b0 + bper < total_bytes ? b0 + bper : total_bytes;
    unsigned long long bits = 0;
    for (unsigned long long i = b0; i < b1; ++i) bits += lit.len[bytes[i]];
    scan[tid] = bits;
    __syncthreads();
    if (tid == 0) {
        unsigned long long run = header_bits_s;
        for (int i = 0; i < kIcThreads; ++i) { const unsigned long long v = scan[i]; scan[i] = run; run += v; }
        const unsigned long long all = run + lit.len[256];
        result[0] = (all + 7) / 8;
        result[1] = total_bytes;
        total_bytes_s = all;                               // reused: bits of the whole stream
        header_bits_s = run;                               // reused: where the end-of-block code starts
    }
    __syncthreads();
    if ((total_bytes_s + 7) / 8 > (unsigned long long)capacity) return;   // does not fit: only the sizes are reported
    {
        const unsigned long long start = scan[tid];
        BitWriter w{out, 0ull, 0, (int64_t)(start >> 5), true};
        w.fill = (int)(start & 31);                        // bits below belong to the previous writer
        for (unsigned long long i = b0; i < b1; ++i) {
            const unsigned char b = bytes[i];
            w.put(lit.code[b], lit.len[b]);
        }
        if (tid == kIcThreads - 1) w.put(lit.code[256], lit.len[256]);
        w.finish();
    }
}

}  // namespace

cudaError_t launch_encode_indices(Ctx &c, int node, unsigned char *out, int64_t capacity, unsigned long long *result)
{
    // the whole row of slots: the autoencoder's layers, then the top-k-only ones, each layer's gaps from its own start
    const int32_t *idx = c.idx + (c.S == 1 ? 0 : (int64_t)node * c.mu_all);
    deflate_indices_kernel<<<1, kIcThreads, 0, c.stream>>>(idx, c.slot_layer, c.koff_dev, c.layer_off_dev, c.mu_all, c.ic_bytes,
                                                          reinterpret_cast<uint32_t *>(out), capacity, result),
        ++g_kernel_launches;
    return cudaGetLastError();
}

// The same coding for a node's innovation positions (parameter server): ascending slots inside each
// layer's run of kept values, gaps counted from the run's first slot.
cudaError_t launch_encode_innovation_positions(Ctx &c, int node, unsigned char *out, int64_t capacity,
                                               unsigned long long *result)
{
    deflate_indices_kernel<<<1, kIcThreads, 0, c.stream>>>(c.inn_pos + (int64_t)node * c.muI, c.inn_slot_layer, c.kioff_dev,
                                                          c.koff64_dev, c.muI, c.ic_bytes, reinterpret_cast<uint32_t *>(out),
                                                          capacity, result),
        ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace lgc
