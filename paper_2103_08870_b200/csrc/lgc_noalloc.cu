// lgc_topk_noalloc: exact top-k by magnitude of one flat fp32 vector for callers that cannot
// provide work space.
//
// Who needs this: code that runs where device allocation is off the table -- inside a region
// that has promised its framework a fixed memory footprint, in a plugin whose host owns the
// allocator and hands out only input and output buffers, or late in a job when the device is
// full and a failed allocation would take the job down.  Such callers can still pass the vector
// and the output array; what they cannot pass is the selection's work space (segment tables,
// radix histogram, per-chunk counts).  Here that work space is a fixed array compiled into the
// library, so the vector length is capped (LGC_NOALLOC_MAX_N) and the array costs its ~60 KB on
// every GPU that loads the library, until the process exits.
//
// The selection itself is done by the same kernels as lgc_topk; only where their tables and
// counters live differs.
#include <mutex>

#include "lgc_internal.cuh"

namespace lgc {
namespace {

constexpr int64_t kMaxN = LGC_NOALLOC_MAX_N;
constexpr int kMaxChunks = (int)(kMaxN / kSelChunk);

// Byte offsets of the pieces inside the static array (each 256-byte aligned).
constexpr size_t kOffErr = 0, kOffSegOff = 256, kOffSegLen = 512, kOffSegK = 768, kOffSegOut = 1024,
                 kOffSmallIds = 1280, kOffLargeIds = 1536, kOffChunk0 = 1792, kOffPrefix = 2048, kOffKRem = 2304,
                 kOffHist = 4096, kOffChunkLarge = kOffHist + kHistBins * sizeof(uint32_t),
                 kOffChunkCnt = kOffChunkLarge + kMaxChunks * sizeof(int32_t),
                 kScratchBytes = kOffChunkCnt + kMaxChunks * sizeof(int2);

// The work space.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
// device address and must never be passed to a kernel as one.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Writes the one-segment tables for this call and clears everything that must start at zero
// (the histogram, the chunk->segment map, the check word): the array still holds whatever the
// previous call left in it.
__global__ void noalloc_setup_kernel(unsigned char *base, int32_t n, int32_t k, int32_t chunks)
{
    const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthreads = gridDim.x * blockDim.x;
    if (tid == 0) {
        *reinterpret_cast<int32_t *>(base + kOffErr) = 0;
        *reinterpret_cast<int64_t *>(base + kOffSegOff) = 0;
        *reinterpret_cast<int32_t *>(base + kOffSegLen) = n;
        *reinterpret_cast<int32_t *>(base + kOffSegK) = k;
        *reinterpret_cast<int32_t *>(base + kOffSegOut) = 0;
        *reinterpret_cast<int32_t *>(base + kOffSmallIds) = 0;
        *reinterpret_cast<int32_t *>(base + kOffLargeIds) = 0;
        reinterpret_cast<int32_t *>(base + kOffChunk0)[0] = 0;
        reinterpret_cast<int32_t *>(base + kOffChunk0)[1] = chunks;
        *reinterpret_cast<uint32_t *>(base + kOffPrefix) = 0;
        *reinterpret_cast<int32_t *>(base + kOffKRem) = 0;
    }
    uint32_t *hist = reinterpret_cast<uint32_t *>(base + kOffHist);
    for (int i = tid; i < kHistBins; i += nthreads) hist[i] = 0;
    int32_t *chunk_large = reinterpret_cast<int32_t *>(base + kOffChunkLarge);
    for (int i = tid; i < chunks; i += nthreads) chunk_large[i] = 0;
}

// Device address of the static array on the current device; looked up once per device.
cudaError_t scratch_address(unsigned char **out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static unsigned char *cached[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        cached[dev] = static_cast<unsigned char *>(p);
    }
    *out = cached[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace lgc

using namespace lgc;

extern "C" lgc_status lgc_topk_noalloc(const float *v, int64_t n, int64_t k, int32_t *idx_out, void *stream)
{
    auto fail = [](lgc_status s, const std::string &msg) { g_last_error = msg; return s; };
    if (!v || !idx_out) return fail(LGC_ERR_INVALID_ARG, "lgc_topk_noalloc: v or idx_out is NULL");
    if (n < 1 || k < 1 || k > n) return fail(LGC_ERR_INVALID_ARG, "lgc_topk_noalloc: need 1 <= k <= n");
    if (n > kMaxN)
        return fail(LGC_ERR_UNSUPPORTED, "lgc_topk_noalloc: n exceeds LGC_NOALLOC_MAX_N (" + std::to_string(kMaxN) +
                                             " elements); use lgc_topk with caller-provided scratch");
    unsigned char *base = nullptr;
    cudaError_t e = scratch_address(&base);
    if (e != cudaSuccess) return fail(LGC_ERR_CUDA, std::string("lgc_topk_noalloc: ") + cudaGetErrorString(e));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool small = n <= kSelChunk;
    const int chunks = small ? 0 : (int)((n + kSelChunk - 1) / kSelChunk);
    noalloc_setup_kernel<<<8, 256, 0, s>>>(base, (int32_t)n, (int32_t)k, chunks), ++g_kernel_launches;
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(LGC_ERR_CUDA, std::string("lgc_topk_noalloc: ") + cudaGetErrorString(e));
    SelectTables t;
    t.num_segments = 1;
    t.num_small = small ? 1 : 0;
    t.num_large = small ? 0 : 1;
    t.num_chunks = chunks;
    t.max_rows = 1;
    t.seg_off = reinterpret_cast<int64_t *>(base + kOffSegOff);
    t.seg_len = reinterpret_cast<int32_t *>(base + kOffSegLen);
    t.seg_k = reinterpret_cast<int32_t *>(base + kOffSegK);
    t.seg_out = reinterpret_cast<int32_t *>(base + kOffSegOut);
    t.small_ids = reinterpret_cast<int32_t *>(base + kOffSmallIds);
    t.large_ids = reinterpret_cast<int32_t *>(base + kOffLargeIds);
    t.large_chunk0 = reinterpret_cast<int32_t *>(base + kOffChunk0);
    t.chunk_large = reinterpret_cast<int32_t *>(base + kOffChunkLarge);
    t.hist = reinterpret_cast<uint32_t *>(base + kOffHist);
    t.prefix = reinterpret_cast<uint32_t *>(base + kOffPrefix);
    t.k_rem = reinterpret_cast<int32_t *>(base + kOffKRem);
    t.chunk_cnt = reinterpret_cast<int2 *>(base + kOffChunkCnt);
    e = launch_select_multipass(t, v, n, 0, 1, idx_out, k, reinterpret_cast<int32_t *>(base + kOffErr), s);
    if (e != cudaSuccess) return fail(LGC_ERR_CUDA, std::string("lgc_topk_noalloc: ") + cudaGetErrorString(e));
    return LGC_OK;
}

// What the kernels of the calls so far recorded in the array's check word on the current device
// (the context-based lgc_check does not see it).  Waits for `stream`, copies four bytes to the
// host, allocates nothing, and clears the word when it was set.
extern "C" lgc_status lgc_topk_noalloc_check(void *stream)
{
    auto fail = [](lgc_status s, const std::string &msg) { g_last_error = msg; return s; };
    unsigned char *base = nullptr;
    cudaError_t e = scratch_address(&base);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&word, base + kOffErr, sizeof word, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail(LGC_ERR_CUDA, std::string("lgc_topk_noalloc_check: ") + cudaGetErrorString(e));
    if (word == 0) return LGC_OK;
    e = cudaMemsetAsync(base + kOffErr, 0, sizeof word, s);
    char buf[112];
    snprintf(buf, sizeof buf, "lgc_topk_noalloc: device check 0x%X: a selection kernel found inconsistent counts", (unsigned)word);
    return fail(LGC_ERR_DEVICE_CHECK, buf);
}
