// Grid-level top-k over result records.  Every pass sorts chunks of kChunk entries in
// shared memory with a bitonic network under the exact ranking order and keeps the k best
// of each chunk; passes repeat until one chunk is left, whose k best are the answer.
#include "common.cuh"

namespace maaso {

constexpr int kChunk = 4096;
constexpr int kTopkThreads = 1024;

struct Entry {
    uint64_t sum_ttft;
    uint32_t n_hit;
    uint32_t n_served;
    uint32_t idx;    // candidate index; 0xFFFFFFFF = padding
    uint32_t valid;  // 1 = scored candidate
};
static_assert(sizeof(Entry) == 24, "entry layout");

// true if a ranks strictly before b: scored first, more hits, lower mean first-token latency
// (exact: sum_a * n_b < sum_b * n_a in 128 bits; nothing served ranks after something served),
// lower index.
__device__ __forceinline__ bool ranks_before(const Entry& a, const Entry& b) {
    if (a.valid != b.valid) return a.valid > b.valid;
    if (a.valid) {
        if (a.n_hit != b.n_hit) return a.n_hit > b.n_hit;
        const bool sa = a.n_served > 0, sb = b.n_served > 0;
        if (sa != sb) return sa;
        if (sa) {
            const uint64_t l_lo = a.sum_ttft * (uint64_t)b.n_served;
            const uint64_t l_hi = __umul64hi(a.sum_ttft, (uint64_t)b.n_served);
            const uint64_t r_lo = b.sum_ttft * (uint64_t)a.n_served;
            const uint64_t r_hi = __umul64hi(b.sum_ttft, (uint64_t)a.n_served);
            if (l_hi != r_hi) return l_hi < r_hi;
            if (l_lo != r_lo) return l_lo < r_lo;
        }
    }
    return a.idx < b.idx;
}

// Order 1 ranks by a score: the entry carries the bit pattern of the score mapped so that
// unsigned order = descending score (as sum_ttft with n_served = 1, n_hit = 0), NaN = not valid.
__device__ __forceinline__ uint64_t descending_key(double s) {
    const uint64_t b = (uint64_t)__double_as_longlong(s);
    const uint64_t ascending = (b >> 63) ? ~b : (b | (1ull << 63));
    return ~ascending;
}

// src_res != null: first pass, entries are built from records [0, n).  Otherwise entries
// come from src_ent[0, n).  Block b sorts its chunk and writes its k best to dst_ent[b*k ..]
// or, when `final`, candidate indices / records to out_idx / out_res.
__global__ void __launch_bounds__(kTopkThreads)
topk_pass_kernel(const maaso_result* src_res, const Entry* src_ent, uint64_t n, uint32_t k,
                 Entry* dst_ent, int final_pass, const maaso_result* all_res, uint32_t* out_idx,
                 maaso_result* out_res, const double* scores) {
    extern __shared__ __align__(16) unsigned char topk_smem[];
    Entry* e = reinterpret_cast<Entry*>(topk_smem);
    const uint64_t base = (uint64_t)blockIdx.x * kChunk;
    for (int i = threadIdx.x; i < kChunk; i += kTopkThreads) {
        const uint64_t g = base + i;
        Entry v;
        v.sum_ttft = 0; v.n_hit = 0; v.n_served = 0; v.idx = 0xFFFFFFFFu; v.valid = 0;
        if (g < n) {
            if (src_res) {
                const uint4 a = reinterpret_cast<const uint4*>(src_res + g)[0];  // status, counted, served, hit
                const uint4 d = reinterpret_cast<const uint4*>(src_res + g)[3];  // .., .., sum_ttft lo, hi
                v.idx = (uint32_t)g;
                v.valid = a.x == 0 ? 1u : 0u;
                v.n_served = a.z;
                v.n_hit = a.w;
                v.sum_ttft = ((uint64_t)d.w << 32) | d.z;
                if (scores) {
                    const double sc = scores[g];
                    v.valid = sc == sc ? 1u : 0u;
                    v.n_hit = 0;
                    v.n_served = 1;
                    v.sum_ttft = descending_key(sc);
                }
            } else {
                v = src_ent[g];
            }
        }
        e[i] = v;
    }
    __syncthreads();
    for (int size = 2; size <= kChunk; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = threadIdx.x; t < kChunk / 2; t += kTopkThreads) {
                const int i = ((t / stride) * stride * 2) + (t % stride);
                const int j = i + stride;
                const bool ascending = (i & size) == 0;
                const Entry a = e[i], b = e[j];
                const bool swap = ascending ? ranks_before(b, a) : ranks_before(a, b);
                if (swap) { e[i] = b; e[j] = a; }
            }
            __syncthreads();
        }
    }
    for (uint32_t i = threadIdx.x; i < k; i += kTopkThreads) {
        if (!final_pass) {
            dst_ent[(uint64_t)blockIdx.x * k + i] = e[i];
        } else {
            const uint32_t idx = e[i].idx;
            out_idx[i] = idx;
            if (out_res) {
                uint4* o = reinterpret_cast<uint4*>(out_res + i);
                if (idx != 0xFFFFFFFFu) {
                    const uint4* s = reinterpret_cast<const uint4*>(all_res + idx);
                    for (int q = 0; q < 8; q++) o[q] = s[q];
                } else {
                    for (int q = 0; q < 8; q++) o[q] = make_uint4(0, 0, 0, 0);
                }
            }
        }
    }
}

size_t topk_scratch_bytes(uint64_t n_cand, uint32_t k) {
    const uint64_t blocks = (n_cand + kChunk - 1) / kChunk;
    return (size_t)(blocks * k * sizeof(Entry)) * 2 + 64;
}

// scratch: at least topk_scratch_bytes(n_cand, k), 16-byte aligned.
cudaError_t launch_topk(const maaso_result* results, uint64_t n_cand, uint32_t k, void* scratch,
                        uint32_t* out_idx, maaso_result* out_res, cudaStream_t stream, int* launches,
                        const double* scores) {
    const size_t smem = (size_t)kChunk * sizeof(Entry);
    cudaError_t err = cudaFuncSetAttribute(topk_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem);
    if (err != cudaSuccess) return err;
    const uint64_t blocks0 = (n_cand + kChunk - 1) / kChunk;
    Entry* buf[2];
    buf[0] = reinterpret_cast<Entry*>(scratch);
    buf[1] = buf[0] + blocks0 * k;
    const maaso_result* src_res = results;
    const Entry* src_ent = nullptr;
    uint64_t n = n_cand;
    int which = 0;
    for (;;) {
        const uint64_t blocks = n == 0 ? 1 : (n + kChunk - 1) / kChunk;
        const int final_pass = blocks == 1;
        topk_pass_kernel<<<(unsigned)blocks, kTopkThreads, smem, stream>>>(
            src_res, src_ent, n, k, buf[which], final_pass, results, out_idx, out_res, scores);
        (*launches)++;
        if (final_pass) break;
        src_res = nullptr;
        src_ent = buf[which];
        n = blocks * k;
        which ^= 1;
    }
    return cudaGetLastError();
}

// ---- top-k for callers that cannot allocate ---------------------------------------------------
// The partial lists of the passes live in a fixed array inside the library image instead of
// memory obtained at run time.  Every pass writes each entry the next pass reads, so nothing
// in the array has to be cleared between calls.
constexpr uint64_t kNoAllocMaxCand = MAASO_NOALLOC_MAX_CAND;
constexpr uint32_t kNoAllocMaxK = MAASO_NOALLOC_MAX_K;
constexpr size_t kNoAllocBytes =
    ((((kNoAllocMaxCand + kChunk - 1) / kChunk) * kNoAllocMaxK * sizeof(Entry) * 2 + 64) + 255) / 256 * 256;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// The device address of the array on the current device: its name is only a host-side handle and
// must not be handed to a kernel.  Looked up on every call (no allocation, no stream work), so no
// cached pointer can go stale when a context is re-created, and host threads share nothing.
static cudaError_t noalloc_scratch(void** out) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    *out = p;
    return cudaSuccess;
}

}  // namespace maaso

extern "C" MAASO_API int maaso_topk_noalloc(const maaso_result* results, uint64_t n_cand, uint32_t k,
                                            uint32_t order, uint32_t* out_idx, maaso_result* out_res,
                                            void* cuda_stream) {
    using namespace maaso;
    if (k == 0) return MAASO_OK;
    if (!out_idx || (!results && n_cand) || order != 0) return MAASO_EINVAL;
    if (n_cand > kNoAllocMaxCand || k > kNoAllocMaxK) return MAASO_ETOOBIG;  // beyond the fixed scratch
    void* scratch = nullptr;
    if (noalloc_scratch(&scratch) != cudaSuccess) {
        cudaGetLastError();
        return MAASO_ECUDA;
    }
    int launches = 0;
    const cudaError_t e = launch_topk(results, n_cand, k, scratch, out_idx, out_res, (cudaStream_t)cuda_stream,
                                      &launches, nullptr);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return MAASO_ECUDA;
    }
    return MAASO_OK;
}
