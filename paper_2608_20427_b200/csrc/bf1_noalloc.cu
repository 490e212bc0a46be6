// bf1_attn_fwd_noalloc: the BF1 forward for callers that cannot allocate device memory.
//
// Some callers run where cudaMalloc is off limits: inside a region whose memory was fixed
// up front (an inference server after start-up, a real-time loop), under an allocator that
// forbids growth, or from a thread that must not take the allocator's locks.  bf1_plan_route
// + bf1_attn_fwd ask such a caller for eight route arrays it has nowhere to put.  This entry
// point keeps them instead in one file-scope device array of fixed size, plans the route into
// it and runs the attention kernel from it.  The caller passes only inputs and outputs.
//
// What to know:
//   - The array is kScratchBytes (about 0.6 MB) of device memory on every GPU that loads the
//     library, held until the process exits.
//   - Limits: at most kMaxQBlocks query blocks in the batch and lists of at most kMaxDegree
//     entries.  The host does not know the individual lengths, so the block count it checks is
//     bf1_route_capacity's upper bound for (batch, total_tokens): one sequence of 262,144 tokens
//     is exactly 4096 blocks and is accepted; a batch of B sequences may hold
//     64 * (4096 - B) + B tokens.  Larger requests return BF1_ERR_CAPACITY and launch nothing.
//   - Host-checkable argument errors (null or misaligned pointers, unsupported geometry) are
//     reported before the planner is launched.
//   - The first call on a device looks up the array's device address (no allocation); make
//     that first call outside any stream capture.
//   - Every call uses the same array and overwrites what the previous call left (the planner
//     rewrites all of it, including the status and hand-out words that must start at zero).
//     Calls that can overlap on the GPU -- different streams without ordering -- race on it.
//   - No cudaMalloc, cudaFree or allocating library routine is called.
#include "bf1_common.cuh"

namespace bf1 {
int check_attn_args(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev, int32_t batch,
                    int64_t total_tokens, int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d, const void* o,
                    const float* lse);   // bf1_attn.cu
}

namespace {

constexpr int kMaxQBlocks = 4096;
constexpr int kMaxDegree = 32;

// Layout of the scratch array, in int32 words.
constexpr size_t kOffSeq = 0;
constexpr size_t kOffBlock = kOffSeq + kMaxQBlocks;
constexpr size_t kOffCount = kOffBlock + kMaxQBlocks;
constexpr size_t kOffPairs = kOffCount + kMaxQBlocks;
constexpr size_t kOffOrder = kOffPairs + kMaxQBlocks;
constexpr size_t kOffIdx = kOffOrder + kMaxQBlocks;
constexpr size_t kOffTotal = kOffIdx + (size_t)kMaxQBlocks * kMaxDegree;   // int64, 8-byte aligned
constexpr size_t kOffNum = kOffTotal + 2;
constexpr size_t kOffStatus = kOffNum + 1;
constexpr size_t kOffSched = kOffStatus + 1;
constexpr size_t kScratchWords = kOffSched + 2;
constexpr size_t kScratchBytes = kScratchWords * sizeof(int32_t);
static_assert(kOffTotal % 2 == 0, "total_pairs must be 8-byte aligned");
static_assert(kScratchBytes < (1u << 20), "the built-in scratch is meant to stay modest");

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) int32_t g_scratch[kScratchWords];

// Device address of g_scratch on the current device, looked up once per device.
int scratch_address(int32_t** out) {
    static int32_t* cache[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return bf1::fail(BF1_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return bf1::fail(BF1_ERR_NO_DEVICE, "device ordinal %d out of range", dev);
    if (!cache[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess || !p)
            return bf1::fail(BF1_ERR_CUDA, "cudaGetSymbolAddress(scratch) failed: %s", cudaGetErrorString(e));
        cache[dev] = static_cast<int32_t*>(p);
    }
    *out = cache[dev];
    return BF1_OK;
}

}  // namespace

extern "C" int bf1_attn_fwd_noalloc(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev,
                                    int32_t batch, int64_t total_tokens, int32_t max_seqlen, int32_t hq,
                                    int32_t hkv, int32_t d, float softmax_scale, const bf1_route_cfg* cfg,
                                    void* o, float* lse, int32_t* status_dev, void* stream) {
    if (int rc = bf1::check_attn_args(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, o, lse))
        return rc;
    int32_t need_blocks = 0, need_degree = 0;
    if (int rc = bf1_route_capacity(batch, total_tokens, max_seqlen, cfg, &need_blocks, &need_degree)) return rc;
    if (need_blocks > kMaxQBlocks)
        return bf1::fail(BF1_ERR_CAPACITY,
                         "bf1_attn_fwd_noalloc: batch may need %d query blocks, the built-in scratch holds %d "
                         "(use bf1_plan_route + bf1_attn_fwd with caller-owned route arrays)",
                         need_blocks, kMaxQBlocks);
    if (need_degree > kMaxDegree)
        return bf1::fail(BF1_ERR_CAPACITY,
                         "bf1_attn_fwd_noalloc: route lists of %d entries, the built-in scratch holds %d per block",
                         need_degree, kMaxDegree);
    int32_t* s = nullptr;
    if (int rc = scratch_address(&s)) return rc;
    bf1_route r;
    r.capacity_qblocks = kMaxQBlocks;
    r.max_degree = kMaxDegree;
    r.qb_seq = s + kOffSeq;
    r.qb_block = s + kOffBlock;
    r.kv_count = s + kOffCount;
    r.pair_count = s + kOffPairs;
    r.order = s + kOffOrder;
    r.kv_idx = s + kOffIdx;
    r.total_pairs = reinterpret_cast<int64_t*>(s + kOffTotal);
    r.num_qblocks = s + kOffNum;
    r.status = status_dev ? status_dev : s + kOffStatus;
    r.sched = s + kOffSched;
    if (int rc = bf1_plan_route(cu_seqlens_dev, batch, total_tokens, max_seqlen, cfg, &r, stream)) return rc;
    return bf1_attn_fwd(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, softmax_scale, &r, o,
                        lse, stream);
}
