// Plans for sequence-sharded prefill: one long sequence cut into contiguous shards of whole blocks,
// one shard per GPU.  The route of the paper is data independent (Section 3.1), so the key/value
// blocks a shard must be sent by the shards in front of it are a pure function of (sequence length,
// shard boundaries, route parameters): block 0, the local window in front of the shard's first
// block, and the dyadic predecessors j - 2^k that fall in front of the shard -- Proposition 1's
// O(log B) per query block.  The exchange itself (point-to-point copies into a landing buffer in the
// receiver's own memory) belongs to the caller's communication library; nothing here touches a peer.
//
//   bf1_shard_needed_blocks   host: which blocks the shard reads but does not own
//   bf1_plan_route_shard      device: the shard's route over its local [needed | own] key/value tensor
// A shard may also own every `stride`-th block (the *_strided entry points): with a power-of-two stride the dyadic
// predecessors j - 2^k, 2^k >= stride, of an owned block are owned too, so that every rank is sent about two
// blocks per block of its own (the window in front of each) and all ranks carry the same work.
#include "bf1_common.cuh"

namespace bf1 {

int check_cfg(const bf1_route_cfg* cfg);   // bf1_plan.cu

// Eq. 1 as a generator: the ascending list P(j), by merging the three ascending candidate streams
// (block 0, dyadic predecessors j - 2^k with k descending, local window j - W .. j).
template <typename F>
__host__ __device__ inline int for_each_selected(const bf1_route_cfg& c, int j, F& f) {
    int deg = 0, last = -1, kmax = -1;
    if (c.dyadic) {
        while ((1 << (kmax + 1)) <= j) ++kmax;
    }
    int a = c.global_first ? 0 : 0x7fffffff;
    int k = kmax;
    int l = j - c.local_blocks;
    if (l < 0) l = 0;
    while (true) {
        const int dcur = (k >= 0) ? j - (1 << k) : 0x7fffffff;
        const int lcur = (l <= j) ? l : 0x7fffffff;
        int m = a < dcur ? a : dcur;
        m = m < lcur ? m : lcur;
        if (m == 0x7fffffff) break;
        if (m == a) a = 0x7fffffff;
        if (m == dcur) --k;
        if (m == lcur) ++l;
        if (m != last) {
            f(m, deg);
            ++deg;
            last = m;
        }
    }
    return deg;
}

// The blocks a shard owns: first, first + stride, ..., `count` of them (stride 1: a contiguous range).
struct Owned {
    int first, stride, count;
    __host__ __device__ bool has(int p) const {
        const int off = p - first;
        return off >= 0 && off % stride == 0 && off / stride < count;
    }
    __host__ __device__ int index(int p) const { return (p - first) / stride; }   // only for owned blocks
    __host__ __device__ int block(int g) const { return first + g * stride; }
};

// Host side: marks the selected blocks that the shard does not own in a bitmap.
struct MarkNotOwned {
    uint64_t* seen;
    Owned own;
    __host__ __device__ void operator()(int p, int) {
        if (!own.has(p)) seen[p >> 6] |= 1ull << (p & 63);
    }
};

// Device side: writes the list entry for block p into the shard's local numbering.
struct WriteLocalEntry {
    int32_t* list;
    const int32_t* needed;
    int num_needed;
    Owned own;
    int max_degree;
    int bad;
    __device__ void operator()(int p, int pos) {
        int idx;
        if (own.has(p)) {
            idx = num_needed + own.index(p);               // an own block: behind the landing area
        } else {
            int lo = 0, hi = num_needed;                    // a received block: its place in the ascending list
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (needed[mid] < p) lo = mid + 1; else hi = mid;
            }
            if (lo >= num_needed || needed[lo] != p) {
                bad |= BF1_DEV_BAD_ROUTE;
                lo = 0;
            }
            idx = lo;
        }
        if (pos < max_degree) list[pos] = idx; else bad |= BF1_DEV_CAPACITY;
    }
};

struct ShardArgs {
    int64_t n_tokens;
    Owned own;
    int32_t num_needed;
    const int32_t* needed;
    bf1_route_cfg cfg;
    bf1_route route;
    int32_t* cu_out;
};

constexpr int kShardThreads = 256;

__global__ void __launch_bounds__(kShardThreads, 1) plan_shard_kernel(const ShardArgs a) {
    __shared__ int32_t s_bad;
    __shared__ unsigned long long s_total;
    __shared__ int32_t s_hist[66];
    const int tid = threadIdx.x;
    const bf1_route& r = a.route;
    const int b = a.cfg.block;
    const int nloc = a.own.count;
    if (tid == 0) {
        s_bad = 0;
        s_total = 0ull;
    }
    for (int i = tid; i < 66; i += kShardThreads) s_hist[i] = 0;
    __syncthreads();
    if (tid == 0 && (nloc > r.capacity_qblocks || r.max_degree > 64)) s_bad = BF1_DEV_CAPACITY;
    __syncthreads();
    if (s_bad) {
        if (tid == 0) {
            *r.status = s_bad;
            *r.num_qblocks = 0;
            *r.total_pairs = 0;
            r.sched[0] = 0;
            r.sched[1] = 0;
            a.cu_out[0] = 0;
            a.cu_out[1] = 0;
        }
        return;
    }
    unsigned long long my_pairs = 0ull;
    for (int g = tid; g < nloc; g += kShardThreads) {
        const int j = a.own.block(g);
        const long long left = a.n_tokens - (long long)j * b;
        const int rows = left < b ? (int)left : b;
        int32_t* list = r.kv_idx + (size_t)g * r.max_degree;
        WriteLocalEntry w{list, a.needed, a.num_needed, a.own, r.max_degree, 0};
        const int deg = for_each_selected(a.cfg, j, w);
        if (w.bad) atomicOr(&s_bad, w.bad);
        const int kept = deg < r.max_degree ? deg : r.max_degree;
        for (int e = kept; e < r.max_degree; ++e) list[e] = -1;
        const int32_t pairs = rows * b * (kept - 1) + rows * (rows + 1) / 2;
        r.qb_seq[g] = 0;
        r.qb_block[g] = a.num_needed + g;
        r.kv_count[g] = kept;
        r.pair_count[g] = pairs;
        my_pairs += (unsigned long long)pairs;
        atomicAdd(&s_hist[kept], 1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) my_pairs += __shfl_down_sync(0xffffffffu, my_pairs, off);
    if ((tid & 31) == 0 && my_pairs) atomicAdd(&s_total, my_pairs);
    __syncthreads();
    // hand-out order: slots by descending list length (counting sort)
    if (tid == 0) {
        int32_t run = 0;
        for (int dg = 65; dg >= 0; --dg) {
            const int32_t c = s_hist[dg];
            s_hist[dg] = run;
            run += c;
        }
    }
    __syncthreads();
    for (int g = tid; g < nloc; g += kShardThreads) {
        const int pos = atomicAdd(&s_hist[r.kv_count[g]], 1);
        r.order[pos] = g;
    }
    if (tid == 0) {
        // every owned block but the last is full (it precedes another block of the sequence)
        const long long last_left = a.n_tokens - (long long)a.own.block(nloc - 1) * b;
        const long long own_tokens = (long long)(nloc - 1) * b + (last_left < b ? last_left : b);
        *r.status = s_bad;
        *r.num_qblocks = s_bad ? 0 : nloc;
        *r.total_pairs = (int64_t)s_total;
        r.sched[0] = 0;
        r.sched[1] = 0;
        a.cu_out[0] = 0;
        a.cu_out[1] = (int32_t)((long long)a.num_needed * b + own_tokens);
    }
}

// A shard is `count` blocks first, first + stride, ... of a sequence of n_tokens tokens.
static int check_shard(int64_t n_tokens, const bf1_route_cfg* cfg, int32_t first, int32_t stride, int32_t count) {
    if (int rc = check_cfg(cfg)) return rc;
    if (cfg->block != 64) return fail(BF1_ERR_UNSUPPORTED, "sequence sharding is built for b = 64 only (block width %d)", cfg->block);
    if (n_tokens < 1 || n_tokens > 0x7fffffffLL - 64) return fail(BF1_ERR_INVALID_ARG, "n_tokens %lld out of range", (long long)n_tokens);
    const int64_t nb = (n_tokens + cfg->block - 1) / cfg->block;
    if (first < 0 || stride < 1 || count < 1 || (int64_t)first + (int64_t)(count - 1) * stride >= nb)
        return fail(BF1_ERR_INVALID_ARG, "shard blocks %d + k * %d, k < %d, are not inside the sequence's %lld blocks", first,
                    stride, count, (long long)nb);
    return BF1_OK;
}

static int needed_blocks(int64_t n_tokens, const bf1_route_cfg* cfg, const Owned& own, int32_t* blocks_out,
                         int32_t capacity, int32_t* count_out) {
    if (!count_out || capacity < 0 || (capacity > 0 && !blocks_out)) return fail(BF1_ERR_INVALID_ARG, "output pointer is null");
    // every needed block lies in front of the shard's last block: mark them in a bitmap, then read it out in order
    const int last = own.block(own.count - 1);
    const size_t words = ((size_t)last + 63) / 64;
    uint64_t* seen = words ? (uint64_t*)calloc(words, sizeof(uint64_t)) : nullptr;
    if (words && !seen) return fail(BF1_ERR_INVALID_ARG, "out of host memory");
    MarkNotOwned mark{seen, own};
    for (int g = 0; g < own.count; ++g) for_each_selected(*cfg, own.block(g), mark);
    int32_t count = 0;
    for (int p = 0; p < last; ++p)
        if (seen[p >> 6] >> (p & 63) & 1) {
            if (count < capacity) blocks_out[count] = p;
            ++count;
        }
    free(seen);
    *count_out = count;
    if (count > capacity) return fail(BF1_ERR_CAPACITY, "the shard needs %d blocks, room for %d", count, capacity);
    return BF1_OK;
}

static int plan_shard(int64_t n_tokens, const Owned& own, const bf1_route_cfg* cfg, const int32_t* needed_blocks_dev,
                      int32_t num_needed, const bf1_route* out, int32_t* cu_seqlens_out_dev, void* stream) {
    if (!out || !cu_seqlens_out_dev || num_needed < 0 || (num_needed > 0 && !needed_blocks_dev))
        return fail(BF1_ERR_INVALID_ARG, "route, cu_seqlens_out or needed_blocks is null");
    if (!out->qb_seq || !out->qb_block || !out->kv_count || !out->kv_idx || !out->pair_count || !out->order ||
        !out->total_pairs || !out->num_qblocks || !out->status || !out->sched)
        return fail(BF1_ERR_INVALID_ARG, "a route array pointer is null");
    if (out->capacity_qblocks < own.count)
        return fail(BF1_ERR_CAPACITY, "route capacity_qblocks %d < %d query blocks of the shard", out->capacity_qblocks,
                    own.count);
    int32_t cap = 0, need_deg = 0;
    if (int rc = bf1_route_capacity(1, n_tokens, (int32_t)n_tokens, cfg, &cap, &need_deg)) return rc;
    if (out->max_degree < need_deg || out->max_degree > 64)
        return fail(BF1_ERR_CAPACITY, "route max_degree %d: need %d .. 64", out->max_degree, need_deg);
    ShardArgs a;
    a.n_tokens = n_tokens;
    a.own = own;
    a.num_needed = num_needed;
    a.needed = needed_blocks_dev;
    a.cfg = *cfg;
    a.route = *out;
    a.cu_out = cu_seqlens_out_dev;
    plan_shard_kernel<<<1, kShardThreads, 0, (cudaStream_t)stream>>>(a);
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}

}  // namespace bf1

using namespace bf1;

extern "C" int bf1_shard_needed_blocks(int64_t n_tokens, const bf1_route_cfg* cfg, int32_t lo_block, int32_t hi_block,
                                       int32_t* blocks_out, int32_t capacity, int32_t* count_out) {
    if (hi_block <= lo_block) return fail(BF1_ERR_INVALID_ARG, "shard blocks [%d, %d) are empty", lo_block, hi_block);
    if (int rc = check_shard(n_tokens, cfg, lo_block, 1, hi_block - lo_block)) return rc;
    return needed_blocks(n_tokens, cfg, Owned{lo_block, 1, hi_block - lo_block}, blocks_out, capacity, count_out);
}

extern "C" int bf1_plan_route_shard(int64_t n_tokens, int32_t lo_block, int32_t hi_block, const bf1_route_cfg* cfg,
                                    const int32_t* needed_blocks_dev, int32_t num_needed, const bf1_route* out,
                                    int32_t* cu_seqlens_out_dev, void* stream) {
    if (hi_block <= lo_block) return fail(BF1_ERR_INVALID_ARG, "shard blocks [%d, %d) are empty", lo_block, hi_block);
    if (int rc = check_shard(n_tokens, cfg, lo_block, 1, hi_block - lo_block)) return rc;
    return plan_shard(n_tokens, Owned{lo_block, 1, hi_block - lo_block}, cfg, needed_blocks_dev, num_needed, out,
                      cu_seqlens_out_dev, stream);
}

extern "C" int bf1_shard_needed_blocks_strided(int64_t n_tokens, const bf1_route_cfg* cfg, int32_t first_block,
                                               int32_t stride, int32_t num_blocks, int32_t* blocks_out,
                                               int32_t capacity, int32_t* count_out) {
    if (int rc = check_shard(n_tokens, cfg, first_block, stride, num_blocks)) return rc;
    return needed_blocks(n_tokens, cfg, Owned{first_block, stride, num_blocks}, blocks_out, capacity, count_out);
}

extern "C" int bf1_plan_route_shard_strided(int64_t n_tokens, int32_t first_block, int32_t stride, int32_t num_blocks,
                                            const bf1_route_cfg* cfg, const int32_t* needed_blocks_dev,
                                            int32_t num_needed, const bf1_route* out, int32_t* cu_seqlens_out_dev,
                                            void* stream) {
    if (int rc = check_shard(n_tokens, cfg, first_block, stride, num_blocks)) return rc;
    return plan_shard(n_tokens, Owned{first_block, stride, num_blocks}, cfg, needed_blocks_dev, num_needed, out,
                      cu_seqlens_out_dev, stream);
}
