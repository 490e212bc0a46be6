// BF1 block-gather flash-attention forward for sm_100a.
//
// Work unit = one query block (64 tokens) of one sequence x one KV head.  The G = 2 query
// heads that share the KV head are stacked into one M = 128 tile (rows 0..63: first head,
// rows 64..127: second head), because they read the same K/V blocks through the same route
// list (the route is per block and the same for all heads, Section 3.1).  For every entry p
// of the unit's list the kernel
//   TMA-loads K[p], V[p] (64 x d each, 128-byte swizzle) into shared memory,
//   S = Q K[p]^T        tcgen05.mma, operands in shared memory, fp32 accumulator in TMEM,
//   online softmax      one thread per row: tcgen05.ld S, mask (self block only), running
//                       max / sum in the exp2 domain, P -> bf16 -> tcgen05.st over S,
//   O += P V[p]         tcgen05.mma with P read from TMEM and V from shared memory,
// and finally writes O / l as bf16 and LSE = max + ln(sum) as fp32.
// With `dense = 1` the list is replaced by 0..j: plain causal attention through the same code.
#include <cuda.h>

#include "bf1_common.cuh"

namespace bf1 {

constexpr int kBlock = 64;      // b: tokens per block
constexpr int kRows = 128;      // MMA M: 2 query heads x 64 tokens
constexpr int kThreads = 128;   // one thread per tile row
constexpr int kStages = 2;      // K/V shared-memory ring

struct AttnArgs {
    const int32_t* cu_seqlens;
    int32_t batch;
    int32_t total_tokens;
    int32_t hq, hkv;
    float scale_log2;      // softmax scale * log2(e)
    int32_t dense;         // 1: every predecessor block, lists ignored
    // route (BF1 mode)
    const int32_t* qb_seq;
    const int32_t* qb_block;
    const int32_t* kv_count;
    const int32_t* kv_idx;
    const int32_t* num_qblocks;
    int32_t max_degree;
    int32_t* status;       // may be null in dense mode
    __nv_bfloat16* o;
    float* lse;
};

template <int D>
struct Smem {
    static constexpr int kChunks = D / 64;                 // 128-byte column chunks per row
    static constexpr int kQBytes = kRows * D * 2;          // 32 KB at d = 128
    static constexpr int kKVBytes = kBlock * D * 2;        // 16 KB at d = 128
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kQBytes;
    static constexpr int kVOff = kKOff + kStages * kKVBytes;
    static constexpr int kBarOff = kVOff + kStages * kKVBytes;
    static constexpr int kTotal = kBarOff + 128;
    static constexpr int kDynamic = kTotal + 1024;         // slack for manual 1024-byte alignment
    static constexpr int kTmemCols = (D == 128) ? 256 : 128;
    static constexpr int kColS = 0;                        // S: 64 fp32 columns; P (bf16) reuses 0..31
    static constexpr int kColO = 64;                       // O: D fp32 columns
};

template <int D>
__global__ void __launch_bounds__(kThreads) attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                            const __grid_constant__ CUtensorMap tm_k,
                                                            const __grid_constant__ CUtensorMap tm_v,
                                                            const AttnArgs args) {
    using L = Smem<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // ---- which unit --------------------------------------------------------------------
    const int slot = blockIdx.x;
    const int kvh = blockIdx.y;
    int seq, j, cnt;
    const int32_t* list = nullptr;
    if (args.status && (*args.status & BF1_DEV_WAIT_TIMEOUT)) return;
    if (!args.dense) {
        if (slot >= *args.num_qblocks) return;
        seq = args.qb_seq[slot];
        j = args.qb_block[slot];
        cnt = args.kv_count[slot];
        list = args.kv_idx + (size_t)slot * args.max_degree;
    } else {
        int acc = 0;
        seq = -1;
        j = 0;
        for (int s = 0; s < args.batch; ++s) {
            const int nb = (args.cu_seqlens[s + 1] - args.cu_seqlens[s] + kBlock - 1) / kBlock;
            if (slot < acc + nb) { seq = s; j = slot - acc; break; }
            acc += nb;
        }
        if (seq < 0) return;
        cnt = j + 1;
    }
    const int seq0 = args.cu_seqlens[seq];
    const int seqlen = args.cu_seqlens[seq + 1] - seq0;
    const int rows_valid = min(kBlock, seqlen - j * kBlock);
    const int tok0 = seq0 + j * kBlock;   // first token row of the query block

    // ---- shared memory carve-up ----------------------------------------------------------
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base + L::kQOff;
    const uint32_t sK = base + L::kKOff;
    const uint32_t sV = base + L::kVOff;
    const uint32_t bar_q = base + L::kBarOff;
    const uint32_t bar_kv = bar_q + 8;            // [kStages]
    const uint32_t bar_s = bar_kv + 8 * kStages;
    const uint32_t bar_o = bar_s + 8;

    if (tid == 0) {
        s_abort = 0;
        mbar_init(bar_q, 1);
        for (int s = 0; s < kStages; ++s) mbar_init(bar_kv + 8 * s, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    __syncwarp();
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem_base), L::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(warp * 32) << 16);  // this warp's 32 lanes
    volatile int* abort_flag = &s_abort;

    // row of this thread: head (tid / 64) of the pair, token (tid % 64) of the block
    const int hl = tid >> 6;
    const int tl = tid & 63;

    auto issue_kv = [&](int it) {
        int p = args.dense ? it : list[it];
        if (p < 0 || p > j || (it == cnt - 1) != (p == j)) {   // never index outside the sequence
            if (args.status) atomicOr(args.status, BF1_DEV_BAD_ROUTE);
            p = (it == cnt - 1) ? j : 0;
        }
        const int st = it % kStages;
        const uint32_t bar = bar_kv + 8 * st;
        mbar_expect_tx(bar, 2 * L::kKVBytes);
        const int row = seq0 + p * kBlock;
#pragma unroll
        for (int c = 0; c < L::kChunks; ++c) {
            tma_load_3d(sK + st * L::kKVBytes + c * (kBlock * 128), &tm_k, c * 64, kvh, row, bar);
            tma_load_3d(sV + st * L::kKVBytes + c * (kBlock * 128), &tm_v, c * 64, kvh, row, bar);
        }
    };

    if (tid == 0) {
        mbar_expect_tx(bar_q, L::kQBytes);
#pragma unroll
        for (int c = 0; c < L::kChunks; ++c)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                tma_load_3d(sQ + c * (kRows * 128) + h * (kBlock * 128), &tm_q, c * 64, kvh * 2 + h, tok0, bar_q);
        issue_kv(0);
    }
    __syncwarp();

    constexpr uint32_t kIdescS = idesc_bf16_f32(kBlock, false);   // 128 x 64 x 16, K-major B
    constexpr uint32_t kIdescO = idesc_bf16_f32(D, true);         // 128 x D x 16, MN-major B

    float m_run = -INFINITY;   // running maximum of the raw (unscaled) scores
    float l_run = 0.f;         // running sum of exp2(scaled score - scaled max)

    for (int it = 0; it < cnt; ++it) {
        const int st = it % kStages;
        const bool diag = (it == cnt - 1);
        if (tid == 0) {
            if (it + 1 < cnt) issue_kv(it + 1);   // stage (it+1)%2 was released by bar_o of it-1
            if (it == 0) mbar_wait(bar_q, 0, abort_flag, args.status);
            mbar_wait(bar_kv + 8 * st, (it / kStages) & 1, abort_flag, args.status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a = sQ + (kk / 4) * (kRows * 128) + (kk % 4) * 32;
                const uint32_t b = sK + st * L::kKVBytes + (kk / 4) * (kBlock * 128) + (kk % 4) * 32;
                mma_ss(tmem + L::kColS, smem_desc_sw128(a, 16, 1024), smem_desc_sw128(b, 16, 1024), kIdescS,
                       kk > 0);
            }
            mma_commit(bar_s);
        }
        __syncwarp();
        mbar_wait(bar_s, it & 1, abort_flag, args.status);
        tc_fence_after();

        // ---- softmax on this thread's row ----------------------------------------------
        uint32_t sreg[2][32];
        tmem_ld32(t_lane + L::kColS, sreg[0]);
        tmem_ld32(t_lane + L::kColS + 32, sreg[1]);
        tmem_wait_ld();
        float mx = m_run;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                float s = __uint_as_float(sreg[h][c]);
                if (diag && (h * 32 + c > tl)) s = -INFINITY;   // causal triangle, self block only
                sreg[h][c] = __float_as_uint(s);
                mx = fmaxf(mx, s);
            }
        const float alpha = ex2_approx((m_run - mx) * args.scale_log2);
        const float msc = mx * args.scale_log2;
        float rowsum = 0.f;
        uint32_t preg[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const int h = c >> 4, cc = (c & 15) * 2;
            const float p0 = ex2_approx(fmaf(__uint_as_float(sreg[h][cc]), args.scale_log2, -msc));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sreg[h][cc + 1]), args.scale_log2, -msc));
            rowsum += p0 + p1;
            preg[c] = pack_bf16x2(p0, p1);
        }
        l_run = l_run * alpha + rowsum;
        m_run = mx;
        tmem_st32(t_lane + L::kColS, preg);   // P overwrites the first 32 columns of S
        if (it > 0) {                         // rescale the running output
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t oreg[32];
                tmem_ld32(t_lane + L::kColO + c * 32, oreg);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
                tmem_st32(t_lane + L::kColO + c * 32, oreg);
            }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < kBlock / 16; ++kk) {
                // V tile: rows = kv tokens (K of this MMA), 128-byte rows of 64 d-elements;
                // 16 kv rows per MMA = two 8-row groups = 2048 bytes; next d chunk 8 KB away
                const uint32_t b = sV + st * L::kKVBytes + kk * 2048;
                mma_ts(tmem + L::kColO, tmem + L::kColS + kk * 8, smem_desc_sw128(b, kBlock * 128, 1024),
                       kIdescO, (it > 0 || kk > 0));
            }
            mma_commit(bar_o);
        }
        __syncwarp();
        mbar_wait(bar_o, it & 1, abort_flag, args.status);
        tc_fence_after();
    }

    // ---- epilogue: O / l -> bf16, LSE ------------------------------------------------------
    const float inv_l = 1.f / l_run;
    const int tok = tok0 + tl;
    const bool store = tl < rows_valid;
    __nv_bfloat16* orow = args.o + ((size_t)tok * args.hq + (kvh * 2 + hl)) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t oreg[32];
        tmem_ld32(t_lane + L::kColO + c * 32, oreg);
        tmem_wait_ld();
        if (store) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
                uint4 w;
                w.x = pack_bf16x2(__uint_as_float(oreg[e + 0]) * inv_l, __uint_as_float(oreg[e + 1]) * inv_l);
                w.y = pack_bf16x2(__uint_as_float(oreg[e + 2]) * inv_l, __uint_as_float(oreg[e + 3]) * inv_l);
                w.z = pack_bf16x2(__uint_as_float(oreg[e + 4]) * inv_l, __uint_as_float(oreg[e + 5]) * inv_l);
                w.w = pack_bf16x2(__uint_as_float(oreg[e + 6]) * inv_l, __uint_as_float(oreg[e + 7]) * inv_l);
                *reinterpret_cast<uint4*>(orow + c * 32 + e) = w;
            }
        }
    }
    if (store) {
        const float lse2 = m_run * args.scale_log2 + lg2_approx(l_run);   // log2 domain
        args.lse[(size_t)(kvh * 2 + hl) * args.total_tokens + tok] = lse2 * 0.6931471805599453f;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, L::kTmemCols);
}

// ---- host side ---------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int get_encode_fn(EncodeTiledFn* fn) {
    static EncodeTiledFn cached = nullptr;
    if (!cached) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        BF1_CUDA_CHECK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres));
        if (!p || qres != cudaDriverEntryPointSuccess)
            return fail(BF1_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        cached = reinterpret_cast<EncodeTiledFn>(p);
    }
    *fn = cached;
    return BF1_OK;
}

// [T, H, d] bf16 tensor, box = 64 tokens x 1 head x 64 elements (128 bytes), 128-byte swizzle.
static int make_map(CUtensorMap* m, const void* ptr, int64_t T, int H, int d) {
    EncodeTiledFn enc;
    if (int rc = get_encode_fn(&enc)) return rc;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)H * d * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)kBlock};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(BF1_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return BF1_OK;
}

static int check_device() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(BF1_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e));
    int major = 0;
    BF1_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return fail(BF1_ERR_NO_DEVICE, "device compute capability %d.x is not sm_100", major);
    return BF1_OK;
}

template <int D>
static int launch(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const AttnArgs& a,
                  int slots, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            Smem<D>::kDynamic));
        configured = true;
    }
    dim3 grid(slots, a.hkv);
    attn_fwd_kernel<D><<<grid, kThreads, Smem<D>::kDynamic, stream>>>(tq, tk, tv, a);
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}

static int attn_common(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev, int32_t batch,
                       int64_t total_tokens, int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d,
                       float softmax_scale, const bf1_route* route, void* o, float* lse, int32_t* status_dev,
                       void* stream) {
    if (!q || !k || !v || !o || !lse || !cu_seqlens_dev)
        return fail(BF1_ERR_INVALID_ARG, "a tensor pointer is null");
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || hq <= 0 || hkv <= 0 || d <= 0)
        return fail(BF1_ERR_INVALID_ARG, "negative or zero size argument");
    if (total_tokens > 0x7fffffffLL - 64)
        return fail(BF1_ERR_UNSUPPORTED, "total_tokens %lld does not fit 32-bit token indices", (long long)total_tokens);
    if (hq % hkv != 0) return fail(BF1_ERR_INVALID_ARG, "hq %d is not a multiple of hkv %d", hq, hkv);
    if (hq / hkv != 2) return fail(BF1_ERR_UNSUPPORTED, "GQA group size %d: only G = 2 is supported", hq / hkv);
    if (d != 64 && d != 128) return fail(BF1_ERR_UNSUPPORTED, "head dimension %d: only 64 and 128 are supported", d);
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15)
        return fail(BF1_ERR_INVALID_ARG, "q, k, v and o must be 16-byte aligned");
    if (hkv > 65535) return fail(BF1_ERR_UNSUPPORTED, "hkv %d exceeds the grid limit", hkv);
    int slots;
    if (route) {
        if (!route->qb_seq || !route->qb_block || !route->kv_count || !route->kv_idx || !route->num_qblocks ||
            !route->status)
            return fail(BF1_ERR_INVALID_ARG, "a route array pointer is null");
        if (route->capacity_qblocks < 1 || route->max_degree < 1)
            return fail(BF1_ERR_CAPACITY, "route capacity_qblocks and max_degree must be >= 1");
        slots = route->capacity_qblocks;
    } else {
        const int64_t cap = total_tokens / kBlock + batch;
        if (cap > 0x7fffffffLL) return fail(BF1_ERR_UNSUPPORTED, "too many query blocks");
        slots = (int)cap;
    }
    if (total_tokens == 0 || batch == 0) return BF1_OK;   // nothing to do
    if (int rc = check_device()) return rc;

    CUtensorMap tq, tk, tv;
    if (int rc = make_map(&tq, q, total_tokens, hq, d)) return rc;
    if (int rc = make_map(&tk, k, total_tokens, hkv, d)) return rc;
    if (int rc = make_map(&tv, v, total_tokens, hkv, d)) return rc;

    AttnArgs a;
    a.cu_seqlens = cu_seqlens_dev;
    a.batch = batch;
    a.total_tokens = (int32_t)total_tokens;
    a.hq = hq;
    a.hkv = hkv;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)d);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.dense = route ? 0 : 1;
    a.qb_seq = route ? route->qb_seq : nullptr;
    a.qb_block = route ? route->qb_block : nullptr;
    a.kv_count = route ? route->kv_count : nullptr;
    a.kv_idx = route ? route->kv_idx : nullptr;
    a.num_qblocks = route ? route->num_qblocks : nullptr;
    a.max_degree = route ? route->max_degree : 0;
    a.status = route ? route->status : status_dev;
    a.o = reinterpret_cast<__nv_bfloat16*>(o);
    a.lse = lse;
    if (d == 128) return launch<128>(tq, tk, tv, a, slots, (cudaStream_t)stream);
    return launch<64>(tq, tk, tv, a, slots, (cudaStream_t)stream);
}

}  // namespace bf1

extern "C" int bf1_attn_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev,
                            int32_t batch, int64_t total_tokens, int32_t max_seqlen, int32_t hq, int32_t hkv,
                            int32_t d, float softmax_scale, const bf1_route* route, void* o, float* lse,
                            void* stream) {
    if (!route) return bf1::fail(BF1_ERR_INVALID_ARG, "route is null");
    return bf1::attn_common(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, softmax_scale,
                            route, o, lse, nullptr, stream);
}

extern "C" int bf1_dense_causal_fwd(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev,
                                    int32_t batch, int64_t total_tokens, int32_t max_seqlen, int32_t hq,
                                    int32_t hkv, int32_t d, float softmax_scale, void* o, float* lse,
                                    int32_t* status_dev, void* stream) {
    return bf1::attn_common(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, softmax_scale,
                            nullptr, o, lse, status_dev, stream);
}
