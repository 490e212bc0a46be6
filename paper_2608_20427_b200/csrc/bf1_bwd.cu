// BF1 attention backward (dQ, dK, dV) over the same route, for sm_100a (head dimension 64 or 128,
// 1, 2 or 4 query heads per KV head).
//
// The paper's correctness gates include a backward pass with finite Q, K and V gradients (Section
// 4.2).  With P = exp(S - LSE) recomputed from the saved LSE and D_i = <dO_i, O_i>:
//     dV_p += P^T dO,   dP = dO V_p^T,   dS = P o (dP - D) * scale,   dQ += dS K_p,   dK_p += dS^T Q.
// Work unit = (query block, KV head) as in the forward pass: the two grouped query heads are the
// 128 rows of every MMA, so their contributions to dK / dV add up inside the tensor core.  Per
// list entry p, five groups of tcgen05 MMAs:
//     S    = Q   K_p^T        (128 x 64 x 128)   A, B K-major from shared memory
//     dP   = dO  V_p^T        (128 x 64 x 128)   same layouts
//     dQ  += dS  K_p          (128 x 128 x 64)   A = dS (bf16, written to shared memory by the threads,
//                                                K-major), B = K_p MN-major; accumulates in TMEM
//     dV^T = dO^T P           (128 x 64 x 128)   A = dO MN-major, B = P MN-major (row-major [q][kv] tile)
//     dK^T = Q^T  dS          (128 x 64 x 128)   A = Q MN-major,  B = dS MN-major
// dV^T / dK^T come out with the head dimension on the TMEM lanes; each thread adds its 64 values
// into fp32 accumulation buffers with coalesced red.global.add.f32 (several query blocks read the
// same KV block), and a second kernel rounds those buffers to bf16.  One CTA per unit and pair of
// query heads (G = 4: two CTAs per unit, whose dK / dV contributions meet in the fp32 buffers; G = 1:
// the second head's rows are cleared and contribute nothing), single-buffered, every step in sequence.
// With d = 64 the transposed products still run as M = 128 MMAs: tensor-memory lanes 64..127 then hold
// nothing of value and are not read.
#include <cuda.h>

#include "bf1_common.cuh"

namespace bf1 {

constexpr int kBlock64 = 64;     // b: tokens per block
constexpr int kBwdThreads = 128;

struct BwdArgs {
    const int32_t* cu_seqlens;
    const int32_t* qb_seq;
    const int32_t* qb_block;
    const int32_t* kv_count;
    const int32_t* kv_idx;
    const int32_t* num_qblocks;
    int32_t max_degree, capacity, total_tokens, hq, hkv, group;
    int32_t* status;
    float scale, scale_log2;
    const __nv_bfloat16* o;
    const __nv_bfloat16* d_o;
    const float* lse;
    __nv_bfloat16* dq;
    float* dk32;   // [T, hkv, d] fp32 accumulation
    float* dv32;
};

template <int D>
struct BwdSmem {
    static constexpr int kQBytes = 128 * D * 2;      // Q / dO tile [D / 64 chunks][128 rows][128 B]
    static constexpr int kKVBytes = 64 * D * 2;      // K / V tile  [D / 64 chunks][64 rows][128 B]
    static constexpr int kQ = 0;
    static constexpr int kDO = kQ + kQBytes;
    static constexpr int kK = kDO + kQBytes;
    static constexpr int kV = kK + kKVBytes;
    // P [128 q rows][64 kv] bf16, 128-byte rows, swizzled (16 KB).  At d = 128 it takes over V's buffer once
    // dP = dO V^T has been computed; at d = 64 the V tile is only 8 KB, so P gets room of its own.
    static constexpr int kP = D == 128 ? kV : kV + kKVBytes;
    static constexpr int kDS = kP + 16384;           // dS same layout
    static constexpr int kBar = kDS + 16384;
    static constexpr int kTotal = kBar + 64;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 2) attn_bwd_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                               const __grid_constant__ CUtensorMap tm_k,
                                                               const __grid_constant__ CUtensorMap tm_v,
                                                               const __grid_constant__ CUtensorMap tm_do,
                                                               const BwdArgs a) {
    using L = BwdSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    // no static shared memory: it would cost a whole extra kilobyte and with it the second CTA per SM
    uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(smem + L::kBar + 32);
    int& s_abort = *reinterpret_cast<int*>(smem + L::kBar + 36);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int slot = blockIdx.x, kvh = blockIdx.y, pair = blockIdx.z;   // pair: which two query heads of the group
    if (a.status && (*a.status & BF1_DEV_WAIT_TIMEOUT)) return;
    if (slot >= min(*a.num_qblocks, a.capacity)) return;
    const int seq = a.qb_seq[slot], j = a.qb_block[slot];
    const int cnt = min(max(a.kv_count[slot], 1), a.max_degree);
    const int32_t* list = a.kv_idx + (size_t)slot * a.max_degree;
    const int seq0 = a.cu_seqlens[seq];
    const int seqlen = a.cu_seqlens[seq + 1] - seq0;
    const int rows_valid = min(kBlock64, seqlen - j * kBlock64);
    const int tok0 = seq0 + j * kBlock64;

    const uint32_t base = smem_u32(smem);
    const uint32_t sQ = base + L::kQ, sDO = base + L::kDO, sK = base + L::kK, sV = base + L::kV;
    const uint32_t sP = base + L::kP, sDS = base + L::kDS;
    const uint32_t bar_q = base + L::kBar, bar_kv = bar_q + 8, bar_a = bar_q + 16, bar_b = bar_q + 24;
    if (tid == 0) {
        s_abort = (base & 1023u) ? 1 : 0;
        if (s_abort && a.status) atomicOr(a.status, BF1_DEV_WAIT_TIMEOUT);
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_a, 1);
        mbar_init(bar_b, 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* abort_flag = &s_abort;
    // dV^T and dK^T reuse the columns of S and dP (which the threads have turned into P and dS by then):
    // 256 columns and 112 KB of shared memory per CTA let two CTAs share an SM
    constexpr uint32_t kColS = 0, kColDP = 64, kColDQ = 128, kColDVt = kColS, kColDKt = kColDP;
    const uint32_t t_lane = tmem + (static_cast<uint32_t>(warp * 32) << 16);

    // rows of this thread: head hl, token tl of the query block
    const int hl = tid >> 6, tl = tid & 63;
    const int h = kvh * a.group + pair * 2 + hl;
    const int tok = tok0 + tl;
    const bool row_ok = tl < rows_valid && pair * 2 + hl < a.group;   // G = 1: rows 64..127 belong to no head

    if (a.group == 1) {
        // one head: rows 64..127 of every column chunk of the Q and dO tiles are never written by a copy; the
        // MMAs still read them, so they are cleared (they then give P = 0 and dS = 0 like rows past a sequence)
        for (int i = tid; i < 2 * (D / 64) * 512; i += kBwdThreads) {
            const int which = i / ((D / 64) * 512), ch = (i / 512) % (D / 64), off = i % 512;
            st_shared_v4((which ? sDO : sQ) + ch * 16384 + 8192 + off * 16, 0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
        __syncthreads();
    }
    if (tid == 0 && !s_abort) {
        if (a.group > 1) {
            mbar_expect_tx(bar_q, 2 * L::kQBytes);
            tma_load_4d(sQ, &tm_q, 0, tok0, h, 0, bar_q);      // h: the pair's first head (hl = 0 here)
            tma_load_4d(sDO, &tm_do, 0, tok0, h, 0, bar_q);
        } else {
            mbar_expect_tx(bar_q, L::kQBytes);                 // 64 rows of each
#pragma unroll
            for (int ch = 0; ch < D / 64; ++ch) {
                tma_load_4d(sQ + ch * 16384, &tm_q, 0, tok0, h, ch, bar_q);
                tma_load_4d(sDO + ch * 16384, &tm_do, 0, tok0, h, ch, bar_q);
            }
        }
    }
    // D_i = <dO_i, O_i> and the row's LSE in the log2 domain
    float Drow = 0.f, lse2 = 0.f;
    if (row_ok) {
        const uint4* op = reinterpret_cast<const uint4*>(a.o + ((size_t)tok * a.hq + h) * D);
        const uint4* gp = reinterpret_cast<const uint4*>(a.d_o + ((size_t)tok * a.hq + h) * D);
#pragma unroll 4
        for (int c = 0; c < D / 8; ++c) {
            const uint4 ov = op[c], gv = gp[c];
            const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                Drow = fmaf(__uint_as_float(ow[e] << 16), __uint_as_float(gw[e] << 16), Drow);
                Drow = fmaf(__uint_as_float(ow[e] & 0xffff0000u), __uint_as_float(gw[e] & 0xffff0000u), Drow);
            }
        }
        lse2 = a.lse[(size_t)h * a.total_tokens + tok] * 1.4426950408889634f;
    }
    mbar_wait(bar_q, 0, abort_flag, a.status);

    constexpr uint32_t kHi = desc_hi_sw128(1024);
    constexpr uint32_t kIdS = idesc_bf16_f32_ab(64, false, false);     // S, dP: 128 x 64, A and B K-major
    constexpr uint32_t kIdQ = idesc_bf16_f32_ab(D, false, true);       // dQ: 128 x 128, B (K tile) MN-major
    constexpr uint32_t kIdT = idesc_bf16_f32_ab(64, true, true);       // dV^T, dK^T: A and B MN-major

    // list entry -> block index, kept inside the sequence whatever the list holds
    auto entry = [&](int it) -> int {
        int p = list[it];
        if (p < 0 || p > j || (it == cnt - 1) != (p == j)) {
            if (tid == 0 && a.status) atomicOr(a.status, BF1_DEV_BAD_ROUTE);
            p = (it == cnt - 1) ? j : 0;
        }
        return p;
    };
    auto load_kv = [&](int p) {   // thread 0 only
        mbar_expect_tx(bar_kv, 2 * L::kKVBytes);
        tma_load_4d(sK, &tm_k, 0, seq0 + p * kBlock64, kvh, 0, bar_kv);
        tma_load_4d(sV, &tm_v, 0, seq0 + p * kBlock64, kvh, 0, bar_kv);
    };
    int p = entry(0);
    if (tid == 0) load_kv(p);
    for (int it = 0; it < cnt; ++it) {
        const int p_next = (it + 1 < cnt) ? entry(it + 1) : 0;
        const bool diag = (it == cnt - 1);
        const int kv_valid = min(kBlock64, seqlen - p * kBlock64);      // key rows of this block inside the sequence
        if (tid == 0) {
            mbar_wait(bar_kv, it & 1, abort_flag, a.status);
            tc_fence_after();
            // S = Q K^T and dP = dO V^T: 8 k-steps of 16 over d
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a_off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4, b_off = ((kk / 4) * 8192 + (kk % 4) * 32) >> 4;
                if (kk == 0) {
                    mma_ss_lohi<false>(tmem + kColS, desc_lo_sw128(sQ, 16) + a_off, desc_lo_sw128(sK, 16) + b_off, kHi, kIdS);
                    mma_ss_lohi<false>(tmem + kColDP, desc_lo_sw128(sDO, 16) + a_off, desc_lo_sw128(sV, 16) + b_off, kHi, kIdS);
                } else {
                    mma_ss_lohi<true>(tmem + kColS, desc_lo_sw128(sQ, 16) + a_off, desc_lo_sw128(sK, 16) + b_off, kHi, kIdS);
                    mma_ss_lohi<true>(tmem + kColDP, desc_lo_sw128(sDO, 16) + a_off, desc_lo_sw128(sV, 16) + b_off, kHi, kIdS);
                }
            }
            mma_commit(bar_a);
        }
        __syncwarp();
        mbar_wait(bar_a, it & 1, abort_flag, a.status);
        tc_fence_after();

        // ---- P and dS for this thread's row, 32 columns at a time, written as bf16 rows ------------
        const uint32_t prow = sP + tid * 128, dsrow = sDS + tid * 128;
        // masked entries get s = -inf (self block, warp-uniform branch) and rows past the end of the
        // sequence an infinite LSE: both give P = 0 exactly, and with it dS = 0
        const float lse_row = row_ok ? lse2 : INFINITY;
        const uint64_t c2p = pack2(a.scale_log2, a.scale_log2), nlp = pack2(-lse_row, -lse_row);
        const uint64_t scp = pack2(a.scale, a.scale), ndp = pack2(-Drow * a.scale, -Drow * a.scale);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t sr[32], dr[32];
            tmem_ld32(t_lane + kColS + half * 32, sr);
            tmem_ld32(t_lane + kColDP + half * 32, dr);
            tmem_wait_ld();
            if (diag) {
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (half * 32 + c > tl) sr[c] = 0xff800000u;   // -inf: causal triangle
            }
            uint32_t pw[16], dw[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint64_t x = fma2(pack2(__uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1])), c2p, nlp);
                float x0, x1;
                unpack2(x, x0, x1);
                const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                // dS = P * (dP - D) * scale
                const uint64_t t = fma2(pack2(__uint_as_float(dr[2 * c]), __uint_as_float(dr[2 * c + 1])), scp, ndp);
                float d0, d1;
                unpack2(mul2(pack2(p0, p1), t), d0, d1);
                pw[c] = pack_bf16x2(p0, p1);
                dw[c] = pack_bf16x2(d0, d1);
            }
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {                          // 16-byte chunk half * 4 + c4 of the 128-byte row
                const int ch = (half * 4 + c4) ^ (tid & 7);
                st_shared_v4(prow + (ch << 4), pw[4 * c4], pw[4 * c4 + 1], pw[4 * c4 + 2], pw[4 * c4 + 3]);
                st_shared_v4(dsrow + (ch << 4), dw[4 * c4], dw[4 * c4 + 1], dw[4 * c4 + 2], dw[4 * c4 + 3]);
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after();
            // dQ += dS K: A = dS [128 q][64 kv] K-major (4 k-steps of 16 kv = 32 bytes), B = K tile MN-major
            // (16 kv rows = 2048 bytes per step, next 64 d columns 8 KB away)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {   // 64 kv rows in steps of 16
                const uint32_t alo = desc_lo_sw128(sDS, 16) + ((kk * 32) >> 4);
                const uint32_t blo = desc_lo_sw128(sK, 8192) + ((kk * 2048) >> 4);
                if (it == 0 && kk == 0) mma_ss_lohi<false>(tmem + kColDQ, alo, blo, kHi, kIdQ);
                else mma_ss_lohi<true>(tmem + kColDQ, alo, blo, kHi, kIdQ);
            }
            // dV^T = dO^T P and dK^T = Q^T dS: A = dO / Q MN-major (M = d: 64 per 128-byte row, next 64 at
            // +16 KB; K = q rows, 16 per step = 2048 bytes), B = P / dS MN-major (N = 64 kv per row)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t ko = (kk * 2048) >> 4;
                if (kk == 0) {
                    mma_ss_lohi<false>(tmem + kColDVt, desc_lo_sw128(sDO, 16384) + ko, desc_lo_sw128(sP, 16) + ko, kHi, kIdT);
                    mma_ss_lohi<false>(tmem + kColDKt, desc_lo_sw128(sQ, 16384) + ko, desc_lo_sw128(sDS, 16) + ko, kHi, kIdT);
                } else {
                    mma_ss_lohi<true>(tmem + kColDVt, desc_lo_sw128(sDO, 16384) + ko, desc_lo_sw128(sP, 16) + ko, kHi, kIdT);
                    mma_ss_lohi<true>(tmem + kColDKt, desc_lo_sw128(sQ, 16384) + ko, desc_lo_sw128(sDS, 16) + ko, kHi, kIdT);
                }
            }
            mma_commit(bar_b);
        }
        __syncwarp();
        mbar_wait(bar_b, it & 1, abort_flag, a.status);
        tc_fence_after();
        // K, V (and P, which lives in V's buffer) are free: fetch the next tile while the sums go out
        if (tid == 0 && it + 1 < cnt) load_kv(p_next);

        // ---- dV^T / dK^T: lane = head-dimension index, 64 key rows along the columns -----------------
        float* dvp = a.dv32 + ((size_t)(seq0 + p * kBlock64) * a.hkv + kvh) * D + tid;
        float* dkp = a.dk32 + ((size_t)(seq0 + p * kBlock64) * a.hkv + kvh) * D + tid;
        const size_t rstride = (size_t)a.hkv * D;
        const bool lane_ok = tid < D;   // d = 64: lanes 64..127 of the transposed products hold nothing (warp-uniform)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t vr[32], kr[32];
            tmem_ld32(t_lane + kColDVt + half * 32, vr);
            tmem_ld32(t_lane + kColDKt + half * 32, kr);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const int kvr = half * 32 + c;
                if (kvr < kv_valid && lane_ok) {
                    atomicAdd(dvp + kvr * rstride, __uint_as_float(vr[c]));
                    atomicAdd(dkp + kvr * rstride, __uint_as_float(kr[c]));
                }
            }
        }
        tc_fence_before();
        __syncthreads();   // dS buffer and the S/dP/dV^T/dK^T columns are free again
        p = p_next;
    }

    // ---- dQ rows -----------------------------------------------------------------------------------
    tc_fence_after();
    __nv_bfloat16* dqrow = a.dq + ((size_t)tok * a.hq + h) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(t_lane + kColDQ + c * 32, r);
        tmem_wait_ld();
        if (row_ok) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
                uint4 w;
                w.x = pack_bf16x2(__uint_as_float(r[e + 0]), __uint_as_float(r[e + 1]));
                w.y = pack_bf16x2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
                w.z = pack_bf16x2(__uint_as_float(r[e + 4]), __uint_as_float(r[e + 5]));
                w.w = pack_bf16x2(__uint_as_float(r[e + 6]), __uint_as_float(r[e + 7]));
                *reinterpret_cast<uint4*>(dqrow + c * 32 + e) = w;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

// fp32 accumulation buffers -> bf16 gradients
__global__ void bwd_round_kernel(const float* __restrict__ src_k, const float* __restrict__ src_v,
                                 __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        dk[i] = __float2bfloat16_rn(src_k[i]);
        dv[i] = __float2bfloat16_rn(src_v[i]);
    }
}

int make_map_4d(CUtensorMap* m, const void* ptr, int64_t T, int H, int d, int heads_per_box, int chunks_per_box);   // bf1_attn.cu

}  // namespace bf1

using namespace bf1;

extern "C" int64_t bf1_attn_bwd_workspace_bytes(int64_t total_tokens, int32_t hkv, int32_t d) {
    if (total_tokens < 0 || hkv <= 0 || d <= 0) return -1;
    return 2 * total_tokens * hkv * d * (int64_t)sizeof(float);
}

extern "C" int bf1_attn_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse,
                            const void* d_o, const int32_t* cu_seqlens_dev, int32_t batch, int64_t total_tokens,
                            int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d, float softmax_scale,
                            const bf1_route* route, void* workspace, void* dq, void* dk, void* dv, void* stream) {
    if (!q || !k || !v || !o || !lse || !d_o || !cu_seqlens_dev || !route || !workspace || !dq || !dk || !dv)
        return fail(BF1_ERR_INVALID_ARG, "a pointer is null");
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || hq <= 0 || hkv <= 0)
        return fail(BF1_ERR_INVALID_ARG, "negative or zero size argument");
    if (total_tokens > 0x7fffffffLL - 64) return fail(BF1_ERR_UNSUPPORTED, "total_tokens does not fit 32-bit token indices");
    if (hq % hkv != 0) return fail(BF1_ERR_INVALID_ARG, "hq %d is not a multiple of hkv %d", hq, hkv);
    const int group = hq / hkv;
    if (group != 1 && group != 2 && group != 4)
        return fail(BF1_ERR_UNSUPPORTED, "GQA group size %d: only G = 1, 2 and 4 are supported", group);
    if (d != 64 && d != 128) return fail(BF1_ERR_UNSUPPORTED, "head dimension %d: only 64 and 128 are supported", d);
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o | (uintptr_t)d_o | (uintptr_t)dq | (uintptr_t)dk |
         (uintptr_t)dv | (uintptr_t)workspace) & 15)
        return fail(BF1_ERR_INVALID_ARG, "tensors and workspace must be 16-byte aligned");
    if (!route->qb_seq || !route->qb_block || !route->kv_count || !route->kv_idx || !route->num_qblocks || !route->status)
        return fail(BF1_ERR_INVALID_ARG, "a route array pointer is null");
    if (route->capacity_qblocks < 1 || route->max_degree < 1 || hkv > 65535)
        return fail(BF1_ERR_CAPACITY, "bad route capacities or hkv");
    if (total_tokens == 0 || batch == 0) return BF1_OK;
    int dev = 0, major = 0;
    BF1_CUDA_CHECK(cudaGetDevice(&dev));
    BF1_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return fail(BF1_ERR_NO_DEVICE, "device compute capability %d.x is not sm_100", major);
    BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<128>::kTotal));
    BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<64>::kTotal));
    // two CTAs per SM need the whole shared-memory carve-out
    BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared));
    BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared));
    CUtensorMap tq, tk, tv, tg;
    // Q and dO: two heads and all column chunks per copy; with one head per KV head, one head and one chunk
    const int q_heads = group == 1 ? 1 : 2, q_chunks = group == 1 ? 1 : d / 64;
    if (int rc = make_map_4d(&tq, q, total_tokens, hq, d, q_heads, q_chunks)) return rc;
    if (int rc = make_map_4d(&tg, d_o, total_tokens, hq, d, q_heads, q_chunks)) return rc;
    if (int rc = make_map_4d(&tk, k, total_tokens, hkv, d, 1, d / 64)) return rc;
    if (int rc = make_map_4d(&tv, v, total_tokens, hkv, d, 1, d / 64)) return rc;
    const size_t n_kv = (size_t)total_tokens * hkv * d;
    BwdArgs a;
    a.cu_seqlens = cu_seqlens_dev;
    a.qb_seq = route->qb_seq;
    a.qb_block = route->qb_block;
    a.kv_count = route->kv_count;
    a.kv_idx = route->kv_idx;
    a.num_qblocks = route->num_qblocks;
    a.max_degree = route->max_degree;
    a.capacity = route->capacity_qblocks;
    a.total_tokens = (int32_t)total_tokens;
    a.hq = hq;
    a.hkv = hkv;
    a.group = group;
    a.status = route->status;
    a.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)d);
    a.scale_log2 = a.scale * 1.4426950408889634f;
    a.o = (const __nv_bfloat16*)o;
    a.d_o = (const __nv_bfloat16*)d_o;
    a.lse = lse;
    a.dq = (__nv_bfloat16*)dq;
    a.dk32 = (float*)workspace;
    a.dv32 = a.dk32 + n_kv;
    cudaStream_t st = (cudaStream_t)stream;
    BF1_CUDA_CHECK(cudaMemsetAsync(workspace, 0, 2 * n_kv * sizeof(float), st));
    dim3 grid(route->capacity_qblocks, hkv, group == 4 ? 2 : 1);   // z: pairs of query heads
    if (d == 128) attn_bwd_kernel<128><<<grid, kBwdThreads, BwdSmem<128>::kTotal, st>>>(tq, tk, tv, tg, a);
    else attn_bwd_kernel<64><<<grid, kBwdThreads, BwdSmem<64>::kTotal, st>>>(tq, tk, tv, tg, a);
    BF1_CUDA_CHECK(cudaGetLastError());
    bwd_round_kernel<<<296, 512, 0, st>>>(a.dk32, a.dv32, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, n_kv);
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}
