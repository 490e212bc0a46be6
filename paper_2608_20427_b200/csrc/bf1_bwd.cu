// BF1 attention backward (dQ, dK, dV) over the same route, for sm_100a (head dimension 64 or 128,
// 1, 2 or 4 query heads per KV head).
//
// The paper's correctness gates include a backward pass with finite Q, K and V gradients (Section
// 4.2).  With P = exp(S - LSE) recomputed from the saved LSE and D_i = <dO_i, O_i>:
//     dV_p += P^T dO,   dP = dO V_p^T,   dS = P o (dP - D) * scale,   dQ += dS K_p,   dK_p += dS^T Q.
// dQ of a query block sums over the KV blocks of its list; dK / dV of a KV block sum over the query
// blocks that read it.  So there are two kernels, each walking the route in the direction in which its
// output stays put, and nothing is ever added in global memory (no atomics, no fp32 gradient buffers,
// the same bits on every run):
//
//   bwd_dq_kernel    unit = (query block, KV head, pair of query heads), as in the forward pass: the two
//                    heads are the 128 rows of every MMA.  Per list entry p:
//                        S  = Q  K_p^T   (128 x 64 x d)    A, B K-major from shared memory
//                        dP = dO V_p^T   (128 x 64 x d)
//                        dQ += dS K_p    (128 x d x 64)    A = dS (bf16, written over S in tensor memory by
//                                                          the threads), B = K_p MN-major; accumulates in TMEM
//                    It also leaves D_i in the workspace for the second kernel.
//   bwd_dkv_kernel   unit = (KV block p, KV head, a run of the query blocks that read p): the INVERSE
//                    route, which a few small kernels derive from the lists on every call (any lists: the
//                    planner's or the caller's).  Per reader j (and pair of heads), S and dP as above, then
//                        dV^T += dO^T P  (d x 64 x 128)    A = dO MN-major, B = P MN-major ([q][kv] tile)
//                        dK^T += Q^T  dS (d x 64 x 128)    A = Q MN-major,  B = dS MN-major
//                    accumulating in tensor memory across all readers (head dimension on the lanes), and
//                    one store at the end.  A block with very many readers (block 0: every query block)
//                    is cut into runs of `chunk` readers handled by different CTAs; their fp32 partial
//                    sums are added in run order by bwd_combine_kernel.
//
// Both compute kernels are persistent: one CTA of 16 warps per SM that takes all of tensor memory (two S/dP
// buffers and two accumulator buffers) and walks through its share of the units, with warps for copies, for
// issuing MMAs, for the arithmetic on S and dP and for reading finished sums out, so that copies, MMAs and
// arithmetic of neighbouring entries and units overlap (see the comment in front of each kernel).  P is rounded
// to bf16 before the MMAs, as in the forward.  With d = 64 the transposed products still run as M = 128 MMAs:
// tensor-memory lanes 64..127 then hold nothing of value and are not read.
#include <cuda.h>

#include <algorithm>

#include "bf1_common.cuh"

namespace bf1 {

constexpr int kBlock64 = 64;     // b: tokens per block
constexpr int kMinChunk = 16;    // readers per dK/dV unit, at least

// The inverse route and the units of bwd_dkv_kernel, all inside the caller's workspace.
struct InvPlan {
    int32_t* count;       // [cap] readers of KV slot g (with multiplicity)
    int32_t* start;       // [cap + 1] first reader of slot g in `readers`
    int32_t* chunks;      // [cap] runs the slot's readers are cut into
    int32_t* part0;       // [cap] first partial-sum slot of a slot with more than one run, else -1
    int32_t* readers;     // [cap * max_degree] query slots, ascending per KV slot
    int32_t* unit_slot;   // [max_units] KV slot of the unit
    int32_t* unit_begin;  // [max_units] its readers: readers[begin .. end)
    int32_t* unit_end;
    int32_t* unit_part;   // [max_units] partial-sum slot it writes, or -1: it writes the final bf16 rows
    int32_t* unit_order;  // [max_units] units, longest first: the order in which the dK/dV kernel deals them out
    int32_t* multi;       // [cap] the KV slots whose readers were cut into more than one run
    int32_t* scalars;     // [8] number of units, total readers, chunk, partial slots, slots in `multi`
    int32_t cap, max_units;
};

struct BwdArgs {
    const int32_t* cu_seqlens;
    const int32_t* qb_seq;
    const int32_t* qb_block;
    const int32_t* kv_count;
    const int32_t* kv_idx;
    const int32_t* num_qblocks;
    const int32_t* order;      // may be null
    int32_t max_degree, capacity, total_tokens, hq, hkv, group;
    int32_t interleave;    // 1: units of all KV heads interleaved (longest first over all heads); 0: KV head by KV head
    int32_t* status;
    float scale, scale_log2;
    const __nv_bfloat16* o;
    const __nv_bfloat16* d_o;
    const float* lse;
    float* delta;          // [hq, T] D_i = <dO_i, O_i>: written by the dQ kernel, read by the dK/dV kernel
    __nv_bfloat16* dq;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    float* partial;        // [partial slots][hkv][2][64][d] fp32 sums of the runs of a many-reader block
    InvPlan inv;
};

// Entry e of a list as every kernel of this library uses it: kept inside [0, j], the last entry the
// query block itself, whatever the array holds (a caller's route may be wrong; the forward flags it).
__device__ __forceinline__ int list_entry(const int32_t* list, int e, int cnt, int j) {
    int p = list[e];
    if (p < 0 || p > j || (e == cnt - 1) != (p == j)) p = (e == cnt - 1) ? j : 0;
    return p;
}

// ---- pieces shared by the two compute kernels ------------------------------------------------------------------

// S = Q K^T (or dP = dO V^T): D / 16 k-steps over the head dimension, 128 x 64 output, A and B K-major (one thread).
template <int D>
__device__ __forceinline__ void issue_qk(uint32_t t_out, uint32_t sA, uint32_t sB) {
    constexpr uint32_t kHi = desc_hi_sw128(1024);
    constexpr uint32_t kIdS = idesc_bf16_f32_ab(64, false, false);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t a_off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4, b_off = ((kk / 4) * 8192 + (kk % 4) * 32) >> 4;
        if (kk == 0) mma_ss_lohi<false>(t_out, desc_lo_sw128(sA, 16) + a_off, desc_lo_sw128(sB, 16) + b_off, kHi, kIdS);
        else mma_ss_lohi<true>(t_out, desc_lo_sw128(sA, 16) + a_off, desc_lo_sw128(sB, 16) + b_off, kHi, kIdS);
    }
}
template <int D>
__device__ __forceinline__ void issue_s_dp(uint32_t t_s, uint32_t t_dp, uint32_t sQ, uint32_t sDO, uint32_t sK, uint32_t sV) {
    issue_qk<D>(t_s, sQ, sK);
    issue_qk<D>(t_dp, sDO, sV);
}

// P and dS of this thread's 32 columns (half = 0 / 1: columns 0..31 / 32..63) of its row, from S and dP in tensor
// memory.  Masked entries get s = -inf (self block, warp-uniform branch) and rows outside the sequence an infinite
// LSE: both give P = 0 exactly, and with it dS = 0.  Results as packed bf16 pairs.
__device__ __forceinline__ void p_and_ds(uint32_t t_s, uint32_t t_dp, int half, int tl, bool diag, float lse_row2, float drow,
                                         float scale, float scale_log2, uint32_t (&pw)[16], uint32_t (&dw)[16]) {
    const uint64_t c2p = pack2(scale_log2, scale_log2), nlp = pack2(-lse_row2, -lse_row2);
    const uint64_t scp = pack2(scale, scale), ndp = pack2(-drow * scale, -drow * scale);
    uint32_t sr[32], dr[32];
    tmem_ld32(t_s + half * 32, sr);
    tmem_ld32(t_dp + half * 32, dr);
    tmem_wait_ld();
    if (diag) {
#pragma unroll
        for (int c = 0; c < 32; ++c)
            if (half * 32 + c > tl) sr[c] = 0xff800000u;   // -inf: causal triangle
    }
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
}

// The same pairs as a bf16 row piece in shared memory: 128-byte rows, 16-byte chunks XOR-swizzled with the row
// (the layout the MMAs read as an MN-major operand).
__device__ __forceinline__ void store_row_piece(uint32_t row_addr, int row, int half, const uint32_t (&w)[16]) {
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {                          // 16-byte chunk half * 4 + c4 of the 128-byte row
        const int ch = (half * 4 + c4) ^ (row & 7);
        st_shared_v4(row_addr + (ch << 4), w[4 * c4], w[4 * c4 + 1], w[4 * c4 + 2], w[4 * c4 + 3]);
    }
}

// One head per KV head: rows 64..127 of every column chunk of the Q and dO tiles are never written by a copy;
// the MMAs still read them, so they are cleared once (they then give P = 0 and dS = 0 like rows past a sequence).
template <int D>
__device__ __forceinline__ void clear_idle_rows(uint32_t sQ, uint32_t sDO, int tid, int threads) {
    for (int i = tid; i < 2 * (D / 64) * 512; i += threads) {
        const int which = i / ((D / 64) * 512), ch = (i / 512) % (D / 64), off = i % 512;
        st_shared_v4((which ? sDO : sQ) + ch * 16384 + 8192 + off * 16, 0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
}

// One Q-shaped tile (Q, dO or O) of a query block and pair of heads (one thread; expect_tx is the caller's).
template <int D>
__device__ __forceinline__ void load_q_tile(uint32_t dst, const CUtensorMap* tm, int tok0, int head, int group, uint32_t bar) {
    if (group > 1) {
        tma_load_4d(dst, tm, 0, tok0, head, 0, bar);
    } else {
#pragma unroll
        for (int ch = 0; ch < D / 64; ++ch) tma_load_4d(dst + ch * 16384, tm, 0, tok0, head, ch, bar);
    }
}

__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t (&w)[4]) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
}

// ---- dQ --------------------------------------------------------------------------------------------------------
//
// One persistent CTA of 16 warps per SM.  Units (query block, KV head, pair of heads) are dealt out statically, in
// the route's longest-list-first order KV head by KV head, back and forth over the CTAs so that each gets the same
// mix.  Everything a unit needs travels through rings whose next entry is under way while the current one is in
// use, across unit boundaries as well:
//     warp 0    copies Q of every unit (two buffers) and the K tile of every list entry (ring of kStages)
//     warp 1    copies dO of every unit, its O tile (into a whole ring stage, ahead of the unit's K/V tiles) and
//               the V tiles
//     warp 2    issues S and dP of every entry into one of two S/dP buffers in tensor memory, as soon as the K / V
//               tiles are there and the dQ MMAs that read the buffer's last dS are done
//     warp 3    issues the dQ MMAs of every entry; dQ accumulates in one of two buffers
//     warps 4-11   the arithmetic on S and dP, two threads per tile row (32 key columns each); dS (bf16) goes back
//               into tensor memory over S, from where the dQ MMAs read it as their A operand
//     warps 12-15   per unit: D_i = <dO_i, O_i> and the LSE of every row into shared memory (and D_i into the
//               workspace, for the dK/dV kernel) one unit ahead; then the finished dQ tile of the unit before,
//               from tensor memory to global memory
// Every wait of a role is on a barrier it waits on once per phase, in phase order: a parity wait is only
// meaningful one phase ahead.
constexpr int kDqThreads = 512;
constexpr int kStages = 3;
// Q / dO buffer (and barrier) of unit n, and the parity of its n-th use
__device__ __forceinline__ int qbuf(int n) { return n & 1; }
__device__ __forceinline__ uint32_t qpar(int n) { return (n >> 1) & 1; }

template <int D>
struct DqSmem {
    static constexpr int kQBytes = 128 * D * 2;      // Q / dO / O tile [D / 64 chunks][128 rows][128 B]
    static constexpr int kKVBytes = 64 * D * 2;      // K / V tile      [D / 64 chunks][64 rows][128 B]
    static constexpr int kQ = 0;                     // [2]
    static constexpr int kDO = kQ + 2 * kQBytes;     // [2]
    static constexpr int kRing = kDO + 2 * kQBytes;  // [kStages] of K | V (or one O tile)
    static constexpr int kRow = kRing + kStages * 2 * kKVBytes;   // D_i [2][128], LSE [2][128] (fp32)
    static constexpr int kBar = kRow + 2048;
    static constexpr int kUsed = kBar + 512;
    // at least this much is requested so that a second CTA never fits an SM: each allocates all of tensor memory
    static constexpr int kTotal = kUsed > 120 * 1024 ? kUsed : 120 * 1024;
};

struct DqUnit {
    int ok, slot, kvh, pair, cnt, seq0, j, tok0, rows_valid;
};

// Unit n of this CTA (see above for the order).
__device__ __forceinline__ DqUnit dq_unit(const BwdArgs& a, int n, int nqb, int pairs) {
    DqUnit u;
    const int per_head = nqb * pairs, total = per_head * a.hkv;
    const int G = gridDim.x;
    const int i = n * G + ((n & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x);
    u.ok = i < total;
    u.slot = u.kvh = u.pair = u.seq0 = u.j = u.tok0 = 0;
    u.cnt = 1;
    u.rows_valid = 0;
    if (u.ok) {
        int rank;
        if (a.interleave) {          // rank-major: the longest lists of all heads first
            const int per_rank = pairs * a.hkv;
            rank = i / per_rank;
            const int rem = i - rank * per_rank;
            u.kvh = rem / pairs;
            u.pair = rem - u.kvh * pairs;
        } else {                     // head-major: a head's K and V stay hot in L2
            u.kvh = i / per_head;
            const int rem = i - u.kvh * per_head;
            rank = rem / pairs;
            u.pair = rem - rank * pairs;
        }
        int slot = a.order ? a.order[rank] : rank;
        slot = min(max(slot, 0), nqb - 1);
        u.slot = slot;
        const int seq = a.qb_seq[slot];
        u.j = a.qb_block[slot];
        u.cnt = min(max(a.kv_count[slot], 1), a.max_degree);
        u.seq0 = a.cu_seqlens[seq];
        u.rows_valid = min(kBlock64, a.cu_seqlens[seq + 1] - u.seq0 - u.j * kBlock64);
        u.tok0 = u.seq0 + u.j * kBlock64;
    }
    return u;
}

__device__ __forceinline__ void named_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kDqThreads, 1) bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                            const __grid_constant__ CUtensorMap tm_k,
                                                            const __grid_constant__ CUtensorMap tm_v,
                                                            const __grid_constant__ CUtensorMap tm_do,
                                                            const __grid_constant__ CUtensorMap tm_o,
                                                            const BwdArgs a) {
    using L = DqSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(smem + L::kBar + 496);
    int& s_abort = *reinterpret_cast<int*>(smem + L::kBar + 500);
    float* s_drow = reinterpret_cast<float*>(smem + L::kRow);          // [2][128]
    float* s_lse = s_drow + 256;                                       // [2][128]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (a.status && (*a.status & BF1_DEV_WAIT_TIMEOUT)) return;
    const int nqb = min(*a.num_qblocks, a.capacity);
    const int pairs = a.group == 4 ? 2 : 1;

    const uint32_t base = smem_u32(smem);
    const uint32_t bars = base + L::kBar;
    // barriers (8 bytes each)
    const uint32_t qdo_full = bars;                          // [2] Q and dO of a unit landed (both copy warps announce bytes)
    const uint32_t qdo_free = qdo_full + 16;                 // [2] the unit's MMAs are done and its D_i computed
    const uint32_t o_full = qdo_free + 16;                   // [2] the unit's O tile landed
    const uint32_t row_full = o_full + 16;                   // [2] D_i and LSE of the unit's rows are in shared memory
    const uint32_t row_free = row_full + 16;                 // [2] ... and have been read by both arithmetic groups (8 warps)
    const uint32_t sdp_full = row_free + 16;                 // [2] S and dP of an entry computed
    const uint32_t ds_ready = sdp_full + 16;                 // [2] dS written (8 warps)
    const uint32_t dq_full = ds_ready + 16;                  // [2] the unit's dQ is complete
    const uint32_t dq_free = dq_full + 16;                   // [2] ... and has been read out of tensor memory
    const uint32_t dq_done = dq_free + 16;                   // [2] the dQ MMAs that read dS from an S / dP buffer are done
    const uint32_t kv_full = dq_done + 16;                   // [kStages] a K and a V tile landed (both copy warps announce bytes)
    const uint32_t ring_free = kv_full + 8 * kStages;        // [kStages] the stage's tiles (or O tile) have been used
    static_assert(160 + 16 * kStages <= 496, "barriers overlap the words behind them");
    if (tid == 0) {
        s_abort = (base & 1023u) ? 1 : 0;
        if (s_abort && a.status) atomicOr(a.status, BF1_DEV_WAIT_TIMEOUT);
        for (int b = 0; b < 2; ++b) {
            mbar_init(qdo_full + 8 * b, 2);
            mbar_init(qdo_free + 8 * b, 2);
            mbar_init(o_full + 8 * b, 1);
            mbar_init(row_full + 8 * b, 1);
            mbar_init(row_free + 8 * b, 8);
            mbar_init(sdp_full + 8 * b, 1);
            mbar_init(ds_ready + 8 * b, 8);
            mbar_init(dq_full + 8 * b, 1);
            mbar_init(dq_free + 8 * b, 1);
            mbar_init(dq_done + 8 * b, 1);
        }
        for (int s = 0; s < kStages; ++s) {
            mbar_init(kv_full + 8 * s, 2);
            mbar_init(ring_free + 8 * s, 1);
        }
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem), 512);
        tmem_relinquish();
    }
    if (a.group == 1) {   // one head per KV head: rows 64..127 of the Q / dO buffers are never written by a copy
        clear_idle_rows<D>(base + L::kQ, base + L::kDO, tid, kDqThreads);
        clear_idle_rows<D>(base + L::kQ + L::kQBytes, base + L::kDO + L::kQBytes, tid, kDqThreads);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* abort_flag = &s_abort;
    if (s_abort) {   // (uniform over the CTA)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, 512);
        return;
    }
    // tensor memory: S | dP of buffer b at columns 128 b (dS takes over columns 0..15 and 32..47 of S), dQ of
    // buffer b at 256 + 128 b
    constexpr uint32_t kColDP = 64, kColDQ = 256;
    const uint32_t q_tx = a.group > 1 ? L::kQBytes : L::kQBytes / 2;   // one head per KV head: half a tile per copy set
    auto stage_k = [&](int s) { return base + L::kRing + s * 2 * L::kKVBytes; };
    auto stage_v = [&](int s) { return base + L::kRing + s * 2 * L::kKVBytes + L::kKVBytes; };

    if (warp == 0 || warp == 1) {
        // ---- copies ----
        const bool first = warp == 0;
        int r = 0;                      // ring entries so far: stage r % kStages, its phase r / kStages
        int rs = 0, rk = 0;             // the same as (stage, phase counter)
        auto ring_wait_free = [&]() {
            if (r >= kStages) mbar_wait(ring_free + 8 * rs, (rk - 1) & 1, abort_flag, a.status);
        };
        auto ring_next = [&]() {
            ++r;
            if (++rs == kStages) { rs = 0; ++rk; }
        };
        DqUnit u = dq_unit(a, 0, nqb, pairs);
        for (int n = 0; u.ok; ++n) {
            const DqUnit un = dq_unit(a, n + 1, nqb, pairs);
            const int b = n & 1, head0 = u.kvh * a.group + u.pair * 2;
            const int32_t* list = a.kv_idx + (size_t)u.slot * a.max_degree;
            const int qb = qbuf(n);
            if (n >= 2) mbar_wait(qdo_free + 8 * qb, qpar(n - 2), abort_flag, a.status);
            if (elect_one()) {
                mbar_expect_tx(qdo_full + 8 * qb, q_tx);
                if (first) load_q_tile<D>(base + L::kQ + qb * L::kQBytes, &tm_q, u.tok0, head0, a.group, qdo_full + 8 * qb);
                else load_q_tile<D>(base + L::kDO + qb * L::kQBytes, &tm_do, u.tok0, head0, a.group, qdo_full + 8 * qb);
            }
            __syncwarp();
            // the O tile's ring entry
            if (!first) {
                ring_wait_free();
                if (elect_one()) {
                    mbar_expect_tx(o_full + 8 * b, q_tx);
                    load_q_tile<D>(stage_k(rs), &tm_o, u.tok0, head0, a.group, o_full + 8 * b);
                }
                __syncwarp();
            }
            ring_next();
            for (int it = 0; it < u.cnt; ++it) {
                const int p = list_entry(list, it, u.cnt, u.j);
                ring_wait_free();
                if (elect_one()) {
                    mbar_expect_tx(kv_full + 8 * rs, L::kKVBytes);
                    if (first) tma_load_4d(stage_k(rs), &tm_k, 0, u.seq0 + p * kBlock64, u.kvh, 0, kv_full + 8 * rs);
                    else tma_load_4d(stage_v(rs), &tm_v, 0, u.seq0 + p * kBlock64, u.kvh, 0, kv_full + 8 * rs);
                }
                __syncwarp();
                ring_next();
            }
            u = un;
        }
    } else if (warp == 2 || warp == 3) {
        // ---- MMAs: warp 2 issues S and dP of every entry, warp 3 its dQ.  Two warps, because what surrounds a batch of
        // MMAs (barrier round trips through shared memory, the unit bookkeeping) costs several hundred cycles per
        // entry, during which a single issuing warp would leave the pipe empty. ----
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        constexpr uint32_t kIdQ = idesc_bf16_f32(D, true);             // dQ: 128 x d, A from tensor memory, B (K tile) MN-major
        DqUnit u = dq_unit(a, 0, nqb, pairs);
        int t = 0, rs = 1 % kStages;       // entries so far; ring stage of the entry (entry 0 of the ring is unit 0's O tile)
        uint32_t kv_phase = 0;             // per stage: parity of the K / V tiles put into it so far
        for (int n = 0; u.ok; ++n) {
            const DqUnit un = dq_unit(a, n + 1, nqb, pairs);
            const int b = n & 1;
            if (warp == 2) mbar_wait(qdo_full + 8 * b, qpar(n), abort_flag, a.status);
            else if (n >= 2) mbar_wait(dq_free + 8 * b, qpar(n - 2), abort_flag, a.status);
            for (int it = 0; it < u.cnt; ++it) {
                const int sb = t & 1;
                if (warp == 2) {
                    // the buffer's last dS must have been read by its dQ MMAs before S overwrites it
                    if (t >= 2) mbar_wait(dq_done + 8 * sb, ((t >> 1) - 1) & 1, abort_flag, a.status);
                    mbar_wait(kv_full + 8 * rs, (kv_phase >> rs) & 1, abort_flag, a.status);
                    tc_fence_after();
                    if (elect_one()) {
                        issue_s_dp<D>(tmem + sb * 128, tmem + sb * 128 + kColDP, base + L::kQ + b * L::kQBytes,
                                      base + L::kDO + b * L::kQBytes, stage_k(rs), stage_v(rs));
                        mma_commit(sdp_full + 8 * sb);
                    }
                    __syncwarp();
                } else {
                    mbar_wait(ds_ready + 8 * sb, (t >> 1) & 1, abort_flag, a.status);
                    tc_fence_after();
                    if (elect_one()) {
                        // dQ += dS K: A = dS [128 q][64 kv] from tensor memory (16 kv = 8 columns per step; keys 0..31 sit in
                        // columns 0..15, keys 32..63 in columns 32..47), B = K tile MN-major (16 kv rows = 2048 bytes per step,
                        // next 64 d columns 8 KB away)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {   // 64 kv rows in steps of 16
                            const uint32_t blo = desc_lo_sw128(stage_k(rs), 8192) + ((kk * 2048) >> 4);
                            const uint32_t a_ds = tmem + sb * 128 + (kk >> 1) * 32 + (kk & 1) * 8;
                            if (kk == 0) {
                                if (it == 0) mma_ts_lohi<false>(tmem + kColDQ + b * 128, a_ds, blo, kHi, kIdQ);
                                else mma_ts_lohi<true>(tmem + kColDQ + b * 128, a_ds, blo, kHi, kIdQ);
                            } else {
                                mma_ts_lohi<true>(tmem + kColDQ + b * 128, a_ds, blo, kHi, kIdQ);
                            }
                        }
                        mma_commit(dq_done + 8 * sb);
                        mma_commit(ring_free + 8 * rs);
                        if (it == u.cnt - 1) {
                            mma_commit(dq_full + 8 * b);
                            mma_commit(qdo_free + 8 * b);
                        }
                    }
                    __syncwarp();
                }
                kv_phase ^= 1u << rs;
                ++t;
                if (++rs == kStages) rs = 0;
            }
            if (++rs == kStages) rs = 0;   // the next unit's O tile
            u = un;
        }
    } else if (warp >= 4 && warp < 12) {
        // ---- arithmetic on S and dP: two threads per tile row (head hl, token tl), warps 4-7 on key columns 0..31 and
        // warps 8-11 on columns 32..63 of every entry ----
        const int half = (warp - 4) >> 2;
        const uint32_t t_lane = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row = tid & 127, tl = row & 63;
        int t = 0;
        DqUnit u = dq_unit(a, 0, nqb, pairs);
        for (int n = 0; u.ok; ++n) {
            const DqUnit un = dq_unit(a, n + 1, nqb, pairs);
            const int b = n & 1;
            mbar_wait(row_full + 8 * b, (n >> 1) & 1, abort_flag, a.status);
            const float Drow = s_drow[b * 128 + row], lse2 = s_lse[b * 128 + row];
            for (int it = 0; it < u.cnt; ++it, ++t) {
                const int sb = t & 1;
                mbar_wait(sdp_full + 8 * sb, (t >> 1) & 1, abort_flag, a.status);
                tc_fence_after();
                uint32_t pw[16], dw[16];
                p_and_ds(t_lane + sb * 128, t_lane + sb * 128 + kColDP, half, tl, it == u.cnt - 1, lse2, Drow, a.scale, a.scale_log2, pw, dw);
                // dS as the A operand of the dQ MMAs: bf16 pairs, written over the first 16 of the 32 S columns just read
                tmem_st16(t_lane + sb * 128 + half * 32, dw);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ds_ready + 8 * sb);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(row_free + 8 * b);
            u = un;
        }
    } else if (warp >= 12) {
        // ---- per unit: D_i and LSE one unit ahead; the finished dQ tile of the unit before ----
        const uint32_t t_lane = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row = tid & 127, hl = row >> 6, tl = row & 63;
        int r = 0;   // ring entry of the current unit's O tile
        auto prologue = [&](const DqUnit& u, int n) {
            const int b = n & 1;
            const int h = u.kvh * a.group + u.pair * 2 + hl, tok = u.tok0 + tl;
            const bool row_ok = tl < u.rows_valid && u.pair * 2 + hl < a.group;   // G = 1: rows 64..127 belong to no head
            float lse2 = INFINITY, Drow = 0.f;
            if (row_ok) lse2 = a.lse[(size_t)h * a.total_tokens + tok] * 1.4426950408889634f;
            mbar_wait(qdo_full + 8 * qbuf(n), qpar(n), abort_flag, a.status);
            mbar_wait(o_full + 8 * b, (n >> 1) & 1, abort_flag, a.status);
            if (n >= 2) mbar_wait(row_free + 8 * b, ((n >> 1) - 1) & 1, abort_flag, a.status);
            const int rs = r % kStages;
            if (row_ok) {
                const uint32_t sO = stage_k(rs), sDO = base + L::kDO + qbuf(n) * L::kQBytes;
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {   // 16-byte pieces of the row: chunk c / 8 of 64 columns, piece c % 8
                    const uint32_t off = (c >> 3) * 16384 + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                    uint32_t ow[4], gw[4];
                    ld_shared_v4(sO + off, ow);
                    ld_shared_v4(sDO + off, gw);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        Drow = fmaf(__uint_as_float(ow[e] << 16), __uint_as_float(gw[e] << 16), Drow);
                        Drow = fmaf(__uint_as_float(ow[e] & 0xffff0000u), __uint_as_float(gw[e] & 0xffff0000u), Drow);
                    }
                }
                a.delta[(size_t)h * a.total_tokens + tok] = Drow;   // for the dK/dV kernel
            }
            s_drow[b * 128 + row] = Drow;
            s_lse[b * 128 + row] = lse2;
            named_sync(1, 128);
            if ((tid & 127) == 0) {
                mbar_arrive(ring_free + 8 * rs);
                mbar_arrive(qdo_free + 8 * qbuf(n));
                mbar_arrive(row_full + 8 * b);
            }
            r += u.cnt + 1;
        };
        DqUnit u = dq_unit(a, 0, nqb, pairs);
        if (u.ok) prologue(u, 0);
        for (int n = 0; u.ok; ++n) {
            const DqUnit un = dq_unit(a, n + 1, nqb, pairs);
            if (un.ok) prologue(un, n + 1);
            const int b = n & 1;
            const int h = u.kvh * a.group + u.pair * 2 + hl, tok = u.tok0 + tl;
            const bool row_ok = tl < u.rows_valid && u.pair * 2 + hl < a.group;
            mbar_wait(dq_full + 8 * b, (n >> 1) & 1, abort_flag, a.status);
            tc_fence_after();
            __nv_bfloat16* dqrow = a.dq + ((size_t)tok * a.hq + h) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(t_lane + kColDQ + b * 128 + c * 32, v);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(v[e + 0]), __uint_as_float(v[e + 1]));
                        w.y = pack_bf16x2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                        w.z = pack_bf16x2(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5]));
                        w.w = pack_bf16x2(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7]));
                        *reinterpret_cast<uint4*>(dqrow + c * 32 + e) = w;
                    }
                }
            }
            tc_fence_before();
            named_sync(1, 128);
            if ((tid & 127) == 0) mbar_arrive(dq_free + 8 * b);
            u = un;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ---- the inverse route -----------------------------------------------------------------------------------------

// The readers of KV slot gp are the query slots of the same sequence whose list names its block (with multiplicity,
// should a caller's list name a block twice).  Transposing the lists is a counting sort by KV slot, linear in the
// number of list entries: count (one thread per entry), scan (inverse_units_kernel), fill in whatever order the
// atomics give, then sort every slot's readers ascending -- the order in which the dK/dV kernel adds is thereby the
// same on every run.
__device__ __forceinline__ bool inverse_entry(const BwdArgs& a, int nqb, int f, int& g, int& kv) {
    g = f / a.max_degree;
    if (g >= nqb) return false;
    const int e = f - g * a.max_degree;
    const int cnt = min(max(a.kv_count[g], 1), a.max_degree);
    if (e >= cnt) return false;
    const int j = a.qb_block[g];
    kv = g - j + list_entry(a.kv_idx + (size_t)g * a.max_degree, e, cnt, j);   // slots of a sequence are consecutive
    return true;
}

// kFill = false: count[kv] += 1 (count is zero on entry).  kFill = true: count[kv] is counted down again and hands out
// the places behind start[kv].
template <bool kFill>
__global__ void __launch_bounds__(256) inverse_route_kernel(const BwdArgs a) {
    const int nqb = min(*a.num_qblocks, a.capacity);
    const int total = nqb * a.max_degree;
    for (int f = blockIdx.x * 256 + threadIdx.x; f < total; f += gridDim.x * 256) {
        int g, kv;
        if (!inverse_entry(a, nqb, f, g, kv)) continue;
        if (!kFill) atomicAdd(a.inv.count + kv, 1);
        else a.inv.readers[a.inv.start[kv] + atomicSub(a.inv.count + kv, 1) - 1] = g;
    }
}

// One CTA per KV slot: its readers ascending.  Up to 32 by ranking inside a warp; more by a bitonic network whose
// comparators all point the same way, so that a length that is no power of two needs no padding (elements past the end
// count as +infinity and never move); in shared memory when they fit, else in place.
constexpr int kSortSmem = 4096;
__global__ void __launch_bounds__(256) inverse_sort_kernel(const BwdArgs a) {
    __shared__ int32_t s_v[kSortSmem];
    const int gp = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    if (gp >= min(*a.num_qblocks, a.capacity) || a.inv.scalars[0] == 0) return;
    const int s0 = a.inv.start[gp], c = a.inv.start[gp + 1] - s0;
    int32_t* r = a.inv.readers + s0;
    if (c <= 1) return;
    if (c <= 32) {
        if (tid >= 32) return;
        const int v = lane < c ? r[lane] : 0x7fffffff;
        int rank = 0;
        for (int j = 0; j < c; ++j) {
            const int vj = __shfl_sync(0xffffffffu, v, j);
            rank += (vj < v) || (vj == v && j < lane);
        }
        if (lane < c) r[rank] = v;
        return;
    }
    int32_t* v = c <= kSortSmem ? s_v : r;
    if (c <= kSortSmem) {
        for (int i = tid; i < c; i += 256) s_v[i] = r[i];
    }
    __syncthreads();
    for (int k = 2; (k >> 1) < c; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < c; i += 256) {
                const int l = (j == (k >> 1)) ? (i ^ (k - 1)) : (i ^ j);   // first step of a merge: mirrored partner
                if (l > i && l < c) {
                    const int x = v[i], y = v[l];
                    if (x > y) { v[i] = y; v[l] = x; }
                }
            }
            __syncthreads();
        }
    }
    if (c <= kSortSmem) {
        for (int i = tid; i < c; i += 256) r[i] = s_v[i];
    }
}

// One CTA: offsets of the reader lists, the run length, and the units of the dK/dV kernel.  kAll: the counting and the
// filling of the readers as well (few list entries: one launch instead of four).
template <bool kAll>
__global__ void __launch_bounds__(1024, 1) inverse_units_kernel(const BwdArgs a) {
    __shared__ int32_t s_warp[32];
    __shared__ int32_t s_carry[5];
    __shared__ int32_t s_chunk;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nqb = min(*a.num_qblocks, a.capacity);
    const InvPlan& v = a.inv;
    // exclusive scan of x over the CTA, with a running carry in s_carry[which]
    auto scan = [&](int x, int which, int& excl) {
        int incl = x;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = s_warp[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += up;
            }
            s_warp[lane] = w;
        }
        __syncthreads();
        const int before = (warp > 0 ? s_warp[warp - 1] : 0) + s_carry[which];
        excl = before + incl - x;
        const int chunk_total = s_warp[31];
        __syncthreads();
        if (tid == 0) s_carry[which] += chunk_total;
        __syncthreads();
    };
    if (tid < 5) s_carry[tid] = 0;
    if (kAll) {
        for (int g = tid; g < nqb; g += 1024) v.count[g] = 0;
        __syncthreads();
        for (int f = tid; f < nqb * a.max_degree; f += 1024) {
            int g, kv;
            if (inverse_entry(a, nqb, f, g, kv)) atomicAdd(v.count + kv, 1);
        }
    }
    __syncthreads();
    // pass 1: where each slot's readers start; the total decides the run length
    for (int b0 = 0; b0 < nqb; b0 += 1024) {
        const int g = b0 + tid;
        const int c = g < nqb ? __ldcg(v.count + g) : 0;   // (written by atomics: read where they were performed)
        int excl;
        scan(c, 0, excl);
        if (g < nqb) v.start[g] = excl;
    }
    if (tid == 0) {
        const int total = s_carry[0];
        v.start[nqb] = total;
        // runs of at least kMinChunk readers, and long enough that the slots with more than one run cannot need
        // more than `cap` partial-sum slots between them (such a slot has fewer than 2 * count / chunk runs)
        s_chunk = max(kMinChunk, (2 * total + max(v.cap, 1) - 1) / max(v.cap, 1));
    }
    __syncthreads();
    const int chunk = s_chunk;
    // pass 2: runs per slot -> unit numbers and partial-sum slots
    for (int b0 = 0; b0 < nqb; b0 += 1024) {
        const int g = b0 + tid;
        const int c = g < nqb ? __ldcg(v.count + g) : 0;   // (written by atomics: read where they were performed)
        const int runs = (c + chunk - 1) / chunk;
        int u0, q0, m0;
        scan(runs, 1, u0);
        scan(runs > 1 ? runs : 0, 2, q0);
        scan(runs > 1 ? 1 : 0, 3, m0);
        if (g < nqb) {
            if (runs > 1) v.multi[m0] = g;
            v.chunks[g] = runs;
            v.part0[g] = runs > 1 ? q0 : -1;
            const int first = v.start[g];
            for (int r = 0; r < runs; ++r) {
                if (u0 + r >= v.max_units) break;
                v.unit_slot[u0 + r] = g;
                v.unit_begin[u0 + r] = first + r * chunk;
                v.unit_end[u0 + r] = min(first + c, first + (r + 1) * chunk);
                v.unit_part[u0 + r] = runs > 1 ? q0 + r : -1;
            }
        }
    }
    // units by descending length (a counting sort; which of two equally long units comes first does not matter: the
    // order only decides which CTA works on which unit)
    __shared__ int32_t s_bin[1024];
    s_bin[tid] = 0;
    __syncthreads();
    const int n_units = min(s_carry[1], v.max_units);
    for (int un = tid; un < n_units; un += 1024) atomicAdd(&s_bin[1023 - min(v.unit_end[un] - v.unit_begin[un], 1023)], 1);
    __syncthreads();
    {
        const int c = s_bin[tid];
        int excl;
        scan(c, 4, excl);
        s_bin[tid] = excl;           // where the units of this length start
    }
    __syncthreads();
    for (int un = tid; un < n_units; un += 1024)
        v.unit_order[atomicAdd(&s_bin[1023 - min(v.unit_end[un] - v.unit_begin[un], 1023)], 1)] = un;
    if (tid == 0) {
        const bool fits = s_carry[1] <= v.max_units && s_carry[2] <= v.cap;
        if (!fits && a.status) atomicOr(a.status, BF1_DEV_CAPACITY);
        v.scalars[0] = fits ? s_carry[1] : 0;
        v.scalars[1] = s_carry[0];
        v.scalars[2] = chunk;
        v.scalars[3] = s_carry[2];
        v.scalars[4] = fits ? s_carry[3] : 0;
    }
    if (kAll) {
        __syncthreads();
        for (int f = tid; f < nqb * a.max_degree; f += 1024) {
            int g, kv;
            if (inverse_entry(a, nqb, f, g, kv)) v.readers[v.start[kv] + atomicSub(v.count + kv, 1) - 1] = g;
        }
    }
}

// ---- dK, dV ----------------------------------------------------------------------------------------------------
//
// One persistent CTA of 16 warps per SM.  A unit is (KV block, KV head, run of the block's readers); units are
// dealt out statically KV head by KV head, back and forth over the CTAs.  K and V of a unit stay in shared memory
// (two buffers: the next unit's arrive early), Q and dO of every step (a reader and a pair of its heads) travel
// through a ring of two stages:
//     warp 0    copies K of every unit and Q of every step;  warp 1: V and dO
//     warp 2    issues S = Q K^T and dP = dO V^T of every step into one of two S/dP buffers in tensor memory
//     warp 3    issues dV^T += dO^T P and dK^T += Q^T dS of every step; the sums stay in one of two accumulator
//               buffers in tensor memory across all steps of the unit
//     warps 4-11   the arithmetic on S and dP (two threads per tile row), P and dS as bf16 tiles to shared memory
//     warps 12-15  the finished sums of the unit before, from tensor memory to global memory
constexpr int kDkvThreads = 512;

template <int D>
struct DkvSmem {
    static constexpr int kQBytes = 128 * D * 2;      // Q / dO tile [D / 64 chunks][128 rows][128 B]
    static constexpr int kKVBytes = 64 * D * 2;      // K / V tile  [D / 64 chunks][64 rows][128 B]
    static constexpr int kQ = 0;                     // [2]
    static constexpr int kDO = kQ + 2 * kQBytes;     // [2]
    static constexpr int kK = kDO + 2 * kQBytes;     // [2]
    static constexpr int kV = kK + 2 * kKVBytes;     // [2]
    static constexpr int kP = kV + 2 * kKVBytes;     // P  [128 q rows][64 kv] bf16, 128-byte rows, swizzled
    static constexpr int kDS = kP + 16384;           // dS likewise
    static constexpr int kBar = kDS + 16384;
    static constexpr int kUsed = kBar + 512;
    // at least this much is requested so that a second CTA never fits an SM: each allocates all of tensor memory
    static constexpr int kTotal = kUsed > 120 * 1024 ? kUsed : 120 * 1024;
};

struct DkvUnit {
    int ok, gp, kvh, r_begin, steps, part, seq0, seqlen, p, kv_valid;
};

// Unit n of this CTA.
__device__ __forceinline__ DkvUnit dkv_unit(const BwdArgs& a, int n, int n_units, int pairs) {
    DkvUnit u;
    const int total = n_units * a.hkv;
    const int G = gridDim.x;
    const int i = n * G + ((n & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x);
    u.ok = i < total;
    u.gp = u.kvh = u.r_begin = u.seq0 = u.seqlen = u.p = u.kv_valid = 0;
    u.steps = 0;
    u.part = -1;
    if (u.ok) {
        int ui;
        if (a.interleave) {
            ui = i / a.hkv;
            u.kvh = i - ui * a.hkv;
        } else {
            u.kvh = i / n_units;
            ui = i - u.kvh * n_units;
        }
        const int unit = a.inv.unit_order[ui];
        u.gp = a.inv.unit_slot[unit];
        u.r_begin = a.inv.unit_begin[unit];
        u.steps = (a.inv.unit_end[unit] - u.r_begin) * pairs;
        u.part = a.inv.unit_part[unit];
        const int seq = a.qb_seq[u.gp];
        u.p = a.qb_block[u.gp];
        u.seq0 = a.cu_seqlens[seq];
        u.seqlen = a.cu_seqlens[seq + 1] - u.seq0;
        u.kv_valid = min(kBlock64, u.seqlen - u.p * kBlock64);      // key rows of this block inside the sequence
    }
    return u;
}

template <int D>
__global__ void __launch_bounds__(kDkvThreads, 1) bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                              const __grid_constant__ CUtensorMap tm_k,
                                                              const __grid_constant__ CUtensorMap tm_v,
                                                              const __grid_constant__ CUtensorMap tm_do,
                                                              const BwdArgs a) {
    using L = DkvSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(smem + L::kBar + 496);
    int& s_abort = *reinterpret_cast<int*>(smem + L::kBar + 500);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (a.status && (*a.status & BF1_DEV_WAIT_TIMEOUT)) return;
    const int n_units = a.inv.scalars[0];
    const int pairs = a.group == 4 ? 2 : 1;

    const uint32_t base = smem_u32(smem);
    const uint32_t bars = base + L::kBar;
    const uint32_t kv_full = bars;                 // [2] K and V of a unit landed (both copy warps announce bytes)
    const uint32_t kv_free = kv_full + 16;         // [2] the unit's S / dP MMAs are done
    const uint32_t q_full = kv_free + 16;          // [2] Q of a step landed
    const uint32_t do_full = q_full + 16;          // [2] dO of a step landed
    const uint32_t q_free = do_full + 16;          // [2] the step's dK^T MMAs are done (they come first: S of the step after
    const uint32_t do_free = q_free + 16;          //     next can then start while its dO is still travelling); [2] its dV^T MMAs
    const uint32_t sdp_full = do_free + 16;        // [2] S and dP of a step computed
    const uint32_t pds_ready = sdp_full + 16;      // [2] P and dS of a step are in shared memory (8 warps); S / dP have been read
    const uint32_t pds_free = pds_ready + 16;      // [1] the MMAs that read P and dS are done
    const uint32_t acc_full = pds_free + 8;        // [2] the unit's sums are complete
    const uint32_t acc_free = acc_full + 16;       // [2] ... and have been read out of tensor memory
    if (tid == 0) {
        s_abort = (base & 1023u) ? 1 : 0;
        if (s_abort && a.status) atomicOr(a.status, BF1_DEV_WAIT_TIMEOUT);
        for (int b = 0; b < 2; ++b) {
            mbar_init(kv_full + 8 * b, 2);
            mbar_init(kv_free + 8 * b, 1);
            mbar_init(q_full + 8 * b, 1);
            mbar_init(do_full + 8 * b, 1);
            mbar_init(q_free + 8 * b, 1);
            mbar_init(do_free + 8 * b, 1);
            mbar_init(sdp_full + 8 * b, 1);
            mbar_init(pds_ready + 8 * b, 8);
            mbar_init(acc_full + 8 * b, 1);
            mbar_init(acc_free + 8 * b, 1);
        }
        mbar_init(pds_free, 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem), 512);
        tmem_relinquish();
    }
    if (a.group == 1) {   // one head per KV head: rows 64..127 of the Q / dO buffers are never written by a copy
        clear_idle_rows<D>(base + L::kQ, base + L::kDO, tid, kDkvThreads);
        clear_idle_rows<D>(base + L::kQ + L::kQBytes, base + L::kDO + L::kQBytes, tid, kDkvThreads);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* abort_flag = &s_abort;
    if (s_abort) {   // (uniform over the CTA)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, 512);
        return;
    }
    // tensor memory: S | dP of buffer b at columns 128 b; dV^T | dK^T (64 columns each: head dimension on the lanes,
    // the block's 64 key rows along the columns) of buffer b at 256 + 128 b
    constexpr uint32_t kColDP = 64, kColAcc = 256, kColDKt = 64;
    const uint32_t q_tx = a.group > 1 ? L::kQBytes : L::kQBytes / 2;   // one head per KV head: half a tile per copy set
    const uint32_t sP = base + L::kP, sDS = base + L::kDS;

    if (warp == 0 || warp == 1) {
        // ---- copies ----
        const bool first = warp == 0;
        int s = 0;   // steps so far
        DkvUnit u = dkv_unit(a, 0, n_units, pairs);
        for (int n = 0; u.ok; ++n) {
            const DkvUnit un = dkv_unit(a, n + 1, n_units, pairs);
            const int b = n & 1;
            if (n >= 2) mbar_wait(kv_free + 8 * b, ((n >> 1) - 1) & 1, abort_flag, a.status);
            if (elect_one()) {
                mbar_expect_tx(kv_full + 8 * b, L::kKVBytes);
                if (first) tma_load_4d(base + L::kK + b * L::kKVBytes, &tm_k, 0, u.seq0 + u.p * kBlock64, u.kvh, 0, kv_full + 8 * b);
                else tma_load_4d(base + L::kV + b * L::kKVBytes, &tm_v, 0, u.seq0 + u.p * kBlock64, u.kvh, 0, kv_full + 8 * b);
            }
            __syncwarp();
            int jq = u.steps > 0 ? a.qb_block[a.inv.readers[u.r_begin]] : 0;
            for (int step = 0; step < u.steps; ++step, ++s) {
                int jq_next = 0;
                if (step + 1 < u.steps) jq_next = a.qb_block[a.inv.readers[u.r_begin + (step + 1) / pairs]];
                const int sb = s & 1;
                const uint32_t full = (first ? q_full : do_full) + 8 * sb;
                if (s >= 2) mbar_wait((first ? q_free : do_free) + 8 * sb, ((s >> 1) - 1) & 1, abort_flag, a.status);
                if (elect_one()) {
                    mbar_expect_tx(full, q_tx);
                    const int head0 = u.kvh * a.group + (step % pairs) * 2;
                    if (first) load_q_tile<D>(base + L::kQ + sb * L::kQBytes, &tm_q, u.seq0 + jq * kBlock64, head0, a.group, full);
                    else load_q_tile<D>(base + L::kDO + sb * L::kQBytes, &tm_do, u.seq0 + jq * kBlock64, head0, a.group, full);
                }
                __syncwarp();
                jq = jq_next;
            }
            u = un;
        }
    } else if (warp == 2 || warp == 3) {
        // ---- MMAs: warp 2 issues S and dP of every step, warp 3 the two transposed products ----
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        constexpr uint32_t kIdT = idesc_bf16_f32_ab(64, true, true);   // dV^T, dK^T: A and B MN-major
        int s = 0;
        DkvUnit u = dkv_unit(a, 0, n_units, pairs);
        for (int n = 0; u.ok; ++n) {
            const DkvUnit un = dkv_unit(a, n + 1, n_units, pairs);
            const int b = n & 1;
            if (warp == 2) mbar_wait(kv_full + 8 * b, (n >> 1) & 1, abort_flag, a.status);
            else if (n >= 2) mbar_wait(acc_free + 8 * b, ((n >> 1) - 1) & 1, abort_flag, a.status);
            for (int step = 0; step < u.steps; ++step, ++s) {
                const int sb = s & 1;
                const uint32_t sQ = base + L::kQ + sb * L::kQBytes, sDO = base + L::kDO + sb * L::kQBytes;
                if (warp == 2) {
                    // the buffer's last S and dP must have been read
                    if (s >= 2) mbar_wait(pds_ready + 8 * sb, ((s >> 1) - 1) & 1, abort_flag, a.status);
                    mbar_wait(q_full + 8 * sb, (s >> 1) & 1, abort_flag, a.status);
                    tc_fence_after();
                    if (elect_one()) issue_qk<D>(tmem + sb * 128, sQ, base + L::kK + b * L::kKVBytes);
                    __syncwarp();
                    mbar_wait(do_full + 8 * sb, (s >> 1) & 1, abort_flag, a.status);
                    if (elect_one()) {
                        issue_qk<D>(tmem + sb * 128 + kColDP, sDO, base + L::kV + b * L::kKVBytes);
                        mma_commit(sdp_full + 8 * sb);
                        if (step == u.steps - 1) mma_commit(kv_free + 8 * b);
                    }
                    __syncwarp();
                } else {
                    mbar_wait(pds_ready + 8 * sb, (s >> 1) & 1, abort_flag, a.status);
                    tc_fence_after();
                    if (elect_one()) {
                        // dK^T += Q^T dS, then dV^T += dO^T P: A = Q / dO MN-major (M = d: 64 per 128-byte row, next 64 at
                        // +16 KB; K = q rows, 16 per step = 2048 bytes), B = P / dS MN-major (N = 64 kv per row)
                        const uint32_t t_acc = tmem + kColAcc + b * 128;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t ko = (kk * 2048) >> 4;
                            if (kk == 0) {
                                if (step == 0) mma_ss_lohi<false>(t_acc + kColDKt, desc_lo_sw128(sQ, 16384) + ko, desc_lo_sw128(sDS, 16) + ko, kHi, kIdT);
                                else mma_ss_lohi<true>(t_acc + kColDKt, desc_lo_sw128(sQ, 16384) + ko, desc_lo_sw128(sDS, 16) + ko, kHi, kIdT);
                            } else {
                                mma_ss_lohi<true>(t_acc + kColDKt, desc_lo_sw128(sQ, 16384) + ko, desc_lo_sw128(sDS, 16) + ko, kHi, kIdT);
                            }
                        }
                        mma_commit(q_free + 8 * sb);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t ko = (kk * 2048) >> 4;
                            if (kk == 0) {
                                if (step == 0) mma_ss_lohi<false>(t_acc, desc_lo_sw128(sDO, 16384) + ko, desc_lo_sw128(sP, 16) + ko, kHi, kIdT);
                                else mma_ss_lohi<true>(t_acc, desc_lo_sw128(sDO, 16384) + ko, desc_lo_sw128(sP, 16) + ko, kHi, kIdT);
                            } else {
                                mma_ss_lohi<true>(t_acc, desc_lo_sw128(sDO, 16384) + ko, desc_lo_sw128(sP, 16) + ko, kHi, kIdT);
                            }
                        }
                        mma_commit(do_free + 8 * sb);
                        mma_commit(pds_free);
                        if (step == u.steps - 1) mma_commit(acc_full + 8 * b);
                    }
                    __syncwarp();
                }
            }
            u = un;
        }
    } else if (warp < 12) {
        // ---- arithmetic on S and dP: two threads per tile row (head hl, token tl of the reader), warps 4-7 on key
        // columns 0..31 and warps 8-11 on columns 32..63 ----
        const int half = (warp - 4) >> 2;
        const uint32_t t_lane = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row = tid & 127, hl = row >> 6, tl = row & 63;
        int s = 0;
        DkvUnit u = dkv_unit(a, 0, n_units, pairs);
        for (int n = 0; u.ok; ++n) {
            const DkvUnit un = dkv_unit(a, n + 1, n_units, pairs);
            // the reader of a step, its block index, the row's LSE (log2 domain) and D_i are fetched one step ahead:
            // dependent global loads that would otherwise sit between the MMAs and the arithmetic
            auto fetch = [&](int step, int& g, float& lse2, float& drow) {
                g = a.inv.readers[u.r_begin + step / pairs];
                const int jq = a.qb_block[g], pr = step % pairs;
                const int rows_valid = min(kBlock64, u.seqlen - jq * kBlock64);
                lse2 = INFINITY;
                drow = 0.f;
                if (tl < rows_valid && pr * 2 + hl < a.group) {
                    const size_t at = (size_t)(u.kvh * a.group + pr * 2 + hl) * a.total_tokens + u.seq0 + jq * kBlock64 + tl;
                    lse2 = a.lse[at] * 1.4426950408889634f;
                    drow = a.delta[at];
                }
            };
            int g = 0, g_next = 0;
            float lse2 = INFINITY, drow = 0.f, lse2_next = INFINITY, drow_next = 0.f;
            if (u.steps > 0) fetch(0, g, lse2, drow);
            for (int step = 0; step < u.steps; ++step, ++s) {
                if (step + 1 < u.steps) fetch(step + 1, g_next, lse2_next, drow_next);
                const int sb = s & 1;
                mbar_wait(sdp_full + 8 * sb, (s >> 1) & 1, abort_flag, a.status);
                tc_fence_after();
                uint32_t pw[16], dw[16];
                p_and_ds(t_lane + sb * 128, t_lane + sb * 128 + kColDP, half, tl, g == u.gp, lse2, drow, a.scale, a.scale_log2, pw, dw);
                if (s >= 1) mbar_wait(pds_free, (s - 1) & 1, abort_flag, a.status);   // the MMAs of the step before have read P and dS
                store_row_piece(sP + row * 128, row, half, pw);
                store_row_piece(sDS + row * 128, row, half, dw);
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pds_ready + 8 * sb);
                g = g_next, lse2 = lse2_next, drow = drow_next;
            }
            u = un;
        }
    } else {
        // ---- the finished dV^T / dK^T of a unit: lane = head-dimension index, 64 key rows along the columns ----
        const uint32_t t_lane = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row = tid & 127;
        DkvUnit u = dkv_unit(a, 0, n_units, pairs);
        for (int n = 0; u.ok; ++n) {
            const DkvUnit un = dkv_unit(a, n + 1, n_units, pairs);
            const int b = n & 1;
            if (u.steps > 0) {
                mbar_wait(acc_full + 8 * b, (n >> 1) & 1, abort_flag, a.status);
                tc_fence_after();
                if (row < D) {   // d = 64: lanes 64..127 hold nothing (warp-uniform)
                    const size_t rstride = (size_t)a.hkv * D;
                    const size_t row0 = ((size_t)(u.seq0 + u.p * kBlock64) * a.hkv + u.kvh) * D + row;
                    float* pk = u.part >= 0 ? a.partial + (((size_t)u.part * a.hkv + u.kvh) * 2) * (kBlock64 * D) + row : nullptr;
#pragma unroll 1
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t vr[32], kr[32];
                        tmem_ld32(t_lane + kColAcc + b * 128 + hh * 32, vr);
                        tmem_ld32(t_lane + kColAcc + b * 128 + kColDKt + hh * 32, kr);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            const int kvr = hh * 32 + c;
                            if (kvr < u.kv_valid) {
                                if (u.part < 0) {
                                    a.dv[row0 + kvr * rstride] = __float2bfloat16_rn(__uint_as_float(vr[c]));
                                    a.dk[row0 + kvr * rstride] = __float2bfloat16_rn(__uint_as_float(kr[c]));
                                } else {
                                    pk[kvr * D] = __uint_as_float(kr[c]);
                                    pk[kBlock64 * D + kvr * D] = __uint_as_float(vr[c]);
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                named_sync(1, 128);
                if ((tid & 127) == 0) mbar_arrive(acc_free + 8 * b);
            }
            u = un;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// KV blocks whose readers were cut into several runs: add the runs' partial sums in run order.  Few blocks
// need it (block 0 of a sequence, with the paper's route); the work items are (such a block, KV head, one of
// its key rows), taken round robin by however many CTAs were launched; a thread adds one element of dK or dV.
template <int D>
__global__ void __launch_bounds__(2 * D) bwd_combine_kernel(const BwdArgs a) {
    const int items = a.inv.scalars[4] * a.hkv * kBlock64;
    const int which = threadIdx.x / D, col = threadIdx.x % D;   // 0: dK, 1: dV
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int row = item % kBlock64, kvh = (item / kBlock64) % a.hkv;
        const int gp = a.inv.multi[item / (kBlock64 * a.hkv)];
        const int runs = a.inv.chunks[gp], q0 = a.inv.part0[gp];
        const int seq = a.qb_seq[gp], p = a.qb_block[gp];
        const int seq0 = a.cu_seqlens[seq];
        if (row >= a.cu_seqlens[seq + 1] - seq0 - p * kBlock64) continue;   // key row outside the sequence
        const float* pk = a.partial + (((size_t)q0 * a.hkv + kvh) * 2 + which) * (kBlock64 * D) + row * D + col;
        const size_t run_stride = (size_t)a.hkv * 2 * kBlock64 * D;
        float sum = 0.f;
#pragma unroll 8
        for (int r = 0; r < runs; ++r) sum += pk[r * run_stride];
        const size_t o = ((size_t)(seq0 + p * kBlock64 + row) * a.hkv + kvh) * D + col;
        (which ? a.dv : a.dk)[o] = __float2bfloat16_rn(sum);
    }
}

int make_map_4d(CUtensorMap* m, const void* ptr, int64_t T, int H, int d, int heads_per_box, int chunks_per_box);   // bf1_attn.cu

// Where everything lives in the caller's workspace (256-byte aligned sections).
struct BwdLayout {
    size_t delta, ints, partial, total;
    size_t n_count, n_start, n_chunks, n_part0, n_readers, n_units, n_multi;   // (n_units: also unit_order)
    BwdLayout(int64_t T, int hq, int hkv, int d, int cap, int max_degree) {
        auto up = [](size_t x) { return (x + 255) / 256 * 256; };
        n_count = (size_t)cap;
        n_start = (size_t)cap + 1;
        n_chunks = (size_t)cap;
        n_part0 = (size_t)cap;
        n_readers = (size_t)cap * max_degree;
        n_units = 2 * (size_t)cap;
        n_multi = (size_t)cap;
        delta = 0;
        ints = up((size_t)T * hq * sizeof(float));
        const size_t n_ints = n_count + n_start + n_chunks + n_part0 + n_readers + 5 * n_units + n_multi + 8;
        partial = ints + up(n_ints * sizeof(int32_t));
        total = partial + up((size_t)cap * hkv * 2 * kBlock64 * d * sizeof(float));
    }
};

}  // namespace bf1

using namespace bf1;

extern "C" int64_t bf1_attn_bwd_workspace_bytes(const bf1_route* route, int64_t total_tokens, int32_t hq, int32_t hkv,
                                                int32_t d) {
    if (!route || total_tokens < 0 || hq <= 0 || hkv <= 0 || d <= 0 || route->capacity_qblocks < 1 || route->max_degree < 1)
        return -1;
    return (int64_t)BwdLayout(total_tokens, hq, hkv, d, route->capacity_qblocks, route->max_degree).total;
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
         (uintptr_t)dv) & 15)
        return fail(BF1_ERR_INVALID_ARG, "tensors must be 16-byte aligned");
    if ((uintptr_t)workspace & 255) return fail(BF1_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    if (!route->qb_seq || !route->qb_block || !route->kv_count || !route->kv_idx || !route->num_qblocks || !route->status)
        return fail(BF1_ERR_INVALID_ARG, "a route array pointer is null");
    if (route->capacity_qblocks < 1 || route->max_degree < 1 || hkv > 65535)
        return fail(BF1_ERR_CAPACITY, "bad route capacities or hkv");
    if (total_tokens == 0 || batch == 0) return BF1_OK;
    int dev = 0, major = 0;
    BF1_CUDA_CHECK(cudaGetDevice(&dev));
    BF1_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return fail(BF1_ERR_NO_DEVICE, "device compute capability %d.x is not sm_100", major);
    static bool configured[64] = {};
    if (dev < 0 || dev >= 64) return fail(BF1_ERR_NO_DEVICE, "device ordinal %d out of range", dev);
    if (!configured[dev]) {
        // two CTAs per SM need the whole shared-memory carve-out
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<128>::kTotal));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<64>::kTotal));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkvSmem<128>::kTotal));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dkv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkvSmem<64>::kTotal));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dq_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dq_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dkv_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(bwd_dkv_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        configured[dev] = true;
    }
    CUtensorMap tq, tk, tv, tg, to;
    // Q and dO: two heads and all column chunks per copy; with one head per KV head, one head and one chunk
    const int q_heads = group == 1 ? 1 : 2, q_chunks = group == 1 ? 1 : d / 64;
    if (int rc = make_map_4d(&tq, q, total_tokens, hq, d, q_heads, q_chunks)) return rc;
    if (int rc = make_map_4d(&tg, d_o, total_tokens, hq, d, q_heads, q_chunks)) return rc;
    if (int rc = make_map_4d(&to, o, total_tokens, hq, d, q_heads, q_chunks)) return rc;
    if (int rc = make_map_4d(&tk, k, total_tokens, hkv, d, 1, d / 64)) return rc;
    if (int rc = make_map_4d(&tv, v, total_tokens, hkv, d, 1, d / 64)) return rc;
    const int cap = route->capacity_qblocks;
    const BwdLayout lay(total_tokens, hq, hkv, d, cap, route->max_degree);
    char* ws = (char*)workspace;
    BwdArgs a;
    a.cu_seqlens = cu_seqlens_dev;
    a.qb_seq = route->qb_seq;
    a.qb_block = route->qb_block;
    a.kv_count = route->kv_count;
    a.kv_idx = route->kv_idx;
    a.num_qblocks = route->num_qblocks;
    a.order = route->order;
    a.max_degree = route->max_degree;
    a.capacity = cap;
    a.total_tokens = (int32_t)total_tokens;
    a.hq = hq;
    a.hkv = hkv;
    a.group = group;
    a.status = route->status;
    a.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)d);
    a.scale_log2 = a.scale * 1.4426950408889634f;
    // The same rule as the forward's hand-out order: while K and V of all heads fit L2 together there is nothing
    // to gain from working head by head, and the longest units of all heads first balance the CTAs better.
    a.interleave = (total_tokens * (int64_t)hkv * d * 4 <= (48LL << 20)) ? 1 : 0;
    a.o = (const __nv_bfloat16*)o;
    a.d_o = (const __nv_bfloat16*)d_o;
    a.lse = lse;
    a.delta = (float*)(ws + lay.delta);
    a.dq = (__nv_bfloat16*)dq;
    a.dk = (__nv_bfloat16*)dk;
    a.dv = (__nv_bfloat16*)dv;
    a.partial = (float*)(ws + lay.partial);
    int32_t* ip = (int32_t*)(ws + lay.ints);
    a.inv.count = ip;            ip += lay.n_count;
    a.inv.start = ip;            ip += lay.n_start;
    a.inv.chunks = ip;           ip += lay.n_chunks;
    a.inv.part0 = ip;            ip += lay.n_part0;
    a.inv.readers = ip;          ip += lay.n_readers;
    a.inv.unit_slot = ip;        ip += lay.n_units;
    a.inv.unit_begin = ip;       ip += lay.n_units;
    a.inv.unit_end = ip;         ip += lay.n_units;
    a.inv.unit_part = ip;        ip += lay.n_units;
    a.inv.unit_order = ip;       ip += lay.n_units;
    a.inv.multi = ip;            ip += lay.n_multi;
    a.inv.scalars = ip;
    a.inv.cap = cap;
    a.inv.max_units = (int32_t)lay.n_units;
    cudaStream_t st = (cudaStream_t)stream;
    int sms = 0;
    BF1_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // the inverse route (readers of every KV block, cut into units) ...
    if ((int64_t)cap * route->max_degree <= 4096) {
        inverse_units_kernel<true><<<1, 1024, 0, st>>>(a);   // few entries: count, scan and fill in one CTA
    } else {
        BF1_CUDA_CHECK(cudaMemsetAsync(a.inv.count, 0, lay.n_count * sizeof(int32_t), st));
        const int grid_inv = (int)std::min<int64_t>(((int64_t)cap * route->max_degree + 255) / 256, 4 * (int64_t)sms);
        inverse_route_kernel<false><<<grid_inv, 256, 0, st>>>(a);
        inverse_units_kernel<false><<<1, 1024, 0, st>>>(a);
        inverse_route_kernel<true><<<grid_inv, 256, 0, st>>>(a);
    }
    inverse_sort_kernel<<<cap, 256, 0, st>>>(a);
    BF1_CUDA_CHECK(cudaGetLastError());
    // ... dQ (and D_i) along the route, dK / dV along its inverse
    const int grid_q = (int)std::min<int64_t>(sms, (int64_t)cap * hkv * (group == 4 ? 2 : 1));   // persistent: one CTA per SM
    const int grid_kv = (int)std::min<int64_t>(sms, (int64_t)lay.n_units * hkv);
    if (d == 128) {
        bwd_dq_kernel<128><<<grid_q, kDqThreads, DqSmem<128>::kTotal, st>>>(tq, tk, tv, tg, to, a);
        bwd_dkv_kernel<128><<<grid_kv, kDkvThreads, DkvSmem<128>::kTotal, st>>>(tq, tk, tv, tg, a);
        bwd_combine_kernel<128><<<4 * sms, 256, 0, st>>>(a);
    } else {
        bwd_dq_kernel<64><<<grid_q, kDqThreads, DqSmem<64>::kTotal, st>>>(tq, tk, tv, tg, to, a);
        bwd_dkv_kernel<64><<<grid_kv, kDkvThreads, DkvSmem<64>::kTotal, st>>>(tq, tk, tv, tg, a);
        bwd_combine_kernel<64><<<4 * sms, 128, 0, st>>>(a);
    }
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}
