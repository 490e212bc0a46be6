// BF1 block-gather flash-attention forward for sm_100a.
//
// Work unit = one query block (64 tokens) of one sequence x one KV head.  The G = 2 query
// heads that share the KV head are stacked into one M = 128 tile (rows 0..63: first head,
// rows 64..127: second head; with G = 4 the tile is 4 heads x 32 tokens and a query block is two
// units; with G = 1 rows 64..127 are idle), because they read the same K/V blocks through the same route
// list (the route is per block and the same for all heads, Section 3.1).  For every entry p
// of the unit's list ("tile"):
//   S = Q K[p]^T        tcgen05.mma, Q and K[p] in shared memory (TMA, 128-byte swizzle),
//                       fp32 accumulator in tensor memory (two S buffers, ping-pong),
//   online softmax      one thread per row: tcgen05.ld S, causal mask on the self block only,
//                       reference maximum (moved lazily) / sum in the exp2 domain, P -> bf16 -> tcgen05.st over S,
//   O += P V[p]         tcgen05.mma with P read from tensor memory and V from shared memory,
// then O / l is written as bf16 and LSE = max + ln(sum) as fp32.
// With `dense = 1` the list is replaced by 0..j: plain causal attention through the same code.
//
// The kernel is persistent (two CTAs per SM; units are handed out KV-head-major, longest list
// first, through an atomic counter) and warp specialised, 12 warps in three warpgroups whose
// register budgets are re-balanced with setmaxnreg:
//   warp 0      TMA producer: Q once per unit, then K and V tiles through a ring of 16 KB slots
//               in the order the MMAs consume them (K0, K1, V0, K2, V1, ...),
//   warp 1      MMA issuer for S = Q K^T: runs up to two tiles ahead of the softmax (two S buffers),
//   warp 3      MMA issuer for O += P V: a separate warp, so that neither kind of MMA waits behind
//               a burst of the other while the tensor pipe's queue is full,
//   warp 2      scheduler: fetches the next unit, decodes it, reads (and range-checks) its list
//               and queues it for the producer -- all of it global-memory latency that must not
//               sit in front of the copies,
//   warps 4-7   softmax, one thread per tile row,
//   warps 8-11  epilogue: take the finished O out of tensor memory into registers (which frees O for the
//               next unit's first PV), normalise, store O and LSE, while the softmax warps are already
//               on the next unit.
// All hand-offs are mbarriers; every wait is bounded (see mbar_wait).
#include <cuda.h>

#include "bf1_common.cuh"

namespace bf1 {

constexpr int kBlock = 64;            // b: tokens per block
constexpr int kRows = 128;            // MMA M: 2 query heads x 64 tokens
constexpr int kThreads = 384;         // 12 warps
// Decoded units queued between scheduler and producer.  One is enough to hide the decode, and every
// unit a CTA holds in advance is a unit another CTA cannot take at the end of the launch: with three
// the last CTAs finished 20 us after the first at 32K, and 8K was 7 % slower.
constexpr int kQueue = 1;
constexpr int kRegsCtl = 40, kRegsSoftmax = 120, kRegsEpilogue = 80;   // registers per thread of each warpgroup
static_assert(kRegsCtl + kRegsSoftmax + kRegsEpilogue <= 240, "register budgets must fit the launch allocation");
constexpr float kSumGuard = 1.152921504606846976e18f;   // 2^60: a tile whose row sum reaches this (or is not finite)
                                                        // is redone against its own maximum

struct AttnArgs {
    const int32_t* cu_seqlens;
    int32_t batch;
    int32_t total_tokens;
    int32_t hq, hkv;
    int32_t group;         // G = hq / hkv query heads per KV head: 1, 2 or 4
    int32_t r_shift;       // log2 of the tile rows per head R = min(64, 128 / G) (6 or 5); a unit covers R query tokens.
                           // With G = 1 only tile rows 0..63 carry a head; rows 64..127 are zero and never stored
    float scale_log2;      // softmax scale * log2(e)
    int32_t dense;         // 1: every predecessor block, lists ignored
    int32_t tail_div;      // the shortest 1 / tail_div of the lists are handed out last, all KV heads interleaved
    // route (BF1 mode)
    const int32_t* qb_seq;
    const int32_t* qb_block;
    const int32_t* kv_count;
    const int32_t* kv_idx;
    const int32_t* order;  // may be null
    const int32_t* num_qblocks;
    int32_t max_degree;
    int32_t capacity;
    int32_t* status;       // may be null in dense mode
    int32_t* sched;        // [2] dynamic hand-out counter + finished-CTA counter; null: static stride
    __nv_bfloat16* o;
    float* lse;
};

// One decoded unit as the scheduler queues it for the producer.
struct QueueEntry {
    int32_t cnt, rows_valid, tok0, kvh, seq0, j, slot, pad;
    int32_t p[32];         // first 32 list entries, range-checked
};

// What the softmax warps leave for the epilogue warps when a unit's last tile is done.
struct Handoff {
    float m[kRows];        // reference maximum per row (raw score units)
    float l[kRows];        // sum of exp2((s - m) * scale_log2) per row
    int32_t cnt, rows_valid, tok0, kvh, g_last, pad[3];
};

template <int D>
struct Cfg {
    static constexpr int kChunks = D / 64;                 // 128-byte column chunks per row
    static constexpr int kQBytes = kRows * D * 2;          // 32 KB at d = 128
    static constexpr int kTileBytes = kBlock * D * 2;      // one K or V block: 16 KB at d = 128
    static constexpr int kRing = (D == 128) ? 4 : 8;       // ring slots
    static constexpr int kQOff = 0;
    static constexpr int kRingOff = kQBytes;
    static constexpr int kStageOff = kRingOff + kRing * kTileBytes;         // O staging: 4 warps x 32 rows x 64 B
    static constexpr int kStageBytes = 4 * 32 * 64;
    static constexpr int kHandOff = kStageOff + kStageBytes;                // Handoff[2]
    static constexpr int kQueueOff = kHandOff + 2 * (int)sizeof(Handoff);   // QueueEntry[kQueue]
    static constexpr int kInfoOff = kQueueOff + kQueue * (int)sizeof(QueueEntry);   // int4[2]
    static constexpr int kBarOff = kInfoOff + 32;
    static constexpr int kNumBars = 2 + 2 * kRing + 2 + 2 + 2 + 1 + 2 + 2 * kQueue + 2 + 2 + 2;
    static constexpr int kMiscOff = kBarOff + 8 * kNumBars;
    static constexpr int kTotal = kMiscOff + 16;
    static constexpr int kTmemCols = 256;
    static constexpr int kColS = 0;                        // S buffers: 2 x 64 fp32 columns
    static constexpr int kColO = 128;                      // O: D fp32 columns
};

struct Unit {
    int seq0, j, cnt, rows_valid, kvh, tok0, slot;
    const int32_t* list;
};

// Unit u of the hand-out order -> what to compute.  KV-head-major (so that the K/V of one head stay hot
// in L2 while its query blocks are processed), inside a head longest list first, then a tail of short units.
// With G = 4 the 128 tile rows are 4 heads x 32 tokens, so a 64-token query block is two units
// (adjacent in the order: they read the same K/V blocks).  `kvh` carries the unit's token offset
// inside its query block in its upper half.
__device__ __forceinline__ void decode_unit(const AttnArgs& a, int nqb, int u, Unit& un) {
    const int halves = kBlock >> a.r_shift;
    const int tok_off = (u % halves) << a.r_shift;
    const int uq = u / halves;
    // Body: KV head by KV head, the longer lists of a head first.  Tail: the shortest lists of ALL heads,
    // longest first across heads, so that the units handed out last are small ones and the CTAs finish
    // together.  The host makes everything tail (tail_div = 1) when K and V fit the L2 cache anyway.
    const int tail_n = nqb / a.tail_div, body_n = nqb - tail_n;
    int idx, head;
    if (uq < body_n * a.hkv) {
        head = uq / body_n;
        idx = uq - head * body_n;
    } else {
        const int ut = uq - body_n * a.hkv;
        idx = body_n + ut / a.hkv;
        head = ut - (ut / a.hkv) * a.hkv;
    }
    un.kvh = head | (tok_off << 16);
    int seq, slot;
    if (!a.dense) {
        slot = a.order ? a.order[idx] : idx;
        seq = a.qb_seq[slot];
        un.j = a.qb_block[slot];
        int c = a.kv_count[slot];
        un.cnt = min(max(c, 1), a.max_degree);
        un.slot = slot;
        un.list = a.kv_idx + (size_t)slot * a.max_degree;
    } else {
        slot = nqb - 1 - idx;
        int acc = 0;
        seq = 0;
        un.j = 0;
        for (int s = 0; s < a.batch; ++s) {
            const int nb = (a.cu_seqlens[s + 1] - a.cu_seqlens[s] + kBlock - 1) / kBlock;
            if (slot < acc + nb) { seq = s; un.j = slot - acc; break; }
            acc += nb;
        }
        un.cnt = un.j + 1;
        un.slot = slot;
        un.list = nullptr;
    }
    un.seq0 = a.cu_seqlens[seq];
    const int seqlen = a.cu_seqlens[seq + 1] - un.seq0;
    un.rows_valid = max(0, min(1 << a.r_shift, seqlen - un.j * kBlock - tok_off));   // of this unit's R tokens
    un.tok0 = un.seq0 + un.j * kBlock + tok_off;
}

template <int REGS>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
}
template <int REGS>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2) attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                               const __grid_constant__ CUtensorMap tm_k,
                                                               const __grid_constant__ CUtensorMap tm_v,
                                                               const __grid_constant__ CUtensorMap tm_o,
                                                               const AttnArgs args) {
    using C = Cfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // Dynamic hand-out: sched[0] is the next unit, sched[1] counts CTAs that are done; the last
    // one to finish puts both back to zero, so the words are ready for the next launch.
    auto retire = [&]() {
        if (args.sched && threadIdx.x == 0) {
            __threadfence();
            if (atomicAdd(args.sched + 1, 1) == (int)gridDim.x - 1) {
                args.sched[0] = 0;
                args.sched[1] = 0;
                __threadfence();
            }
        }
    };
    const uint32_t base = smem_u32(smem);
    const uint32_t sQ = base + C::kQOff;
    const uint32_t sRing = base + C::kRingOff;
    const uint32_t bar_q_full = base + C::kBarOff;
    const uint32_t bar_q_free = bar_q_full + 8;
    const uint32_t bar_full = bar_q_free + 8;                 // [kRing]
    const uint32_t bar_free = bar_full + 8 * C::kRing;        // [kRing]
    const uint32_t bar_s_full = bar_free + 8 * C::kRing;      // [2]
    const uint32_t bar_p_full = bar_s_full + 16;              // [2]
    const uint32_t bar_pv_done = bar_p_full + 16;             // [2]
    const uint32_t bar_o_free = bar_pv_done + 16;
    const uint32_t bar_info = bar_o_free + 8;                 // [2]
    const uint32_t bar_sq_full = bar_info + 16;               // [kQueue]
    const uint32_t bar_sq_free = bar_sq_full + 8 * kQueue;    // [kQueue]
    const uint32_t bar_ho_full = bar_sq_free + 8 * kQueue;    // [2]
    const uint32_t bar_ho_free = bar_ho_full + 16;            // [2]
    const uint32_t bar_info_free = bar_ho_free + 16;          // [2]
    volatile int4* s_info = reinterpret_cast<volatile int4*>(smem + C::kInfoOff);   // {cnt, rows_valid, tok0, kvh}
    volatile QueueEntry* s_queue = reinterpret_cast<volatile QueueEntry*>(smem + C::kQueueOff);
    volatile Handoff* s_hand = reinterpret_cast<volatile Handoff*>(smem + C::kHandOff);
    uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem + C::kMiscOff);
    int* s_abort = reinterpret_cast<int*>(smem + C::kMiscOff + 4);
    int* s_nqb = reinterpret_cast<int*>(smem + C::kMiscOff + 8);

    if (tid == 0) {
        // The status word and the block count are read together (two independent loads in flight), and no other
        // warp waits for them before its own set-up.  If an earlier launch on this status word gave up, this one
        // raises its abort flag: every role then sees an empty queue and the CTA leaves through the normal exit.
        const int earlier = args.status ? *args.status : 0;
        int nqb = 0;
        if (!args.dense) {
            nqb = min(*args.num_qblocks, args.capacity);
        }
        *s_abort = (earlier & BF1_DEV_WAIT_TIMEOUT) ? 1 : 0;
        if (base & 1023u) {   // the swizzled tiles need a 1024-byte aligned window
            *s_abort = 1;
            if (args.status) atomicOr(args.status, BF1_DEV_WAIT_TIMEOUT);
        }
        if (args.dense) {
            for (int s = 0; s < args.batch; ++s)
                nqb += (args.cu_seqlens[s + 1] - args.cu_seqlens[s] + kBlock - 1) / kBlock;
        }
        *s_nqb = nqb;
        s_nqb[1] = 0;
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_free, 1);
        for (int s = 0; s < C::kRing; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_free + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_s_full + 8 * s, 1);
            mbar_init(bar_p_full + 8 * s, 4);    // one arrival per softmax warp
            mbar_init(bar_pv_done + 8 * s, 1);
            mbar_init(bar_info + 8 * s, 1);
            mbar_init(bar_ho_full + 8 * s, 4);   // softmax warps
            mbar_init(bar_ho_free + 8 * s, 4);   // epilogue warps
            mbar_init(bar_info_free + 8 * s, 5); // softmax warps + PV issuer have read the unit descriptor
        }
        for (int s = 0; s < kQueue; ++s) {
            mbar_init(bar_sq_full + 8 * s, 1);
            mbar_init(bar_sq_free + 8 * s, 1);
        }
        mbar_init(bar_o_free, 4);                // epilogue warps
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_o);
    }
    __syncwarp();
    // The scheduler warp decodes this CTA's first unit (unit blockIdx.x; the shared counter hands
    // out the units after the first gridDim.x) while the others set up barriers and tensor memory:
    // the decode is a chain of dependent global loads that would otherwise delay the first copy.
    auto fetch_unit = [&](int u, int nqb_, Unit& un, int& my_p) {
        decode_unit(args, nqb_, u, un);
        my_p = 0;
        if (lane < un.cnt) {   // entries 0..31, one per lane, made safe to use
            int p = args.dense ? lane : un.list[lane];
            if (p < 0 || p > un.j || (lane == un.cnt - 1) != (p == un.j)) {
                if (args.status) atomicOr(args.status, BF1_DEV_BAD_ROUTE);
                p = (lane == un.cnt - 1) ? un.j : 0;
            }
            my_p = p;
        }
    };
    Unit un0 = {};
    int my_p0 = 0;
    bool have0 = false;
    if (warp == 2) {
        int nqb0 = 0;
        if (!args.dense) {
            nqb0 = min(*args.num_qblocks, args.capacity);
        } else {
            for (int s = 0; s < args.batch; ++s)
                nqb0 += (args.cu_seqlens[s + 1] - args.cu_seqlens[s] + kBlock - 1) / kBlock;
        }
        have0 = (int)blockIdx.x < nqb0 * args.hkv * (kBlock >> args.r_shift);
        if (have0) fetch_unit(blockIdx.x, nqb0, un0, my_p0);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem_base), C::kTmemCols);
        tmem_relinquish();
    }
    if (args.group == 1) {
        // one query head per KV head: the lower half of the 128-row tile is unused; the MMAs still read it, so
        // it is cleared once (the Q copies only ever write rows 0..63 of each column chunk)
        for (int i = tid; i < C::kChunks * (kBlock * 128 / 16); i += kThreads) {
            const int ch = i / (kBlock * 128 / 16), off = i % (kBlock * 128 / 16);
            st_shared_v4(sQ + ch * (kRows * 128) + kBlock * 128 + off * 16, 0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem_base;
    volatile int* abort_flag = s_abort;
    const int nqb = *s_nqb;
    const int total_units = nqb * args.hkv * (kBlock >> args.r_shift);

    if (warp < 4) {
        setmaxnreg_dec<kRegsCtl>();
        if (warp == 2) {
            // ================================ scheduler =======================================
            for (int n = 0;; ++n) {
                Unit un = un0;
                int my_p = my_p0;
                bool have = have0 && !*abort_flag;
                if (n > 0) {
                    int u = 0;
                    if (lane == 0)
                        u = (args.sched ? atomicAdd(args.sched, 1) + (int)gridDim.x : (int)(blockIdx.x + n * gridDim.x));
                    u = __shfl_sync(0xffffffffu, u, 0);
                    have = u < total_units && !*abort_flag;
                    if (have) fetch_unit(u, nqb, un, my_p);
                }
                const int qs = n % kQueue;
                if (n >= kQueue) mbar_wait(bar_sq_free + 8 * qs, ((n / kQueue) - 1) & 1, abort_flag, args.status);
                volatile QueueEntry* e = s_queue + qs;
                e->p[lane] = my_p;
                if (lane == 0) {
                    e->cnt = have ? un.cnt : 0;
                    e->rows_valid = un.rows_valid;
                    e->tok0 = un.tok0;
                    e->kvh = un.kvh;
                    e->seq0 = un.seq0;
                    e->j = un.j;
                    e->slot = un.slot;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sq_full + 8 * qs);
                if (!have) break;
            }
        } else if (warp == 0) {
            // ================================ TMA producer ====================================
            // The whole warp walks the loop; one elected lane issues the copies.
            int slot = 0, pass = 0;
            for (int n = 0;; ++n) {
                const int qs = n % kQueue;
                mbar_wait(bar_sq_full + 8 * qs, (n / kQueue) & 1, abort_flag, args.status);
                volatile QueueEntry* e = s_queue + qs;
                int cnt = e->cnt;
                const int rows_valid = e->rows_valid, tok0 = e->tok0, kvh_packed = e->kvh, seq0 = e->seq0, j = e->j;
                const int kvh = kvh_packed & 0xffff;
                const int rslot = e->slot;
                int my_p = e->p[lane];
                if (*abort_flag) cnt = 0;
                auto load_tile = [&](int p, bool is_v) {
                    if (pass > 0) mbar_wait(bar_free + 8 * slot, (pass - 1) & 1, abort_flag, args.status);
                    const uint32_t bar = bar_full + 8 * slot;
                    if (elect_one()) {
                        mbar_expect_tx(bar, C::kTileBytes);
                        // one copy per tile: box = 64 elements x 64 tokens x 1 head x all column chunks
                        tma_load_4d(sRing + slot * C::kTileBytes, is_v ? &tm_v : &tm_k, 0, seq0 + p * kBlock, kvh, 0, bar);
                    }
                    __syncwarp();
                    if (++slot == C::kRing) { slot = 0; ++pass; }
                };
                // One loop body for every step keeps the producer's code small and hot in the
                // instruction cache.  Step s loads K(s) and then V(s-1): K0, [Q], K1, V0, K2, V1, ...,
                // the order in which the MMA warp consumes them.  K0 only needs a ring slot, so it
                // is started before the wait for the Q buffer.
                int base_i = 0;
                int p_prev = 0;
                for (int st = 0; st <= cnt; ++st) {
                    int p_cur = 0;
                    if (st < cnt) {
                        if (st - base_i == 32) {   // lists longer than a warp: fetch the next 32 entries
                            base_i += 32;
                            const int ii = base_i + lane;
                            int p = 0;
                            if (ii < cnt) {
                                p = args.dense ? ii : args.kv_idx[(size_t)rslot * args.max_degree + ii];
                                if (p < 0 || p > j || (ii == cnt - 1) != (p == j)) {
                                    if (args.status) atomicOr(args.status, BF1_DEV_BAD_ROUTE);
                                    p = (ii == cnt - 1) ? j : 0;
                                }
                            }
                            my_p = p;
                        }
                        p_cur = __shfl_sync(0xffffffffu, my_p, st - base_i);
                        load_tile(p_cur, false);
                    }
                    if (st == 0) {
                        if (n > 0) mbar_wait(bar_q_free, (n - 1) & 1, abort_flag, args.status);
                        // slot n & 1 of the descriptor was last used by unit n - 2: every reader has let go of it
                        if (n >= 2) mbar_wait(bar_info_free + 8 * (n & 1), ((n >> 1) - 1) & 1, abort_flag, args.status);
                        if (elect_one()) {
                            // publish the unit (or the end marker cnt = 0) to the MMA and softmax warps
                            s_info[n & 1].x = cnt;
                            s_info[n & 1].y = rows_valid;
                            s_info[n & 1].z = tok0;
                            s_info[n & 1].w = kvh_packed;
                            mbar_arrive(bar_info + 8 * (n & 1));
                            if (cnt == 0) {
                                mbar_arrive(bar_q_full);
                            } else if (args.group > 1) {
                                mbar_expect_tx(bar_q_full, C::kQBytes);
                                // one copy: box = 64 elements x R tokens x G heads x all column chunks
                                tma_load_4d(sQ, &tm_q, 0, tok0, kvh * args.group, 0, bar_q_full);
                            } else {
                                // G = 1: one head, 64 rows per column chunk; each chunk goes to the place the
                                // 128-row tile layout gives it (rows 64..127 stay zero)
                                mbar_expect_tx(bar_q_full, C::kQBytes / 2);
#pragma unroll
                                for (int ch = 0; ch < C::kChunks; ++ch)
                                    tma_load_4d(sQ + ch * (kRows * 128), &tm_q, 0, tok0, kvh, ch, bar_q_full);
                            }
                        }
                        __syncwarp();
                    } else {
                        load_tile(p_prev, true);
                    }
                    p_prev = p_cur;
                }
                if (cnt == 0) break;
                if (elect_one()) mbar_arrive(bar_sq_free + 8 * qs);
                __syncwarp();
            }
        } else if (warp == 1) {
            // ================================ MMA issuer: S = Q K^T ============================
            // The whole warp walks the loop (so that addresses and descriptors stay warp-uniform and
            // cheap); one elected lane issues the MMAs and commits.  S and PV have separate issuing
            // warps: an issuer stalls while the tensor pipe's queue is full, and with one issuer a
            // stalled burst of S MMAs would keep a ready PV (which frees an S buffer and feeds the
            // epilogue) waiting behind it, and the other way round.
            constexpr uint32_t kIdescS = idesc_bf16_f32(kBlock, false);   // 128 x 64 x 16, K-major B
            static_assert((C::kRing & (C::kRing - 1)) == 0, "ring size must be a power of two");
            uint32_t g = 0;    // tiles before this unit; S buffer of tile t = t & 1
            uint32_t e0 = 0;   // ring fills before this unit
            // Descriptor halves that never change: the high word (SBO = 1024, version, swizzle) and
            // the low words of Q's eight k-slices; a ring slot only adds slot * kTileBytes / 16.
            constexpr uint32_t kDescHi = desc_hi_sw128(1024);
            const uint32_t q_lo = desc_lo_sw128(sQ, 16);
            const uint32_t k_lo0 = desc_lo_sw128(sRing, 16);
            for (int n = 0;; ++n) {
                mbar_wait(bar_q_full, n & 1, abort_flag, args.status);
                const int cnt = s_info[n & 1].x;
                if (cnt == 0 || *abort_flag) break;
                for (int st = 0; st < cnt; ++st) {
                    const uint32_t t = g + st;
                    const uint32_t e = e0 + (st == 0 ? 0 : 2 * st - 1);   // ring fill holding K(st): K0, K1, V0, K2, V1, ...
                    const uint32_t slot = e & (C::kRing - 1);
                    mbar_wait(bar_full + 8 * slot, (e / C::kRing) & 1, abort_flag, args.status);   // K landed
                    // S(t) overwrites the buffer that held P(t-2): PV(t-2) must have finished with it
                    if (t >= 2) mbar_wait(bar_pv_done + 8 * (t & 1), ((t - 2) >> 1) & 1, abort_flag, args.status);
                    tc_fence_after();
                    const uint32_t k_lo = k_lo0 + slot * (C::kTileBytes >> 4);
                    const uint32_t d_s = tmem + C::kColS + (t & 1) * 64;
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t a_off = ((kk / 4) * (kRows * 128) + (kk % 4) * 32) >> 4;
                            const uint32_t b_off = ((kk / 4) * (kBlock * 128) + (kk % 4) * 32) >> 4;
                            if (kk == 0) mma_ss_lohi<false>(d_s, q_lo + a_off, k_lo + b_off, kDescHi, kIdescS);
                            else mma_ss_lohi<true>(d_s, q_lo + a_off, k_lo + b_off, kDescHi, kIdescS);
                        }
                        mma_commit(bar_free + 8 * slot);
                        mma_commit(bar_s_full + 8 * (t & 1));
                        if (st == cnt - 1) mma_commit(bar_q_free);   // last S of the unit: Q may be replaced
                    }
                    __syncwarp();
                }
                g += cnt;
                e0 += 2 * cnt;
            }
        } else if (warp == 3) {
            // ================================ MMA issuer: O += P V =============================
            constexpr uint32_t kIdescO = idesc_bf16_f32(D, true);         // 128 x D x 16, MN-major B
            constexpr uint32_t kDescHi = desc_hi_sw128(1024);
            const uint32_t v_lo0 = desc_lo_sw128(sRing, kBlock * 128);
            uint32_t g = 0, e0 = 0;
            for (int n = 0;; ++n) {
                mbar_wait(bar_info + 8 * (n & 1), (n >> 1) & 1, abort_flag, args.status);
                const int cnt = s_info[n & 1].x;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_info_free + 8 * (n & 1));
                if (cnt == 0 || *abort_flag) break;
                for (int st = 0; st < cnt; ++st) {
                    const uint32_t t = g + st;
                    const uint32_t e = e0 + (st == cnt - 1 ? 2 * cnt - 1 : 2 * st + 2);   // ring fill holding V(st)
                    const uint32_t slot = e & (C::kRing - 1);
                    mbar_wait(bar_full + 8 * slot, (e / C::kRing) & 1, abort_flag, args.status);       // V landed
                    mbar_wait(bar_p_full + 8 * (t & 1), (t >> 1) & 1, abort_flag, args.status);        // P written
                    if (st == 0 && n > 0) mbar_wait(bar_o_free, (n - 1) & 1, abort_flag, args.status);
                    tc_fence_after();
                    // V tile: rows = kv tokens (the K of this MMA), 128-byte rows of 64 d-elements;
                    // 16 kv rows per MMA = two 8-row groups = 2048 bytes; next d chunk 8 KB away
                    const uint32_t v_lo = v_lo0 + slot * (C::kTileBytes >> 4);
                    const uint32_t a_p = tmem + C::kColS + (t & 1) * 64;
                    if (elect_one()) {
                        if (st == 0) mma_ts_lohi<false>(tmem + C::kColO, a_p, v_lo, kDescHi, kIdescO);
                        else mma_ts_lohi<true>(tmem + C::kColO, a_p, v_lo, kDescHi, kIdescO);
#pragma unroll
                        for (int kk = 1; kk < kBlock / 16; ++kk)
                            mma_ts_lohi<true>(tmem + C::kColO, a_p + kk * 8, v_lo + kk * (2048 >> 4), kDescHi, kIdescO);
                        mma_commit(bar_free + 8 * slot);
                        mma_commit(bar_pv_done + 8 * (t & 1));
                    }
                    __syncwarp();
                }
                g += cnt;
                e0 += 2 * cnt;
            }
        }
        __syncwarp();
    } else if (warp < 8) {
        // ================================ softmax ==========================================
        setmaxnreg_inc<kRegsSoftmax>();
        const int quarter = warp & 3;                     // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;              // tile row of this thread: head row / R, token row % R
        const uint32_t t_lane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c2 = args.scale_log2;
        uint32_t g = 0;
        for (int n = 0;; ++n) {
            mbar_wait(bar_info + 8 * (n & 1), (n >> 1) & 1, abort_flag, args.status);
            const int cnt = *abort_flag ? 0 : s_info[n & 1].x;
            const int rows_valid = s_info[n & 1].y, tok0 = s_info[n & 1].z, kvh = s_info[n & 1].w;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_info_free + 8 * (n & 1));
            const int tl = (kvh >> 16) + (row & ((1 << args.r_shift) - 1));   // token inside the 64-token query block
            float m_used = 0.f;    // reference maximum (raw score units) the exponentials are taken against
            float l_run = 0.f;     // running sum of exp2((s - m_used) * c2)
            for (int i = 0; i < cnt; ++i, ++g) {
                const uint32_t t_s = t_lane + C::kColS + (g & 1) * 64;
                mbar_wait(bar_s_full + 8 * (g & 1), (g >> 1) & 1, abort_flag, args.status);
                tc_fence_after();
                // The exponentials of a tile are taken against the row's current reference maximum m_used; the
                // tile's own maximum is only computed for the first tile of a unit, and again (second pass) when
                // a row's sum shows that the reference has fallen too far behind (sum >= 2^60, or not finite).
                // Any reference gives the same softmax as long as nothing overflows: P (bf16), l and O (fp32) are
                // floating point, so their relative accuracy does not depend on the scale.  The second pass is
                // entered by the whole warp (its tensor-memory accesses are warp-wide), but only a row whose own
                // sum tripped moves its reference; every other row multiplies by exactly 1 and recomputes the
                // values it already had, so a row's arithmetic depends on that row alone (later tokens of the
                // block cannot change it).
                uint32_t preg[32];
                float tile_sum = 0.f;
                bool tripped = false;
#pragma unroll 1
                for (int pass = 0; pass < 2; ++pass) {
                    uint32_t sreg[64];
                    {
                        uint32_t (&lo)[32] = *reinterpret_cast<uint32_t (*)[32]>(&sreg[0]);
                        uint32_t (&hi)[32] = *reinterpret_cast<uint32_t (*)[32]>(&sreg[32]);
                        tmem_ld32(t_s, lo);
                        tmem_ld32(t_s + 32, hi);
                    }
                    tmem_wait_ld();
                    if (i == cnt - 1) {   // self block: causal triangle (warp-uniform branch)
#pragma unroll
                        for (int c = 0; c < 64; ++c)
                            if (c > tl) sreg[c] = 0xff800000u;   // -inf
                    }
                    if (i == 0 || pass == 1) {
                        float mxa = -INFINITY, mxb = -INFINITY;
#pragma unroll
                        for (int c = 0; c < 64; c += 4) {
                            mxa = fmax3(mxa, __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]));
                            mxb = fmax3(mxb, __uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3]));
                        }
                        const float mx = fmaxf(mxa, mxb);
                        if (i == 0) {
                            m_used = mx;
                        } else {
                            const float alpha = tripped ? ex2_approx((m_used - mx) * c2) : 1.0f;
                            l_run *= alpha;
                            m_used = tripped ? mx : m_used;
                            // O holds the sum up to tile i-1 once PV(g-1) has completed
                            mbar_wait(bar_pv_done + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1, abort_flag, args.status);
                            tc_fence_after();
#pragma unroll
                            for (int c = 0; c < D / 16; ++c) {
                                uint32_t oreg[16];
                                tmem_ld16(t_lane + C::kColO + c * 16, oreg);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
                                tmem_st16(t_lane + C::kColO + c * 16, oreg);
                            }
                        }
                    }
                    const float msc = m_used * c2;
                    const uint64_t c2p = pack2(c2, c2), mscp = pack2(-msc, -msc);
                    uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const uint64_t x = fma2(pack2(__uint_as_float(sreg[2 * c]), __uint_as_float(sreg[2 * c + 1])), c2p, mscp);
                        float x0, x1;
                        unpack2(x, x0, x1);
                        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
                        if (c & 1) sum_b = add2(sum_b, pack2(p0, p1)); else sum_a = add2(sum_a, pack2(p0, p1));
                        preg[c] = pack_bf16x2(p0, p1);
                    }
                    float r0, r1;
                    unpack2(add2(sum_a, sum_b), r0, r1);
                    tile_sum = r0 + r1;
                    if (i == 0 || pass == 1) break;
                    tripped = !(tile_sum < kSumGuard);
                    if (!__any_sync(0xffffffffu, tripped)) break;
                }
                l_run += tile_sum;
                tmem_st32(t_s, preg);   // P overwrites the first 32 columns of this S buffer
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p_full + 8 * (g & 1));
            }
            // ---- hand the unit over to the epilogue warps -------------------------------------
            if (n >= 2) mbar_wait(bar_ho_free + 8 * (n & 1), ((n >> 1) - 1) & 1, abort_flag, args.status);
            volatile Handoff* h = s_hand + (n & 1);
            h->m[row] = m_used;
            h->l[row] = l_run;
            if (row == 0) {
                h->cnt = cnt;
                h->rows_valid = rows_valid;
                h->tok0 = tok0;
                h->kvh = kvh;
                h->g_last = (int)(g - 1);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ho_full + 8 * (n & 1));
            if (cnt == 0) break;
        }
    } else {
        // ================================ epilogue =========================================
        setmaxnreg_dec<kRegsEpilogue>();
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int hl = row >> args.r_shift;               // which head of the group (uniform in a warp: R >= 32)
        const int tl = row & ((1 << args.r_shift) - 1);   // token inside the unit
        const uint32_t t_lane = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c2 = args.scale_log2;
        for (int n = 0;; ++n) {
            mbar_wait(bar_ho_full + 8 * (n & 1), (n >> 1) & 1, abort_flag, args.status);
            volatile Handoff* h = s_hand + (n & 1);
            const float m_used = h->m[row], l_run = h->l[row];
            const int cnt = *abort_flag ? 0 : h->cnt;
            const int rows_valid = h->rows_valid, tok0 = h->tok0, kvh = h->kvh & 0xffff;
            const uint32_t gl = (uint32_t)h->g_last;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ho_free + 8 * (n & 1));
            if (cnt == 0) break;
            mbar_wait(bar_pv_done + 8 * (gl & 1), (gl >> 1) & 1, abort_flag, args.status);
            tc_fence_after();
            const float inv_l = 1.f / l_run;
            const int tok = tok0 + tl;
            const bool head_ok = hl < args.group;      // G = 1: tile rows 64..127 belong to no head (warp-uniform)
            const bool store = tl < rows_valid && head_ok;
            __nv_bfloat16* orow = args.o + ((size_t)tok * args.hq + (kvh * args.group + hl)) * D;
            // O leaves tensor memory first, all of it, normalised and packed to bf16 in registers: the
            // next unit's first PV overwrites O and waits for exactly this, so nothing slow (staging,
            // copy-engine waits) may sit in front of the release.
            uint32_t pk[D / 2];
#pragma unroll
            for (int c = 0; c < D / 16; ++c) {
                uint32_t oreg[16];
                tmem_ld16(t_lane + C::kColO + c * 16, oreg);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    pk[c * 8 + e] = pack_bf16x2(__uint_as_float(oreg[2 * e]) * inv_l, __uint_as_float(oreg[2 * e + 1]) * inv_l);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_o_free);
            // Full blocks then go through shared memory and TMA stores: each warp packs 32 rows x 32
            // columns into its own 2 KB staging tile (64-byte swizzle, conflict-free) and one lane
            // hands it to the copy engine.  Scattered 16-byte global stores from here would sit in the
            // same load/store path as every other warp's mbarrier and shared-memory traffic and
            // slow the whole SM down.
            const bool full_tile = rows_valid == (1 << args.r_shift) && head_ok;   // warp-uniform
            const uint32_t stage_w = base + C::kStageOff + (warp & 3) * 2048;
            const uint32_t srow = stage_w + lane * 64;
            if (full_tile) {
                const int sw = (lane >> 1) & 3;       // 64-byte swizzle: chunk ^= (row / 2) % 4
#pragma unroll
                for (int c2 = 0; c2 < D / 32; ++c2) {   // 32 columns = 16 packed registers per store
                    if (lane == 0) bulk_wait_read0();   // the previous store has finished reading the tile
                    __syncwarp();
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
                        st_shared_v4(srow + ((ch ^ sw) << 4), pk[c2 * 16 + ch * 4 + 0], pk[c2 * 16 + ch * 4 + 1],
                                     pk[c2 * 16 + ch * 4 + 2], pk[c2 * 16 + ch * 4 + 3]);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_3d(&tm_o, c2 * 32, kvh * args.group + hl, tok0 + ((quarter * 32) & ((1 << args.r_shift) - 1)),
                                     stage_w);
                        bulk_commit_group();
                    }
                }
            } else if (store) {
                // partial last block of a sequence: the rows after it belong to someone else
#pragma unroll
                for (int c = 0; c < D / 8; ++c)
                    *reinterpret_cast<uint4*>(orow + c * 8) = make_uint4(pk[c * 4], pk[c * 4 + 1], pk[c * 4 + 2], pk[c * 4 + 3]);
            }
            if (store) {
                const float lse2 = m_used * c2 + lg2_approx(l_run);   // log2 domain
                args.lse[(size_t)(kvh * args.group + hl) * args.total_tokens + tok] = lse2 * 0.6931471805599453f;
            }
        }
    }

    if (warp >= 8 && lane == 0) bulk_wait0();   // this thread's output stores have landed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, C::kTmemCols);
    retire();
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

// Encoding a tensor map costs a driver call of a microsecond or two, and a forward call needs four.
// A map is a pure function of (pointer, extents, box, swizzle), so each host thread keeps the last
// few it built; a layer that is called again with the same buffers (every step of a serving loop,
// every repetition of a benchmark) then launches without touching the driver.
struct MapKey {
    const void* ptr;
    int64_t T;
    int32_t H, d, heads_per_box, tokens_per_box, kind;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && T == o.T && H == o.H && d == o.d && heads_per_box == o.heads_per_box &&
               tokens_per_box == o.tokens_per_box && kind == o.kind;
    }
};
struct MapCache {
    static constexpr int kEntries = 64;
    MapKey key[kEntries];
    CUtensorMap map[kEntries];
    bool used[kEntries] = {};
    static uint32_t slot_of(const MapKey& k) {
        uint64_t h = (uint64_t)(uintptr_t)k.ptr * 0x9E3779B97F4A7C15ull;
        h ^= (uint64_t)k.T * 0xC2B2AE3D27D4EB4Full + (uint64_t)(k.H * 131 + k.d * 31 + k.heads_per_box * 7 + k.tokens_per_box * 3 + k.kind);
        return (uint32_t)(h >> 40) % kEntries;
    }
    const CUtensorMap* find(const MapKey& k) const {
        const uint32_t i = slot_of(k);
        return used[i] && key[i] == k ? &map[i] : nullptr;
    }
    void put(const MapKey& k, const CUtensorMap& m) {
        const uint32_t i = slot_of(k);
        key[i] = k;
        map[i] = m;
        used[i] = true;
    }
};
static thread_local MapCache g_map_cache;

// [T, H, d] bf16 tensor seen as 4-D {64 elements, T tokens, H heads, d/64 column chunks}; box = 64
// elements (128 bytes) x 64 tokens x `heads_per_box` heads x all chunks, 128-byte swizzle.  In shared
// memory that is [chunk][head][token][128 B]: one K-major (or, for V, MN-major) 64-row tile per
// chunk and head, which is what the MMA descriptors walk.
static int make_map(CUtensorMap* m, const void* ptr, int64_t T, int H, int d, int heads_per_box, int tokens_per_box = kBlock,
                    int chunks_per_box = 0) {
    if (chunks_per_box == 0) chunks_per_box = d / 64;
    const MapKey key{ptr, T, H, d, heads_per_box, tokens_per_box, chunks_per_box == d / 64 ? 0 : 2};
    if (const CUtensorMap* hit = g_map_cache.find(key)) {
        *m = *hit;
        return BF1_OK;
    }
    EncodeTiledFn enc;
    if (int rc = get_encode_fn(&enc)) return rc;
    cuuint64_t dims[4] = {64, (cuuint64_t)T, (cuuint64_t)H, (cuuint64_t)(d / 64)};
    cuuint64_t strides[3] = {(cuuint64_t)H * d * 2, (cuuint64_t)d * 2, 128};
    cuuint32_t box[4] = {64, (cuuint32_t)tokens_per_box, (cuuint32_t)heads_per_box, (cuuint32_t)chunks_per_box};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(BF1_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    g_map_cache.put(key, *m);
    return BF1_OK;
}

// O [T, Hq, d] bf16 for the epilogue's TMA stores: box = 32 elements (64 bytes) x 1 head x 32 tokens,
// 64-byte swizzle.
static int make_store_map(CUtensorMap* m, void* ptr, int64_t T, int H, int d) {
    const MapKey key{ptr, T, H, d, 1, 32, 1};
    if (const CUtensorMap* hit = g_map_cache.find(key)) {
        *m = *hit;
        return BF1_OK;
    }
    EncodeTiledFn enc;
    if (int rc = get_encode_fn(&enc)) return rc;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)H * d * 2};
    cuuint32_t box[3] = {32, 1, 32};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptr, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(BF1_ERR_CUDA, "cuTensorMapEncodeTiled (O) failed with CUresult %d", (int)r);
    g_map_cache.put(key, *m);
    return BF1_OK;
}

// the same map for the other translation units of the library
int make_map_4d(CUtensorMap* m, const void* ptr, int64_t T, int H, int d, int heads_per_box, int chunks_per_box) {
    return make_map(m, ptr, T, H, d, heads_per_box, kBlock, chunks_per_box);
}

struct DeviceInfo {
    int sm_count = 0;
    bool ok = false;
};

static int device_info(DeviceInfo* out) {
    static DeviceInfo cache[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(BF1_ERR_NO_DEVICE, "no CUDA device: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return fail(BF1_ERR_NO_DEVICE, "device ordinal %d out of range", dev);
    if (!cache[dev].ok) {
        int major = 0, sms = 0;
        BF1_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return fail(BF1_ERR_NO_DEVICE, "device compute capability %d.x is not sm_100", major);
        BF1_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            Cfg<128>::kTotal));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(attn_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            Cfg<64>::kTotal));
        cache[dev].sm_count = sms;
        cache[dev].ok = true;
    }
    *out = cache[dev];
    return BF1_OK;
}

// Everything about a forward call that the host can check without a device or a route.
int check_attn_args(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev, int32_t batch,
                    int64_t total_tokens, int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d, const void* o,
                    const float* lse) {
    if (!q || !k || !v || !o || !lse || !cu_seqlens_dev)
        return fail(BF1_ERR_INVALID_ARG, "a tensor pointer is null");
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || hq <= 0 || hkv <= 0 || d <= 0)
        return fail(BF1_ERR_INVALID_ARG, "negative or zero size argument");
    if (total_tokens > 0x7fffffffLL - 64)
        return fail(BF1_ERR_UNSUPPORTED, "total_tokens %lld does not fit 32-bit token indices", (long long)total_tokens);
    if (hq % hkv != 0) return fail(BF1_ERR_INVALID_ARG, "hq %d is not a multiple of hkv %d", hq, hkv);
    const int group = hq / hkv;
    if (group != 1 && group != 2 && group != 4)
        return fail(BF1_ERR_UNSUPPORTED, "GQA group size %d: only G = 1, 2 and 4 are supported", group);
    if (d != 64 && d != 128) return fail(BF1_ERR_UNSUPPORTED, "head dimension %d: only 64 and 128 are supported", d);
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15)
        return fail(BF1_ERR_INVALID_ARG, "q, k, v and o must be 16-byte aligned");
    return BF1_OK;
}

static int attn_common(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_dev, int32_t batch,
                       int64_t total_tokens, int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d,
                       float softmax_scale, const bf1_route* route, void* o, float* lse, int32_t* work_dev,
                       void* stream) {
    if (int rc = check_attn_args(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, o, lse)) return rc;
    const int group = hq / hkv;
    int64_t slots;
    if (route) {
        if (!route->qb_seq || !route->qb_block || !route->kv_count || !route->kv_idx || !route->num_qblocks ||
            !route->status)
            return fail(BF1_ERR_INVALID_ARG, "a route array pointer is null");
        if (route->capacity_qblocks < 1 || route->max_degree < 1)
            return fail(BF1_ERR_CAPACITY, "route capacity_qblocks and max_degree must be >= 1");
        slots = route->capacity_qblocks;
    } else {
        slots = total_tokens / kBlock + batch;
    }
    if (slots * hkv * 2 > 0x7fffffffLL) return fail(BF1_ERR_UNSUPPORTED, "too many work units");
    if (total_tokens == 0 || batch == 0) return BF1_OK;   // nothing to do
    DeviceInfo info;
    if (int rc = device_info(&info)) return rc;

    CUtensorMap tq, tk, tv, to;
    if (int rc = make_store_map(&to, o, total_tokens, hq, d)) return rc;
    if (group == 1) {   // one head, one column chunk per copy
        if (int rc = make_map(&tq, q, total_tokens, hq, d, 1, kBlock, 1)) return rc;
    } else {
        if (int rc = make_map(&tq, q, total_tokens, hq, d, group, kRows / group)) return rc;
    }
    if (int rc = make_map(&tk, k, total_tokens, hkv, d, 1)) return rc;
    if (int rc = make_map(&tv, v, total_tokens, hkv, d, 1)) return rc;

    AttnArgs a;
    a.cu_seqlens = cu_seqlens_dev;
    a.batch = batch;
    a.total_tokens = (int32_t)total_tokens;
    a.hq = hq;
    a.hkv = hkv;
    a.group = group;
    a.r_shift = group == 4 ? 5 : 6;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)d);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.dense = route ? 0 : 1;
    // Hand-out order.  One KV head at a time keeps that head's K and V hot in L2 while its query blocks are
    // processed, which matters once K and V of all heads together outgrow the cache (32K tokens x 8 heads x 128:
    // 134 MB; interleaving the heads there cost 6 %).  Below that, longest-first over all heads balances the
    // CTAs better (4K: 23.5 -> 21.6 us, 8K: 41.0 -> 38.6 us, dense 8K: 280 -> 222 us).
    const int64_t kv_bytes = total_tokens * (int64_t)hkv * d * 4;
    a.tail_div = kv_bytes <= (48LL << 20) ? 1 : 8;
    a.qb_seq = route ? route->qb_seq : nullptr;
    a.qb_block = route ? route->qb_block : nullptr;
    a.kv_count = route ? route->kv_count : nullptr;
    a.kv_idx = route ? route->kv_idx : nullptr;
    a.order = route ? route->order : nullptr;
    a.num_qblocks = route ? route->num_qblocks : nullptr;
    a.max_degree = route ? route->max_degree : 0;
    a.capacity = route ? route->capacity_qblocks : 0;
    a.status = route ? route->status : work_dev;
    a.sched = route ? route->sched : (work_dev ? work_dev + 1 : nullptr);
    a.o = reinterpret_cast<__nv_bfloat16*>(o);
    a.lse = lse;

    const int64_t units = slots * hkv * (group == 4 ? 2 : 1);
    const int grid = (int)(units < 2LL * info.sm_count ? units : 2LL * info.sm_count);
    if (d == 128)
        attn_fwd_kernel<128><<<grid, kThreads, Cfg<128>::kTotal, (cudaStream_t)stream>>>(tq, tk, tv, to, a);
    else
        attn_fwd_kernel<64><<<grid, kThreads, Cfg<64>::kTotal, (cudaStream_t)stream>>>(tq, tk, tv, to, a);
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
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
                                    int32_t* work_dev, void* stream) {
    return bf1::attn_common(q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, hq, hkv, d, softmax_scale,
                            nullptr, o, lse, work_dev, stream);
}
