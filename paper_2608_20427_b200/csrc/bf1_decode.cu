// BF1 cached one-token decode over selected KV pages (paper Section 3.2 and 5.4).
//
// The newest token of a sequence of n cached tokens (position n-1, block j = (n-1) / 64) reads
// the pages of P(j) -- O(log B) pages, O(b d log B) key/value elements per head -- out of a paged
// KV cache: page = 64 tokens, [page, 64, Hkv, d] bf16, logical block -> physical page through a
// page table.  The page list only changes when n crosses a block boundary, so the plan
// (bf1_plan_decode) is made once per 64-token "route epoch" and reused by every decode step in
// it; the attention call reads the current lengths itself to find how many tokens of the self
// page are valid.  The paper measures planning at 100-121 us against 12-23 us of execution and
// names plan reuse across the epoch as the open problem; here the plan is a ~4 us kernel and is
// off the per-token path.
//
// The work is memory-bound (every selected K/V byte is read once, 2*G MACs per element): one kernel,
// decode_fused_kernel, in which a CTA serves one KV head and one pair of query heads and walks a page
// list, or a run of it, with an online softmax over a ring of cp.async page pairs.  With enough lists
// to fill the GPU a CTA takes a whole list; with fewer, every list is cut into runs (about two CTAs per
// SM in all, down to one page per CTA), each CTA leaves a partial (max, sum, O) in the workspace and
// the last CTA of a list to finish (atomic ticket, reset by the kernel) adds the runs up in run order.
#include <algorithm>

#include "bf1_common.cuh"

namespace bf1 {

constexpr int kPage = 64;             // tokens per page = block width b
constexpr int kDecThreads = 128;
constexpr int kDecStages = 3;          // page-pair buffers per CTA
constexpr int kDecCtasPerSm = 2;       // CTAs aimed at when a list is cut into runs (measured: 1 -> 11.4, 2 -> 10.8, 3 -> 11.7, 6 -> 14.5 us at batch 8)

struct DecodeArgs {
    const __nv_bfloat16* q;           // [batch, hq, d]
    const __nv_bfloat16* k_pages;     // [pages, 64, hkv, d]
    const __nv_bfloat16* v_pages;
    const int32_t* seqlens;           // [batch] current cached lengths (>= 0)
    const int32_t* count;             // plan: [batch] pages to read
    const int32_t* page;              // plan: [batch, max_degree] physical pages, self page last
    const int32_t* block;             // plan: [batch] block index the plan was made for
    int32_t* status;
    int32_t max_degree, hq, hkv, num_pages;
    int32_t group, pairs;             // G = hq / hkv (1, 2 or 4) and ceil(G / 2): a CTA serves one pair of query heads
    float scale_log2;
    float* part;                      // [batch, hkv * pairs, max_degree, 2, d + 2] partial (o[d], m, l)
    int32_t* ticket;                  // [batch, hkv * pairs], zero before and after every call
    __nv_bfloat16* o;                 // [batch, hq, d]
    float* lse;                       // [hq, batch]
    int32_t batch;
    int32_t nsplit;                   // decode_fused_kernel: CTAs a page list is cut over (1: no partial results)
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// cp.async that writes zeros when src_bytes is 0 (rows behind the newest token: unwritten cache memory
// that may hold anything, NaN included, and must not reach a multiply)
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// One CTA per (sequence, KV head, pair of query heads[, run of the list]).  Pages stream in through a
// kDecStages-deep cp.async ring with ONE block-wide synchronisation per page; inside a page each of the
// four warps owns 16 keys and keeps its own online-softmax state (max, sum, O) for both grouped heads,
// merged once at the end.  The arithmetic uses warp-level mma (m16n8k16: the two heads are rows 0 and 1
// of the 16-row operand, the rest is zero): the work is memory-bound, but as scalar FMAs it was a chain
// of 1500 dependent instructions and five synchronisations per page, which is what bounded the kernel.
template <int D, bool kSplit>
__global__ void __launch_bounds__(kDecThreads) decode_fused_kernel(const DecodeArgs a) {
    constexpr int kRowBytes = D * 2;
    constexpr int kVecPerRow = D / 8;                   // 16-byte chunks per row
    constexpr int kVecPerThread = kPage * kVecPerRow / kDecThreads;
    constexpr int kPageBytes = kPage * D * 2;
    // [stage][K | V][64 rows][D bf16]; the 16-byte chunks of every row are XOR-swizzled with (row & 7), which
    // keeps both the B-fragment loads of K (8 rows, same chunk) and the ldmatrix rows of V conflict-free
    extern __shared__ __align__(128) uint8_t dsmem[];
    __shared__ float sM[4][2], sL[4][2];
    __shared__ float sO[4][2][D];
    __shared__ float sW[2][64];                         // combine: weight of every partial
    __shared__ float sRed[2][2];
    __shared__ int sLast;
    __shared__ int sPages[64];                          // the sequence's page list (max_degree <= 64)

    const int kvp = blockIdx.x, s = blockIdx.y, tid = threadIdx.x;
    const int kvh = kvp / a.pairs, hbase = kvh * a.group + (kvp % a.pairs) * 2;   // first query head of this CTA's pair
    const int nheads = min(2, a.group - (kvp % a.pairs) * 2);                      // 1 when G = 1
    const int warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
    // The page list is fetched together with the plan's count and the length (independent loads in flight at
    // once), not after them: at small batch the kernel is one chain of dependent memory round trips.
    if (tid < a.max_degree) sPages[tid] = a.page[(size_t)s * a.max_degree + tid];
    const int cnt = a.count[s];
    const int n = a.seqlens[s];
    if (cnt <= 0) return;
    const int j = (n - 1) / kPage;
    if (j != a.block[s]) {            // the plan belongs to another route epoch
        if (tid == 0 && kvp == 0) atomicOr(a.status, BF1_DEV_BAD_ROUTE);
        return;
    }
    const int tail = n - j * kPage;   // valid tokens of the self page (the last list entry)
    __syncthreads();                  // sPages is complete (every exit above is taken by the whole CTA)
    const int* pages = sPages;
    // the part of the list this CTA walks: all of it, or the z-th run of `per` entries
    const int per = kSplit ? (cnt + a.nsplit - 1) / a.nsplit : cnt;
    const int e_lo = kSplit ? (int)blockIdx.z * per : 0, e_hi = min(cnt, e_lo + per);
    if (e_lo >= cnt) return;          // fewer runs than CTAs for this sequence
    auto issue_page = [&](int e, int stage) {
        int pg = pages[e];
        if (pg < 0 || pg >= a.num_pages) {
            if (tid == 0) atomicOr(a.status, BF1_DEV_BAD_ROUTE);
            pg = 0;
        }
        const int valid = (e == cnt - 1) ? tail : kPage;
        const size_t row_stride = (size_t)a.hkv * D;
        const __nv_bfloat16* kp = a.k_pages + ((size_t)pg * kPage * a.hkv + kvh) * D;
        const __nv_bfloat16* vp = a.v_pages + ((size_t)pg * kPage * a.hkv + kvh) * D;
        const uint32_t kb = smem_u32(dsmem) + stage * 2 * kPageBytes, vb = kb + kPageBytes;
#pragma unroll
        for (int q = 0; q < kVecPerThread; ++q) {
            const int i = tid + q * kDecThreads, rr = i / kVecPerRow, c = i % kVecPerRow;
            const uint32_t off = rr * kRowBytes + ((c ^ (rr & 7)) << 4);
            const uint32_t nbytes = rr < valid ? 16u : 0u;
            cp_async16_zfill(kb + off, kp + rr * row_stride + c * 8, nbytes);
            cp_async16_zfill(vb + off, vp + rr * row_stride + c * 8, nbytes);
        }
    };
#pragma unroll
    for (int i = 0; i < kDecStages - 1; ++i) {
        if (e_lo + i < e_hi) issue_page(e_lo + i, i);
        cp_async_commit();                               // possibly empty: keeps the group count uniform
    }
    // A fragments of Q: rows 0 and 1 of the 16-row operand are the two grouped heads, the rest zero
    uint32_t qa[D / 16][2];
    {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(a.q + ((size_t)s * a.hq + hbase + (gid < nheads ? gid : 0)) * D);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            qa[kk][0] = gid < nheads ? qrow[kk * 8 + tig] : 0u;          // columns kk*16 + 2*tig, +1
            qa[kk][1] = gid < nheads ? qrow[kk * 8 + tig + 4] : 0u;      // columns kk*16 + 8 + 2*tig, +1
        }
    }
    float m_run = -INFINITY, l_run = 0.f;                // per lane: head gid (lanes with gid >= 2 carry dummies)
    float acc[D / 8][4];
#pragma unroll
    for (int dn = 0; dn < D / 8; ++dn) acc[dn][0] = acc[dn][1] = acc[dn][2] = acc[dn][3] = 0.f;
    const int key0 = warp * 16;                          // this warp's 16 keys of every page

    for (int e = e_lo; e < e_hi; ++e) {
        cp_async_wait<kDecStages - 2>();                 // page e has landed (for this thread's copies)
        __syncthreads();                                 // ... for everybody's; and page e-1 is no longer read
        if (e + kDecStages - 1 < e_hi) issue_page(e + kDecStages - 1, (e - e_lo + kDecStages - 1) % kDecStages);
        cp_async_commit();
        const int valid = (e == cnt - 1) ? tail : kPage;
        if (key0 >= valid) continue;                     // warp-uniform: none of this warp's keys exists
        const uint32_t kb = smem_u32(dsmem) + ((e - e_lo) % kDecStages) * 2 * kPageBytes, vb = kb + kPageBytes;
        // ---- scores of 16 keys: two n-tiles of 8 keys, D / 16 k-steps ----------------------------
        float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                const int key = key0 + nt * 8 + gid;     // B fragment: n = gid, k = 2*tig (+8)
                const uint32_t row = kb + key * kRowBytes + tig * 4;
                uint32_t b0, b1;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b0) : "r"(row + (((2 * kk) ^ (key & 7)) << 4)));
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b1) : "r"(row + (((2 * kk + 1) ^ (key & 7)) << 4)));
                mma_16816(sc[nt], qa[kk][0], 0u, qa[kk][1], 0u, b0, b1);
            }
        }
        // lane (gid < 2, tig) holds head gid's scores of keys key0 + nt*8 + 2*tig, +1
        float sv[4];
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int key = key0 + (i >> 1) * 8 + 2 * tig + (i & 1);
            sv[i] = (gid < 2) ? ((key < valid) ? sc[i >> 1][i & 1] * a.scale_log2 : -INFINITY) : 0.f;
            mx = fmaxf(mx, sv[i]);
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));       // finite: key0 < valid
        const float m_new = fmaxf(m_run, mx);
        const float alpha = exp2f(m_run - m_new);                   // 0 on the warp's first page
        float pv[4], psum = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            pv[i] = exp2f(sv[i] - m_new);
            psum += pv[i];
        }
        psum += __shfl_xor_sync(0xffffffffu, psum, 1);
        psum += __shfl_xor_sync(0xffffffffu, psum, 2);
        l_run = l_run * alpha + psum;
        m_run = m_new;
        // P as the A operand of the second mma: the C layout of the scores is the A layout of the next k-step
        const uint32_t pa0 = gid < 2 ? pack_bf16x2(pv[0], pv[1]) : 0u;   // keys 2*tig, +1
        const uint32_t pa2 = gid < 2 ? pack_bf16x2(pv[2], pv[3]) : 0u;   // keys 8 + 2*tig, +1
        // ---- O = alpha * O + P V: D / 8 n-tiles of 8 columns, V fragments by ldmatrix.trans ---------
        const int lrow = key0 + (lane & 7) + ((lane >> 3) & 1) * 8;      // ldmatrix: lane supplies row (lane % 8) of matrix lane / 8
        const uint32_t vrow = vb + lrow * kRowBytes;
#pragma unroll
        for (int dn = 0; dn < D / 8; dn += 2) {
            acc[dn][0] *= alpha;
            acc[dn][1] *= alpha;
            acc[dn + 1][0] *= alpha;
            acc[dn + 1][1] *= alpha;
            uint32_t r0, r1, r2, r3;   // matrices: (keys 0-7, dn), (keys 8-15, dn), (keys 0-7, dn+1), (keys 8-15, dn+1)
            ldmatrix_x4_trans(vrow + (((dn + (lane >> 4)) ^ (lrow & 7)) << 4), r0, r1, r2, r3);
            mma_16816(acc[dn], pa0, 0u, pa2, 0u, r0, r1);
            mma_16816(acc[dn + 1], pa0, 0u, pa2, 0u, r2, r3);
        }
    }
    cp_async_wait<0>();
    // ---- merge the four warps' states ------------------------------------------------------------------
    if (gid < 2) {
        if (tig == 0) { sM[warp][gid] = m_run; sL[warp][gid] = l_run; }
#pragma unroll
        for (int dn = 0; dn < D / 8; ++dn) {
            sO[warp][gid][dn * 8 + 2 * tig] = acc[dn][0];
            sO[warp][gid][dn * 8 + 2 * tig + 1] = acc[dn][1];
        }
    }
    __syncthreads();
    const int h = tid >> 6, r = tid & 63;
    float m_all = fmaxf(fmaxf(sM[0][h], sM[1][h]), fmaxf(sM[2][h], sM[3][h]));   // warp 0 always has key 0
    float wgt[4], l_all = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        wgt[w] = exp2f(sM[w][h] - m_all);                // 0 for a warp that never saw a valid key
        l_all = fmaf(wgt[w], sL[w][h], l_all);
    }
    constexpr int kColsPerThread = D / 64;
    float out[kColsPerThread];
#pragma unroll
    for (int c = 0; c < kColsPerThread; ++c) {
        const int col = r * kColsPerThread + c;
        float o = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) o = fmaf(wgt[w], sO[w][h][col], o);
        out[c] = o;
    }
    if (kSplit) {
        // ---- this run's (max, sum, O) goes to the workspace; the last CTA of the list to finish adds the runs up in
        //      run order (fixed and data-independent) ------------------------------------------------------------
        const int runs = (cnt + per - 1) / per;
        const int c0 = r * kColsPerThread;
        const size_t list_id = (size_t)s * a.hkv * a.pairs + kvp;
        float* my = a.part + ((list_id * a.max_degree + blockIdx.z) * 2 + h) * (D + 2);
#pragma unroll
        for (int c = 0; c < kColsPerThread; ++c) my[c0 + c] = out[c];
        if (r == 0) { my[D] = m_all; my[D + 1] = l_all; }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int t = atomicAdd(a.ticket + list_id, 1);
            sLast = (t == runs - 1);
            if (sLast) a.ticket[list_id] = 0;            // ready for the next call
        }
        __syncthreads();
        if (!sLast) return;
        __threadfence();
        const float* base = a.part + (list_id * a.max_degree * 2 + h) * (D + 2);
        const size_t estride = 2 * (D + 2);
        if (r < runs) sW[h][r] = base[r * estride + D];  // every run's max is fetched by its own thread
        __syncthreads();
        m_all = -INFINITY;
        for (int i = 0; i < runs && i < 64; ++i) m_all = fmaxf(m_all, sW[h][i]);
        float w_mine = 0.f, lpart = 0.f;
        if (r < runs) {
            w_mine = exp2f(sW[h][r] - m_all);
            lpart = w_mine * base[r * estride + D + 1];
        }
        __syncthreads();
        if (r < runs) sW[h][r] = w_mine;
        l_all = lpart;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) l_all += __shfl_xor_sync(0xffffffffu, l_all, off);
        if ((tid & 31) == 0) sRed[h][(tid >> 5) & 1] = l_all;
        __syncthreads();
        l_all = sRed[h][0] + sRed[h][1];
#pragma unroll
        for (int c = 0; c < kColsPerThread; ++c) out[c] = 0.f;
#pragma unroll 4
        for (int i = 0; i < runs; ++i) {
            const float w = sW[h][i];
#pragma unroll
            for (int c = 0; c < kColsPerThread; ++c) out[c] = fmaf(w, base[i * estride + c0 + c], out[c]);
        }
    }
    if (h >= nheads) return;                             // G = 1: the second head of the pair does not exist
    const float inv = 1.f / l_all;
    __nv_bfloat16* orow = a.o + ((size_t)s * a.hq + hbase + h) * D;
#pragma unroll
    for (int c = 0; c < kColsPerThread; ++c) orow[r * kColsPerThread + c] = __float2bfloat16_rn(out[c] * inv);
    if (r == 0) a.lse[(size_t)(hbase + h) * a.batch + s] = (m_all + log2f(l_all)) * 0.6931471805599453f;
}

// One thread per sequence: Eq. 1 for the block of the newest token, mapped through the page table.
__global__ void plan_decode_kernel(const int32_t* seqlens, const int32_t* page_table, int max_pages_per_seq,
                                   int batch, bf1_route_cfg cfg, bf1_decode_plan plan) {
    // One CTA walks the batch: error bits are collected in shared memory and the status word is
    // WRITTEN once at the end, so no thread's bit can be lost to another thread's clearing store.
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    for (int s = threadIdx.x; s < batch; s += blockDim.x) {
        const int n = seqlens[s];
        int32_t* list = plan.page + (size_t)s * plan.max_degree;
        int deg = 0;
        int bad = 0;
        // Pages are 64 tokens whatever the route block width b: with b = 128 a listed block is two pages, and
        // the newest token's own block is its pages up to the one that holds the token.
        const int f = cfg.block / kPage;
        const int jt = n > 0 ? (n - 1) / kPage : -1;      // logical page of the newest token
        const int j = jt >= 0 ? jt / f : -1;              // its route block
        if (n < 0 || jt >= max_pages_per_seq) bad = BF1_DEV_BAD_SEQLENS;
        if (n > 0 && !bad) {
            int last = -1, kmax = -1;
            if (cfg.dyadic) while ((1 << (kmax + 1)) <= j) ++kmax;
            int g = cfg.global_first ? 0 : 0x7fffffff;
            int k = kmax;
            int l = max(j - cfg.local_blocks, 0);
            while (true) {                                   // merge of the three ascending candidate streams
                const int dcur = (k >= 0) ? j - (1 << k) : 0x7fffffff;
                const int lcur = (l <= j) ? l : 0x7fffffff;
                const int m = min(g, min(dcur, lcur));
                if (m == 0x7fffffff) break;
                if (m == g) g = 0x7fffffff;
                if (m == dcur) --k;
                if (m == lcur) ++l;
                if (m != last) {
                    const int t1 = (m < j) ? m * f + f - 1 : jt;
                    for (int t = m * f; t <= t1; ++t) {
                        if (deg < plan.max_degree) list[deg] = page_table[(size_t)s * max_pages_per_seq + t];
                        else bad |= BF1_DEV_CAPACITY;
                        ++deg;
                    }
                    last = m;
                }
            }
            if (deg > plan.max_degree) deg = plan.max_degree;
        }
        for (int e2 = deg; e2 < plan.max_degree; ++e2) list[e2] = -1;
        plan.count[s] = bad ? 0 : deg;
        plan.block[s] = jt;
        if (bad) atomicOr(&s_bad, bad);
    }
    __syncthreads();
    if (threadIdx.x == 0) *plan.status = s_bad;
}

int check_cfg(const bf1_route_cfg* cfg);   // bf1_plan.cu

}  // namespace bf1

using namespace bf1;

extern "C" int64_t bf1_decode_workspace_bytes(int32_t batch, int32_t hq, int32_t hkv, int32_t max_degree, int32_t d) {
    if (batch < 0 || hq <= 0 || hkv <= 0 || hq % hkv != 0 || max_degree <= 0 || d <= 0) return -1;
    const int64_t pairs = (hq / hkv + 1) / 2;   // CTAs (and partial-result slots) per KV head
    const int64_t part = (int64_t)batch * hkv * pairs * max_degree * 2 * (d + 2) * (int64_t)sizeof(float);
    const int64_t tick = (int64_t)batch * hkv * pairs * (int64_t)sizeof(int32_t);
    return ((part + 255) / 256) * 256 + tick;
}

extern "C" int bf1_plan_decode(const int32_t* seqlens_dev, const int32_t* page_table_dev, int32_t max_pages_per_seq,
                               int32_t batch, const bf1_route_cfg* cfg, const bf1_decode_plan* out, void* stream) {
    if (int rc = check_cfg(cfg)) return rc;
    if (!seqlens_dev || !page_table_dev || !out || !out->count || !out->page || !out->block || !out->status)
        return fail(BF1_ERR_INVALID_ARG, "a decode-plan pointer is null");
    if (batch < 0 || max_pages_per_seq < 1 || out->max_degree < 1)
        return fail(BF1_ERR_INVALID_ARG, "bad batch, max_pages_per_seq or max_degree");
    int32_t cap = 0, need = 0;
    if (int rc = bf1_route_capacity(1, (int64_t)max_pages_per_seq * kPage, max_pages_per_seq * kPage, cfg, &cap, &need))
        return rc;
    if (out->max_degree < need)
        return fail(BF1_ERR_CAPACITY, "decode plan max_degree %d < %d needed for %d pages per sequence", out->max_degree,
                    need, max_pages_per_seq);
    if (batch == 0) return BF1_OK;
    const int threads = batch >= 1024 ? 1024 : ((batch + 31) / 32) * 32;
    plan_decode_kernel<<<1, threads, 0, (cudaStream_t)stream>>>(seqlens_dev, page_table_dev,
                                                                               max_pages_per_seq, batch, *cfg, *out);
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}

extern "C" int bf1_decode_fwd(const void* q, const void* k_pages, const void* v_pages, int32_t num_pages,
                              const int32_t* seqlens_dev, int32_t batch, int32_t hq, int32_t hkv, int32_t d,
                              float softmax_scale, const bf1_decode_plan* plan, void* workspace, void* o, float* lse,
                              void* stream) {
    if (!q || !k_pages || !v_pages || !seqlens_dev || !plan || !workspace || !o || !lse)
        return fail(BF1_ERR_INVALID_ARG, "a pointer is null");
    if (!plan->count || !plan->page || !plan->block || !plan->status)
        return fail(BF1_ERR_INVALID_ARG, "a decode-plan pointer is null");
    if (batch < 0 || num_pages < 0 || hq <= 0 || hkv <= 0) return fail(BF1_ERR_INVALID_ARG, "negative or zero size argument");
    if (hq % hkv != 0) return fail(BF1_ERR_INVALID_ARG, "hq %d is not a multiple of hkv %d", hq, hkv);
    const int group = hq / hkv, pairs = (group + 1) / 2;
    if (group != 1 && group != 2 && group != 4)
        return fail(BF1_ERR_UNSUPPORTED, "GQA group size %d: only G = 1, 2 and 4 are supported", group);
    if (d != 64 && d != 128) return fail(BF1_ERR_UNSUPPORTED, "head dimension %d: only 64 and 128 are supported", d);
    if (((uintptr_t)q | (uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)o | (uintptr_t)workspace) & 15)
        return fail(BF1_ERR_INVALID_ARG, "q, k_pages, v_pages, o and workspace must be 16-byte aligned");
    if (plan->max_degree < 1 || plan->max_degree > 64 || hkv * pairs > 65535 || batch > 65535)
        return fail(BF1_ERR_UNSUPPORTED, "max_degree must be <= 64; hkv and batch must fit the grid (<= 65535)");
    if (batch == 0) return BF1_OK;
    DecodeArgs a;
    a.q = (const __nv_bfloat16*)q;
    a.k_pages = (const __nv_bfloat16*)k_pages;
    a.v_pages = (const __nv_bfloat16*)v_pages;
    a.seqlens = seqlens_dev;
    a.count = plan->count;
    a.page = plan->page;
    a.block = plan->block;
    a.status = plan->status;
    a.max_degree = plan->max_degree;
    a.hq = hq;
    a.hkv = hkv;
    a.num_pages = num_pages;
    a.group = group;
    a.pairs = pairs;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)d);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.part = (float*)workspace;
    const int64_t part = (int64_t)batch * hkv * pairs * plan->max_degree * 2 * (d + 2) * (int64_t)sizeof(float);
    a.ticket = (int32_t*)((char*)workspace + ((part + 255) / 256) * 256);
    a.o = (__nv_bfloat16*)o;
    a.lse = lse;
    a.batch = batch;
    static int sm_count[64] = {};
    int dev = 0;
    BF1_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return fail(BF1_ERR_NO_DEVICE, "device ordinal %d out of range", dev);
    constexpr int kSmem128 = kDecStages * 2 * 64 * 128 * 2, kSmem64 = kDecStages * 2 * 64 * 64 * 2;
    if (!sm_count[dev]) {
        BF1_CUDA_CHECK(cudaFuncSetAttribute(decode_fused_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem128));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(decode_fused_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem128));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(decode_fused_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem64));
        BF1_CUDA_CHECK(cudaFuncSetAttribute(decode_fused_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem64));
        BF1_CUDA_CHECK(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    }
    const int64_t lists = (int64_t)batch * hkv * pairs;
    if (lists >= sm_count[dev]) {
        // enough (sequence, KV head) pairs to fill the GPU: one CTA walks a whole list
        a.nsplit = 1;
        dim3 grid(hkv * pairs, batch);
        if (d == 128) decode_fused_kernel<128, false><<<grid, kDecThreads, kSmem128, (cudaStream_t)stream>>>(a);
        else decode_fused_kernel<64, false><<<grid, kDecThreads, kSmem64, (cudaStream_t)stream>>>(a);
    } else {
        // few lists: every list is cut into runs of pages, one CTA each (about two CTAs per SM in all, down to one
        // page per CTA), and the last CTA of a list to finish adds the runs' partial results up
        const int64_t want = (kDecCtasPerSm * (int64_t)sm_count[dev] + lists - 1) / lists;
        a.nsplit = (int)std::min<int64_t>(std::min<int64_t>(want, plan->max_degree), 64);
        // a run of fewer pages than the ring has stages needs that much less shared memory (more CTAs per SM)
        const int per_max = (plan->max_degree + a.nsplit - 1) / a.nsplit;
        const int stages = std::min(per_max, kDecStages);
        dim3 grid(hkv * pairs, batch, a.nsplit);
        if (d == 128) decode_fused_kernel<128, true><<<grid, kDecThreads, kSmem128 / kDecStages * stages, (cudaStream_t)stream>>>(a);
        else decode_fused_kernel<64, true><<<grid, kDecThreads, kSmem64 / kDecStages * stages, (cudaStream_t)stream>>>(a);
    }
    BF1_CUDA_CHECK(cudaGetLastError());
    return BF1_OK;
}
