/*
 * BF1 oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow CPU statement of what the BF1 forward operator computes: exact softmax
 * attention over the key set that the causal dyadic block route selects (Section 3.1,
 * Eq. 1).  It shares no code with the CUDA path and must never be called from it; only
 * the tests, the smoke check and the benchmark's cpu-baseline leg may load this file.
 *
 * Everything here is written out from the definitions:
 *   - blocks:   B = ceil(n / b), token i lives in block floor(i / b)          (Section 3.1)
 *   - route:    P(j) = {j, j-1, j-2, 0} u {j - 2^r : r >= 2}, invalid and duplicate
 *               indices removed                                               (Eq. 1)
 *   - mask:     token pair (i, c) is selected iff block(c) is in P(block(i)) and c <= i
 *               (self block: token-level causal triangle; every other selected block is
 *               strictly earlier)                                             (Section 3.1)
 *   - counting: a non-self block pair contributes rows*b token pairs, the self block
 *               rows*(rows+1)/2                                               (Prop. 1)
 *   - attention: s_c = scale * <q_i, k_c>, softmax over the selected c, O_i = sum p_c v_c,
 *               LSE_i = ln sum exp(s_c); no score bias                        (Section 3.1)
 *
 * Arithmetic is fp32 (the _f32 entry points) or fp64 (the _f64 ones, used to show that
 * the fp32 rounding noise is far below the parity tolerance).  Loops run in ascending
 * column order and are never blocked, fused or reordered; OpenMP only spreads
 * independent (head, row) pairs over cores.
 *
 * Pins (see tests/test_oracle_*.py): the 26.98x interaction reduction at 32K (Table 2),
 * the maximum shortest path of eight at B = 512 (Prop. 2), the 4 + floor(log2 j) degree
 * bound (Prop. 1), closed-form totals, Q = 0 / constant-V / one-hot-V special cases, the
 * dense special case against a library SDPA, brute force on tiny inputs, future-token
 * isolation.  GQA head mapping (query head h reads KV head floor(h / G)) is a convention
 * the paper does not state: it is pinned only to the library's grouped-query convention.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t block;        /* b: block width in tokens                                   */
    int32_t local_blocks; /* W: number of immediately preceding blocks always read      */
    int32_t global_first; /* 1: block 0 is always read                                  */
    int32_t dyadic;       /* 1: blocks j - 2^k are read for every k >= 0 with j-2^k >= 0 */
} bf1o_cfg;

/* ---- route ------------------------------------------------------------------------ */

static int is_pow2(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }

/* Eq. 1 as a predicate on a (query block, key block) pair.  With W = 2 the offsets 2^0
 * and 2^1 coincide with the local window, so "every k >= 0" and the paper's "r >= 2"
 * select the same set. */
int bf1o_sel(const bf1o_cfg *cfg, int64_t jq, int64_t jk)
{
    if (jk < 0 || jk > jq) return 0;                 /* invalid index / not causal */
    int64_t delta = jq - jk;
    if (delta <= cfg->local_blocks) return 1;        /* j, j-1, ..., j-W           */
    if (cfg->global_first && jk == 0) return 1;      /* block 0                    */
    if (cfg->dyadic && is_pow2(delta)) return 1;     /* j - 2^k                    */
    return 0;
}

int64_t bf1o_num_blocks(const bf1o_cfg *cfg, int64_t n)
{
    return (n + cfg->block - 1) / cfg->block;
}

/* Ascending list P(j) for every query block of one sequence of n tokens, its length,
 * the token-pair count of the query block, and the total.  kv_idx is [B, max_degree],
 * unused slots set to -1.  Returns the total selected token pairs, or -1 if a list
 * does not fit in max_degree. */
int64_t bf1o_route(const bf1o_cfg *cfg, int64_t n, int32_t max_degree,
                   int32_t *kv_idx, int32_t *kv_count, int64_t *pair_count)
{
    const int64_t b = cfg->block, B = bf1o_num_blocks(cfg, n);
    int64_t total = 0;
    for (int64_t jq = 0; jq < B; ++jq) {
        int32_t len = 0;
        for (int64_t jk = 0; jk <= jq; ++jk) {
            if (!bf1o_sel(cfg, jq, jk)) continue;
            if (len >= max_degree) return -1;
            kv_idx[jq * max_degree + len++] = (int32_t)jk;
        }
        for (int32_t e = len; e < max_degree; ++e) kv_idx[jq * max_degree + e] = -1;
        int64_t rows = n - jq * b < b ? n - jq * b : b;
        int64_t pairs = rows * b * (len - 1) + rows * (rows + 1) / 2;
        kv_count[jq] = len;
        pair_count[jq] = pairs;
        total += pairs;
    }
    return total;
}

/* B x B boolean block mask. */
void bf1o_block_mask(const bf1o_cfg *cfg, int64_t n, uint8_t *bm)
{
    const int64_t B = bf1o_num_blocks(cfg, n);
    for (int64_t jq = 0; jq < B; ++jq)
        for (int64_t jk = 0; jk < B; ++jk)
            bm[jq * B + jk] = (uint8_t)bf1o_sel(cfg, jq, jk);
}

/* n x n boolean token mask: M[i, c] = sel(block(i), block(c)) and c <= i. */
void bf1o_token_mask(const bf1o_cfg *cfg, int64_t n, uint8_t *m)
{
    const int64_t b = cfg->block;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t c = 0; c < n; ++c)
            m[i * n + c] = (uint8_t)(bf1o_sel(cfg, i / b, c / b) && c <= i);
}

/* Longest shortest path, in layers, from any block i to any later block j when one
 * layer carries information from every p in P(j) to j (Prop. 2).  Plain BFS from each
 * source.  Returns -1 if some later block is unreachable. */
int32_t bf1o_max_shortest_path(const bf1o_cfg *cfg, int32_t B)
{
    int32_t *dist = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    int32_t *queue = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    int32_t worst = 0;
    for (int32_t src = 0; src < B; ++src) {
        for (int32_t x = 0; x < B; ++x) dist[x] = -1;
        int32_t head = 0, tail = 0;
        dist[src] = 0;
        queue[tail++] = src;
        while (head < tail) {
            int32_t x = queue[head++];
            for (int32_t y = x + 1; y < B; ++y) {      /* y reads x in one layer? */
                if (dist[y] < 0 && bf1o_sel(cfg, y, x)) {
                    dist[y] = dist[x] + 1;
                    queue[tail++] = y;
                }
            }
        }
        for (int32_t y = src; y < B; ++y) {
            if (dist[y] < 0) { worst = -1; goto done; }
            if (dist[y] > worst) worst = dist[y];
        }
    }
done:
    free(dist);
    free(queue);
    return worst;
}

/* ---- attention --------------------------------------------------------------------- */

static inline float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* The same three routines are instantiated once in fp32 and once in fp64. */
#define REAL float
#define SUFFIX(name) name##_f32
#define R_EXP expf
#define R_LOG logf
#include "bf1_oracle_attn.inc"
#undef REAL
#undef SUFFIX
#undef R_EXP
#undef R_LOG

#define REAL double
#define SUFFIX(name) name##_f64
#define R_EXP exp
#define R_LOG log
#include "bf1_oracle_attn.inc"
#undef REAL
#undef SUFFIX
#undef R_EXP
#undef R_LOG

#ifdef _OPENMP
#include <omp.h>
int bf1o_threads(void) { return omp_get_max_threads(); }
#else
int bf1o_threads(void) { return 1; }
#endif
