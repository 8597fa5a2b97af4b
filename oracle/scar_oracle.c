/*
 * CPU oracle for the SCAR checkpoint-and-recover parameter pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the paper defines, used to check the CUDA library.  It is not part of the
 * product: nothing in the library, its binding or its kernels may call it, and
 * it shares no code, header, table or helper with them.  Every function is
 * pinned by CPU tests against closed forms, invariants of Theorems 4.1/4.2,
 * special cases and brute force; none is "parity unpinned".
 *
 * Arithmetic: element values are taken exactly as stored (fp32 or int32 bit
 * patterns) and widened without rounding; floating-point sums run in fp64 in
 * ascending element order, integer sums in 64-bit integers.  There is no
 * blocking, vectorisation or reordering.
 *
 * The same file also builds with -fopenmp, only to time the oracle on all host
 * cores: the loops over blocks (scores, pack, cache update, recovery) then run
 * in parallel, the selection stays the serial sort.  Per-block sums keep their
 * element order either way; only the recovery's sum ACROSS blocks changes its
 * order in that build.  Every pin and every parity test uses the plain build.
 *
 * Notation follows the paper's appendix proof of Theorem 4.1:
 *   x = live parameters x^(T), z = running checkpoint, S = lost set.
 * A "parameter" for distance, selection and loss is one block of contiguous
 * elements (Section 5.1 partitions by rows, layers or shards); block b covers
 * elements [boff[b], boff[b+1]).
 */

#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#define SCAR_PRAGMA(x) _Pragma(#x)
#define SCAR_OVER_BLOCKS SCAR_PRAGMA(omp parallel for schedule(static))
#define SCAR_OVER_BLOCKS_SUM(...) SCAR_PRAGMA(omp parallel for schedule(static) reduction(+ : __VA_ARGS__))
int scar_oracle_threads(void) { return omp_get_max_threads(); }
#else
#define SCAR_OVER_BLOCKS
#define SCAR_OVER_BLOCKS_SUM(...)
int scar_oracle_threads(void) { return 1; }
#endif

/* ---- geometry ----------------------------------------------------------- */

/* Number of blocks of a row-structured layout: rows of row_elems (0 = one row
 * of n_elems), blocks of block_elems that never cross a row end. */
uint64_t scar_oracle_count_blocks(uint64_t n_elems, uint64_t row_elems, uint64_t block_elems)
{
    if (n_elems == 0 || block_elems == 0) return 0;
    uint64_t row = row_elems ? row_elems : n_elems;
    uint64_t per_row = (row + block_elems - 1) / block_elems;
    return (n_elems / row) * per_row;
}

/* Writes the B+1 element offsets of that layout. */
void scar_oracle_layout_offsets(uint64_t n_elems, uint64_t row_elems, uint64_t block_elems, uint64_t *boff)
{
    uint64_t b = 0;
    if (n_elems && block_elems) {
        uint64_t row = row_elems ? row_elems : n_elems;
        for (uint64_t r0 = 0; r0 < n_elems; r0 += row)
            for (uint64_t e = 0; e < row; e += block_elems)
                boff[b++] = r0 + e;
    }
    boff[b] = n_elems;
}

/* Section 4.3: any number of parameter-server nodes may fail; a node is a
 * contiguous shard of blocks here.  Shard s owns blocks
 * [floor(s*B/S), floor((s+1)*B/S)).  Mask bytes: 0 alive, non-zero lost. */
void scar_oracle_expand_shards(uint64_t n_blocks, uint64_t n_shards, const uint8_t *lost_shards,
                               uint8_t *lost_blocks)
{
    memset(lost_blocks, 0, n_blocks);
    for (uint64_t s = 0; s < n_shards; ++s) {
        if (!lost_shards[s]) continue;
        uint64_t lo = (uint64_t)(((unsigned __int128)s * n_blocks) / n_shards);
        uint64_t hi = (uint64_t)(((unsigned __int128)(s + 1) * n_blocks) / n_shards);
        for (uint64_t b = lo; b < hi; ++b) lost_blocks[b] = 1;
    }
}

/* ---- checkpoint step 1: distance of every parameter to its saved value -- */

/* Section 4.3, checkpoint step 1, with the l2 norm of the appendix proofs:
 * score_b = sum_{i in b} (x_i - z_i)^2  (the squared distance; ranking by it
 * equals ranking by the distance). */
void scar_oracle_scores_f32(const float *x, const float *z, const uint64_t *boff, uint64_t n_blocks,
                            double *score)
{
    SCAR_OVER_BLOCKS
    for (uint64_t b = 0; b < n_blocks; ++b) {
        double acc = 0.0;
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) {
            double d = (double)x[i] - (double)z[i];
            acc += d * d;
        }
        score[b] = acc;
    }
}

/* Appendix C: for parameters that are distributions the distance is the total
 * variation, (1/2) sum |x_i - z_i|, scaled per block; this is the plain l1 sum of
 * float data, the scale (weight) is applied by the caller. */
void scar_oracle_scores_f32_l1(const float *x, const float *z, const uint64_t *boff, uint64_t n_blocks,
                               double *score)
{
    SCAR_OVER_BLOCKS
    for (uint64_t b = 0; b < n_blocks; ++b) {
        double acc = 0.0;
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i)
            acc += fabs((double)x[i] - (double)z[i]);
        score[b] = acc;
    }
}

/* Appendix C (LDA): distances between count rows use a length-scaled total
 * variation, which for counts is half the l1 distance; the factor 1/2 is
 * dropped so that score_b = sum_{i in b} |x_i - z_i| stays an integer. */
void scar_oracle_scores_i32(const int32_t *x, const int32_t *z, const uint64_t *boff, uint64_t n_blocks,
                            uint64_t *score)
{
    SCAR_OVER_BLOCKS
    for (uint64_t b = 0; b < n_blocks; ++b) {
        uint64_t acc = 0;
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) {
            int64_t d = (int64_t)x[i] - (int64_t)z[i];
            acc += (uint64_t)(d < 0 ? -d : d);
        }
        score[b] = acc;
    }
}

/* ---- checkpoint step 3: the fraction r with the largest distances ------- */

/* Section 4.2 checkpoints a fraction r of the parameters at a time; the
 * paper leaves the rounding open.  Reading used: k = round(r*B) (halves away
 * from zero), at least one block when r > 0, never more than B.
 * Returns -1 when r is outside [0, 1] or NaN. */
int64_t scar_oracle_k_from_r(double r, uint64_t n_blocks)
{
    if (!(r >= 0.0 && r <= 1.0)) return -1;
    double t = r * (double)n_blocks;
    uint64_t k = (uint64_t)round(t);
    if (k > n_blocks) k = n_blocks;
    if (k == 0 && r > 0.0 && n_blocks > 0) k = 1;
    return (int64_t)k;
}

typedef struct { double s; uint32_t id; } rank_f64;
typedef struct { uint64_t s; uint32_t id; } rank_u64;

static int cmp_rank_f64(const void *pa, const void *pb)
{
    const rank_f64 *a = (const rank_f64 *)pa, *b = (const rank_f64 *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    return (a->id > b->id) - (a->id < b->id);
}
static int cmp_rank_u64(const void *pa, const void *pb)
{
    const rank_u64 *a = (const rank_u64 *)pa, *b = (const rank_u64 *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    return (a->id > b->id) - (a->id < b->id);
}
static int cmp_u32(const void *pa, const void *pb)
{
    uint32_t a = *(const uint32_t *)pa, b = *(const uint32_t *)pb;
    return (a > b) - (a < b);
}

/* Section 4.2 prioritisation heuristic (largest change since last saved) and
 * Section 4.3 checkpoint step 3: order all blocks by (score descending, block
 * id ascending), keep the first k, return their ids in ascending order.  A
 * score that is NaN or infinite ranks as +infinity (such a block is saved
 * first); *nonfinite receives how many blocks had one.  Returns 0, or -1 if
 * memory ran out. */
int scar_oracle_select_f64(const double *score, uint64_t n_blocks, uint64_t k, uint32_t *sel,
                           uint64_t *nonfinite)
{
    rank_f64 *a = (rank_f64 *)malloc((n_blocks ? n_blocks : 1) * sizeof *a);
    if (!a) return -1;
    uint64_t bad = 0;
    for (uint64_t b = 0; b < n_blocks; ++b) {
        double s = score[b];
        if (isnan(s) || isinf(s)) { s = INFINITY; ++bad; }
        a[b].s = s;
        a[b].id = (uint32_t)b;
    }
    qsort(a, n_blocks, sizeof *a, cmp_rank_f64);
    for (uint64_t j = 0; j < k; ++j) sel[j] = a[j].id;
    qsort(sel, k, sizeof *sel, cmp_u32);
    if (nonfinite) *nonfinite = bad;
    free(a);
    return 0;
}

int scar_oracle_select_u64(const uint64_t *score, uint64_t n_blocks, uint64_t k, uint32_t *sel)
{
    rank_u64 *a = (rank_u64 *)malloc((n_blocks ? n_blocks : 1) * sizeof *a);
    if (!a) return -1;
    for (uint64_t b = 0; b < n_blocks; ++b) { a[b].s = score[b]; a[b].id = (uint32_t)b; }
    qsort(a, n_blocks, sizeof *a, cmp_rank_u64);
    for (uint64_t j = 0; j < k; ++j) sel[j] = a[j].id;
    qsort(sel, k, sizeof *sel, cmp_u32);
    free(a);
    return 0;
}

/* ---- checkpoint step 4: update the cache, save the selected parameters -- */

/* Section 4.3 step 4, the part written to storage: the payload is the
 * concatenation, in ascending block id, of the stored bytes of x over every
 * selected block; poff[j] is the element offset of block sel[j] inside the
 * payload and poff[k] the payload length.  Elements are 4 bytes wide. */
void scar_oracle_pack(const uint32_t *x, const uint64_t *boff, const uint32_t *sel, uint64_t k,
                      uint32_t *payload, uint64_t *poff)
{
    uint64_t out = 0;
    for (uint64_t j = 0; j < k; ++j) {
        poff[j] = out;
        out += boff[sel[j] + 1] - boff[sel[j]];
    }
    poff[k] = out;
    SCAR_OVER_BLOCKS
    for (uint64_t j = 0; j < k; ++j) {
        uint64_t b = sel[j], at = poff[j];
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) payload[at++] = x[i];
    }
}

/* Section 4.3 step 4, the cache refresh: z_b := x_b bytewise for
 * every selected block; all other blocks of z keep their bytes. */
void scar_oracle_update(uint32_t *z, const uint32_t *x, const uint64_t *boff, const uint32_t *sel, uint64_t k)
{
    SCAR_OVER_BLOCKS
    for (uint64_t j = 0; j < k; ++j) {
        uint64_t b = sel[j];
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) z[i] = x[i];
    }
}

/* ---- recovery ----------------------------------------------------------- */

/* Appendix proof of Theorem 4.1: partial recovery replaces x_S by z_S and
 * leaves x_{S^c} alone; its perturbation is ||z_S - x_S||.  Returns the sum of
 * squares over the lost blocks (taken before anything is overwritten), counts
 * the lost blocks/elements, and, when write != 0, performs x_b := z_b bytewise
 * for the lost blocks.  lost_blocks == NULL means every block is lost, i.e.
 * full recovery with perturbation x^(T) - x^(C) (Example 2.3). */
double scar_oracle_recover_f32(float *x, const float *z, const uint64_t *boff, uint64_t n_blocks,
                               const uint8_t *lost_blocks, int write, uint64_t *n_lost_blocks,
                               uint64_t *n_lost_elems)
{
    double acc = 0.0;
    uint64_t nb = 0, ne = 0;
    SCAR_OVER_BLOCKS_SUM(acc, nb, ne)
    for (uint64_t b = 0; b < n_blocks; ++b) {
        if (lost_blocks && !lost_blocks[b]) continue;
        ++nb;
        ne += boff[b + 1] - boff[b];
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) {
            double d = (double)z[i] - (double)x[i];
            acc += d * d;
        }
    }
    if (write)
        SCAR_OVER_BLOCKS
        for (uint64_t b = 0; b < n_blocks; ++b) {
            if (lost_blocks && !lost_blocks[b]) continue;
            memcpy(x + boff[b], z + boff[b], (boff[b + 1] - boff[b]) * sizeof(float));
        }
    if (n_lost_blocks) *n_lost_blocks = nb;
    if (n_lost_elems) *n_lost_elems = ne;
    return acc;
}

/* Integer form of the same: l1 perturbation sum_{i in S} |z_i - x_i|. */
uint64_t scar_oracle_recover_i32(int32_t *x, const int32_t *z, const uint64_t *boff, uint64_t n_blocks,
                                 const uint8_t *lost_blocks, int write, uint64_t *n_lost_blocks,
                                 uint64_t *n_lost_elems)
{
    uint64_t acc = 0, nb = 0, ne = 0;
    SCAR_OVER_BLOCKS_SUM(acc, nb, ne)
    for (uint64_t b = 0; b < n_blocks; ++b) {
        if (lost_blocks && !lost_blocks[b]) continue;
        ++nb;
        ne += boff[b + 1] - boff[b];
        for (uint64_t i = boff[b]; i < boff[b + 1]; ++i) {
            int64_t d = (int64_t)z[i] - (int64_t)x[i];
            acc += (uint64_t)(d < 0 ? -d : d);
        }
    }
    if (write)
        SCAR_OVER_BLOCKS
        for (uint64_t b = 0; b < n_blocks; ++b) {
            if (lost_blocks && !lost_blocks[b]) continue;
            memcpy(x + boff[b], z + boff[b], (boff[b + 1] - boff[b]) * sizeof(int32_t));
        }
    if (n_lost_blocks) *n_lost_blocks = nb;
    if (n_lost_elems) *n_lost_elems = ne;
    return acc;
}
