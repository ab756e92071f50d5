/*
 * CPU oracle for the distributed sparse-embedding lookup served by the
 * bounded-lag-synchronous (BLS) alltoallv.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
 * statement of what the hot path computes.  It shares no code with the CUDA
 * library and must never be linked, imported or called from the product path;
 * only the test-suite, the smoke check and the benchmark's CPU-baseline leg
 * use it.
 *
 * What it states (paper passages in brackets):
 *   - batch row-block partition: sample g of the global batch belongs to
 *     requester rank g / b                                    [Section I, par. 6]
 *   - the paper leaves the table partitioning strategy open; the two used
 *     here are table-wise round-robin (owner = t mod P) and row-wise blocks
 *     (owner = id / ceil(N_t / P))                            [Section I, par. 6]
 *   - every rank determines the vector IDs it needs from every other rank and
 *     exchanges them with an alltoallv; with bound k = 0 this is semantically
 *     MPI_Alltoallv, i.e. a stable sort of each rank's requests by destination
 *     with counts and displacements             [Section I par. 6; Section III-D]
 *   - the owner performs the embedding-bag lookup (sum pooling) [Listing 1]
 *   - pooled vectors travel back to the requester's layout     [Listing 1]
 *
 * Floating point: sums are formed in fp64 from the stored values (fp32, bf16
 * or fp16 widened exactly) and rounded once to fp32.
 *
 * Pins (tests/test_oracle_*.py): closed-form counts for one-hot table-wise
 * inputs, numpy stable argsort / cumsum, torch embedding_bag for P = 1,
 * exact-valued tables, brute force on tiny inputs, definition-vs-routed
 * agreement.  No function here is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

enum { PART_TABLE_RR = 0, PART_ROW_BLOCK = 1 };
enum { DT_F32 = 0, DT_BF16 = 1, DT_F16 = 2 };

/* ---------------------------------------------------------------- values */

/* IEEE binary16 -> double, from the format definition. */
static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0)        v = ldexp((double)m, -24);            /* subnormal / zero */
    else if (e == 31)  v = m ? NAN : INFINITY;
    else               v = ldexp((double)(m | 0x400), e - 25);
    return sign ? -v : v;
}

/* bfloat16 = upper half of a binary32. */
static double bf16_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* binary32 -> binary16, round to nearest even, from the format definition. */
static uint16_t float_to_half(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t sign = (u >> 16) & 0x8000u;
    int32_t e = (int32_t)((u >> 23) & 0xFF) - 127;
    uint32_t m = u & 0x7FFFFFu;
    if (e == 128) return (uint16_t)(sign | 0x7C00u | (m ? 0x200u : 0));
    if (e > 15) return (uint16_t)(sign | 0x7C00u);
    if (e >= -14) {                                  /* normal half */
        uint32_t h = ((uint32_t)(e + 15) << 10) | (m >> 13);
        uint32_t rem = m & 0x1FFFu;
        if (rem > 0x1000u || (rem == 0x1000u && (h & 1))) h++;   /* may carry into exponent: correct */
        return (uint16_t)(sign | h);
    }
    if (e < -25) return (uint16_t)sign;              /* underflow to zero */
    m |= 0x800000u;                                  /* subnormal half */
    int shift = -e - 14 + 13;                        /* 14..24 */
    uint32_t h = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1), halfway = 1u << (shift - 1);
    if (rem > halfway || (rem == halfway && (h & 1))) h++;
    return (uint16_t)(sign | h);
}

static uint16_t float_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* SplitMix64 (Steele, Lea, Flood 2014): n-th output for a given seed. */
static uint64_t splitmix64_nth(uint64_t seed, uint64_t n)
{
    uint64_t z = seed + n * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

/* Counter-hash table element before rounding to the storage type:
 * four 16-bit fields summed, centred, one fp32 multiply. */
static float hash_value_f32(uint64_t seed, int t, int64_t row, int c)
{
    uint64_t counter = ((uint64_t)t << 48) | ((uint64_t)row << 16) | (uint64_t)c;
    uint64_t z = splitmix64_nth(seed, counter + 1);
    int32_t s = (int32_t)(z & 0xFFFF) + (int32_t)((z >> 16) & 0xFFFF)
              + (int32_t)((z >> 32) & 0xFFFF) + (int32_t)((z >> 48) & 0xFFFF) - 131070;
    const float scale = (float)(1.0 / sqrt(4.0 * (65536.0 * 65536.0 - 1.0) / 12.0));
    volatile float v = (float)s * scale;             /* a single fp32 product */
    return v;
}

/* A table is either materialised (data != NULL) or given by its hash seed. */
typedef struct {
    const void *data;
    int64_t rows;
    int32_t dim;
    int32_t dtype;
    uint64_t seed;
    int32_t index;
} oracle_table_t;

static double table_elem(const oracle_table_t *tb, int64_t row, int c)
{
    if (tb->data) {
        int64_t i = row * tb->dim + c;
        switch (tb->dtype) {
        case DT_F32:  return (double)((const float *)tb->data)[i];
        case DT_BF16: return bf16_to_double(((const uint16_t *)tb->data)[i]);
        default:      return half_to_double(((const uint16_t *)tb->data)[i]);
        }
    }
    float v = hash_value_f32(tb->seed, tb->index, row, c);
    switch (tb->dtype) {
    case DT_F32:  return (double)v;
    case DT_BF16: return bf16_to_double(float_to_bf16(v));
    default:      return half_to_double(float_to_half(v));
    }
}

/* Materialise rows [row_lo, row_lo + nrows) of a hash table into `out`
 * (float for fp32, uint16 bit patterns otherwise). */
int oracle_fill_table(uint64_t seed, int t, int64_t row_lo, int64_t nrows, int dim, int dtype,
                      void *out, int nthreads)
{
    if (nthreads < 1) nthreads = 1;
    #pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t r = 0; r < nrows; r++)
        for (int c = 0; c < dim; c++) {
            float v = hash_value_f32(seed, t, row_lo + r, c);
            int64_t i = r * dim + c;
            if (dtype == DT_F32)       ((float *)out)[i] = v;
            else if (dtype == DT_BF16) ((uint16_t *)out)[i] = float_to_bf16(v);
            else                       ((uint16_t *)out)[i] = float_to_half(v);
        }
    return 0;
}

/* ------------------------------------------------------------- owner map */

static int64_t row_block(int64_t rows, int P) { return (rows + P - 1) / P; }

/* Owner rank and owner-local row of (table t, row id). */
static void owner_of(int part, int P, int t, int64_t rows, int32_t id, int *dst, int32_t *local)
{
    if (part == PART_TABLE_RR) { *dst = t % P; *local = id; }
    else { int64_t blk = row_block(rows, P); *dst = (int)(id / blk); *local = (int32_t)(id - (int64_t)*dst * blk); }
}

/* Does owner `dst` hold any part of table t? (defines which bags get a sub-bag entry) */
static int involves(int part, int P, int t, int dst)
{
    return part == PART_TABLE_RR ? (t % P == dst) : 1;
}

/* Number of sub-bag entries in the message src -> dst. */
int64_t oracle_subbags_per_pair(int part, int P, int T, int b, int dst)
{
    int64_t n = 0;
    for (int t = 0; t < T; t++) if (involves(part, P, t, dst)) n += b;
    return n;
}

/* ------------------------------------------------------------ step 1: route */

/*
 * Routing artefacts of one iteration, i.e. the arguments an alltoallv of the
 * requests would be called with and the buffers on both sides of it.
 *
 *   sendcounts[src*P+dst]  lookups of src owned by dst
 *   sdispls   [src*P+dst]  exclusive scan of sendcounts over dst
 *   recvcounts[dst*P+src]  = sendcounts[src*P+dst]
 *   rdispls   [dst*P+src]  exclusive scan of recvcounts over src
 *   sendbuf[L]  concatenation over src (rank src starts at offsets[src*T*b]) of
 *               src's owner-local rows, sorted by dst, ties in original order
 *               (bag order, then position inside the bag): a stable counting sort
 *   recvbuf[L]  concatenation over dst (rank dst starts at the sum of the
 *               receive totals of lower ranks) of what dst receives: the
 *               segment of src at rdispls[dst][src]
 *   sublen[...] concatenation over dst, then src, of one length per bag of src
 *               that can involve dst (table-wise: bags of dst's tables; row-wise:
 *               all bags), in bag order (t, s)
 *
 * Returns 0, or -1 if an id is out of range / offsets are not monotone.
 */
int oracle_route(int P, int T, int b, int part, const int64_t *rows,
                 const int32_t *ids, const int32_t *offsets,
                 int32_t *sendcounts, int32_t *sdispls, int32_t *recvcounts, int32_t *rdispls,
                 int32_t *sendbuf, int32_t *recvbuf, int32_t *sublen, int nthreads)
{
    int bad = 0;
    int64_t bags_per_rank = (int64_t)T * b;
    if (nthreads < 1) nthreads = 1;

    /* per requester: histogram, scan, stable placement */
    #pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
    for (int src = 0; src < P; src++) {
        int32_t *cnt = sendcounts + (int64_t)src * P, *dsp = sdispls + (int64_t)src * P;
        int64_t g0 = (int64_t)src * bags_per_rank;
        int64_t base = offsets[g0];
        for (int d = 0; d < P; d++) cnt[d] = 0;
        for (int t = 0; t < T; t++)
            for (int s = 0; s < b; s++) {
                int64_t g = g0 + (int64_t)t * b + s;
                if (offsets[g + 1] < offsets[g]) { bad = 1; continue; }
                for (int64_t l = offsets[g]; l < offsets[g + 1]; l++) {
                    if (ids[l] < 0 || ids[l] >= rows[t]) { bad = 1; continue; }
                    int dst; int32_t loc;
                    owner_of(part, P, t, rows[t], ids[l], &dst, &loc);
                    cnt[dst]++;
                }
            }
        int32_t run = 0;
        for (int d = 0; d < P; d++) { dsp[d] = run; run += cnt[d]; }
        int32_t *next = (int32_t *)malloc(sizeof(int32_t) * P);
        for (int d = 0; d < P; d++) next[d] = dsp[d];
        for (int t = 0; t < T; t++)
            for (int s = 0; s < b; s++) {
                int64_t g = g0 + (int64_t)t * b + s;
                for (int64_t l = offsets[g]; l < offsets[g + 1]; l++) {
                    if (ids[l] < 0 || ids[l] >= rows[t]) continue;
                    int dst; int32_t loc;
                    owner_of(part, P, t, rows[t], ids[l], &dst, &loc);
                    sendbuf[base + next[dst]++] = loc;
                }
            }
        free(next);
    }
    if (bad) return -1;

    /* the exchange: receive-side counts, displacements and buffers */
    int64_t *rbase = (int64_t *)malloc(sizeof(int64_t) * (P + 1));
    int64_t *sbbase = (int64_t *)malloc(sizeof(int64_t) * (P + 1));
    rbase[0] = 0; sbbase[0] = 0;
    for (int dst = 0; dst < P; dst++) {
        int32_t run = 0;
        for (int src = 0; src < P; src++) {
            recvcounts[(int64_t)dst * P + src] = sendcounts[(int64_t)src * P + dst];
            rdispls[(int64_t)dst * P + src] = run;
            run += recvcounts[(int64_t)dst * P + src];
        }
        rbase[dst + 1] = rbase[dst] + run;
        sbbase[dst + 1] = sbbase[dst] + (int64_t)P * oracle_subbags_per_pair(part, P, T, b, dst);
    }
    #pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
    for (int dst = 0; dst < P; dst++) {
        int64_t per_pair = oracle_subbags_per_pair(part, P, T, b, dst);
        for (int src = 0; src < P; src++) {
            int64_t sbase = offsets[(int64_t)src * bags_per_rank];
            const int32_t *seg = sendbuf + sbase + sdispls[(int64_t)src * P + dst];
            int32_t n = sendcounts[(int64_t)src * P + dst];
            memcpy(recvbuf + rbase[dst] + rdispls[(int64_t)dst * P + src], seg, sizeof(int32_t) * (size_t)n);
            /* sub-bag lengths: count, per bag, the ids owned by dst */
            int32_t *sl = sublen + sbbase[dst] + (int64_t)src * per_pair;
            int64_t q = 0;
            for (int t = 0; t < T; t++) {
                if (!involves(part, P, t, dst)) continue;
                for (int s = 0; s < b; s++) {
                    int64_t g = (int64_t)src * bags_per_rank + (int64_t)t * b + s;
                    int32_t c = 0;
                    for (int64_t l = offsets[g]; l < offsets[g + 1]; l++) {
                        int d2; int32_t loc;
                        owner_of(part, P, t, rows[t], ids[l], &d2, &loc);
                        c += (d2 == dst);
                    }
                    sl[q++] = c;
                }
            }
        }
    }
    free(rbase); free(sbbase);
    return 0;
}

/* ------------------------------------------- result by the plain definition */

/*
 * out[((src*b + s)*T + t)*D + c] = sum over the ids of bag (src,t,s) of
 * W_t[id][c], in fp64, rounded once to fp32.  If n_sel > 0 only the bags listed
 * in sel[] (flat bag indices g) are computed, into out[i*D + c] for i-th entry.
 */
int oracle_pool_definition(int P, int T, int b, const oracle_table_t *tables,
                           const int32_t *ids, const int32_t *offsets,
                           int64_t n_sel, const int64_t *sel, float *out, int nthreads)
{
    int64_t G = (int64_t)P * T * b;
    int64_t n = n_sel > 0 ? n_sel : G;
    if (nthreads < 1) nthreads = 1;
    #pragma omp parallel for num_threads(nthreads) schedule(static)
    for (int64_t i = 0; i < n; i++) {
        int64_t g = n_sel > 0 ? sel[i] : i;
        int src = (int)(g / ((int64_t)T * b));
        int t = (int)((g / b) % T);
        int s = (int)(g % b);
        const oracle_table_t *tb = &tables[t];
        int D = tb->dim;
        float *o = n_sel > 0 ? out + i * D : out + (((int64_t)src * b + s) * T + t) * D;
        for (int c = 0; c < D; c++) {
            double acc = 0.0;
            for (int64_t l = offsets[g]; l < offsets[g + 1]; l++)
                acc += table_elem(tb, ids[l], c);
            o[c] = (float)acc;
        }
    }
    return 0;
}

/* ------------------------ result by following the routed buffers: steps 2, 3 */

/*
 * Owner-side gather and sum-pool over what each owner received (recvbuf,
 * recvcounts, rdispls, sublen as produced by oracle_route), then the return
 * scatter into the requester layout.  Table-wise: a bag has one owner, the
 * pooled vector is copied.  Row-wise: the owners' partial sums of one bag are
 * added in owner order.  fp64 throughout, one rounding to fp32 at the end.
 */
int oracle_pool_routed(int P, int T, int b, int part, const oracle_table_t *tables,
                       const int32_t *recvbuf, const int32_t *recvcounts, const int32_t *rdispls,
                       const int32_t *sublen, float *out)
{
    int D = tables[0].dim;
    int64_t G = (int64_t)P * T * b;
    double *acc = (double *)calloc((size_t)(G * D), sizeof(double));
    if (!acc) return -2;
    int64_t rbase = 0, sbbase = 0;
    for (int dst = 0; dst < P; dst++) {
        int64_t per_pair = oracle_subbags_per_pair(part, P, T, b, dst);
        int64_t total = 0;
        for (int src = 0; src < P; src++) {
            const int32_t *seg = recvbuf + rbase + rdispls[(int64_t)dst * P + src];
            const int32_t *sl = sublen + sbbase + (int64_t)src * per_pair;
            int64_t pos = 0, q = 0;
            for (int t = 0; t < T; t++) {
                if (!involves(part, P, t, dst)) continue;
                int64_t blk = part == PART_ROW_BLOCK ? row_block(tables[t].rows, P) : 0;
                for (int s = 0; s < b; s++) {
                    int32_t n = sl[q++];
                    double *a = acc + ((((int64_t)src * b + s) * T + t) * D);
                    for (int32_t j = 0; j < n; j++) {
                        int64_t row = (int64_t)seg[pos + j] + (int64_t)dst * blk;   /* owner-local -> table row */
                        for (int c = 0; c < D; c++) a[c] += table_elem(&tables[t], row, c);
                    }
                    pos += n;
                }
            }
            if (pos != recvcounts[(int64_t)dst * P + src]) { free(acc); return -1; }
            total += pos;
        }
        rbase += total;
        sbbase += (int64_t)P * per_pair;
    }
    for (int64_t i = 0; i < G * D; i++) out[i] = (float)acc[i];
    free(acc);
    return 0;
}
