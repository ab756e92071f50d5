// Hot-row staging for Zipf-skewed lookups (table-wise placement).
//
// Under power-law access a few hundred rows of a table receive most of the
// lookups, but an LRU L1 keeps only the few dozen hottest because every SM sees
// just a thin slice of the requests.  Here the hot set is made explicit: request
// counts are gathered from ID batches the caller shows us (bls_hot_observe), the K
// most requested rows of every table are selected (bls_hot_build), the router then
// marks each lookup with its slot in that list, and the gather kernel keeps the
// list's rows in shared memory while it works on a table.  Results are unchanged:
// a staged row is a copy of the table row.  The paper treats caching as orthogonal
// to its collective (Section II); this is an internal optimisation of step 2.
#include "bls_internal.h"

namespace {

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct HotLayout {
    size_t counts, bitmap, prefix, row_base, word_base, rows, count, hotslot, pair_ctr, total;
    long long n_rows, n_words;
};

HotLayout hot_layout(const bls_plan_t *pl, int K)
{
    const BlsParams &p = pl->prm;
    HotLayout L;
    L.n_rows = 0; L.n_words = 0;
    for (int t = 0; t < p.T; t++) { L.n_rows += pl->h_rows[t]; L.n_words += (pl->h_rows[t] + 31) / 32; }
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align256(o + bytes); return at; };
    L.counts = take(sizeof(unsigned) * (size_t)L.n_rows);
    L.bitmap = take(sizeof(unsigned) * (size_t)L.n_words);
    L.prefix = take(sizeof(unsigned) * (size_t)L.n_words);
    L.row_base = take(sizeof(long long) * (p.T + 1));
    L.word_base = take(sizeof(long long) * (p.T + 1));
    L.rows = take(sizeof(int) * (size_t)p.T * K);
    L.count = take(sizeof(int) * p.T);
    L.hotslot = take(sizeof(unsigned short) * (size_t)p.S * p.P * p.cap);
    L.pair_ctr = take(sizeof(int) * p.NI);
    L.total = o;
    return L;
}

// One thread per lookup of the batch: count requests per (table, row).
__global__ void __launch_bounds__(256) bls_hot_count_kernel(BlsParams p, const int *ids, const int *off, long long n_ids)
{
    // grid (tiles, T, P): tile of 256*8 lookups of the (src, table) chunk
    const int t = blockIdx.y, src = blockIdx.z;
    const long long g0 = ((long long)src * p.T + t) * p.b;
    long long lo = off[g0], hi = off[g0 + p.b];
    if (lo < 0 || hi > n_ids || hi < lo) return;
    const unsigned rows = (unsigned)p.tab[t].rows;
    unsigned *cnt = p.hot.counts + p.hot.row_base[t];
    for (long long l = lo + (long long)blockIdx.x * blockDim.x + threadIdx.x; l < hi; l += (long long)gridDim.x * blockDim.x) {
        const unsigned id = (unsigned)ids[l];
        if (id < rows) atomicAdd(&cnt[id], 1u);
    }
}

// One block per table: the largest count threshold that keeps at most K rows,
// then bitmap, per-word prefix counts and the slot-ordered row list.
__global__ void __launch_bounds__(1024) bls_hot_select_kernel(BlsParams p)
{
    constexpr int BINS = 4096;
    __shared__ unsigned hist[BINS];
    __shared__ unsigned s_thr;
    __shared__ unsigned warp_tot[32];
    __shared__ unsigned s_carry, s_round;
    const int t = blockIdx.x;
    const long long rows = p.tab[t].rows;
    const unsigned *cnt = p.hot.counts + p.hot.row_base[t];
    for (int i = threadIdx.x; i < BINS; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (long long r = threadIdx.x; r < rows; r += blockDim.x) {
        const unsigned c = cnt[r];
        if (c) atomicAdd(&hist[c < BINS ? c : BINS - 1], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned acc = 0, thr = BINS;                      // rows with count >= thr are hot
        for (int c = BINS - 1; c >= 1; c--) {
            if (acc + hist[c] > (unsigned)p.hot.K) break;
            acc += hist[c];
            thr = c;
        }
        s_thr = thr;
        s_carry = 0;
    }
    __syncthreads();
    const unsigned thr = s_thr;
    const long long words = (rows + 31) / 32;
    unsigned *bm = p.hot.bitmap + p.hot.word_base[t], *pf = p.hot.prefix + p.hot.word_base[t];
    int *list = p.hot.rows + (size_t)t * p.hot.K;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (long long w0 = 0; w0 < words; w0 += blockDim.x) {
        const long long w = w0 + threadIdx.x;
        unsigned bits = 0;
        if (w < words)
            for (int b = 0; b < 32; b++) {
                const long long r = w * 32 + b;
                if (r < rows) { unsigned c = cnt[r]; c = c < BINS ? c : BINS - 1; if (c >= thr && c > 0) bits |= 1u << b; }
            }
        const unsigned n = __popc(bits);
        unsigned inc = n;                                  // block-wide exclusive scan of the popcounts
        for (int o = 1; o < 32; o <<= 1) { unsigned y = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += y; }
        if (lane == 31) warp_tot[wid] = inc;
        __syncthreads();
        if (wid == 0) {
            unsigned v = warp_tot[lane], x = v;
            for (int o = 1; o < 32; o <<= 1) { unsigned y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
            warp_tot[lane] = x - v;
            if (lane == 31) s_round = x;                   // hot rows found in this round of words
        }
        __syncthreads();
        const unsigned before = s_carry + warp_tot[wid] + inc - n;
        if (w < words) {
            bm[w] = bits;
            pf[w] = before;
            unsigned rest = bits, k = before;
            while (rest) {
                const int b = __ffs(rest) - 1;
                rest &= rest - 1;
                if (k < (unsigned)p.hot.K) list[k] = (int)(w * 32 + b);
                k++;
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) s_carry += s_round;
        __syncthreads();
    }
    if (threadIdx.x == 0) p.hot.count[t] = (int)min(s_carry, (unsigned)p.hot.K);
}

}  // namespace

extern "C" {

bls_status_t bls_hot_bytes(bls_plan_t *pl, int rows_per_table, size_t *bytes)
{
    if (!pl || !bytes || rows_per_table < 1 || rows_per_table > 65534) return BLS_EINVAL;
    if (pl->prm.part != BLS_PART_TABLE_RR) return BLS_ESTATE;
    *bytes = hot_layout(pl, rows_per_table).total;
    return BLS_OK;
}

bls_status_t bls_hot_attach(bls_plan_t *pl, int rows_per_table, void *buffer, size_t bytes)
{
    if (!pl || !buffer || ((uintptr_t)buffer & 255) || rows_per_table < 1 || rows_per_table > 65534) return BLS_EINVAL;
    if (pl->prm.part != BLS_PART_TABLE_RR || pl->t_handed != pl->t_next) return BLS_ESTATE;
    // the staged copy must fit in one SM's shared memory next to the kernel's own needs
    if ((size_t)rows_per_table * pl->prm.row_bytes > 200 * 1024) return BLS_ENOSPC;
    HotLayout L = hot_layout(pl, rows_per_table);
    if (bytes < L.total) return BLS_ENOSPC;
    BlsParams &p = pl->prm;
    char *b = (char *)buffer;
    p.hot.enabled = 0;
    p.hot.K = rows_per_table;
    p.hot.counts = (unsigned *)(b + L.counts);
    p.hot.bitmap = (unsigned *)(b + L.bitmap);
    p.hot.prefix = (unsigned *)(b + L.prefix);
    p.hot.row_base = (const long long *)(b + L.row_base);
    p.hot.word_base = (const long long *)(b + L.word_base);
    p.hot.rows = (int *)(b + L.rows);
    p.hot.count = (int *)(b + L.count);
    p.hot.hotslot = (unsigned short *)(b + L.hotslot);
    p.hot.pair_ctr = (int *)(b + L.pair_ctr);
    long long *rb = (long long *)malloc(sizeof(long long) * 2 * (p.T + 1));
    if (!rb) return BLS_ENOSPC;
    long long *wb = rb + p.T + 1;
    rb[0] = wb[0] = 0;
    for (int t = 0; t < p.T; t++) { rb[t + 1] = rb[t] + pl->h_rows[t]; wb[t + 1] = wb[t] + (pl->h_rows[t] + 31) / 32; }
    bool ok = cudaMemcpyAsync(b + L.row_base, rb, sizeof(long long) * (p.T + 1), cudaMemcpyHostToDevice, pl->stream) == cudaSuccess &&
              cudaMemcpyAsync(b + L.word_base, wb, sizeof(long long) * (p.T + 1), cudaMemcpyHostToDevice, pl->stream) == cudaSuccess &&
              cudaMemsetAsync(b + L.counts, 0, sizeof(unsigned) * (size_t)L.n_rows, pl->stream) == cudaSuccess &&
              cudaMemsetAsync(b + L.hotslot, 0xFF, sizeof(unsigned short) * (size_t)p.S * p.P * p.cap, pl->stream) == cudaSuccess &&
              cudaStreamSynchronize(pl->stream) == cudaSuccess;
    free(rb);
    pl->hot_attached = ok ? 1 : 0;
    return ok ? BLS_OK : BLS_ECUDA;
}

bls_status_t bls_hot_observe(bls_plan_t *pl, const int32_t *ids, const int32_t *offsets, int64_t n_ids)
{
    if (!pl || !offsets || (!ids && n_ids > 0) || n_ids < 0) return BLS_EINVAL;
    if (!pl->hot_attached) return BLS_ESTATE;
    const BlsParams &p = pl->prm;
    long long per_chunk = n_ids / ((long long)p.P * p.T) + 1;
    int tiles = (int)((per_chunk + 2047) / 2048);
    if (tiles > 1024) tiles = 1024;
    bls_hot_count_kernel<<<dim3(tiles, p.T, p.P), 256, 0, pl->stream>>>(p, ids, offsets, n_ids);
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}

bls_status_t bls_hot_build(bls_plan_t *pl)
{
    if (!pl) return BLS_EINVAL;
    if (!pl->hot_attached || pl->t_handed != pl->t_next) return BLS_ESTATE;
    bls_hot_select_kernel<<<pl->prm.T, 1024, 0, pl->stream>>>(pl->prm);
    if (cudaGetLastError() != cudaSuccess) return BLS_ECUDA;
    pl->prm.hot.enabled = 1;
    return BLS_OK;
}

bls_status_t bls_hot_view(bls_plan_t *pl, const int32_t **rows, const int32_t **count, int *rows_per_table)
{
    if (!pl) return BLS_EINVAL;
    if (!pl->hot_attached) return BLS_ESTATE;
    if (rows) *rows = pl->prm.hot.rows;
    if (count) *count = pl->prm.hot.count;
    if (rows_per_table) *rows_per_table = pl->prm.hot.K;
    return BLS_OK;
}

}  // extern "C"
