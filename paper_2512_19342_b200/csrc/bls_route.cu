// Step 1, the router: every requester rank sorts the rows it needs by owner rank
// (Section I: "each process determines the vector IDs required from other
// processes, and retrieves them through an alltoallv").  Output per requester:
// sendcounts / sdispls, the stably packed send buffer of owner-local rows, and
// the start of every sub-bag inside it (the owner rebuilds bag boundaries from
// consecutive differences).
//
// Positions never depend on the order in which atomics land: counts come from
// histograms, positions from exclusive scans, so the packed buffer is the unique
// stable counting sort by destination.
//
// Table-wise placement: the owner depends on the table only, so a requester's
// (table) chunks move as a whole; counts follow from the offsets alone.
// Row-wise placement: a real multisplit, done per tile of 128 bags of one table.
#include "bls_device.cuh"

// ------------------------------------------------------------------ table-wise
// First half (chunk lengths, scan, counts, displacements): tw_meta_warp, run by the
// gate kernel.  Second half, here: move every ID to its place and write the sub-bag
// starts.
// grid (NT, P): tile = 128 bags of one (requester, table) chunk.  Copies the
// chunk's IDs to their place in the send buffer (coalesced) and writes the
// sub-bag starts.
__global__ void __launch_bounds__(256) bls_tw_copy_kernel(BlsParams p)
{
    const int src = blockIdx.y;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int i = blockIdx.x / p.tiles_per_table;
    const int s0 = (blockIdx.x % p.tiles_per_table) * BLS_ROUTE_TB;
    const int nb = min(BLS_ROUTE_TB, p.b - s0);
    const int t = p.pair[i].t;
    const long long g0 = ((long long)src * p.T + t) * p.b;
    const int *cbp = p.chunk_base + (size_t)src * (p.NI + 1);
    const int cb = cbp[i];
    const int cn = cbp[i + 1] - cb;              // chunk length accepted by the meta kernel
    const long long off0 = c.off[g0];
    __shared__ int s_lo, s_hi;
    if (threadIdx.x < nb) {
        int st, en;
        if (!bag_range(c, g0 + s0 + threadIdx.x, off0, cn, st, en)) flag(p, BLS_ST_EINVAL);
        int pos = cb + st;
        c.sub_start[(size_t)i * p.b + s0 + threadIdx.x] = pos > p.cap ? p.cap : pos;
        if (threadIdx.x == 0) s_lo = st;
        if (threadIdx.x == nb - 1) s_hi = en;
    }
    __syncthreads();
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int lo = s_lo, hi = max(s_lo, s_hi);
    const int *in = c.ids + off0;
    if (!p.hot.enabled) {
        for (int l0 = lo + threadIdx.x; l0 < hi; l0 += 4 * blockDim.x) {
            int id[4];
            #pragma unroll
            for (int q = 0; q < 4; q++) {
                const int l = l0 + q * blockDim.x;
                id[q] = l < hi ? __ldcs(in + l) : 0;
            }
            #pragma unroll
            for (int q = 0; q < 4; q++) {
                const int l = l0 + q * blockDim.x;
                if (l >= hi) continue;
                int v = id[q];
                if ((unsigned)v >= rows) { v = 0; flag(p, BLS_ST_ERANGE); }
                const int pos = cb + l;
                if (pos < p.cap) c.sendbuf[pos] = v;
            }
        }
    } else {
        // also tell the owner which lookups hit its staged copy of the table's hot rows:
        // slot = number of hot rows before this one (bitmap + per-word prefix counts)
        const unsigned *bm = p.hot.bitmap + p.hot.word_base[t], *pf = p.hot.prefix + p.hot.word_base[t];
        unsigned short *hs = p.hot.hotslot + ((size_t)c.slot * p.P + src) * (size_t)p.cap;
        for (int l = lo + threadIdx.x; l < hi; l += blockDim.x) {
            int id = __ldcs(in + l);
            if ((unsigned)id >= rows) { id = 0; flag(p, BLS_ST_ERANGE); }
            const unsigned w = __ldg(bm + (id >> 5)), bit = 1u << (id & 31);
            const unsigned slot = (w & bit) ? __ldg(pf + (id >> 5)) + __popc(w & (bit - 1u)) : 0xFFFFu;
            int pos = cb + l;
            if (pos < p.cap) { c.sendbuf[pos] = id; hs[pos] = (unsigned short)slot; }
        }
    }
}

// -------------------------------------------------------------------- row-wise

// grid (NT, P), one thread per bag: per-tile histogram over destinations.
__global__ void __launch_bounds__(BLS_ROUTE_TB) bls_rw_count_kernel(BlsParams p)
{
    __shared__ int cnt[BLS_MAX_RANKS];
    const int src = blockIdx.y;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int t = blockIdx.x / p.tiles_per_table;
    const int s0 = (blockIdx.x % p.tiles_per_table) * BLS_ROUTE_TB;
    const int nb = min(BLS_ROUTE_TB, p.b - s0);
    if (threadIdx.x < BLS_MAX_RANKS) cnt[threadIdx.x] = 0;
    __syncthreads();
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    if (threadIdx.x < nb) {
        int st, en;
        long long g = ((long long)src * p.T + t) * p.b + s0 + threadIdx.x;
        if (!bag_range(c, g, 0, c.n_ids, st, en)) flag(p, BLS_ST_EINVAL);
        for (int l = st; l < en; l++) {
            int id = c.ids[l];
            if ((unsigned)id >= rows) { id = 0; flag(p, BLS_ST_ERANGE); }
            atomicAdd(&cnt[id / blk], 1);
        }
    }
    __syncthreads();
    if (threadIdx.x < p.P)
        p.tile_cnt[((size_t)src * p.NT + blockIdx.x) * p.P + threadIdx.x] = cnt[threadIdx.x];
}

// One block per requester: exclusive scan of the tile counts in (destination,
// tile) order, in place; send counts and displacements.
__global__ void __launch_bounds__(1024) bls_rw_scan_kernel(BlsParams p)
{
    __shared__ long long warp_tot[32];
    __shared__ long long s_total;
    const int src = blockIdx.x;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    int *tc = p.tile_cnt + (size_t)src * p.NT * p.P;
    const long long N = (long long)p.P * p.NT;
    const long long per = (N + blockDim.x - 1) / blockDim.x;
    const long long e0 = min(N, (long long)threadIdx.x * per), e1 = min(N, e0 + per);
    long long sum = 0;
    for (long long e = e0; e < e1; e++) sum += tc[(e % p.NT) * p.P + (e / p.NT)];
    // block exclusive scan of the per-thread sums
    long long inc = sum;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        long long v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    if (w == 0) {
        long long v = warp_tot[lane], x = v;
        for (int o = 1; o < 32; o <<= 1) {
            long long y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        warp_tot[lane] = x - v;
        if (lane == 31) s_total = x;
    }
    __syncthreads();
    long long run = warp_tot[w] + inc - sum;
    for (long long e = e0; e < e1; e++) {
        int *cell = &tc[(e % p.NT) * p.P + (e / p.NT)];
        int v = *cell;
        if (e % p.NT == 0) c.sdispls[e / p.NT] = (int)run;
        *cell = (int)(run > p.cap ? p.cap : run);
        run += v;
    }
    __syncthreads();
    if (threadIdx.x < p.P) {
        int d = threadIdx.x;
        long long end = d + 1 < p.P ? c.sdispls[d + 1] : s_total;
        c.sendcounts[d] = (int)(end - c.sdispls[d]);
        // sub-bag starts are kept bag-major [table][sample][dst]: the entry after the last bag
        // closes every destination's region
        c.sub_start[(size_t)p.T * p.b * p.P + d] = (int)(end > p.cap ? p.cap : end);
    }
    if (threadIdx.x == 0 && s_total > p.cap) flag(p, BLS_ST_ENOSPC);
}

// grid (NT, P), one thread per bag.  Inside a tile, the lookups of one
// destination keep their original order: position = tile base + number of
// same-destination lookups in earlier bags of the tile + rank inside the bag.
__global__ void __launch_bounds__(BLS_ROUTE_TB) bls_rw_scatter_kernel(BlsParams p)
{
    __shared__ int cnt[BLS_MAX_RANKS][BLS_ROUTE_TB + 1];
    const int src = blockIdx.y;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int t = blockIdx.x / p.tiles_per_table;
    const int s0 = (blockIdx.x % p.tiles_per_table) * BLS_ROUTE_TB;
    const int nb = min(BLS_ROUTE_TB, p.b - s0);
    const int s = threadIdx.x;
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    for (int d = 0; d < p.P; d++) cnt[d][s] = 0;
    int st = 0, en = 0;
    if (s < nb) {
        long long g = ((long long)src * p.T + t) * p.b + s0 + s;
        bag_range(c, g, 0, c.n_ids, st, en);
        for (int l = st; l < en; l++) {
            int id = c.ids[l];
            if ((unsigned)id >= rows) id = 0;
            cnt[id / blk][s]++;
        }
    }
    __syncthreads();
    // exclusive scan over the bags of the tile, one warp per destination
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int *tb = p.tile_cnt + ((size_t)src * p.NT + blockIdx.x) * p.P;
    for (int d = w; d < p.P; d += BLS_ROUTE_TB / 32) {
        int v[BLS_ROUTE_TB / 32], tot = 0;
        #pragma unroll
        for (int q = 0; q < BLS_ROUTE_TB / 32; q++) { v[q] = cnt[d][lane * (BLS_ROUTE_TB / 32) + q]; tot += v[q]; }
        int inc = tot;
        for (int o = 1; o < 32; o <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        int run = tb[d] + inc - tot;
        #pragma unroll
        for (int q = 0; q < BLS_ROUTE_TB / 32; q++) { cnt[d][lane * (BLS_ROUTE_TB / 32) + q] = run; run += v[q]; }
    }
    __syncthreads();
    if (s < nb) {
        for (int d = 0; d < p.P; d++) {
            int pos = cnt[d][s];
            c.sub_start[((size_t)t * p.b + s0 + s) * p.P + d] = pos > p.cap ? p.cap : pos;
        }
        for (int l = st; l < en; l++) {
            int id = c.ids[l];
            if ((unsigned)id >= rows) id = 0;
            int d = id / blk;
            int pos = cnt[d][s]++;
            if (pos < p.cap) c.sendbuf[pos] = id - d * blk;
        }
    }
}

int bls_route_kernels(const bls_plan_t *pl) { return pl->prm.part == BLS_PART_TABLE_RR ? 1 : 3; }

void bls_launch_route(const bls_plan_t *pl)
{
    const BlsParams &p = pl->prm;
    dim3 grid(p.NT, p.P);
    if (p.part == BLS_PART_TABLE_RR) {
        bls_tw_copy_kernel<<<grid, 256, 0, pl->stream>>>(p);
    } else {
        bls_rw_count_kernel<<<grid, BLS_ROUTE_TB, 0, pl->stream>>>(p);
        bls_rw_scan_kernel<<<p.P, 1024, 0, pl->stream>>>(p);
        bls_rw_scatter_kernel<<<grid, BLS_ROUTE_TB, 0, pl->stream>>>(p);
    }
}
