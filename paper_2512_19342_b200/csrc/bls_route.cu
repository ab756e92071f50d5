// Step 1, the router: every requester rank sorts the rows it needs by owner rank
// (Section I: every rank works out which vector IDs it needs from which other rank and
// fetches them with an alltoallv).  Output per requester:
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

// id / blk without a division: q = floor(id * floor(2^32/blk) / 2^32) is the quotient
// or one less (the error term is below id / 2^32 < 1/2), one correction step fixes it.
__device__ __forceinline__ int owner_of_row(unsigned id, int blk, unsigned magic, int &local)
{
    unsigned q = __umulhi(id, magic);
    unsigned r = id - q * (unsigned)blk;
    if (r >= (unsigned)blk) { q++; r -= (unsigned)blk; }
    local = (int)r;
    return (int)q;
}

// A tile (128 bags of one table of one requester) is routed only if all its bags are
// well-formed; otherwise it is treated as empty and BLS_EINVAL is latched.  Returns the
// tile's ID range [lo, hi).
__device__ __forceinline__ bool tile_range(const BlsParams &p, const RouteCtx &c, long long g0, int nb, int &lo, int &hi)
{
    bool ok = true;
    if ((int)threadIdx.x < nb) {
        const long long a = c.off[g0 + threadIdx.x], e = c.off[g0 + threadIdx.x + 1];
        ok = a >= 0 && a <= e && e <= c.n_ids;
    }
    ok = __syncthreads_and(ok);
    if (!ok) { if (threadIdx.x == 0) flag(p, BLS_ST_EINVAL); lo = hi = 0; return false; }
    lo = c.off[g0];
    hi = c.off[g0 + nb];
    return true;
}

// grid (NT, P): per-tile histogram over destinations, one thread per lookup (coalesced);
// lanes with the same destination are counted together.
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
    int lo, hi;
    tile_range(p, c, ((long long)src * p.T + t) * p.b + s0, nb, lo, hi);      // contains a barrier
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    const unsigned magic = p.tab[t].magic;
    const int lane = threadIdx.x & 31;
    for (int l0 = lo + (threadIdx.x & ~31); l0 < hi; l0 += BLS_ROUTE_TB) {
        const int l = l0 + lane;
        int d = 64 + lane;                                  // no lookup: matches nobody
        if (l < hi) {
            unsigned id = (unsigned)__ldcs(c.ids + l);
            if (id >= rows) { id = 0; flag(p, BLS_ST_ERANGE); }
            int local;
            d = owner_of_row(id, blk, magic, local);
        }
        const unsigned same = __match_any_sync(0xffffffffu, d);
        if (l < hi && lane == __ffs(same) - 1) atomicAdd(&cnt[d], __popc(same));
    }
    __syncthreads();
    if (threadIdx.x < p.P)
        p.tile_cnt[((size_t)src * p.NT + blockIdx.x) * p.P + threadIdx.x] = cnt[threadIdx.x];
}

// One block per requester: exclusive scan of the tile counts in (destination, tile)
// order, in place; send counts, displacements and the closing sub-bag entries.
// Warp w owns destinations w, w+32, ...: totals first, then the displacements, then the
// per-tile bases 32 tiles at a time.
__global__ void __launch_bounds__(1024) bls_rw_scan_kernel(BlsParams p)
{
    __shared__ long long tot[BLS_MAX_RANKS], disp[BLS_MAX_RANKS + 1];
    const int src = blockIdx.x;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    int *tc = p.tile_cnt + (size_t)src * p.NT * p.P;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int d = w; d < p.P; d += 32) {
        long long sum = 0;
        for (int tile = lane; tile < p.NT; tile += 32) sum += tc[(size_t)tile * p.P + d];
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) tot[d] = sum;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long run = 0;
        for (int d = 0; d < p.P; d++) { disp[d] = run; run += tot[d]; }
        disp[p.P] = run;
        if (run > p.cap) flag(p, BLS_ST_ENOSPC);
    }
    __syncthreads();
    if (threadIdx.x < p.P) {
        const int d = threadIdx.x;
        c.sdispls[d] = (int)min(disp[d], (long long)0x7fffffff);
        c.sendcounts[d] = (int)tot[d];
        // sub-bag starts are kept bag-major [table][sample][dst]: the entry after the last bag
        // closes every destination's region
        c.sub_start[(size_t)p.T * p.b * p.P + d] = (int)min(disp[d + 1], (long long)p.cap);
    }
    for (int d = w; d < p.P; d += 32) {
        long long run = disp[d];
        for (int t0 = 0; t0 < p.NT; t0 += 128) {           // four independent loads per lane in flight
            int v[4];
            #pragma unroll
            for (int q = 0; q < 4; q++) {
                const int tile = t0 + q * 32 + lane;
                v[q] = tile < p.NT ? tc[(size_t)tile * p.P + d] : 0;
            }
            #pragma unroll
            for (int q = 0; q < 4; q++) {
                int inc = v[q];
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += y;
                }
                const int tile = t0 + q * 32 + lane;
                if (tile < p.NT) tc[(size_t)tile * p.P + d] = (int)min(run + inc - v[q], (long long)p.cap);
                run += __shfl_sync(0xffffffffu, inc, 31);
            }
        }
    }
}

// grid (NT, P), one thread per bag.  Inside a tile, the lookups of one
// destination keep their original order: position = tile base + number of
// same-destination lookups in earlier bags of the tile + rank inside the bag.
// The tile's IDs are first staged in shared memory (coalesced) with their owner
// already computed, so the two per-bag passes run out of shared memory.
#define BLS_RW_STAGE 2048
__global__ void __launch_bounds__(BLS_ROUTE_TB) bls_rw_scatter_kernel(BlsParams p)
{
    __shared__ int cnt[BLS_MAX_RANKS][BLS_ROUTE_TB + 1];
    __shared__ int s_local[BLS_RW_STAGE], s_out[BLS_RW_STAGE];
    __shared__ unsigned char s_dst[BLS_RW_STAGE];
    __shared__ int s_tcount[BLS_MAX_RANKS], s_toff[BLS_MAX_RANKS];
    const int src = blockIdx.y;
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int t = blockIdx.x / p.tiles_per_table;
    const int s0 = (blockIdx.x % p.tiles_per_table) * BLS_ROUTE_TB;
    const int nb = min(BLS_ROUTE_TB, p.b - s0);
    const int s = threadIdx.x;
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    const unsigned magic = p.tab[t].magic;
    const long long g0 = ((long long)src * p.T + t) * p.b + s0;
    for (int d = 0; d < p.P; d++) cnt[d][s] = 0;
    int lo, hi;
    const bool ok = tile_range(p, c, g0, nb, lo, hi);
    const bool staged = hi - lo <= BLS_RW_STAGE;
    if (staged)
        for (int l = lo + threadIdx.x; l < hi; l += BLS_ROUTE_TB) {
            unsigned id = (unsigned)__ldcs(c.ids + l);
            if (id >= rows) id = 0;
            int local;
            s_dst[l - lo] = (unsigned char)owner_of_row(id, blk, magic, local);
            s_local[l - lo] = local;
        }
    __syncthreads();
    int st = 0, en = 0;
    if (ok && s < nb) { st = c.off[g0 + s]; en = c.off[g0 + s + 1]; }
    auto look = [&](int l, int &local) {                    // owner and owner-local row of lookup l
        if (staged) { local = s_local[l - lo]; return (int)s_dst[l - lo]; }
        unsigned id = (unsigned)c.ids[l];
        if (id >= rows) id = 0;
        return owner_of_row(id, blk, magic, local);
    };
    for (int l = st; l < en; l++) { int local; cnt[look(l, local)][s]++; }
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
        if (lane == 31) s_tcount[d] = run - tb[d];          // lookups of this tile that go to d
    }
    __syncthreads();
    // sub-bag starts of the tile: nb rows of P entries, contiguous in the bag-major layout
    {
        int *rows_out = c.sub_start + ((size_t)t * p.b + s0) * p.P;
        for (int e = threadIdx.x; e < nb * p.P; e += BLS_ROUTE_TB) rows_out[e] = min(cnt[e % p.P][e / p.P], p.cap);
    }
    if (!staged) {                                          // oversized tile: write straight to the send buffer
        for (int l = st; l < en; l++) {
            int local;
            const int d = look(l, local);
            const int pos = cnt[d][s]++;
            if (pos < p.cap) c.sendbuf[pos] = local;
        }
        return;
    }
    // reorder inside shared memory (destination-major, order kept), then copy each
    // destination's segment to the send buffer with coalesced stores
    if (threadIdx.x == 0) {
        int run = 0;
        for (int d = 0; d < p.P; d++) { s_toff[d] = run; run += s_tcount[d]; }
    }
    __syncthreads();
    for (int l = st; l < en; l++) {
        int local;
        const int d = look(l, local);
        const int pos = cnt[d][s]++;
        s_out[s_toff[d] + (pos - tb[d])] = local;
    }
    __syncthreads();
    for (int d = 0; d < p.P; d++) {
        const int base_d = tb[d], n_d = s_tcount[d], o_d = s_toff[d];
        for (int k2 = threadIdx.x; k2 < n_d; k2 += BLS_ROUTE_TB)
            if (base_d + k2 < p.cap) c.sendbuf[base_d + k2] = s_out[o_d + k2];
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
