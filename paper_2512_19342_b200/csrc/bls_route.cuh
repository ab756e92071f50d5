// Device code of the router (step 1), shared by the stand-alone router kernels and the
// persistent ring kernel.  Every function works on one tile with a block of
// BLS_ROUTE_TB threads.
#pragma once
#include "bls_device.cuh"

// Which tile a block works on: taken from the grid (stand-alone kernels; the special
// registers cost nothing to re-read) or handed over (ring kernel).
struct TileFromGrid {
    __device__ __forceinline__ unsigned tile() const { return blockIdx.x; }
    __device__ __forceinline__ unsigned src() const { return blockIdx.y; }
};
struct TileGiven {
    unsigned tile_, src_;
    __device__ __forceinline__ unsigned tile() const { return tile_; }
    __device__ __forceinline__ unsigned src() const { return src_; }
};


// ------------------------------------------------------------------ table-wise
// First half (chunk lengths, scan, counts, displacements): tw_meta_warp, run by the
// gate kernel.  Second half, here: move every ID to its place and write the sub-bag
// starts.
// A tile = p.tile_bags bags of one (requester, table) chunk (128 for long bags, up to the
// whole chunk for short ones, so that a block always has a few thousand IDs to move); the
// stand-alone kernel runs on a grid (NT, P).  A block copies the tile's IDs to their place
// in the send buffer (coalesced) and writes the sub-bag starts.
// The work on one tile, given the requester's context, the tile (pair i, bags s0 .. s0 + nb - 1 of table t)
// and the chunk's place (cb) and accepted length (cn) in the send buffer.  Returns the end of the
// tile's IDs relative to the start of the chunk.
template <int INFLIGHT>
__device__ __forceinline__ int tw_copy_ctx(const BlsParams &p, const RouteCtx &c, int src, int i, int t, int s0, int nb,
                                           int cb, int cn)
{
    const long long g0 = ((long long)src * p.T + t) * p.b;
    const long long off0 = c.off[g0];
    __shared__ int s_lo, s_hi;
    for (int s = threadIdx.x; s < nb; s += blockDim.x) {
        int st, en;
        if (!bag_range(c, g0 + s0 + s, off0, cn, st, en)) flag(p, BLS_ST_EINVAL);
        int pos = cb + st;
        c.sub_start[(size_t)i * p.b + s0 + s] = pos > p.cap ? p.cap : pos;
        if (s == 0) s_lo = st;
        if (s == nb - 1) s_hi = en;
    }
    __syncthreads();                             // s_lo, s_hi
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int lo = s_lo, hi = max(s_lo, s_hi);
    const int *in = c.ids + off0;
    if (!p.hot.enabled) {
        for (int l0 = lo + threadIdx.x; l0 < hi; l0 += INFLIGHT * blockDim.x) {
            int id[INFLIGHT];
            #pragma unroll
            for (int q = 0; q < INFLIGHT; q++) {
                const int l = l0 + q * blockDim.x;
                id[q] = l < hi ? __ldcs(in + l) : 0;
            }
            #pragma unroll
            for (int q = 0; q < INFLIGHT; q++) {
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
    return hi;
}

template <int INFLIGHT, class Where>
__device__ __forceinline__ void tw_copy_tile(const BlsParams &p, const Where where)
{
    const int src = where.src();
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int i = where.tile() / p.tiles_per_table;
    const int s0 = (where.tile() % p.tiles_per_table) * p.tile_bags;
    const int *cbp = p.chunk_base + (size_t)src * (p.NI + 1);
    const int cb = cbp[i];
    tw_copy_ctx<INFLIGHT>(p, c, src, i, p.pair[i].t, s0, min(p.tile_bags, p.b - s0), cb, cbp[i + 1] - cb);
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

// Range of lookups [lo, hi) of a tile (BLS_ROUTE_TB bags of one table of one requester).
// A tile whose ends are not ordered or leave the ID array is treated as empty and
// BLS_EINVAL is latched; both row-wise kernels apply the same rule, so the counts
// and the positions derived from them always agree.
__device__ __forceinline__ void tile_ends(const BlsParams &p, const RouteCtx &c, long long g0, int nb, int &lo, int &hi)
{
    const long long a = c.off[g0], e = c.off[g0 + nb];
    if (a >= 0 && a <= e && e <= c.n_ids) { lo = (int)a; hi = (int)e; return; }
    flag(p, BLS_ST_EINVAL);
    lo = hi = 0;
}

// grid (NT, P), 128 threads: per-tile histogram over destinations (a tile is p.tile_bags
// bags of one table of one requester, up to a whole chunk).  The tile's IDs are read 2048
// at a time; the next 2048 are requested before the current ones are counted.  Every
// lookup is one shared-memory atomic on its warp's own histogram (measured: much cheaper
// than finding the lanes with equal destinations by a warp match first).
#define BLS_RW_PER_THREAD 16
#define BLS_RW_CHUNK (BLS_RW_PER_THREAD * BLS_ROUTE_TB)
template <class Where>
__device__ __forceinline__ void rw_count_tile(const BlsParams &p, const Where where)
{
    __shared__ int wcnt[BLS_ROUTE_TB / 32][BLS_MAX_RANKS];     // one histogram per warp
    const int src = where.src();
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int tid = threadIdx.x;
    const int t = where.tile() / p.tiles_per_table;
    const int s0 = (where.tile() - t * p.tiles_per_table) * p.tile_bags;
    const int nb = min(p.tile_bags, p.b - s0);
    (&wcnt[0][0])[tid] = 0;
    int lo, hi;
    tile_ends(p, c, ((long long)src * p.T + t) * p.b + s0, nb, lo, hi);
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    const unsigned magic = p.tab[t].magic;
    __syncthreads();
    bool bad = false;
    int cur[BLS_RW_PER_THREAD], nxt[BLS_RW_PER_THREAD];
    #pragma unroll
    for (int q = 0; q < BLS_RW_PER_THREAD; q++) {
        const int l = lo + q * BLS_ROUTE_TB + tid;
        cur[q] = l < hi ? __ldcs(c.ids + l) : 0;
    }
    for (int l0 = lo; l0 < hi; l0 += BLS_RW_CHUNK) {
        #pragma unroll
        for (int q = 0; q < BLS_RW_PER_THREAD; q++) {
            const int l = l0 + BLS_RW_CHUNK + q * BLS_ROUTE_TB + tid;
            nxt[q] = l < hi ? __ldcs(c.ids + l) : 0;
        }
        #pragma unroll
        for (int q = 0; q < BLS_RW_PER_THREAD; q++) {
            const int l = l0 + q * BLS_ROUTE_TB + tid;
            if (l < hi) {
                unsigned id = (unsigned)cur[q];
                if (id >= rows) { id = 0; bad = true; }
                int local;
                atomicAdd(&wcnt[tid >> 5][owner_of_row(id, blk, magic, local)], 1);
            }
        }
        #pragma unroll
        for (int q = 0; q < BLS_RW_PER_THREAD; q++) cur[q] = nxt[q];
    }
    if (bad) flag(p, BLS_ST_ERANGE);
    __syncthreads();
    if (tid < p.P) {
        const int n = wcnt[0][tid] + wcnt[1][tid] + wcnt[2][tid] + wcnt[3][tid];
        p.tile_cnt[((size_t)src * p.NT + where.tile()) * p.P + tid] = n;
        if (n) atomicAdd(&p.rw_total[src * p.P + tid], n);
    }
}

// grid (P destinations, P requesters), 128 threads: displacement of the destination's
// region (the totals of the destinations before it), send count, and the exclusive scan
// of the destination's tile counts in tile order, in place.
#define BLS_RW_SCAN_PER_THREAD 4
template <class Where>
__device__ __forceinline__ void rw_scan_tile(const BlsParams &p, const Where where)
{
    __shared__ long long s_disp;
    __shared__ int s_warp[4];
    const int d = where.tile(), src = where.src();       // here the "tile" is the destination rank
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    if (w == 0) {
        long long before = 0, all = 0;
        for (int dd = lane; dd < p.P; dd += 32) {
            const int x = p.rw_total[src * p.P + dd];
            all += x;
            if (dd < d) before += x;
        }
        for (int o = 16; o > 0; o >>= 1) {
            before += __shfl_xor_sync(0xffffffffu, before, o);
            all += __shfl_xor_sync(0xffffffffu, all, o);
        }
        if (lane == 0) {
            s_disp = before;
            c.sdispls[d] = (int)min(before, (long long)0x7fffffff);
            c.sendcounts[d] = p.rw_total[src * p.P + d];
            if (d == 0 && all > p.cap) flag(p, BLS_ST_ENOSPC);
        }
    }
    __syncthreads();
    long long run = s_disp;
    int *tc = p.tile_cnt + (size_t)src * p.NT * p.P + d;
    for (int t0 = 0; t0 < p.NT; t0 += 128 * BLS_RW_SCAN_PER_THREAD) {
        int v[BLS_RW_SCAN_PER_THREAD], sum = 0;
        #pragma unroll
        for (int q = 0; q < BLS_RW_SCAN_PER_THREAD; q++) {
            const int tile = t0 + tid * BLS_RW_SCAN_PER_THREAD + q;
            v[q] = tile < p.NT ? tc[(size_t)tile * p.P] : 0;
            sum += v[q];
        }
        int inc = sum;
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) s_warp[w] = inc;
        __syncthreads();
        long long base = run + inc - sum;
        for (int ww = 0; ww < w; ww++) base += s_warp[ww];
        #pragma unroll
        for (int q = 0; q < BLS_RW_SCAN_PER_THREAD; q++) {
            const int tile = t0 + tid * BLS_RW_SCAN_PER_THREAD + q;
            if (tile < p.NT) tc[(size_t)tile * p.P] = (int)min(base, (long long)p.cap);
            base += v[q];
        }
        run += (long long)s_warp[0] + s_warp[1] + s_warp[2] + s_warp[3];
        __syncthreads();
    }
}

// grid (NT, P), 128 threads: places the lookups of one tile and writes its sub-bag starts.
// The tile's lookups are classified BLS_RW_CHUNK at a time, one thread per lookup
// (coalesced).  For every destination d a bit mask over the chunk's lookups is built
// with shared-memory atomics (bit i set: lookup i goes to d) together with the number of set bits
// before each 32-bit word.  Everything else is a rank query on those masks:
//   position of lookup i       = base[d] + set bits of d's mask below i   (stable by construction)
//   start of sub-bag (bag s, d) = base[d] + set bits of d's mask below the bag's first lookup
// so neither needs a per-bag loop, an atomic or a second pass over the IDs, and the
// sub-bag starts (bag-major [table][sample][dst]) are written with coalesced stores.
#define BLS_RW_WORDS (BLS_RW_CHUNK / 32)
template <class Where>
__device__ __forceinline__ void rw_scatter_tile(const BlsParams p, const Where where)   // by value: the compiler then knows that no store changes a field
{
    extern __shared__ __align__(8) unsigned rw_smem[];  // the block's dynamic shared memory (rw_scatter_smem bytes)
    // layout: mp[P][WORDS + 1] (x = mask word, y = set bits before it) | id[CHUNK] | off[tile_bags + 1] | base[P]
    uint2 (*s_mp)[BLS_RW_WORDS + 1] = reinterpret_cast<uint2 (*)[BLS_RW_WORDS + 1]>(rw_smem);
    int *s_id = reinterpret_cast<int *>(rw_smem + 2 * (size_t)p.P * (BLS_RW_WORDS + 1));
    int *s_off = s_id + BLS_RW_CHUNK;
    int *s_base = s_off + p.tile_bags + 1;

    const int src = where.src();
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int t = where.tile() / p.tiles_per_table;
    const int s0 = (where.tile() - t * p.tiles_per_table) * p.tile_bags;
    const int nb = min(p.tile_bags, p.b - s0);
    const unsigned rows = (unsigned)p.tab[t].rows;
    const int blk = p.tab[t].blk;
    const unsigned magic = p.tab[t].magic;
    const long long g0 = ((long long)src * p.T + t) * p.b + s0;
    int lo, hi;
    tile_ends(p, c, g0, nb, lo, hi);
    const int n = hi - lo;
    // the IDs of a chunk are requested one chunk ahead and parked in registers
    int idr[BLS_RW_PER_THREAD];
    auto request = [&](int c0) {
        #pragma unroll
        for (int q = 0; q < BLS_RW_PER_THREAD; q++) {
            const int i = c0 + q * BLS_ROUTE_TB + tid;
            idr[q] = i < n ? __ldcs(c.ids + lo + i) : 0;
        }
    };
    request(0);
    // bag starts relative to the tile, forced into [0, n]; a bag that ends before it starts is reported
    for (int s = tid; s <= nb; s += BLS_ROUTE_TB) {
        const long long a = c.off[g0 + s];
        if (s < nb && n > 0 && a > (long long)c.off[g0 + s + 1]) flag(p, BLS_ST_EINVAL);
        s_off[s] = (int)min(max(a - lo, 0LL), (long long)n);
    }
    if (tid < p.P) s_base[tid] = p.tile_cnt[((size_t)src * p.NT + where.tile()) * p.P + tid];
    int *rows_out = c.sub_start + ((size_t)t * p.b + s0) * p.P;
    const unsigned lt = (1u << lane) - 1u;
    int s_lo = 0;                                       // first bag that starts in the current chunk

    for (int c0 = 0; c0 == 0 || c0 < n; c0 += BLS_RW_CHUNK) {
        const int nc = min(BLS_RW_CHUNK, n - c0);
        const int nw = (nc + 31) >> 5;
        const bool last = c0 + nc >= n;
        // classify: the chunk's IDs go to shared memory (range-checked), then per warp step
        // the lanes that share a destination find one another and one of them stores their
        // mask; destinations nobody goes to keep the zero written just before
        #pragma unroll
        for (int q = 0; q < BLS_RW_PER_THREAD; q++) {
            const int i = q * BLS_ROUTE_TB + tid;
            if (i < nc) s_id[i] = (unsigned)idr[q] < rows ? idr[q] : 0;   // out of range: reported by the count kernel
        }
        if (!last) request(c0 + BLS_RW_CHUNK);
        __syncthreads();                                // also: s_off and s_base are in place
        // bags that start in [c0, c0 + nc): the starts are sorted, so they are s_lo .. s_hi - 1
        // (the last chunk also takes the bags that start at its end)
        int s_hi = nb;
        if (!last) {
            int a = s_lo, e = nb;                       // first bag whose start is >= c0 + nc
            while (a < e) {
                const int m = (a + e) >> 1;
                if (s_off[m] < c0 + nc) a = m + 1; else e = m;
            }
            s_hi = a;
        }
        #pragma unroll 1
        for (int i = tid; i - lane < nc; i += BLS_ROUTE_TB) {           // the bound is the same for a whole warp
            if (lane < p.P) s_mp[lane][i >> 5].x = 0u;
            __syncwarp();
            if (i < nc) {
                int local;
                const int d = owner_of_row((unsigned)s_id[i], blk, magic, local);
                atomicOr(&s_mp[d][i >> 5].x, 1u << lane);                // measured: far cheaper than a warp match
            }
        }
        __syncthreads();
        // set bits before every word, one warp per destination (two words per lane)
        for (int d = w; d < p.P; d += BLS_ROUTE_TB / 32) {
            const int v0 = 2 * lane < nw ? __popc(s_mp[d][2 * lane].x) : 0;
            const int v1 = 2 * lane + 1 < nw ? __popc(s_mp[d][2 * lane + 1].x) : 0;
            int inc = v0 + v1;
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += y;
            }
            const int excl = inc - v0 - v1;
            if (2 * lane < nw) s_mp[d][2 * lane].y = (unsigned)excl;
            if (2 * lane + 1 < nw) s_mp[d][2 * lane + 1].y = (unsigned)(excl + v0);
            if (lane == 31) s_mp[d][nw] = make_uint2(0u, (unsigned)inc);   // closing entry: the chunk's total
        }
        __syncthreads();
        for (int i = tid; i < nc; i += BLS_ROUTE_TB) {
            int local;
            const int d = owner_of_row((unsigned)s_id[i], blk, magic, local);
            const uint2 mp = s_mp[d][i >> 5];
            const int pos = s_base[d] + (int)mp.y + __popc(mp.x & lt);
            if (pos < p.cap) c.sendbuf[pos] = local;    // measured: grouping in shared memory first is slower
        }
        // sub-bag starts of those bags (a bag's P entries are contiguous in the bag-major
        // layout).  P a multiple of 4: one thread per four destinations of a bag, so that a
        // warp's 16-byte stores cover one contiguous piece of the array; else one thread per entry.
        if ((p.P & 3) == 0) {
            const int qpb = p.P >> 2;                           // 16-byte pieces per bag
            for (int e = tid; e < (s_hi - s_lo) * qpb; e += BLS_ROUTE_TB) {
                const int s = s_lo + e / qpb, d = (e % qpb) * 4;
                const int x = min(max(s_off[s] - c0, 0), nc);
                const int wd = x >> 5;
                const unsigned below = (1u << (x & 31)) - 1u;
                auto start_of = [&](int dd) {
                    const uint2 mp = s_mp[dd][wd];
                    return min(s_base[dd] + (int)mp.y + __popc(mp.x & below), p.cap);
                };
                *reinterpret_cast<int4 *>(rows_out + (size_t)s * p.P + d) =
                    make_int4(start_of(d), start_of(d + 1), start_of(d + 2), start_of(d + 3));
            }
        } else {
            for (int e = tid; e < (s_hi - s_lo) * p.P; e += BLS_ROUTE_TB) {
                const int s = s_lo + e / p.P, d = e % p.P;
                const int x = min(max(s_off[s] - c0, 0), nc);
                const uint2 mp = s_mp[d][x >> 5];
                rows_out[(size_t)s * p.P + d] = min(s_base[d] + (int)mp.y + __popc(mp.x & ((1u << (x & 31)) - 1u)), p.cap);
            }
        }
        s_lo = s_hi;
        __syncthreads();
        if (tid < p.P) s_base[tid] += (int)s_mp[tid][nw].y;
        __syncthreads();
    }
    // the entries after the last bag of the requester close every destination's region
    if (where.tile() == p.NT - 1 && tid < p.P) c.sub_start[(size_t)p.T * p.b * p.P + tid] = min(s_base[tid], p.cap);
}


__host__ __device__ __forceinline__ size_t rw_scatter_smem(const BlsParams &p)
{
    return sizeof(uint2) * (size_t)p.P * (BLS_RW_WORDS + 1) + sizeof(int) * (BLS_RW_CHUNK + p.tile_bags + 1 + p.P);
}
