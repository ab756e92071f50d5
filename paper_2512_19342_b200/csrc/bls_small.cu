// Small iterations in one launch.  An iteration of a few thousand lookups (the one-ID-per-table
// click-log shapes of Section V-F at small batch sizes) takes a few microseconds of memory
// latency, and a wave of three dependent kernels spends most of its time between launches.
// When the logical ranks move in lockstep (no injected delays) and placement is table-wise,
// nothing in an iteration needs a grid-wide barrier:
//   * the place of a (requester, table) chunk in the send buffer follows from the requester's
//     offsets alone, so every block works it out for itself (one warp, a scan over the
//     requester's tables) instead of waiting for a block that publishes it;
//   * a block routes its tile (IDs to the packed send buffer, sub-bag starts: the same
//     artefacts, bit for bit, as the stand-alone router) and then answers the same tile: its
//     lane groups stream the sub-bags they have just written, pool them and store the vectors
//     into the requester's output slot (the same device code as the stand-alone gather
//     kernel, so the sums carry the same bits);
//   * the block that finishes last publishes the iteration for all ranks: receive-side
//     counts, the three counters of every rank, the time stamps.
// Every block first checks that all ranks have completed exactly the iterations before this
// one; if not, nothing is written and BLS_ESTATE is latched.
#include "bls_route.cuh"
#include "bls_gather.cuh"

template <int LANES, int DT>
__global__ void __launch_bounds__(BLS_ROUTE_TB)
bls_small_tw_kernel(BlsParams p, long long t, const int *ids, const int *off, long long n_ids)
{
    __shared__ int s_meta[3];                          // ranks in lockstep?  start and end of the block's chunk
    __shared__ int s_last;
    stream_order_enter();                              // launched with launch_serialised()
    BlsDev *d = p.dev;
    const int src = blockIdx.y;
    const int i = blockIdx.x / p.tiles_per_table;      // (owner, table) pair of the tile
    const int s0 = (blockIdx.x % p.tiles_per_table) * p.tile_bags;
    const int nb = min(p.tile_bags, p.b - s0);
    const int slot = (int)(t % p.S);
    RouteCtx c;
    c.ids = ids;
    c.off = off;
    c.n_ids = n_ids;
    c.slot = slot;
    {
        int *cnt = p.counts + (size_t)slot * 4 * p.P * p.P;
        c.sendcounts = cnt + src * p.P;
        c.sdispls = cnt + p.P * p.P + src * p.P;
        c.sendbuf = p.sendbuf + ((size_t)slot * p.P + src) * (size_t)p.cap;
        c.sub_start = p.sub_start + ((size_t)slot * p.P + src) * (size_t)p.sub_stride;
    }

    if (threadIdx.x < 32) {
        const int r = threadIdx.x;
        const bool in_step = r >= p.P || (d->posted[r] == t && d->served[r] == t && d->done[r] == t);
        const bool ok = __all_sync(0xffffffffu, in_step);
        int cb = 0, ce = 0;
        if (ok) tw_meta_ctx(p, c, src, r, blockIdx.x == 0, i, cb, ce);   // the requester's first block also publishes
        if (r == 0) { s_meta[0] = ok; s_meta[1] = cb; s_meta[2] = ce; }
    }
    __syncthreads();
    const bool ok = s_meta[0] != 0;
    if (ok) {
        const BlsPairDesc pr = p.pair[i];
        const int cb = s_meta[1];
        const int hi = tw_copy_ctx<8>(p, c, src, i, pr.t, s0, nb, cb, s_meta[2] - cb);
        __syncthreads();                               // the tile's IDs and sub-bag starts are in place
        constexpr int G = BLS_ROUTE_TB / LANES;        // lane groups of the block
        const int R = (nb + G - 1) / G;                // consecutive sub-bags per lane group
        const int r0 = (threadIdx.x / LANES) * R;
        if (r0 < nb) {
            const int n = min(R, nb - r0);
            // the sub-bag after the tile belongs to another block: the tile's end is known here
            const int end_pos = r0 + n == nb ? (int)min((long long)cb + hi, (long long)p.cap) : -1;
            stream_run<LANES, DT, 4, false>(p, pr, i, slot, src, s0 + r0, n, threadIdx.x % LANES, nullptr, end_pos);
        }
    }

    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&d->small_ctr, 1) == (int)(gridDim.x * gridDim.y) - 1;
    }
    __syncthreads();
    if (!s_last || threadIdx.x >= 32) return;
    __threadfence();
    const int r = threadIdx.x;
    const unsigned long long now = __shfl_sync(0xffffffffu, globaltimer_ns(), 0);   // one time for all ranks
    if (!ok) {
        if (r == 0) flag(p, BLS_ST_ESTATE);
    } else if (r < p.P) {
        write_recv_side(p, r, t);
        d->posted[r] = t + 1;
        d->served[r] = t + 1;
        d->done[r] = t + 1;
        stamp(p, t, r, 0, now);
        stamp(p, t, r, 1, now);
        stamp(p, t, r, 2, now);
    }
    if (r == 0) {
        d->in_ids[slot] = ids;
        d->in_off[slot] = off;
        d->in_n[slot] = n_ids;
        d->small_ctr = 0;
    }
}

template <int LANES, int DT>
static void launch_small_kernel(const bls_plan_t *pl, long long t, const int *ids, const int *off, long long n_ids)
{
    launch_serialised(bls_small_tw_kernel<LANES, DT>, dim3(pl->prm.NT, pl->prm.P), dim3(BLS_ROUTE_TB), pl->stream,
                      pl->prm, t, ids, off, n_ids);
}

template <int DT>
static void launch_small_dt(const bls_plan_t *pl, long long t, const int *ids, const int *off, long long n_ids)
{
    switch (pl->prm.lanes) {
    case 1: launch_small_kernel<1, DT>(pl, t, ids, off, n_ids); break;
    case 2: launch_small_kernel<2, DT>(pl, t, ids, off, n_ids); break;
    case 4: launch_small_kernel<4, DT>(pl, t, ids, off, n_ids); break;
    case 8: launch_small_kernel<8, DT>(pl, t, ids, off, n_ids); break;
    case 16: launch_small_kernel<16, DT>(pl, t, ids, off, n_ids); break;
    default: launch_small_kernel<32, DT>(pl, t, ids, off, n_ids); break;
    }
}

void bls_launch_small(const bls_plan_t *pl, long long t, const int *ids, const int *off, long long n_ids)
{
    switch (pl->prm.dtype) {
    case BLS_F32: launch_small_dt<BLS_F32>(pl, t, ids, off, n_ids); break;
    case BLS_BF16: launch_small_dt<BLS_BF16>(pl, t, ids, off, n_ids); break;
    default: launch_small_dt<BLS_F16>(pl, t, ids, off, n_ids); break;
    }
}
