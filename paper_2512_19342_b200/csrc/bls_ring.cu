// Slot ring of the bounded-lag-synchronous exchange: per-rank progress counters
// in device memory, the gate that decides what every logical rank may do in the
// next wave of kernels, and the commit that publishes the wave's progress.
//
// Reading of the paper (Section III-C, III-D, Section IV / Listing 2):
//   * iteration j uses slot j mod S, S = k_max + 1 buffers created at plan time;
//   * a rank may put the requests of iteration j only when every rank has
//     completed iteration j - k - 1, i.e. min(done) >= j - k (Listing 2 notes that a
//     rank too far ahead would overwrite a buffer);
//   * an owner answers iteration j once all P sources have posted it (tagged
//     messages are counted per iteration);
//   * a rank completes iteration j once all owners have answered it; completion
//     is oldest first; the oldest request must complete once more than k are
//     outstanding; the last batch drains everything.
// Without injected delays all ranks act together, one wave of stand-alone kernels per
// step, planned by the gate below.  With injected delays the ranks act on their own,
// inside the persistent ring kernel of bls_event.cu, under the same rules.
#include "bls_device.cuh"

// Warp 0 decides (lane r is logical rank r).  With table-wise placement the block has
// one more warp per rank, which then runs the first half of the router for the ranks
// that were told to post (saves a launch on the critical path of every step).
// This gate plans one wave of stand-alone kernels and never waits: injected delays are
// the business of the event-driven ring kernel (bls_event.cu).
__device__ __forceinline__ void gate_warp(const BlsParams &p, int mode, long long t_last, long long floor_, int k,
                                          const int *ids, const int *off, long long n_ids, int overlapped)
{
    BlsDev *d = p.dev;
    const int r = threadIdx.x;
    const bool act = r < p.P;
    const long long BIG = 0x7fffffffffffffffLL;

    if (r == 0) { d->work_ctr = 0; d->done_ctr = 0; }
    if (p.hot.enabled)
        for (int i = r; i < p.NI; i += 32) p.hot.pair_ctr[i] = 0;
    if (p.part == BLS_PART_ROW_BLOCK && mode != BLS_MODE_LOOKUP_ONLY)
        for (int i = r; i < p.P * p.P; i += 32) p.rw_total[i] = 0;      // the count kernel adds the tiles' counts
    if (r == 0 && off != nullptr && (mode == BLS_MODE_STEP || mode == BLS_MODE_ROUTE_ONLY)) {
        int slot = (int)(t_last % p.S);
        d->in_ids[slot] = ids;
        d->in_off[slot] = off;
        d->in_n[slot] = n_ids;
    }
    __syncwarp();

    const long long posted = act ? d->posted[r] : BIG;
    const long long served = act ? d->served[r] : BIG;
    const long long done = act ? d->done[r] : BIG;
    const bool sync_mode = (mode == BLS_MODE_ROUTE_ONLY || mode == BLS_MODE_LOOKUP_ONLY);
    const long long min_done = warp_min_ll(done);

    // post: slot of iteration `posted` is free once every rank completed posted - k - 1
    bool go_r = act && mode != BLS_MODE_LOOKUP_ONLY && posted <= t_last && min_done >= posted - k;
    long long posted2 = act ? posted + (go_r ? 1 : 0) : BIG;
    const long long min_posted2 = warp_min_ll(posted2);
    const long long max_posted2 = warp_max_ll(act ? posted2 : -1);

    // serve: all P sources (self included) have posted the iteration.  In overlapped mode the
    // router of this wave runs beside the gather kernel, so only iterations posted by earlier
    // waves can be answered.
    const long long min_posted = warp_min_ll(posted);
    bool go_s = act && mode != BLS_MODE_ROUTE_ONLY && served < (overlapped ? min_posted : min_posted2);
    long long served2 = act ? served + (go_s ? 1 : 0) : BIG;
    const long long min_served2 = warp_min_ll(served2);

    // complete: all owners have answered; oldest first
    bool go_c = act && mode != BLS_MODE_ROUTE_ONLY && done < min_served2;
    long long done2 = act ? done + (go_c ? 1 : 0) : BIG;
    const long long min_done2 = warp_min_ll(done2);

    if (act) {
        d->route_iter[r] = go_r ? posted : -1;
        d->serve_iter[r] = go_s ? served : -1;
        d->consume_iter[r] = go_c ? done : -1;
    }
    if (r == 0) {
        long long lag = max_posted2 - 1 - min_done;
        if (lag > d->max_lag) d->max_lag = lag;
        // the wave must satisfy the bound: everything up to the floor completes
        if (!sync_mode && floor_ >= 0 && min_done2 <= floor_) atomicOr(&d->status, BLS_ST_ESTATE);
        if (mode == BLS_MODE_ROUTE_ONLY && min_posted2 <= t_last) atomicOr(&d->status, BLS_ST_ESTATE);
        if (mode == BLS_MODE_LOOKUP_ONLY && min_done2 <= t_last) atomicOr(&d->status, BLS_ST_ESTATE);
    }
}

__global__ void __launch_bounds__(1024) bls_gate_kernel(BlsParams p, int mode, long long t_last,
                                                        long long floor_, int k, const int *ids,
                                                        const int *off, long long n_ids, int overlapped)
{
    if (threadIdx.x < 32) gate_warp(p, mode, t_last, floor_, k, ids, off, n_ids, overlapped);
    // overlapped mode: the router's first half runs on the second stream too (bls_tw_meta_kernel)
    if (p.part != BLS_PART_TABLE_RR || mode == BLS_MODE_LOOKUP_ONLY || overlapped) return;
    __threadfence_block();
    __syncthreads();                                   // the wave plan is visible to the other warps
    const int w = threadIdx.x >> 5;
    if (w < p.P) tw_meta_warp(p, w, threadIdx.x & 31);
}

// The router's first half on its own (one warp per requester), for the overlapped mode.
__global__ void __launch_bounds__(1024) bls_tw_meta_kernel(BlsParams p)
{
    const int w = threadIdx.x >> 5;
    if (w < p.P) tw_meta_warp(p, w, threadIdx.x & 31);
}

void bls_launch_meta(const bls_plan_t *pl, cudaStream_t stream)
{
    bls_tw_meta_kernel<<<1, 32 * pl->prm.P, 0, stream>>>(pl->prm);
}

// One warp; publishes the progress of a wave that has no gather kernel at its end
// (bls_route); otherwise the last block of the gather kernel does this.
__global__ void __launch_bounds__(32) bls_commit_kernel(BlsParams p) { commit_lane(p, threadIdx.x); }

void bls_launch_gate(const bls_plan_t *pl, int mode, long long t_last, long long forced_floor, int k,
                     const int *ids, const int *off, long long n_ids, int overlapped)
{
    // table-wise: one warp per rank for the router's first half (warp 0 is also the gate)
    const bool meta = pl->prm.part == BLS_PART_TABLE_RR && mode != BLS_MODE_LOOKUP_ONLY && !overlapped;
    bls_gate_kernel<<<1, meta ? 32 * pl->prm.P : 32, 0, pl->stream>>>(pl->prm, mode, t_last, forced_floor, k, ids, off, n_ids, overlapped);
}

void bls_launch_commit(const bls_plan_t *pl)
{
    bls_commit_kernel<<<1, 32, 0, pl->stream>>>(pl->prm);
}
