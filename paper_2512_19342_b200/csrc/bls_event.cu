// Event-driven mode of the slot ring: one persistent kernel per bls_step / bls_drain call
// in which every logical rank advances on its own.
//
// Reading of the paper (Section III-C: initiation never synchronises two processes;
// Section III-D: any two processes are at most k iterations apart; Section IV, Listing 2:
// the loop of a BLS-enabled rank).  Each rank r runs Listing 2's loop as a small state
// machine: spend the injected delay of iteration j (Section V-E setting 2: a delay models
// a slowdown of any nature) -> complete every outstanding request whose data has arrived,
// oldest first -> wait until the slot of j is free (every rank has completed j - k - 1)
// -> post j (route its IDs) -> complete what has arrived and, while more than k requests
// are outstanding, block on the oldest -> next iteration.  An owner answers iteration j
// (gather, pool, return) as soon as all P ranks have posted it, whatever its own loop is
// doing: the data "arrives" the way a one-sided put does.  After the last iteration the
// outstanding requests complete in order as they arrive.
//
// On one GPU the ranks cannot be separate kernels that wait for one another.  They are
// one cooperative launch instead: warp 0 of block 0 is the scheduler (lane r = rank r);
// it watches the clock, the counters and the actions in flight, and publishes *actions*
// - the router's phases for one requester, the gather of one owner - into a queue in
// device memory; every other block is a worker that claims tiles of published actions
// and runs the same device code as the stand-alone kernels.  Nothing waits on another
// launch; every wait in here is bounded by the clock and ends in BLS_ETIMEOUT.
#include "bls_route.cuh"
#include "bls_gather.cuh"

namespace {

constexpr int RING_GATHER_CHUNK = 8;    // warp-sized pieces of work per gather tile (a block has 4 warps)

struct RingArgs {
    int mode;                   // BLS_MODE_STEP or BLS_MODE_DRAIN
    int k;
    long long t_last;           // newest iteration whose inputs exist
    long long floor_;           // iteration that must be complete on every rank before the launch ends, or -1
    const int *ids, *off;       // inputs of iteration t_last (BLS_MODE_STEP)
    long long n_ids;
    int R, rpc;                 // gather: bags per run, runs per (owner, table, requester) chunk
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned *p, unsigned v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_relaxed(const int *p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Every block leaves through here; the last one clears the queue header for the next launch.
__device__ __forceinline__ void ring_leave(const BlsParams &p)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        BlsQueue *q = p.queue;
        __threadfence();
        if (atomicAdd(&q->exited, 1) == (int)gridDim.x - 1) {
            q->tail = 0;
            q->exit = 0;
            __threadfence();
            q->exited = 0;
        }
    }
}

// ------------------------------------------------------------------ workers
template <int LANES, int DT, int PART>
__device__ __forceinline__ void ring_worker(const BlsParams &p, const RingArgs &a)
{
    constexpr int GPW = 32 / LANES;                    // runs per warp
    constexpr int RPT = RING_GATHER_CHUNK * GPW;       // runs per gather tile
    __shared__ int s_q, s_tile, s_ctr;
    BlsQueue *q = p.queue;
    unsigned cur = 0;                                  // oldest action that may still have tiles (thread 0 only)
    unsigned acquired = 0;                             // actions below this index were published before this block's last acquire
    // a worker gives up long after the scheduler would have (its limit covers the scheduler's two stages)
    const unsigned long long limit = 4ull * p.dev->wait_limit_ns + 1000000000ull;
    const int lane = threadIdx.x % LANES;
    const int g = (threadIdx.x & 31) / LANES;
    for (;;) {
        if (threadIdx.x == 0) {
            int got = -1, tile = 0;
            const unsigned long long t0 = globaltimer_ns();
            unsigned spins = 0;
            for (;;) {
                // The tail is polled with a relaxed load; an acquire (which also drops the SM's L1 lines, and
                // with them the cached hot rows of every block on this SM) is paid once per action, before
                // the first tile of an action published after this block's last acquire.
                unsigned tail = (unsigned)ld_relaxed((const int *)&q->tail);
                if (cur < tail) {
                    if (cur >= acquired) {
                        tail = ld_acquire(&q->tail);
                        acquired = tail;
                    }
                    BlsAct *e = &q->act[cur];
                    const int n = e->n_tiles;
                    int t = n;
                    if (ld_relaxed(&e->next) < n) t = atomicAdd(&e->next, 1);
                    if (t < n) { got = (int)cur; tile = t; break; }
                    cur++;
                    continue;
                }
                if (ld_relaxed(&q->exit)) break;
                __nanosleep(spins < 32 ? 20 : 200);
                if ((++spins & 255u) == 0 && globaltimer_ns() - t0 > limit) {
                    flag(p, BLS_ST_ETIMEOUT);
                    break;
                }
            }
            s_q = got;
            s_tile = tile;
            s_ctr = 0;
        }
        __syncthreads();
        const int qi = s_q;
        const unsigned tile = (unsigned)s_tile;
        if (qi < 0) break;
        const BlsAct *e = &q->act[qi];
        const int kind = e->kind, rank = e->rank;
        if constexpr (PART == BLS_PART_TABLE_RR) {
            if (kind == BLS_ACT_TW_META) {
                if (threadIdx.x < 32) tw_meta_warp(p, rank, threadIdx.x);
            } else if (kind == BLS_ACT_TW_COPY) {
                tw_copy_tile<8>(p, TileGiven{tile, (unsigned)rank});
            } else if (kind == BLS_ACT_GATHER_TW) {
                // a gather tile is RING_GATHER_CHUNK warp-sized pieces; the block's warps take them one by one
                // (runs differ in length: a fixed split would leave warps idle behind the longest)
                for (;;) {
                    int piece = 0;
                    if ((threadIdx.x & 31) == 0) piece = atomicAdd(&s_ctr, 1);
                    piece = __shfl_sync(0xffffffffu, piece, 0);
                    if (piece >= RING_GATHER_CHUNK) break;
                    const int run = (int)tile * RPT + piece * GPW + g;   // among the owner's runs, pair-major
                    if (run < e->aux) {
                        const int chunk = run / a.rpc;                   // (pair of the owner, requester)
                        const int s0 = (run - chunk * a.rpc) * a.R;
                        const int i = e->first + chunk / p.P, src = chunk % p.P;
                        const BlsPairDesc pr = p.pair[i];
                        stream_run<LANES, DT, 4, false>(p, pr, i, e->slot, src, s0, min(a.R, p.b - s0), lane, nullptr);
                    }
                    __syncwarp();
                }
            }
        } else {
            if (kind == BLS_ACT_RW_COUNT) rw_count_tile(p, TileGiven{tile, (unsigned)rank});
            else if (kind == BLS_ACT_RW_SCAN) rw_scan_tile(p, TileGiven{tile, (unsigned)rank});
            else if (kind == BLS_ACT_RW_SCATTER) rw_scatter_tile(p, TileGiven{tile, (unsigned)rank});
            else if (kind == BLS_ACT_GATHER_RW) {
                for (;;) {
                    int piece = 0;
                    if ((threadIdx.x & 31) == 0) piece = atomicAdd(&s_ctr, 1);
                    piece = __shfl_sync(0xffffffffu, piece, 0);
                    if (piece >= RING_GATHER_CHUNK) break;
                    const int run = (int)tile * RPT + piece * GPW + g;
                    if (run < e->aux) rowwise_run<LANES, DT>(p, e->slot, run, a.R, a.rpc, lane, g);
                    __syncwarp();
                }
            }
        }
        __syncthreads();                               // the whole tile is done (and s_q, s_tile have been read)
        if (threadIdx.x == 0) {
            __threadfence();
            atomicAdd(&q->act[qi].finished, 1);
        }
    }
}

// ---------------------------------------------------------------- scheduler
// Publish one action per lane that has one (warp-collective).  Returns the lane's queue
// index, or -1.  The entries are written first, then the new tail is released.
__device__ __forceinline__ int ring_publish(const BlsParams &p, unsigned &tail, bool has, int kind, int rank, int slot,
                                            int n_tiles, int aux, int first, bool &fatal)
{
    const unsigned m = __ballot_sync(0xffffffffu, has);
    if (!m) return -1;
    const unsigned lane = threadIdx.x & 31;
    const unsigned idx = tail + __popc(m & ((1u << lane) - 1u));
    const unsigned new_tail = tail + __popc(m);
    if (new_tail > BLS_Q_CAP) {                        // cannot happen within the plan's limits; never overrun the queue
        if (lane == 0) flag(p, BLS_ST_ESTATE);
        fatal = true;
        return -1;
    }
    if (has) {
        BlsAct *e = &p.queue->act[idx];
        e->kind = kind; e->rank = rank; e->slot = slot; e->n_tiles = n_tiles;
        e->next = 0; e->finished = 0; e->aux = aux; e->first = first;
        __threadfence();
    }
    __syncwarp();
    tail = new_tail;
    if (lane == 0) st_release(&p.queue->tail, tail);
    return has ? (int)idx : -1;
}

template <int LANES, int PART>
__device__ __forceinline__ void ring_scheduler(const BlsParams &p, const RingArgs &a)
{
    constexpr bool TW = PART == BLS_PART_TABLE_RR;
    constexpr int RPT = RING_GATHER_CHUNK * (32 / LANES);
    BlsDev *d = p.dev;
    BlsQueue *q = p.queue;
    const int r = threadIdx.x;                         // lane = logical rank
    const bool act = r < p.P;
    const long long BIG = 0x7fffffffffffffffLL;
    const int k = a.k;

    if (r == 0 && a.off != nullptr && a.mode == BLS_MODE_STEP) {
        const int slot = (int)(a.t_last % p.S);
        d->in_ids[slot] = a.ids;
        d->in_off[slot] = a.off;
        d->in_n[slot] = a.n_ids;
    }
    long long posted = act ? d->posted[r] : BIG;
    long long served = act ? d->served[r] : BIG;
    long long done = act ? d->done[r] : BIG;
    int rstate = act ? d->rstate[r] : BLS_RS_DELAY;
    unsigned long long ready_ns = act ? d->ready_ns[r] : ~0ull;
    const unsigned long long wait_limit = d->wait_limit_ns;
    // the owner's share of the gather (table-wise): its (owner, table) pairs
    int own_first = 0, own_runs = 0;
    if (TW && act) {
        own_first = p.pair_first[r];
        own_runs = (p.pair_first[r + 1] - own_first) * p.P * a.rpc;
    }
    const int rw_runs = TW ? 0 : p.T * p.P * a.rpc;
    int post_q = -1, post_n = 0, post_phase = 0;       // router action in flight for this rank
    int serve_q = -1, serve_n = 0;                     // gather action in flight (row-wise: lane 0 holds the one action)
    unsigned tail = 0;
    bool fatal = false, ignore_delays = false;
    unsigned long long t_progress = globaltimer_ns();
    long long fin_seen = 0;
    __syncwarp();

    for (;;) {
        const unsigned long long now = globaltimer_ns();
        bool changed = false;

        // (1) router phases that have finished: next phase, or the post is complete
        bool next_phase = false;
        long long fin_sum = 0;
        if (post_q >= 0) {
            const int f = ld_acquire(&q->act[post_q].finished);
            fin_sum += f;
            if (f >= post_n) {
                const int last_phase = TW ? 1 : 2;
                if (post_phase < last_phase) {
                    post_phase++;
                    next_phase = true;
                } else {
                    stamp(p, posted, r, 0, now);
                    posted++;
                    d->posted[r] = posted;
                    post_q = -1;
                    rstate = BLS_RS_AFTER_POST;
                }
                changed = true;
            }
        }
        // (2) gathers that have finished: the owner has answered the iteration
        bool serve_fin = false;
        if (serve_q >= 0) {
            const int f = ld_acquire(&q->act[serve_q].finished);
            fin_sum += f;
            serve_fin = f >= serve_n;
        }
        if (!TW) serve_fin = __shfl_sync(0xffffffffu, serve_fin, 0);   // one action for all owners
        if (act && serve_fin) {
            write_recv_side(p, r, served);
            stamp(p, served, r, 1, now);
            served++;
            d->served[r] = served;
            serve_q = -1;
            changed = true;
        }

        // (3) the end of a delay, and the completions a rank makes at the points of its loop
        if (rstate == BLS_RS_DELAY && (now >= ready_ns || ignore_delays)) {
            rstate = BLS_RS_WANT_POST;
            changed = true;
        }
        const long long min_served = warp_min_ll(served);
        const bool loop_point = rstate != BLS_RS_DELAY && rstate != BLS_RS_POSTING;
        const bool all_posted = a.mode == BLS_MODE_DRAIN && posted > a.t_last;   // last batch: the rest completes as it arrives
        if (act && (loop_point || all_posted)) {
            while (done < min_served) {                // oldest first
                stamp(p, done, r, 2, now);
                done++;
                changed = true;
            }
            d->done[r] = done;
        }
        // (4) after a post: go on once at most k requests are outstanding, and start the next delay
        if (rstate == BLS_RS_AFTER_POST && posted - done <= k) rstate = BLS_RS_IDLE;
        if (act && rstate == BLS_RS_IDLE) {
            const unsigned long long dl = ignore_delays ? 0ull : stall_draw(d, r, posted);
            ready_ns = now + dl;
            rstate = dl ? BLS_RS_DELAY : BLS_RS_WANT_POST;
            changed = true;
        }
        // (5) post: the slot of iteration `posted` is free once every rank has completed posted - k - 1
        const long long min_done = warp_min_ll(done);
        const bool go_post = act && rstate == BLS_RS_WANT_POST && posted <= a.t_last && min_done >= posted - k;
        if (go_post) {
            d->route_iter[r] = posted;
            if (!TW)
                for (int i = 0; i < p.P; i++) p.rw_total[r * p.P + i] = 0;   // the count tiles add to these
            post_phase = 0;
            rstate = BLS_RS_POSTING;
            changed = true;
        }
        {
            const bool has = go_post || next_phase;
            int kind, n;
            if (TW) { kind = post_phase == 0 ? BLS_ACT_TW_META : BLS_ACT_TW_COPY; n = post_phase == 0 ? 1 : p.NT; }
            else {
                kind = post_phase == 0 ? BLS_ACT_RW_COUNT : post_phase == 1 ? BLS_ACT_RW_SCAN : BLS_ACT_RW_SCATTER;
                n = post_phase == 1 ? p.P : p.NT;
            }
            const int idx = ring_publish(p, tail, has, kind, r, (int)(posted % p.S), n, 0, 0, fatal);
            if (has) { post_q = idx; post_n = n; }
        }
        // (6) serve: all P sources (self included) have posted the iteration
        const long long min_posted = warp_min_ll(posted);
        {
            bool go = act && serve_q < 0 && served < min_posted;
            if (!TW) go = __shfl_sync(0xffffffffu, go, 0) && r == 0;
            const int runs = TW ? own_runs : rw_runs;
            const int n = (runs + RPT - 1) / RPT;
            const int idx = ring_publish(p, tail, go, TW ? BLS_ACT_GATHER_TW : BLS_ACT_GATHER_RW, r, (int)(served % p.S), n,
                                         runs, own_first, fatal);
            if (go) { serve_q = idx; serve_n = n; changed = true; }   // an owner without tables: n = 0, finished at once
        }
        // (7) the largest distance between the newest posted and the oldest incomplete iteration
        {
            const long long newest = warp_max_ll(act ? posted + (post_q >= 0 ? 1 : 0) : -1);
            if (r == 0 && newest - 1 - min_done > d->max_lag) d->max_lag = newest - 1 - min_done;
        }
        // (8) leave once the call's obligation is met, nothing is in flight and nobody can act right now
        const bool any_changed = __any_sync(0xffffffffu, changed);
        const bool inflight = __any_sync(0xffffffffu, post_q >= 0 || serve_q >= 0);
        const bool obliged = a.floor_ >= 0 && min_done <= a.floor_;
        if (fatal || (!obliged && !inflight && !any_changed)) break;
        // (9) bounded waiting: no progress for longer than the limit -> report, stop honouring delays;
        //     still none after that -> give up
        fin_sum = __reduce_add_sync(0xffffffffu, (int)fin_sum);
        if (any_changed || fin_sum != fin_seen) {
            t_progress = now;
            fin_seen = fin_sum;
        } else if (now - t_progress > wait_limit) {
            if (r == 0) flag(p, BLS_ST_ETIMEOUT);
            if (ignore_delays) break;
            ignore_delays = true;
            t_progress = now;
        } else {
            __nanosleep(100);
        }
    }
    if (act) {
        d->rstate[r] = rstate == BLS_RS_POSTING ? BLS_RS_WANT_POST : rstate;   // (only after a give-up)
        d->ready_ns[r] = ready_ns;
    }
    __syncwarp();
    if (r == 0) {
        __threadfence();
        atomicExch(&q->exit, 1);
    }
}

template <int LANES, int DT, int PART>
__global__ void __launch_bounds__(BLS_ROUTE_TB, PART == BLS_PART_TABLE_RR ? 6 : 8)
bls_ring_kernel(BlsParams p, RingArgs a)
{
    if (blockIdx.x == 0) {
        if (threadIdx.x < 32) ring_scheduler<LANES, PART>(p, a);
    } else {
        ring_worker<LANES, DT, PART>(p, a);
    }
    ring_leave(p);
}

template <int LANES, int DT, int PART>
cudaError_t launch_ring(bls_plan_t *pl, RingArgs &a)
{
    const BlsParams &p = pl->prm;
    auto kernel = bls_ring_kernel<LANES, DT, PART>;
    const size_t smem = PART == BLS_PART_ROW_BLOCK ? rw_scatter_smem(p) : 0;
    if (!pl->ring_blocks_per_sm) {
        int nb = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kernel, BLS_ROUTE_TB, smem);
        if (e != cudaSuccess) return e;
        if (nb < 1) return cudaErrorLaunchOutOfResources;
        pl->ring_blocks_per_sm = nb;
    }
    // as many blocks as stay resident together (a cooperative launch: the workers wait for the
    // scheduler), fewer when the iteration has fewer tiles than that
    constexpr int RPT = RING_GATHER_CHUNK * (32 / LANES);
    const long long gather_tiles = ((long long)(PART == BLS_PART_TABLE_RR ? p.NI : p.T) * p.P * a.rpc + RPT - 1) / RPT + p.P;
    const long long route_tiles = (long long)p.NT * p.P;
    long long want = (gather_tiles > route_tiles ? gather_tiles : route_tiles) + 1;
    const long long most = (long long)pl->ring_blocks_per_sm * pl->sm_count;
    if (want > most) want = most;
    if (want < 2) want = 2;
    void *args[] = {(void *)&pl->prm, (void *)&a};
    return cudaLaunchCooperativeKernel((void *)kernel, dim3((unsigned)want), dim3(BLS_ROUTE_TB), args, smem, pl->stream);
}

template <int LANES, int DT>
cudaError_t launch_ring_part(bls_plan_t *pl, RingArgs &a)
{
    return pl->prm.part == BLS_PART_TABLE_RR ? launch_ring<LANES, DT, BLS_PART_TABLE_RR>(pl, a)
                                             : launch_ring<LANES, DT, BLS_PART_ROW_BLOCK>(pl, a);
}

template <int DT>
cudaError_t launch_ring_dt(bls_plan_t *pl, RingArgs &a)
{
    switch (pl->prm.lanes) {
    case 1: return launch_ring_part<1, DT>(pl, a);
    case 2: return launch_ring_part<2, DT>(pl, a);
    case 4: return launch_ring_part<4, DT>(pl, a);
    case 8: return launch_ring_part<8, DT>(pl, a);
    case 16: return launch_ring_part<16, DT>(pl, a);
    default: return launch_ring_part<32, DT>(pl, a);
    }
}

}  // namespace

int bls_launch_ring(bls_plan_t *pl, int mode, long long t_last, long long floor_, int k, const int *ids,
                    const int *off, long long n_ids)
{
    RingArgs a;
    a.mode = mode; a.k = k; a.t_last = t_last; a.floor_ = floor_;
    a.ids = ids; a.off = off; a.n_ids = n_ids;
    bls_gather_tiling(pl, &a.R, &a.rpc);
    switch (pl->prm.dtype) {
    case BLS_F32: return (int)launch_ring_dt<BLS_F32>(pl, a);
    case BLS_BF16: return (int)launch_ring_dt<BLS_BF16>(pl, a);
    default: return (int)launch_ring_dt<BLS_F16>(pl, a);
    }
}
