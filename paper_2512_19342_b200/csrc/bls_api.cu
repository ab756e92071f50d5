// Host side of the C ABI: workspace layout, plan construction, and the calls
// that enqueue one wave of kernels (gate -> route -> gather/pool/return -> commit).
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <vector>
#include "bls_internal.h"

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    size_t dev, tab, pair, pair_of, pair_first, counts, sendbuf, sub_start, out, chunk_base, tile_cnt, rw_total, queue,
        stamps, stage_ids, stage_off, total;
};

int dtype_bytes(int dt) { return dt == BLS_F32 ? 4 : 2; }

bls_status_t check_shape(const bls_table_t *tables, int T, int part, int P, int b, int k_max,
                         int64_t cap)
{
    if (!tables || T < 1 || P < 1 || P > BLS_MAX_RANKS || b < 1 || k_max < 0 ||
        k_max + 1 > BLS_MAX_SLOTS || cap < 1 || cap > 0x7ffffff0)
        return BLS_EINVAL;
    if (part != BLS_PART_TABLE_RR && part != BLS_PART_ROW_BLOCK) return BLS_EINVAL;
    const int D = tables[0].dim, dt = tables[0].dtype;
    if (dt != BLS_F32 && dt != BLS_BF16 && dt != BLS_F16) return BLS_EINVAL;
    const int rb = D * dtype_bytes(dt);
    if (rb != 16 && rb != 32 && rb != 64 && rb != 128 && rb != 256 && rb != 512) return BLS_EINVAL;
    for (int t = 0; t < T; t++) {
        if (tables[t].dim != D || tables[t].dtype != dt) return BLS_EINVAL;
        if (tables[t].rows < 1 || tables[t].rows > 0x7fffffff) return BLS_EINVAL;
    }
    const long long NI = part == BLS_PART_TABLE_RR ? T : (long long)T * P;
    if (NI * b > 0x7ffffff0LL || (long long)P * T * b > 0x7ffffff0LL) return BLS_EINVAL;
    return BLS_OK;
}

void fill_params(BlsParams &p, const bls_table_t *tables, int T, int part, int P, int b, int k_max,
                 int64_t cap)
{
    memset(&p, 0, sizeof(p));
    p.P = P; p.T = T; p.b = b; p.part = part; p.S = k_max + 1;
    p.D = tables[0].dim; p.dtype = tables[0].dtype;
    p.row_bytes = p.D * dtype_bytes(p.dtype);
    p.lanes = p.row_bytes / 16;
    p.NI = part == BLS_PART_TABLE_RR ? T : T * P;
    p.NQ = p.NI * b;
    p.cap = (int)((cap + 3) / 4 * 4);          // every rank's send buffer starts on a 16-byte boundary
    // Routing tiles of BLS_ROUTE_TB bags or a power-of-two multiple.
    // Table-wise: a tile is only copied, so it grows for short bags until a block moves
    // 2048 IDs or more, as long as enough tiles remain to fill the GPU.
    // Row-wise: up to 2048 bags (a tile is routed 2048 lookups at a time by one block, which
    // requests the next 2048 while it works), fewer when the tiles would not fill the GPU.
    p.tile_bags = BLS_ROUTE_TB;
    if (part == BLS_PART_ROW_BLOCK) {
        while (p.tile_bags < b && p.tile_bags < 2048 &&
               (long long)T * P * ((b + 2 * p.tile_bags - 1) / (2 * p.tile_bags)) >= 1024)
            p.tile_bags *= 2;
    }
    if (part == BLS_PART_TABLE_RR) {
        const double avg = (double)cap / ((double)p.NI * b);
        while (p.tile_bags < b && p.tile_bags * avg < 2048.0 &&
               (long long)T * P * ((b + 2 * p.tile_bags - 1) / (2 * p.tile_bags)) >= 2048)
            p.tile_bags *= 2;
    }
    p.tiles_per_table = (b + p.tile_bags - 1) / p.tile_bags;
    p.NT = T * p.tiles_per_table;
    // table-wise: NQ starts + 1 terminal entry; row-wise (bag-major): NQ starts + P terminal entries
    p.sub_stride = (long long)align_up((size_t)p.NQ + (part == BLS_PART_TABLE_RR ? 1 : P), 4);
    p.out_slot_elems = (long long)P * b * T * p.D;
}

Layout make_layout(const BlsParams &p)
{
    Layout L;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const size_t S = p.S, P = p.P;
    L.dev = take(sizeof(BlsDev));
    L.tab = take(sizeof(BlsTableDesc) * p.T);
    L.pair = take(sizeof(BlsPairDesc) * p.NI);
    L.pair_of = take(sizeof(int) * p.T);
    L.pair_first = take(sizeof(int) * (p.P + 1));
    L.counts = take(sizeof(int) * S * 4 * P * P);
    L.sendbuf = take(sizeof(int) * S * P * (size_t)p.cap);
    L.sub_start = take(sizeof(int) * S * P * (size_t)p.sub_stride);
    L.out = take(sizeof(float) * S * (size_t)p.out_slot_elems);
    L.chunk_base = take(sizeof(int) * P * (size_t)(p.NI + 1));
    L.tile_cnt = take(p.part == BLS_PART_ROW_BLOCK ? sizeof(int) * P * (size_t)p.NT * P : 0);
    L.rw_total = take(p.part == BLS_PART_ROW_BLOCK ? sizeof(int) * P * P : 0);
    L.queue = take(sizeof(BlsQueue));
    L.stamps = take(sizeof(unsigned long long) * BLS_TL_ITERS * P * 3);
    L.stage_ids = take(sizeof(int) * S * P * (size_t)p.cap);
    L.stage_off = take(sizeof(int) * S * ((size_t)P * p.T * p.b + 1));
    L.total = o;
    return L;
}

bool cuda_ok(cudaError_t e) { return e == cudaSuccess; }

}  // namespace

extern "C" {

const char *bls_strerror(int s)
{
    switch (s) {
    case BLS_OK: return "ok";
    case BLS_EINVAL: return "invalid argument or malformed offsets";
    case BLS_ENOSPC: return "workspace or per-rank ID capacity too small";
    case BLS_ECUDA: return "CUDA runtime error";
    case BLS_ERANGE: return "ID out of range";
    case BLS_ETIMEOUT: return "bounded device-side wait expired";
    case BLS_ESTATE: return "call order violated or bound out of range";
    default: return "unknown status";
    }
}

bls_status_t bls_plan_bytes(const bls_table_t *tables, int T, int part, int P, int local_batch,
                            int k_max, int64_t max_ids_per_rank, size_t *bytes)
{
    if (!bytes) return BLS_EINVAL;
    bls_status_t st = check_shape(tables, T, part, P, local_batch, k_max, max_ids_per_rank);
    if (st != BLS_OK) return st;
    BlsParams p;
    fill_params(p, tables, T, part, P, local_batch, k_max, max_ids_per_rank);
    *bytes = make_layout(p).total;
    return BLS_OK;
}

bls_status_t bls_plan(const bls_table_t *tables, int T, int part, int P, int local_batch, int k_max,
                      int64_t max_ids_per_rank, void *workspace, size_t bytes, void *cuda_stream,
                      bls_plan_t **plan)
{
    if (!plan || !workspace || ((uintptr_t)workspace & 255)) return BLS_EINVAL;
    bls_status_t st = check_shape(tables, T, part, P, local_batch, k_max, max_ids_per_rank);
    if (st != BLS_OK) return st;
    for (int t = 0; t < T; t++)
        if (!tables[t].weight || ((uintptr_t)tables[t].weight & 15)) return BLS_EINVAL;
    bls_plan_t *pl = (bls_plan_t *)calloc(1, sizeof(bls_plan_t));
    if (!pl) return BLS_ENOSPC;
    BlsParams &p = pl->prm;
    fill_params(p, tables, T, part, P, local_batch, k_max, max_ids_per_rank);
    Layout L = make_layout(p);
    if (bytes < L.total) { free(pl); return BLS_ENOSPC; }
    char *ws = (char *)workspace;
    p.dev = (BlsDev *)(ws + L.dev);
    p.tab = (const BlsTableDesc *)(ws + L.tab);
    p.pair = (const BlsPairDesc *)(ws + L.pair);
    p.pair_of_table = (const int *)(ws + L.pair_of);
    p.pair_first = (const int *)(ws + L.pair_first);
    p.counts = (int *)(ws + L.counts);
    p.sendbuf = (int *)(ws + L.sendbuf);
    p.sub_start = (int *)(ws + L.sub_start);
    p.out = (float *)(ws + L.out);
    p.chunk_base = (int *)(ws + L.chunk_base);
    p.tile_cnt = (int *)(ws + L.tile_cnt);
    p.rw_total = (int *)(ws + L.rw_total);
    p.queue = (BlsQueue *)(ws + L.queue);
    p.stamps = (unsigned long long *)(ws + L.stamps);
    p.stage_ids = (int *)(ws + L.stage_ids);
    p.stage_off = (int *)(ws + L.stage_off);
    pl->stream = (cudaStream_t)cuda_stream;
    pl->k_max = k_max;
    pl->k_cur = -1;
    pl->routed_only = -1;
    pl->bytes = L.total;
    pl->h_rows = (long long *)malloc(sizeof(long long) * T);
    if (!pl->h_rows) { free(pl); return BLS_ENOSPC; }
    for (int t = 0; t < T; t++) pl->h_rows[t] = tables[t].rows;
    {   // Run length: long enough to amortise the start of a run, short enough to balance the
        // tail.  Measured optima: about 160 rows (8 bags) for 20-row bags, 16-32 bags for 2-row
        // bags, 4-6 bags of 10 rows for row-wise placement.
        const bool tw = part == BLS_PART_TABLE_RR;
        double avg = (double)max_ids_per_rank / ((double)(tw ? p.NI : T) * local_batch);
        int R = (int)((tw ? 160.0 : 50.0) / (avg < 0.5 ? 0.5 : avg) + 0.5);
        pl->bags_per_run = R < 4 ? 4 : (R > 24 ? 24 : R);
        pl->rows_in_flight = 4;
        pl->ring_mode = -1;
    }
    int devid = 0;
    if (!cuda_ok(cudaGetDevice(&devid)) ||
        !cuda_ok(cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, devid))) {
        free(pl->h_rows);
        free(pl);
        return BLS_ECUDA;
    }

    // descriptors
    std::vector<BlsTableDesc> tab(T);
    std::vector<BlsPairDesc> pair(p.NI);
    std::vector<int> pair_of(T, 0);
    std::vector<int> pair_first(P + 1, 0);
    for (int t = 0; t < T; t++) {
        tab[t].weight = tables[t].weight;
        tab[t].rows = tables[t].rows;
        tab[t].blk = part == BLS_PART_ROW_BLOCK ? (int)((tables[t].rows + P - 1) / P) : 0;
        tab[t].magic = tab[t].blk <= 1 ? 0xFFFFFFFFu : (unsigned)((1ull << 32) / (unsigned long long)tab[t].blk);
    }
    int n = 0;
    for (int d = 0; d < P; d++) {
        pair_first[d] = n;
        for (int t = 0; t < T; t++) {
            BlsPairDesc q;
            memset(&q, 0, sizeof(q));
            q.t = t; q.dst = d;
            if (part == BLS_PART_TABLE_RR) {
                if (t % P != d) continue;
                q.base = tables[t].weight;
                q.nrows = (int)tables[t].rows;
                pair_of[t] = n;
            } else {
                long long first = (long long)d * tab[t].blk;
                long long have = tables[t].rows - first;
                if (have > tab[t].blk) have = tab[t].blk;
                if (have < 1) { have = 1; first = 0; }      // owner holds nothing: never addressed
                q.base = (const char *)tables[t].weight + (size_t)first * p.row_bytes;
                q.nrows = (int)have;
            }
            pair[n++] = q;
        }
    }
    pair_first[P] = n;
    BlsDev hd;
    memset(&hd, 0, sizeof(hd));
    for (int r = 0; r < BLS_MAX_RANKS; r++) hd.route_iter[r] = hd.serve_iter[r] = hd.consume_iter[r] = -1;
    hd.wait_limit_ns = 2000000000ull;
    bool ok = cuda_ok(cudaMemcpyAsync(ws + L.dev, &hd, sizeof(hd), cudaMemcpyHostToDevice, pl->stream)) &&
              cuda_ok(cudaMemcpyAsync(ws + L.tab, tab.data(), sizeof(BlsTableDesc) * T,
                                      cudaMemcpyHostToDevice, pl->stream)) &&
              cuda_ok(cudaMemcpyAsync(ws + L.pair, pair.data(), sizeof(BlsPairDesc) * p.NI,
                                      cudaMemcpyHostToDevice, pl->stream)) &&
              cuda_ok(cudaMemcpyAsync(ws + L.pair_of, pair_of.data(), sizeof(int) * T,
                                      cudaMemcpyHostToDevice, pl->stream)) &&
              cuda_ok(cudaMemcpyAsync(ws + L.pair_first, pair_first.data(), sizeof(int) * (P + 1),
                                      cudaMemcpyHostToDevice, pl->stream)) &&
              cuda_ok(cudaMemsetAsync(ws + L.counts, 0, sizeof(int) * p.S * 4 * P * P, pl->stream)) &&
              cuda_ok(cudaMemsetAsync(ws + L.queue, 0, 16, pl->stream)) &&            // the queue's header
              cuda_ok(cudaMemsetAsync(ws + L.stamps, 0, sizeof(unsigned long long) * BLS_TL_ITERS * P * 3, pl->stream)) &&
              // the vectors above are pageable: make sure the copies have left them
              cuda_ok(cudaStreamSynchronize(pl->stream));
    if (!ok) { free(pl->h_rows); free(pl); return BLS_ECUDA; }
    *plan = pl;
    return BLS_OK;
}

void bls_destroy(bls_plan_t *plan)
{
    if (!plan) return;
    if (plan->prof_ev) {
        for (int i = 0; i < BLS_PROF_MAX * 4; i++) cudaEventDestroy(plan->prof_ev[i]);
        free(plan->prof_ev);
    }
    if (plan->side_ready) {
        cudaStreamDestroy(plan->s_side);
        cudaEventDestroy(plan->e_fork);
        cudaEventDestroy(plan->e_join);
    }
    if (plan->host_path) {
        cudaStreamDestroy(plan->s_in);
        cudaStreamDestroy(plan->s_out);
        cudaEventDestroy(plan->e_in);
        cudaEventDestroy(plan->e_comp);
        cudaEventDestroy(plan->e_out);
    }
    free(plan->h_rows);
    free(plan);
}

bls_status_t bls_profile(bls_plan_t *pl, int enable)
{
    if (!pl) return BLS_EINVAL;
    if (enable && !pl->prof_ev) {
        pl->prof_ev = (cudaEvent_t *)calloc((size_t)BLS_PROF_MAX * 4, sizeof(cudaEvent_t));
        if (!pl->prof_ev) return BLS_ENOSPC;
        for (int i = 0; i < BLS_PROF_MAX * 4; i++) cudaEventCreate(&pl->prof_ev[i]);
    }
    pl->prof_on = enable ? 1 : 0;
    return BLS_OK;
}

bls_status_t bls_profile_read(bls_plan_t *pl, double *ms_route, double *ms_gather, double *ms_ring,
                              int64_t *calls, int64_t *kernels)
{
    if (!pl) return BLS_EINVAL;
    if (cudaStreamSynchronize(pl->stream) != cudaSuccess) return BLS_ECUDA;
    double r = 0, g = 0, c = 0;
    for (int i = 0; i < pl->prof_n; i++) {
        cudaEvent_t *ev = pl->prof_ev + (size_t)i * 4;
        float a = 0, b = 0, d = 0;
        if (cudaEventElapsedTime(&a, ev[0], ev[1]) != cudaSuccess ||
            cudaEventElapsedTime(&b, ev[1], ev[2]) != cudaSuccess ||
            cudaEventElapsedTime(&d, ev[2], ev[3]) != cudaSuccess)
            return BLS_ECUDA;
        r += a; g += b; c += d;
    }
    if (ms_route) *ms_route = r;
    if (ms_gather) *ms_gather = g;
    if (ms_ring) *ms_ring = c;
    if (calls) *calls = pl->prof_n;
    if (kernels) *kernels = pl->kernels_launched;
    pl->prof_n = 0;
    return BLS_OK;
}

static bls_status_t launch_check()
{
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}

// One wave: gate -> router -> gather/pool/return -> commit, with optional stage events.
static void enqueue_wave(bls_plan_t *pl, int mode, long long t_last, long long floor_, int k,
                         const int *ids, const int *off, long long n_ids)
{
    cudaEvent_t *ev = nullptr;
    if (pl->prof_on && pl->prof_n < BLS_PROF_MAX && pl->prof_ev) ev = pl->prof_ev + (size_t)pl->prof_n++ * 4;
    if (ev) cudaEventRecord(ev[0], pl->stream);
    bls_launch_gate(pl, mode, t_last, floor_, k, ids, off, n_ids);
    bls_launch_route(pl);
    if (ev) cudaEventRecord(ev[1], pl->stream);
    bls_launch_gather(pl);                             // its last block commits the wave
    if (ev) { cudaEventRecord(ev[2], pl->stream); cudaEventRecord(ev[3], pl->stream); }
    pl->kernels_launched += 2 + bls_route_kernels(pl);
}

// Overlapped wave (bound >= 1): the requesters post iteration t while the owners answer
// iteration t - 1, which is in another slot, so the two do not depend on each other
// (Table I of the paper: communication of one batch beside computation of another).  The
// gate plans both; then the gather kernel (answer t - 1, commit) goes to the plan's stream
// and the router's two kernels (post t) to a second stream: the router's first half and the launch
// gap between router and gather kernel leave the critical path, and the copy kernel's small blocks
// fill the gather kernel's tail as its blocks retire (measured: they are not resident together before that, and making
// them so by equal L1 / shared-memory splits gains nothing).  (Row-wise placement stays sequential:
// its router needs shared memory and several blocks per SM to hide its load latency,
// neither of which the resident gather blocks leave.)  The plan's stream waits for the copy
// kernel, so everything enqueued on it afterwards sees the wave complete.
static bool side_stream_ready(bls_plan_t *pl)
{
    if (pl->side_ready) return true;
    if (cudaStreamCreateWithFlags(&pl->s_side, cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaEventCreateWithFlags(&pl->e_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&pl->e_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaStreamDestroy(pl->s_side);
        return false;
    }
    pl->side_ready = 1;
    return true;
}

static void enqueue_wave_overlapped(bls_plan_t *pl, long long t_last, long long floor_, int k, const int *ids,
                                    const int *off, long long n_ids)
{
    cudaEvent_t *ev = nullptr;
    if (pl->prof_on && pl->prof_n < BLS_PROF_MAX && pl->prof_ev) ev = pl->prof_ev + (size_t)pl->prof_n++ * 4;
    if (ev) cudaEventRecord(ev[0], pl->stream);
    bls_launch_gate(pl, BLS_MODE_STEP, t_last, floor_, k, ids, off, n_ids, 1);
    cudaEventRecord(pl->e_fork, pl->stream);
    if (ev) cudaEventRecord(ev[1], pl->stream);
    bls_launch_gather(pl);                             // first, so that its blocks are resident first
    cudaStreamWaitEvent(pl->s_side, pl->e_fork, 0);
    bls_launch_meta(pl, pl->s_side);                   // chunk bases, send counts and displacements of iteration t
    bls_launch_route_beside(pl, pl->s_side);
    cudaEventRecord(pl->e_join, pl->s_side);
    cudaStreamWaitEvent(pl->stream, pl->e_join, 0);
    if (ev) { cudaEventRecord(ev[2], pl->stream); cudaEventRecord(ev[3], pl->stream); }
    pl->kernels_launched += 3 + bls_route_kernels(pl);
}

// Event-driven mode: the whole call is one launch of the persistent ring kernel, in which
// every logical rank posts, is answered and completes on its own (bls_event.cu).  Used
// whenever delays are injected, and for iterations so small that the launches of a wave
// would dominate.
static bool ring_applies(const bls_plan_t *pl)
{
    if (pl->any_stall || pl->ring_mode > 0) return true;
    // small iterations (below about 128 K lookups): one launch instead of three dependent ones,
    // unless the caller asked for the overlapped mode of the stand-alone kernels
    return pl->ring_mode == 0 && pl->overlap_mode <= 0 && !pl->prm.hot.enabled &&
           (long long)pl->prm.P * pl->prm.cap < (1 << 17);
}

// Table-wise iterations with the ranks in lockstep, the whole iteration in one launch (bls_small.cu).
// Measured against the wave of stand-alone kernels: 2.5 times faster at 50 K lookups per iteration
// and 1.7 times at 200 K whatever the bag lengths; level from about 350 K lookups with 20-ID bags;
// with short bags (one ID per bag, or the 2.4 of a Pareto law; 64- and 256-byte rows) still 10-30 %
// faster at 0.5-1 M lookups, level at 2 M, slower beyond.  At a million lookups the overlapped mode
// takes over for bounds >= 1 anyway.
static bool small_applies(const bls_plan_t *pl)
{
    const BlsParams &p = pl->prm;
    if (pl->fused_mode < 0 || p.part != BLS_PART_TABLE_RR || p.hot.enabled || pl->rows_in_flight != 4) return false;
    if (pl->fused_mode > 0) return true;
    const long long room = (long long)p.P * p.cap;     // lookups an iteration can hold
    const bool short_bags = (long long)p.cap <= 4LL * p.T * p.b;
    return room < (1 << 18) || (short_bags && room < (1 << 20));
}

static void enqueue_small(bls_plan_t *pl, long long t, const int *ids, const int *off, long long n_ids)
{
    cudaEvent_t *ev = nullptr;
    if (pl->prof_on && pl->prof_n < BLS_PROF_MAX && pl->prof_ev) ev = pl->prof_ev + (size_t)pl->prof_n++ * 4;
    if (ev) { cudaEventRecord(ev[0], pl->stream); cudaEventRecord(ev[1], pl->stream); }
    bls_launch_small(pl, t, ids, off, n_ids);
    if (ev) { cudaEventRecord(ev[2], pl->stream); cudaEventRecord(ev[3], pl->stream); }
    pl->kernels_launched += 1;
}

static bls_status_t enqueue_ring(bls_plan_t *pl, int mode, long long t_last, long long floor_, int k, const int *ids,
                                 const int *off, long long n_ids)
{
    cudaEvent_t *ev = nullptr;
    if (pl->prof_on && pl->prof_n < BLS_PROF_MAX && pl->prof_ev) ev = pl->prof_ev + (size_t)pl->prof_n++ * 4;
    if (ev) { cudaEventRecord(ev[0], pl->stream); cudaEventRecord(ev[1], pl->stream); }
    const int err = bls_launch_ring(pl, mode, t_last, floor_, k, ids, off, n_ids);
    if (ev) { cudaEventRecord(ev[2], pl->stream); cudaEventRecord(ev[3], pl->stream); }
    pl->kernels_launched += 1;
    pl->unserved = 0;                                  // whatever the owners still owe is answered inside the launch
    pl->ring_used = 1;
    return err == (int)cudaSuccess ? BLS_OK : BLS_ECUDA;
}

// Debug aid: a slot that is about to receive iteration `iter` holds an iteration that has
// been handed back already; filling it with 0xFF bytes (NaN) makes any bag the gather
// kernel fails to write, and any read of a slot before its data has arrived, visible.
static void poison_slot(const bls_plan_t *pl, long long iter)
{
    if (!pl->poison) return;
    cudaMemsetAsync(pl->prm.out + (size_t)(iter % pl->prm.S) * pl->prm.out_slot_elems, 0xFF,
                    sizeof(float) * (size_t)pl->prm.out_slot_elems, pl->stream);
}

static const float *slot_out(const bls_plan_t *pl, long long iter)
{
    return pl->prm.out + (size_t)(iter % pl->prm.S) * pl->prm.out_slot_elems;
}

bls_status_t bls_route(bls_plan_t *pl, int64_t iter, const int32_t *ids, const int32_t *offsets,
                       int64_t n_ids)
{
    if (!pl || !offsets || (!ids && n_ids > 0) || n_ids < 0) return BLS_EINVAL;
    if (iter != pl->t_next || pl->t_handed != pl->t_next || pl->routed_only >= 0) return BLS_ESTATE;
    poison_slot(pl, iter);
    bls_launch_gate(pl, BLS_MODE_ROUTE_ONLY, iter, -1, 0, ids, offsets, n_ids);
    bls_launch_route(pl);
    bls_launch_commit(pl);
    pl->kernels_launched += 2 + bls_route_kernels(pl);
    pl->routed_only = iter;
    pl->t_next = iter + 1;
    return launch_check();
}

bls_status_t bls_lookup(bls_plan_t *pl, int64_t iter)
{
    if (!pl) return BLS_EINVAL;
    if (pl->routed_only != iter) return BLS_ESTATE;
    bls_launch_gate(pl, BLS_MODE_LOOKUP_ONLY, iter, -1, 0, nullptr, nullptr, 0);
    bls_launch_gather(pl);                             // its last block commits the wave
    pl->kernels_launched += 2;
    pl->routed_only = -1;
    pl->t_handed = iter + 1;
    return launch_check();
}

bls_status_t bls_step(bls_plan_t *pl, int k, const int32_t *ids, const int32_t *offsets, int64_t n_ids,
                      const float **out, int64_t *out_iter)
{
    if (!pl || !offsets || (!ids && n_ids > 0) || n_ids < 0 || !out || !out_iter) return BLS_EINVAL;
    if (k < 0 || k > pl->k_max || pl->routed_only >= 0) return BLS_ESTATE;
    if (pl->k_cur >= 0 && pl->k_cur != k && pl->t_handed != pl->t_next) return BLS_ESTATE;
    pl->k_cur = k;
    const long long t = pl->t_next++;
    poison_slot(pl, t);
    // (iterations below about a million lookups are bound by the launch rate, of the host or of
    // the GPU, and the second stream costs five more driver calls per step: they stay on one stream)
    const bool ring = ring_applies(pl);
    const bool overlapped = !ring && k >= 1 && pl->prm.part == BLS_PART_TABLE_RR && !pl->prm.hot.enabled &&
                            pl->overlap_mode >= 0 &&
                            (pl->overlap_mode > 0 || (long long)pl->prm.P * pl->prm.cap >= (1 << 20)) && side_stream_ready(pl);
    if (ring) {
        const bls_status_t st = enqueue_ring(pl, BLS_MODE_STEP, t, t - k, k, ids, offsets, n_ids);
        if (st != BLS_OK) return st;
    } else if (!overlapped && !pl->unserved && small_applies(pl)) {
        enqueue_small(pl, t, ids, offsets, n_ids);     // posts, answers and completes iteration t on every rank
    } else if (overlapped) {
        enqueue_wave_overlapped(pl, t, t - k, k, ids, offsets, n_ids);
        pl->unserved = 1;                              // iteration t is answered by the next wave
    } else {
        enqueue_wave(pl, BLS_MODE_STEP, t, t - k, k, ids, offsets, n_ids);
    }
    if (t - k >= pl->t_handed) {                       // (an iteration of an earlier loop has been handed back already)
        *out = slot_out(pl, t - k);
        *out_iter = t - k;
        pl->t_handed = t - k + 1;
    } else {
        *out = nullptr;
        *out_iter = -1;
    }
    return launch_check();
}

bls_status_t bls_drain(bls_plan_t *pl, const float **out, int64_t *out_iter)
{
    if (!pl || !out || !out_iter) return BLS_EINVAL;
    if (pl->routed_only >= 0) return BLS_ESTATE;
    if (pl->t_handed == pl->t_next) {
        *out = nullptr;
        *out_iter = -1;
        pl->k_cur = -1;
        pl->ring_used = 0;
        return BLS_OK;
    }
    const long long f = pl->t_handed;
    // In a wave every rank completes an iteration in the step that issues it (in overlapped
    // mode: in the step after it, so the newest one is still to be answered).  In event-driven
    // mode ranks may be behind: the launch ends once iteration f is complete on every rank.
    if (pl->any_stall || pl->ring_used) {
        const bls_status_t st = enqueue_ring(pl, BLS_MODE_DRAIN, pl->t_next - 1, f, pl->k_cur < 0 ? 0 : pl->k_cur, nullptr, nullptr, 0);
        if (st != BLS_OK) return st;
    } else if (pl->unserved) {
        enqueue_wave(pl, BLS_MODE_DRAIN, pl->t_next - 1, f, pl->k_cur < 0 ? 0 : pl->k_cur, nullptr, nullptr, 0);
        pl->unserved = 0;
    }
    *out = slot_out(pl, f);
    *out_iter = f;
    pl->t_handed = f + 1;
    if (pl->t_handed == pl->t_next) { pl->k_cur = -1; pl->ring_used = 0; }
    return launch_check();
}

// Host-buffer path: the copies run on two streams of their own so that the upload of the
// next iteration and the download of the previous result overlap (PCIe is full duplex); with a
// bound >= 1 the download of iteration t - k also runs beside the kernels of iteration t.  The plan's stream waits for both, so work enqueued
// on it afterwards, and a synchronisation of it, see the copies complete.
static bool host_path_ready(bls_plan_t *pl)
{
    if (pl->host_path) return true;
    if (cudaStreamCreateWithFlags(&pl->s_in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&pl->s_out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&pl->e_in, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&pl->e_comp, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&pl->e_out, cudaEventDisableTiming) != cudaSuccess)
        return false;
    // nothing has been enqueued on the copy streams yet: order them after what the plan's stream holds
    if (cudaEventRecord(pl->e_comp, pl->stream) != cudaSuccess) return false;
    pl->comp_iter = pl->t_next;
    pl->host_path = 1;
    return true;
}

// Copy a handed-back iteration to the host.  `early`: the iteration was complete before the kernels
// that the current call has just enqueued (a bound >= 1; >= 2 in overlapped mode, where an iteration
// is answered one step after it was posted), and those kernels write another slot of the ring, so
// the copy only has to wait for the previous call's kernels and runs beside the current ones.
static bls_status_t download(bls_plan_t *pl, const float *out, float *host_out, bool early)
{
    const bool copy = out && host_out;
    if (!early && cudaEventRecord(pl->e_comp, pl->stream) != cudaSuccess) return BLS_ECUDA;
    if (copy) {
        // (early: e_comp still marks the end of the previous call's kernels)
        if (cudaStreamWaitEvent(pl->s_out, pl->e_comp, 0) != cudaSuccess ||
            cudaMemcpyAsync(host_out, out, sizeof(float) * (size_t)pl->prm.out_slot_elems, cudaMemcpyDeviceToHost,
                            pl->s_out) != cudaSuccess ||
            cudaEventRecord(pl->e_out, pl->s_out) != cudaSuccess)
            return BLS_ECUDA;
    }
    if (early && cudaEventRecord(pl->e_comp, pl->stream) != cudaSuccess) return BLS_ECUDA;
    pl->comp_iter = pl->t_next;
    if (copy && cudaStreamWaitEvent(pl->stream, pl->e_out, 0) != cudaSuccess) return BLS_ECUDA;
    return BLS_OK;
}

bls_status_t bls_step_host(bls_plan_t *pl, int k, const int32_t *ids, const int32_t *offsets,
                           int64_t n_ids, float *host_out, int64_t *out_iter)
{
    if (!pl || !offsets || (!ids && n_ids > 0) || n_ids < 0 || !out_iter) return BLS_EINVAL;
    const BlsParams &p = pl->prm;
    if (n_ids > (long long)p.P * p.cap) return BLS_ENOSPC;
    if (k < 0 || k > pl->k_max || pl->routed_only >= 0) return BLS_ESTATE;
    if (!host_path_ready(pl)) return BLS_ECUDA;
    const int slot = (int)(pl->t_next % p.S);
    const size_t G1 = (size_t)p.P * p.T * p.b + 1;
    int *d_ids = p.stage_ids + (size_t)slot * p.P * p.cap;
    int *d_off = p.stage_off + (size_t)slot * G1;
    // upload after the previous step's kernels (the staging slot's last user finished long before them)
    if (cudaStreamWaitEvent(pl->s_in, pl->e_comp, 0) != cudaSuccess ||
        cudaMemcpyAsync(d_off, offsets, sizeof(int) * G1, cudaMemcpyHostToDevice, pl->s_in) != cudaSuccess ||
        (n_ids > 0 &&
         cudaMemcpyAsync(d_ids, ids, sizeof(int) * (size_t)n_ids, cudaMemcpyHostToDevice, pl->s_in) != cudaSuccess) ||
        cudaEventRecord(pl->e_in, pl->s_in) != cudaSuccess ||
        cudaStreamWaitEvent(pl->stream, pl->e_in, 0) != cudaSuccess)
        return BLS_ECUDA;
    // e_comp marks the end of the previous iteration's kernels only if that iteration came through this path too
    const bool fresh = pl->comp_iter == pl->t_next;
    const float *out = nullptr;
    bls_status_t st = bls_step(pl, k, d_ids, d_off, n_ids, &out, out_iter);
    if (st != BLS_OK) return st;
    // with injected delays (ring kernel) an iteration may complete inside the launch that hands it back
    const bool early = out && fresh && !ring_applies(pl) && !pl->ring_used && k >= (pl->unserved ? 2 : 1);
    return download(pl, out, host_out, early);
}

bls_status_t bls_drain_host(bls_plan_t *pl, float *host_out, int64_t *out_iter)
{
    if (!pl || !out_iter) return BLS_EINVAL;
    if (!host_path_ready(pl)) return BLS_ECUDA;
    const float *out = nullptr;
    bls_status_t st = bls_drain(pl, &out, out_iter);
    if (st != BLS_OK) return st;
    return download(pl, out, host_out, false);
}

bls_status_t bls_view(bls_plan_t *pl, int64_t iter, bls_route_view_t *v)
{
    if (!pl || !v) return BLS_EINVAL;
    if (iter < 0 || iter >= pl->t_next || iter < pl->t_next - pl->prm.S) return BLS_ESTATE;
    const BlsParams &p = pl->prm;
    const size_t slot = (size_t)(iter % p.S), PP = (size_t)p.P * p.P;
    const int *cnt = p.counts + slot * 4 * PP;
    v->sendcounts = cnt;
    v->sdispls = cnt + PP;
    v->recvcounts = cnt + 2 * PP;
    v->rdispls = cnt + 3 * PP;
    v->sendbuf = p.sendbuf + slot * p.P * (size_t)p.cap;
    v->sendbuf_stride = p.cap;
    v->sub_start = p.sub_start + slot * p.P * (size_t)p.sub_stride;
    v->sub_stride = p.sub_stride;
    v->subbags_per_rank = p.NQ;
    v->sub_entries = p.NQ + (p.part == BLS_PART_TABLE_RR ? 1 : p.P);
    v->sub_bag_major = p.part == BLS_PART_TABLE_RR ? 0 : 1;
    v->out = p.out + slot * (size_t)p.out_slot_elems;
    return BLS_OK;
}

bls_status_t bls_counters(bls_plan_t *pl, int64_t *posted, int64_t *served, int64_t *done)
{
    if (!pl) return BLS_EINVAL;
    BlsDev hd;
    if (cudaStreamSynchronize(pl->stream) != cudaSuccess ||
        cudaMemcpy(&hd, pl->prm.dev, sizeof(hd), cudaMemcpyDeviceToHost) != cudaSuccess)
        return BLS_ECUDA;
    for (int r = 0; r < pl->prm.P; r++) {
        if (posted) posted[r] = hd.posted[r];
        if (served) served[r] = hd.served[r];
        if (done) done[r] = hd.done[r];
    }
    return BLS_OK;
}

bls_status_t bls_status(bls_plan_t *pl, int64_t *max_lag)
{
    if (!pl) return BLS_EINVAL;
    BlsDev hd;
    if (cudaStreamSynchronize(pl->stream) != cudaSuccess ||
        cudaMemcpy(&hd, pl->prm.dev, sizeof(hd), cudaMemcpyDeviceToHost) != cudaSuccess)
        return BLS_ECUDA;
    if (max_lag) *max_lag = hd.max_lag;
    if (hd.status & BLS_ST_EINVAL) return BLS_EINVAL;
    if (hd.status & BLS_ST_ENOSPC) return BLS_ENOSPC;
    if (hd.status & BLS_ST_ERANGE) return BLS_ERANGE;
    if (hd.status & BLS_ST_ESTATE) return BLS_ESTATE;
    if (hd.status & BLS_ST_ETIMEOUT) return BLS_ETIMEOUT;
    return BLS_OK;
}

bls_status_t bls_set_stall(bls_plan_t *pl, int rank, int64_t ns)
{
    if (!pl || rank < 0 || rank >= pl->prm.P || ns < 0) return BLS_EINVAL;
    unsigned long long v = (unsigned long long)ns;
    if (ns > 0) pl->any_stall = 1;
    return cudaMemcpyAsync(&pl->prm.dev->stall_ns[rank], &v, sizeof(v), cudaMemcpyHostToDevice,
                           pl->stream) == cudaSuccess &&
                   cudaStreamSynchronize(pl->stream) == cudaSuccess
               ? BLS_OK
               : BLS_ECUDA;
}

bls_status_t bls_set_random_stall(bls_plan_t *pl, int rank, int64_t max_ns, uint64_t seed)
{
    if (!pl || rank < 0 || rank >= pl->prm.P || max_ns < 0) return BLS_EINVAL;
    unsigned long long v = (unsigned long long)max_ns, sd = seed;
    if (max_ns > 0) pl->any_stall = 1;
    return cudaMemcpyAsync(&pl->prm.dev->stall_rand_ns[rank], &v, sizeof(v), cudaMemcpyHostToDevice, pl->stream) == cudaSuccess &&
                   cudaMemcpyAsync(&pl->prm.dev->stall_seed, &sd, sizeof(sd), cudaMemcpyHostToDevice, pl->stream) == cudaSuccess &&
                   cudaStreamSynchronize(pl->stream) == cudaSuccess
               ? BLS_OK
               : BLS_ECUDA;
}

bls_status_t bls_set_poison(bls_plan_t *pl, int enable)
{
    if (!pl) return BLS_EINVAL;
    pl->poison = enable ? 1 : 0;
    return BLS_OK;
}

bls_status_t bls_set_overlap(bls_plan_t *pl, int mode)
{
    if (!pl || mode < -1 || mode > 1) return BLS_EINVAL;
    pl->overlap_mode = mode;
    return BLS_OK;
}

bls_status_t bls_set_fused(bls_plan_t *pl, int mode)
{
    if (!pl || mode < -1 || mode > 1) return BLS_EINVAL;
    pl->fused_mode = mode;
    return BLS_OK;
}

bls_status_t bls_set_ring(bls_plan_t *pl, int mode)
{
    if (!pl || mode < -1 || mode > 1) return BLS_EINVAL;
    if (pl->t_handed != pl->t_next) return BLS_ESTATE;      // only between loops
    pl->ring_mode = mode;
    return BLS_OK;
}

bls_status_t bls_timeline(bls_plan_t *pl, int64_t first_iter, int n_iter, uint64_t *post_ns, uint64_t *serve_ns,
                          uint64_t *done_ns)
{
    if (!pl || first_iter < 0 || n_iter < 0) return BLS_EINVAL;
    if (first_iter + n_iter > pl->t_next || first_iter + BLS_TL_ITERS < pl->t_next) return BLS_ESTATE;
    if (cudaStreamSynchronize(pl->stream) != cudaSuccess) return BLS_ECUDA;
    const int P = pl->prm.P;
    std::vector<unsigned long long> h((size_t)BLS_TL_ITERS * P * 3);
    if (cudaMemcpy(h.data(), pl->prm.stamps, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
        return BLS_ECUDA;
    for (int i = 0; i < n_iter; i++)
        for (int r = 0; r < P; r++) {
            const unsigned long long *e = &h[((size_t)((first_iter + i) % BLS_TL_ITERS) * P + r) * 3];
            if (post_ns) post_ns[(size_t)i * P + r] = e[0];
            if (serve_ns) serve_ns[(size_t)i * P + r] = e[1];
            if (done_ns) done_ns[(size_t)i * P + r] = e[2];
        }
    return BLS_OK;
}

bls_status_t bls_set_tuning(bls_plan_t *pl, int bags_per_run, int rows_in_flight)
{
    if (!pl || bags_per_run < 0 || bags_per_run > 4096 || (rows_in_flight != 0 && rows_in_flight != 4 && rows_in_flight != 8 && rows_in_flight != 16 && rows_in_flight != 32))
        return BLS_EINVAL;
    if (bags_per_run) pl->bags_per_run = bags_per_run;
    if (rows_in_flight) pl->rows_in_flight = rows_in_flight;
    return BLS_OK;
}

bls_status_t bls_set_wait_limit(bls_plan_t *pl, int64_t ns)
{
    if (!pl || ns < 0) return BLS_EINVAL;
    unsigned long long v = (unsigned long long)ns;
    return cudaMemcpyAsync(&pl->prm.dev->wait_limit_ns, &v, sizeof(v), cudaMemcpyHostToDevice,
                           pl->stream) == cudaSuccess &&
                   cudaStreamSynchronize(pl->stream) == cudaSuccess
               ? BLS_OK
               : BLS_ECUDA;
}

}  // extern "C"
