// Steps 2 and 3 fused: the owner-side embedding-bag lookup (gather rows, sum-pool
// per bag with fp32 accumulation; Listing 1's apply_emb) writes each pooled vector
// straight into the requester's output slot out[src][s][t][:], so the pooled
// vectors never make a round trip through memory.
//
// The work is random row reads, bound by memory latency unless enough loads are in
// flight.  A group of LANES = row_bytes/16 lanes streams a *run* of consecutive
// sub-bags of one (owner, table, requester) chunk: their IDs are contiguous in the
// requester's packed send buffer, so the group walks one ID stream and keeps
// batches of U row loads in flight across bag boundaries (two batches are
// outstanding while a third batch's IDs are being fetched, 16 bytes at a time from
// aligned addresses); a bag boundary only costs a store of the accumulator.  Rows of one bag are added in their original
// order, so the result does not depend on how runs are cut.  Runs are handed out
// through an atomic counter in table-major order: at any moment the SMs work on
// one or two tables, whose Zipf-hot rows stay in L1/L2.  IDs and outputs use
// streaming loads/stores so that they do not evict table rows.
#include "bls_gather.cuh"
#include "bls_gather_bulk.cuh"

// The run loop of the table-wise gather kernel: runs are handed out by an atomic counter.
template <int LANES, int DT, int U>
__device__ __forceinline__ void pool_runs(const BlsParams &p, int R, int runs_per_chunk, int n_runs)
{
    constexpr int GPW = 32 / LANES;                    // groups (runs) per warp
    const int lane = threadIdx.x % LANES;
    const int g = (threadIdx.x & 31) / LANES;
    BlsDev *dev = p.dev;
    int base = 0;
    if ((threadIdx.x & 31) == 0) base = atomicAdd(&dev->work_ctr, GPW);
    base = __shfl_sync(0xffffffffu, base, 0);
    while (base < n_runs) {
        int next_base = 0;                             // grab the next runs now, use them later
        if ((threadIdx.x & 31) == 0) next_base = atomicAdd(&dev->work_ctr, GPW);
        const int run = base + g;
        if (run < n_runs) {
            const int chunk = run / runs_per_chunk;    // (pair, requester), pair-major
            const int s0 = (run - chunk * runs_per_chunk) * R;
            const int i = chunk / p.P, src = chunk - i * p.P;
            const BlsPairDesc pr = p.pair[i];
            const long long j = dev->serve_iter[pr.dst];
            if (j >= 0)                                // else: this owner does not serve in this wave
                stream_run<LANES, DT, U, false>(p, pr, i, (int)(j % p.S), src, s0, min(R, p.b - s0), lane, nullptr);
        }
        __syncwarp();
        base = __shfl_sync(0xffffffffu, next_base, 0);
    }
}

template <int LANES, int DT, int U>
__global__ void __launch_bounds__(256, (U >= 8 ? 2 : 3))
bls_gather_pool_kernel(BlsParams p, int R, int runs_per_chunk, int n_runs)
{
    pool_runs<LANES, DT, U>(p, R, runs_per_chunk, n_runs);
    finish_wave(p);
}

// Bulk-copy variant of the table-wise gather kernel (optional, bls_set_tuning): rows are staged
// in shared memory by cp.async.bulk, NST stages of BR rows per lane group.  Blocks of 128
// threads; persistent, runs handed out by the same counter.
template <int LANES, int DT, int BR, int NST>
__global__ void __launch_bounds__(128)
bls_gather_bulk_kernel(BlsParams p, int R, int runs_per_chunk, int n_runs)
{
    extern __shared__ __align__(128) unsigned char bulk_smem[];
    constexpr int GPW = 32 / LANES;
    constexpr int GPB = 4 * GPW;                       // lane groups per block
    constexpr int ROW = LANES * 16;
    const int lane = threadIdx.x % LANES;
    const int g = (threadIdx.x & 31) / LANES;
    const int gb = threadIdx.x / LANES;                // group within the block
    const unsigned gmask = LANES == 32 ? 0xffffffffu : (((1u << LANES) - 1u) << (g * LANES));
    BlsDev *dev = p.dev;
    BulkRing<LANES, BR, NST> ring;
    ring.rows = smem_addr(bulk_smem) + (unsigned)gb * (NST * BR * ROW);
    ring.bars = smem_addr(bulk_smem) + (unsigned)GPB * (NST * BR * ROW) + (unsigned)gb * (NST * 8);
    ring.kb_issue = ring.kb_wait = 0;
    if (lane == 0) {
        for (int s = 0; s < NST; s++) mbar_init(ring.bars + s * 8u, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    int timed_out = 0;

    int base = 0;
    if ((threadIdx.x & 31) == 0) base = atomicAdd(&dev->work_ctr, GPW);
    base = __shfl_sync(0xffffffffu, base, 0);
    while (base < n_runs) {
        int next_base = 0;
        if ((threadIdx.x & 31) == 0) next_base = atomicAdd(&dev->work_ctr, GPW);
        const int run = base + g;
        if (run < n_runs) {
            const int chunk = run / runs_per_chunk;    // (pair, requester), pair-major
            const int s0 = (run - chunk * runs_per_chunk) * R;
            const int i = chunk / p.P, src = chunk - i * p.P;
            const BlsPairDesc pr = p.pair[i];
            const long long j = dev->serve_iter[pr.dst];
            if (j >= 0)
                bulk_run<LANES, DT, BR, NST>(p, pr, i, (int)(j % p.S), src, s0, min(R, p.b - s0), lane, gmask, ring, timed_out);
        }
        __syncwarp();
        base = __shfl_sync(0xffffffffu, next_base, 0);
    }
    if (timed_out) flag(p, BLS_ST_ETIMEOUT);
    finish_wave(p);
}

// Hot-row variant: one persistent block per SM.  Blocks start spread over the
// (owner, table) pairs; a block copies its pair's hot rows into shared memory once
// and takes runs from the pair's counter until the pair is used up.  After that its
// warps help with whatever the other pairs have left, without staging (leftovers
// are small, and a fresh copy would cost more than it saves).
template <int LANES, int DT>
__global__ void __launch_bounds__(768, 1)
bls_gather_hot_kernel(BlsParams p, int R, int runs_per_chunk)
{
    extern __shared__ uint4 hot_rows[];                // [K][LANES]
    constexpr int GPW = 32 / LANES;
    const int lane = threadIdx.x % LANES;
    const int wl = threadIdx.x & 31;
    const int g = wl / LANES;
    BlsDev *dev = p.dev;
    const int runs_in_pair = p.P * runs_per_chunk;
    const int i0 = (int)(((long long)blockIdx.x * p.NI) / gridDim.x);

    auto take_runs = [&](int i, auto hot_tag) {        // all runs this warp can get from pair i
        constexpr bool HOT = decltype(hot_tag)::value;
        const BlsPairDesc pr = p.pair[i];
        const long long j = dev->serve_iter[pr.dst];
        if (j < 0) return;                             // this owner does not serve in this wave
        int base = 0;
        if (wl == 0) base = atomicAdd(&p.hot.pair_ctr[i], GPW);
        base = __shfl_sync(0xffffffffu, base, 0);
        while (base < runs_in_pair) {
            int next_base = 0;
            if (wl == 0) next_base = atomicAdd(&p.hot.pair_ctr[i], GPW);
            const int run = base + g;
            if (run < runs_in_pair) {
                const int src = run / runs_per_chunk;
                const int s0 = (run - src * runs_per_chunk) * R;
                stream_run<LANES, DT, 4, HOT>(p, pr, i, (int)(j % p.S), src, s0, min(R, p.b - s0), lane, hot_rows);
            }
            __syncwarp();
            base = __shfl_sync(0xffffffffu, next_base, 0);
        }
    };

    {   // stage the hot rows of the block's own pair: eight independent loads per thread at a time
        const BlsPairDesc pr = p.pair[i0];
        const int tot = min(p.hot.count[pr.t], p.hot.K) * LANES;
        const int *list = p.hot.rows + (size_t)pr.t * p.hot.K;
        const uint4 *tbl = reinterpret_cast<const uint4 *>(pr.base);
        for (int e0 = 0; e0 < tot; e0 += 8 * blockDim.x) {
            uint4 tmp[8];
            #pragma unroll
            for (int k = 0; k < 8; k++) {
                const int e = e0 + k * blockDim.x + threadIdx.x;
                if (e < tot) {
                    const unsigned row = min((unsigned)list[e / LANES], (unsigned)pr.nrows - 1u);
                    tmp[k] = __ldg(tbl + (size_t)row * LANES + (e % LANES));
                }
            }
            #pragma unroll
            for (int k = 0; k < 8; k++) {
                const int e = e0 + k * blockDim.x + threadIdx.x;
                if (e < tot) hot_rows[e] = tmp[k];
            }
        }
    }
    __syncthreads();
    take_runs(i0, std::true_type{});
    // leftovers of the other pairs: each lane looks at one pair's counter, the warp visits those with work
    for (int q0 = 1; q0 < p.NI; q0 += 32) {
        const int q = q0 + wl;
        bool has = false;
        if (q < p.NI) has = *(volatile int *)&p.hot.pair_ctr[(i0 + q) % p.NI] < runs_in_pair;
        unsigned m = __ballot_sync(0xffffffffu, has);
        while (m) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            take_runs((i0 + q0 + b) % p.NI, std::false_type{});
        }
    }
    finish_wave(p);
}

// Row-wise gather kernel: persistent blocks, runs of bags handed out by an atomic counter.
template <int LANES, int DT>
__global__ void __launch_bounds__(256, 4)
bls_gather_rowwise_kernel(BlsParams p, int R, int runs_per_chunk, int n_runs)
{
    constexpr int GPW = 32 / LANES;
    const int lane = threadIdx.x % LANES;
    const int g = (threadIdx.x & 31) / LANES;
    BlsDev *dev = p.dev;

    int base = 0;
    if ((threadIdx.x & 31) == 0) base = atomicAdd(&dev->work_ctr, GPW);
    base = __shfl_sync(0xffffffffu, base, 0);
    while (base < n_runs) {
        int next_base = 0;
        if ((threadIdx.x & 31) == 0) next_base = atomicAdd(&dev->work_ctr, GPW);
        const int run = base + g;
        const long long j = dev->serve_iter[0];        // row-wise: all owners answer the same iteration
        if (run < n_runs && j >= 0) rowwise_run<LANES, DT>(p, (int)(j % p.S), run, R, runs_per_chunk, lane, g);
        __syncwarp();
        base = __shfl_sync(0xffffffffu, next_base, 0);
    }
    finish_wave(p);
}

// Runs are as long as the plan asks for, but short enough that every resident lane
// group gets at least two: small workloads are latency-bound and need the parallelism.
void bls_gather_tiling(const bls_plan_t *pl, int *R_out, int *rpc_out)
{
    const BlsParams &p = pl->prm;
    const bool rowwise = p.part == BLS_PART_ROW_BLOCK;
    const int groups_per_warp = 32 / p.lanes;
    const long long bags = (long long)(rowwise ? p.T : p.NI) * p.P * p.b;
    const long long resident_groups = (long long)pl->sm_count * 24 * groups_per_warp;
    long long fit = bags / (2 * resident_groups);
    int R = (int)(fit < 1 ? 1 : (fit < pl->bags_per_run ? fit : pl->bags_per_run));
    while ((long long)(rowwise ? p.T : p.NI) * p.P * ((p.b + R - 1) / R) > 0x7fffffffLL) R *= 2;   // run numbers are 32-bit
    *R_out = R;
    *rpc_out = (p.b + R - 1) / R;
}

template <int LANES, int DT, int U>
static void launch_gather(const bls_plan_t *pl)
{
    const BlsParams &p = pl->prm;
    const bool rowwise = p.part == BLS_PART_ROW_BLOCK;
    int R, rpc;
    bls_gather_tiling(pl, &R, &rpc);
    // table-wise: runs of sub-bags of one (owner, table, requester); row-wise: runs of bags of one (table, requester)
    const long long n_runs = (long long)(rowwise ? p.T : p.NI) * p.P * rpc;
    // persistent blocks: as many as stay resident (table-wise: 3 per SM at 80 registers; row-wise: 4 at 64
    // registers, measured faster than 3 or 5), fewer for small workloads
    const long long want = (n_runs + 8 * (32 / LANES) - 1) / (8 * (32 / LANES));
    const int per_sm = rowwise ? 4 : 3;
    const int blocks = (int)(want < 1 ? 1 : (want > pl->sm_count * per_sm ? pl->sm_count * per_sm : want));
    if (rowwise) {
        bls_gather_rowwise_kernel<LANES, DT><<<blocks, 256, 0, pl->stream>>>(p, R, rpc, (int)n_runs);
    } else if (pl->rows_in_flight >= 16 && LANES >= 4 && !p.hot.enabled) {
        if constexpr (LANES >= 4) {
            // rows staged in shared memory by the bulk-copy engine: 4 stages of 8 rows (or 2 of 8) per lane group
            constexpr int BR = 8;
            const bool deep = pl->rows_in_flight >= 32;
            const size_t smem = (size_t)(4 * (32 / LANES)) * ((deep ? 4 : 2) * BR * LANES * 16 + (deep ? 4 : 2) * 8);
            auto kernel = deep ? bls_gather_bulk_kernel<LANES, DT, BR, 4> : bls_gather_bulk_kernel<LANES, DT, BR, 2>;
            cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   // per device, cheap: every launch
            int per = 1;
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, kernel, 128, smem);
            const long long want2 = (n_runs + 4 * (32 / LANES) - 1) / (4 * (32 / LANES));
            const long long most = (long long)pl->sm_count * (per < 1 ? 1 : per);
            kernel<<<(unsigned)(want2 < 1 ? 1 : (want2 > most ? most : want2)), 128, smem, pl->stream>>>(p, R, rpc, (int)n_runs);
        }
    } else if (p.hot.enabled) {
        const size_t smem = (size_t)p.hot.K * p.row_bytes;
        static size_t configured = 0;                  // per instantiation: shared memory size it was set up for
        if (configured != smem) {
            cudaFuncSetAttribute(bls_gather_hot_kernel<LANES, DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            // leave the rest of the SM's on-chip memory to L1
            int pct = (int)((smem + 2048) * 100 / (228 * 1024)) + 1;
            cudaFuncSetAttribute(bls_gather_hot_kernel<LANES, DT>, cudaFuncAttributePreferredSharedMemoryCarveout, pct > 100 ? 100 : pct);
            configured = smem;
        }
        bls_gather_hot_kernel<LANES, DT><<<pl->sm_count, 768, smem, pl->stream>>>(p, R, rpc);
    } else
        bls_gather_pool_kernel<LANES, DT, U><<<blocks, 256, 0, pl->stream>>>(p, R, rpc, (int)n_runs);
}

template <int LANES, int DT>
static void launch_gather_u(const bls_plan_t *pl)
{
    if (pl->rows_in_flight == 8) launch_gather<LANES, DT, 8>(pl);
    else launch_gather<LANES, DT, 4>(pl);
}

template <int DT>
static void launch_gather_dt(const bls_plan_t *pl)
{
    switch (pl->prm.lanes) {
    case 1: launch_gather_u<1, DT>(pl); break;
    case 2: launch_gather_u<2, DT>(pl); break;
    case 4: launch_gather_u<4, DT>(pl); break;
    case 8: launch_gather_u<8, DT>(pl); break;
    case 16: launch_gather_u<16, DT>(pl); break;
    default: launch_gather_u<32, DT>(pl); break;
    }
}

void bls_launch_gather(const bls_plan_t *pl)
{
    switch (pl->prm.dtype) {
    case BLS_F32: launch_gather_dt<BLS_F32>(pl); break;
    case BLS_BF16: launch_gather_dt<BLS_BF16>(pl); break;
    default: launch_gather_dt<BLS_F16>(pl); break;
    }
}
