// Device-side helpers shared by the kernels of libbls (inline: the library is built
// without relocatable device code).
#pragma once
#include "bls_internal.h"

__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Programmatic stream serialisation, for chains of very short kernels.  A kernel launched with
// launch_serialised() may have its blocks made resident while the previous kernel of the stream is
// still running; stream_order_enter(), the first statement of every such kernel, holds them until
// that kernel has completed and its writes are visible, and then lets the next kernel of the stream
// be brought in the same way.  The order of the stream is unchanged; the launch latency between
// dependent kernels is hidden.  Because every kernel launched this way waits before anything
// else, completion stays transitive along the stream.
__device__ __forceinline__ void stream_order_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <class... Params, class... Args>
static inline cudaError_t launch_serialised(void (*kernel)(Params...), dim3 grid, dim3 block, cudaStream_t stream,
                                            Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

__device__ __forceinline__ void flag(const BlsParams &p, int bit) { atomicOr(&p.dev->status, bit); }

// Injected delay of rank r before it posts iteration j: the fixed part plus a uniform draw
// from [0, span], the SplitMix64 output for (seed, rank, iteration) - a counter-based
// generator, so a run can be repeated and reproduced on the host.
__device__ __forceinline__ unsigned long long stall_draw(const BlsDev *d, int r, long long j)
{
    unsigned long long stall = d->stall_ns[r];
    const unsigned long long span = d->stall_rand_ns[r];
    if (span) {
        unsigned long long z = d->stall_seed + (((unsigned long long)r << 40) + (unsigned long long)j + 1ull) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z ^= z >> 31;
        stall += z % (span + 1ull);
    }
    return stall;
}

// Time stamp of an event of (iteration j, rank r): what = 0 post, 1 serve, 2 completion.
__device__ __forceinline__ void stamp(const BlsParams &p, long long j, int r, int what, unsigned long long now)
{
    p.stamps[((size_t)(j % BLS_TL_ITERS) * p.P + r) * 3 + what] = now;
}

// Receive-side counts and displacements of the request leg for owner r, iteration j
// (recvcounts = sendcounts transposed, rdispls = exclusive scan over sources).
__device__ __forceinline__ void write_recv_side(const BlsParams &p, int r, long long j)
{
    int *cnt = p.counts + (size_t)(j % p.S) * 4 * p.P * p.P;
    const int *sendcounts = cnt;
    int *recvcounts = cnt + 2 * p.P * p.P, *rdispls = cnt + 3 * p.P * p.P;
    int run = 0;
    for (int src = 0; src < p.P; src++) {
        const int c = sendcounts[src * p.P + r];
        recvcounts[r * p.P + src] = c;
        rdispls[r * p.P + src] = run;
        run += c;
    }
}

__device__ __forceinline__ long long warp_min_ll(long long v)
{
    for (int o = 16; o > 0; o >>= 1) {
        long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w < v ? w : v;
    }
    return v;
}
__device__ __forceinline__ long long warp_max_ll(long long v)
{
    for (int o = 16; o > 0; o >>= 1) {
        long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w > v ? w : v;
    }
    return v;
}

// What a requester needs to route the iteration the gate assigned to it.
struct RouteCtx {
    const int *ids, *off;
    long long n_ids;
    int slot;
    int *sendcounts, *sdispls, *sendbuf, *sub_start;
};

__device__ __forceinline__ bool route_ctx(const BlsParams &p, int src, RouteCtx &c)
{
    long long j = p.dev->route_iter[src];
    if (j < 0) return false;
    c.slot = (int)(j % p.S);
    c.ids = p.dev->in_ids[c.slot];
    c.off = p.dev->in_off[c.slot];
    c.n_ids = p.dev->in_n[c.slot];
    int *cnt = p.counts + (size_t)c.slot * 4 * p.P * p.P;
    c.sendcounts = cnt + src * p.P;
    c.sdispls = cnt + p.P * p.P + src * p.P;
    c.sendbuf = p.sendbuf + ((size_t)c.slot * p.P + src) * (size_t)p.cap;
    c.sub_start = p.sub_start + ((size_t)c.slot * p.P + src) * (size_t)p.sub_stride;
    return true;
}

// Sanitised range of bag g relative to `off0`: 0 <= st <= en <= limit.
__device__ __forceinline__ bool bag_range(const RouteCtx &c, long long g, long long off0, long long limit,
                                          int &st, int &en)
{
    long long a = (long long)c.off[g] - off0, e = (long long)c.off[g + 1] - off0;
    bool ok = a >= 0 && a <= e && e <= limit;
    if (!ok) { a = 0; e = 0; }
    st = (int)a;
    en = (int)e;
    return ok;
}

// Table-wise router, first half, by one warp for requester `src`: the owner depends
// on the table only, so the (requester, table) chunks move as a whole.  Chunk
// lengths come from the offsets alone; an exclusive scan in (owner, table) order
// gives every chunk its place in the packed send buffer, and the send counts and
// displacements follow.  With `publish` the results go to memory (chunk bases, send
// counts, displacements, end of the last sub-bag); in any case the warp learns where
// the chunk of pair `want` starts and ends (the fused kernel for small iterations lets
// every block work that out for itself instead of waiting for another block).
__device__ __forceinline__ void tw_meta_ctx(const BlsParams &p, const RouteCtx &c, int src, int lane, bool publish,
                                            int want, int &cb_want, int &cb_after)
{
    const long long g_rank = (long long)src * p.T * p.b;
    int *cb = p.chunk_base + (size_t)src * (p.NI + 1);
    long long run = 0;
    int mine = 0, after = 0;
    for (int i0 = 0; i0 < p.NI; i0 += 32) {
        const int i = i0 + lane;
        long long n = 0;
        if (i < p.NI) {
            const long long g0 = g_rank + (long long)p.pair[i].t * p.b;
            const long long a = c.off[g0], e = c.off[g0 + p.b];
            n = e - a;
            if (a < 0 || n < 0 || e > c.n_ids) { n = 0; if (publish) flag(p, BLS_ST_EINVAL); }
        }
        long long incl = n;
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        const int base = (int)min(run + incl - n, (long long)0x7fffffff);
        if (i < p.NI && publish) cb[i] = base;
        if (i == want) mine = base;
        if (i == want + 1) after = base;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    const int total = (int)min(run, (long long)0x7fffffff);
    cb_want = __shfl_sync(0xffffffffu, mine, want & 31);
    cb_after = want + 1 < p.NI ? __shfl_sync(0xffffffffu, after, (want + 1) & 31) : total;
    if (!publish) return;
    if (lane == 0) {
        cb[p.NI] = total;
        if (run > p.cap) flag(p, BLS_ST_ENOSPC);
        c.sub_start[p.NQ] = (int)(run > p.cap ? p.cap : run);
    }
    __syncwarp();
    for (int d = lane; d < p.P; d += 32) {
        const int lo = cb[p.pair_first[d]], hi = cb[p.pair_first[d + 1]];
        c.sdispls[d] = lo;
        c.sendcounts[d] = hi - lo;
    }
}

__device__ __forceinline__ void tw_meta_warp(const BlsParams &p, int src, int lane)
{
    RouteCtx c;
    if (!route_ctx(p, src, c)) return;
    int first, second;
    tw_meta_ctx(p, c, src, lane, true, 0, first, second);
}

// Publish the progress of the wave that has just run (lane r = rank r).  For every
// answered iteration also write the receive-side counts and displacements.
__device__ __forceinline__ void commit_lane(const BlsParams &p, int r)
{
    BlsDev *d = p.dev;
    if (r >= p.P) return;
    const unsigned long long now = globaltimer_ns();
    long long j = d->route_iter[r];
    if (j >= 0) {
        d->posted[r] = j + 1;
        stamp(p, j, r, 0, now);
        // route_iter stays as it is until the next gate rewrites it: in overlapped mode the
        // router of this wave may still be running beside the kernel that commits
    }
    j = d->serve_iter[r];
    if (j >= 0) {
        write_recv_side(p, r, j);
        d->served[r] = j + 1;
        d->serve_iter[r] = -1;
        stamp(p, j, r, 1, now);
    }
    j = d->consume_iter[r];
    if (j >= 0) {
        d->done[r] = j + 1;
        d->consume_iter[r] = -1;
        stamp(p, j, r, 2, now);
    }
}

// Called by every thread of every block at the end of the last kernel of a wave:
// the block that finishes last commits the wave.
__device__ __forceinline__ void finish_wave(const BlsParams &p)
{
    __shared__ int s_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&p.dev->done_ctr, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (s_last && threadIdx.x < 32) {
        __threadfence();
        commit_lane(p, threadIdx.x);
    }
}
