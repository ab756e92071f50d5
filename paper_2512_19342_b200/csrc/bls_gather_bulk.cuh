// Table-wise gather with the rows staged in shared memory by the bulk-copy engine
// (cp.async.bulk, one copy per embedding row, completion counted in bytes on an mbarrier).
//
// Same streaming scheme as stream_run: a group of LANES lanes walks the ID stream of a
// run of consecutive sub-bags and adds the rows of a bag in their original order, so the
// results are bit-identical to the register path.  What differs is how a row travels:
// a lane reads one ID and issues ONE bulk copy for the whole row into a ring of
// NST stages x BR rows per lane group; the lanes then add the row from shared memory,
// 16 bytes each.  A row costs one copy instruction instead of LANES load instructions,
// and rows in flight live in shared memory instead of in registers.  The copies read
// this GPU's own tables only and are never multicast.
#pragma once
#include "bls_gather.cuh"

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_arrive(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// One embedding row, global -> shared, completion reported to the mbarrier in bytes.
// Both addresses are 16-byte aligned and the size is a multiple of 16 (rows are 16..512 bytes).
__device__ __forceinline__ void bulk_row(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Per lane group: ring memory and its NST barriers; kb counts the batches the group has
// issued since the kernel started (stage = kb mod NST, phase parity = (kb / NST) & 1).
template <int LANES, int BR, int NST>
struct BulkRing {
    static constexpr int ROW = LANES * 16;
    unsigned rows;          // shared-memory address of the group's NST * BR row slots
    unsigned bars;          // shared-memory address of its NST barriers
    unsigned kb_issue, kb_wait;
};

template <int LANES, int DT, int BR, int NST>
__device__ __forceinline__ void bulk_run(const BlsParams &p, const BlsPairDesc &pr, int i, int slot, int src, int s0,
                                         int nb, int lane, unsigned gmask, BulkRing<LANES, BR, NST> &ring, int &timed_out)
{
    constexpr int ROW = LANES * 16;
    const size_t bag_stride = (size_t)p.T * p.D;
    const int *ss = p.sub_start + ((size_t)slot * p.P + src) * (size_t)p.sub_stride + (size_t)i * p.b + s0;
    const int p0 = min(max(ss[0], 0), p.cap);
    const int n = min(max(ss[nb], p0), p.cap) - p0;    // rows in this run
    auto bag_end = [&](int c) { return c < nb - 1 ? min(max(ss[c + 1] - p0, 0), n) : c == nb - 1 ? n : 0x7fffffff; };
    int cur = 0;
    int e_cur = bag_end(0), e_nxt = bag_end(1);
    const int *sb = p.sendbuf + ((size_t)slot * p.P + src) * (size_t)p.cap + p0;
    const char *tbl = reinterpret_cast<const char *>(pr.base);
    const unsigned nrows_m1 = (unsigned)pr.nrows - 1u;
    float *o = p.out + (size_t)slot * p.out_slot_elems +
               (((size_t)src * p.b + s0) * p.T + pr.t) * p.D + lane * Acc<DT>::N;
    Acc<DT> acc;
    acc.zero();
    const int nbat = (n + BR - 1) / BR;
    constexpr int PER = (BR + LANES - 1) / LANES;      // rows a lane issues per batch
    constexpr int AHEAD = 1;                           // the IDs of a batch are requested this many batches before its copies are issued (measured: 4 is slower)
    int idq[AHEAD][PER];                               // idq[0]: IDs of the batch to be issued next, idq[1]: of the one after, ...

    auto load_ids = [&](int k) {                       // IDs of batch k enter the queue's last place; the queue moves up
        #pragma unroll
        for (int d = 0; d + 1 < AHEAD; d++)
            #pragma unroll
            for (int q = 0; q < PER; q++) idq[d][q] = idq[d + 1][q];
        #pragma unroll
        for (int q = 0; q < PER; q++) {
            const int x = k * BR + q * LANES + lane;
            idq[AHEAD - 1][q] = (k < nbat && q * LANES + lane < BR && x < n) ? __ldcs(sb + x) : 0;
        }
    };
    auto issue = [&](int k) {                          // batch k of the run goes to the next free stage
        if (k >= nbat) return;
        const unsigned st = ring.kb_issue % NST;
        const unsigned bar = ring.bars + st * 8u;
        const int valid = min(BR, n - k * BR);
        if (lane == 0) mbar_expect_tx_arrive(bar, (unsigned)valid * ROW);
        __syncwarp(gmask);
        #pragma unroll
        for (int q = 0; q < PER; q++) {
            const int u = q * LANES + lane;
            if (u < valid)
                bulk_row(ring.rows + (st * BR + u) * ROW, tbl + (size_t)min((unsigned)idq[0][q], nrows_m1) * ROW, ROW, bar);
        }
        ring.kb_issue++;
    };
    auto consume = [&](int k) {
        const unsigned st = ring.kb_wait % NST;
        const unsigned bar = ring.bars + st * 8u;
        const unsigned parity = (ring.kb_wait / NST) & 1u;
        ring.kb_wait++;
        if (!timed_out) {                              // bounded: two seconds on the clock, then no more waiting
            unsigned tries = 0;
            unsigned long long t0 = 0;
            while (!mbar_try_wait(bar, parity)) {
                if ((++tries & 255u) == 0) {
                    const unsigned long long now = globaltimer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > 2000000000ull) { timed_out = 1; break; }
                }
            }
        }
        const unsigned base = ring.rows + st * BR * ROW + lane * 16u;
        const int valid = min(BR, n - k * BR);
        auto lds = [&](int u) {
            uint4 v;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(base + u * ROW));
            return v;
        };
        if (valid == BR && e_cur >= k * BR + BR) {     // a full batch inside one bag
            uint4 v[BR];
            #pragma unroll
            for (int u = 0; u < BR; u++) v[u] = lds(u);
            #pragma unroll
            for (int u = 0; u < BR; u++) acc.add(v[u]);
        } else {
            for (int u = 0; u < valid; u++) {
                const int x = k * BR + u;
                while (x == e_cur) {                   // bags that end here (possibly empty ones)
                    flush<DT>(o, acc);
                    o += bag_stride;
                    acc.zero();
                    cur++;
                    e_cur = e_nxt;
                    e_nxt = bag_end(cur + 1);
                }
                acc.add(lds(u));
            }
        }
        __syncwarp(gmask);                             // every lane has read the stage: it may be refilled
    };

    #pragma unroll
    for (int d = 0; d < AHEAD; d++) load_ids(d);       // the queue holds batches 0 .. AHEAD-1
    for (int k = 0; k < NST && k < nbat; k++) {
        issue(k);
        load_ids(k + AHEAD);
    }
    for (int k = 0; k < nbat; k++) {
        consume(k);
        issue(k + NST);                                // its IDs were requested AHEAD batches ago
        load_ids(k + NST + AHEAD);
    }
    for (; cur < nb; cur++) {                          // the bags after the last row (the last one, and empty ones)
        flush<DT>(o, acc);
        o += bag_stride;
        acc.zero();
    }
}
