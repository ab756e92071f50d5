// Device code of steps 2 and 3 (gather, sum-pool, return), shared by the stand-alone
// gather kernels and the persistent ring kernel.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <type_traits>
#include "bls_device.cuh"

// fp32 accumulators as packed pairs: sm_100 adds two fp32 lanes per instruction
// (round-to-nearest, identical to two scalar adds).
template <int DT> struct Acc;
template <> struct Acc<BLS_F32> {
    static constexpr int N = 4;
    float2 a, b;
    __device__ __forceinline__ void zero() { a = b = make_float2(0.f, 0.f); }
    __device__ __forceinline__ void add(const uint4 &u)
    {
        a = __fadd2_rn(a, make_float2(__uint_as_float(u.x), __uint_as_float(u.y)));
        b = __fadd2_rn(b, make_float2(__uint_as_float(u.z), __uint_as_float(u.w)));
    }
    __device__ __forceinline__ float4 lo() const { return make_float4(a.x, a.y, b.x, b.y); }
    __device__ __forceinline__ float4 hi() const { return make_float4(0.f, 0.f, 0.f, 0.f); }
};
template <> struct Acc<BLS_BF16> {
    static constexpr int N = 8;
    float2 a, b, c, d;
    __device__ __forceinline__ void zero() { a = b = c = d = make_float2(0.f, 0.f); }
    // a bf16 is the upper half of an fp32: widening is exact
    static __device__ __forceinline__ float2 w(unsigned u)
    {
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
    }
    __device__ __forceinline__ void add(const uint4 &u)
    {
        a = __fadd2_rn(a, w(u.x)); b = __fadd2_rn(b, w(u.y));
        c = __fadd2_rn(c, w(u.z)); d = __fadd2_rn(d, w(u.w));
    }
    __device__ __forceinline__ float4 lo() const { return make_float4(a.x, a.y, b.x, b.y); }
    __device__ __forceinline__ float4 hi() const { return make_float4(c.x, c.y, d.x, d.y); }
};
template <> struct Acc<BLS_F16> {
    static constexpr int N = 8;
    float2 a, b, c, d;
    __device__ __forceinline__ void zero() { a = b = c = d = make_float2(0.f, 0.f); }
    static __device__ __forceinline__ float2 w(unsigned u)
    {
        return __half22float2(*reinterpret_cast<const __half2 *>(&u));
    }
    __device__ __forceinline__ void add(const uint4 &u)
    {
        a = __fadd2_rn(a, w(u.x)); b = __fadd2_rn(b, w(u.y));
        c = __fadd2_rn(c, w(u.z)); d = __fadd2_rn(d, w(u.w));
    }
    __device__ __forceinline__ float4 lo() const { return make_float4(a.x, a.y, b.x, b.y); }
    __device__ __forceinline__ float4 hi() const { return make_float4(c.x, c.y, d.x, d.y); }
};

// A lane's share of a pooled vector: 16 bytes for fp32 tables, 32 bytes (two 16-byte stores) for
// 16-bit tables.  Streaming stores: outputs are not read again by this kernel.  (One 256-bit
// store per lane, which writes each 32-byte sector once instead of twice, was measured and is
// no faster: the store path does not limit these kernels.)
template <int DT>
__device__ __forceinline__ void flush(float *o, const Acc<DT> &acc)
{
    __stcs(reinterpret_cast<float4 *>(o), acc.lo());
    if (Acc<DT>::N == 8) __stcs(reinterpret_cast<float4 *>(o) + 1, acc.hi());
}

// One run: nb consecutive sub-bags of pair `pr` requested by rank `src`, starting at
// sample s0, in ring slot `slot`.  With HOT, lookups whose slot number (written by
// the router) is below K read their row from the staged copy in shared memory.
// `end_pos` >= 0 gives the send-buffer position where the run's IDs end, for a caller that
// knows it while the start of the sub-bag after the run may not be in memory yet.
template <int LANES, int DT, int U, bool HOT>
__device__ __forceinline__ void stream_run(const BlsParams &p, const BlsPairDesc &pr, int i, int slot, int src,
                                           int s0, int nb, int lane, const uint4 *hot_rows, int end_pos = -1)
{
    constexpr int Q = U / 4;                           // 16-byte ID quads per batch
    const size_t bag_stride = (size_t)p.T * p.D;       // floats between consecutive samples in out
    const int *ss = p.sub_start + ((size_t)slot * p.P + src) * (size_t)p.sub_stride + (size_t)i * p.b + s0;
    const int p0 = min(max(ss[0], 0), p.cap);
    const int n = min(max(end_pos >= 0 ? end_pos : ss[nb], p0), p.cap) - p0;    // rows in this run
    // The ID stream is read in aligned 16-byte quads and processed in whole batches
    // of U rows: stream coordinate y = a + x, where x counts the run's rows and
    // a = p0 mod 4.  The a IDs before the run and the IDs after it up to the end of
    // the last batch belong to other bags (or to nobody); their rows are loaded
    // (clamped, so always in bounds) and accumulated into a "bag" that is never
    // stored.  That keeps the inner loop free of validity predicates.
    const int a = p0 & 3;
    const int yend = a + n;
    const int org = a - p0;                            // y coordinate of send-buffer position 0
    // bag c of the run ends at bag_end(c); c = -1 is the part before the run, c = nb the part after
    auto bag_end = [&](int c) {
        return c < 0 ? a : c < nb - 1 ? min(max(ss[c + 1] + org, a), yend) : c == nb - 1 ? yend : 0x7fffffff;
    };
    int cur = -1;
    int e_cur = a, e_nxt = bag_end(0);
    const size_t row0 = ((size_t)slot * p.P + src) * (size_t)p.cap + (p0 - a);
    const int4 *sq = reinterpret_cast<const int4 *>(p.sendbuf + row0);
    const uint2 *hq = HOT ? reinterpret_cast<const uint2 *>(p.hot.hotslot + row0) : nullptr;
    const uint4 *rowbase = reinterpret_cast<const uint4 *>(pr.base) + lane;
    const unsigned nrows_m1 = (unsigned)pr.nrows - 1u;
    const unsigned K = HOT ? (unsigned)p.hot.K : 0u;
    float *o = p.out + (size_t)slot * p.out_slot_elems +
               (((size_t)src * p.b + s0) * p.T + pr.t) * p.D + lane * Acc<DT>::N;

    Acc<DT> acc;
    acc.zero();
    int4 ida[Q], idb[Q];                               // IDs of the next batch for va / for vb
    uint2 ha[Q], hb[Q];                                // and their staged-copy slots
    uint4 va[U], vb[U];
    const int nbat = (yend + U - 1) / U;

    auto load_ids = [&](int4(&idq)[Q], uint2(&hsq)[Q], int k) {
        if (k >= nbat) return;
        #pragma unroll
        for (int q = 0; q < Q; q++) {
            idq[q] = __ldcs(sq + k * Q + q);
            if (HOT) hsq[q] = __ldcs(hq + k * Q + q);
        }
    };
    auto issue = [&](uint4(&v)[U], const int4(&idq)[Q], const uint2(&hsq)[Q], int k) {
        if (k >= nbat) return;
        #pragma unroll
        for (int u = 0; u < U; u++) {
            const unsigned id = (unsigned)(&idq[u / 4].x)[u & 3];
            if constexpr (HOT) {
                const unsigned w = (&hsq[u / 4].x)[(u & 3) >> 1];
                const unsigned hs = (u & 1) ? (w >> 16) : (w & 0xffffu);
                // one generic load, no branch: the address is in shared memory for a staged row,
                // in the table otherwise (lane groups of a warp differ, a branch would diverge)
                const uint4 *src_row = hs < K ? hot_rows + hs * LANES + lane : rowbase + (size_t)min(id, nrows_m1) * LANES;
                v[u] = *src_row;
            } else {
                v[u] = __ldg(rowbase + (size_t)min(id, nrows_m1) * LANES);
            }
        }
    };
    auto consume = [&](const uint4(&v)[U], int k) {
        if (k >= nbat) return;
        if (e_cur >= k * U + U) {                      // no bag ends inside this batch
            #pragma unroll
            for (int u = 0; u < U; u++) acc.add(v[u]);
            return;
        }
        #pragma unroll
        for (int u = 0; u < U; u++) {
            const int y = k * U + u;
            while (y == e_cur) {                       // bags that end here (possibly empty ones)
                if (cur >= 0) {
                    flush<DT>(o, acc);
                    o += bag_stride;
                }
                acc.zero();
                cur++;
                e_cur = e_nxt;
                e_nxt = bag_end(cur + 1);
            }
            acc.add(v[u]);
        }
    };

    // Pipeline: the IDs of a batch are fetched two batches before its rows are
    // requested, and its rows one batch before they are added, so that neither the ID
    // latency nor the row latency sits on the critical path.
    load_ids(ida, ha, 0);
    load_ids(idb, hb, 1);
    issue(va, ida, ha, 0);
    load_ids(ida, ha, 2);
    for (int k = 0; k < nbat; k += 2) {
        issue(vb, idb, hb, k + 1);
        load_ids(idb, hb, k + 3);
        consume(va, k);
        issue(va, ida, ha, k + 2);
        load_ids(ida, ha, k + 4);
        consume(vb, k + 1);
    }
    // bags not closed by a row after them: the last one when the run ends on a batch
    // boundary, and everything when the run has no rows at all
    if (cur < 0) { cur = 0; acc.zero(); }
    for (; cur < nb; cur++) {
        flush<DT>(o, acc);
        o += bag_stride;
        acc.zero();
    }
}

// Row-wise placement: the IDs of one bag are spread over the owners' regions of the
// requester's send buffer, a handful per owner.  One lane group takes a bag, walks
// the owners in rank order (their sub-bag starts are stored bag-major, so the P
// starts and P ends of a bag are two contiguous reads), gathers every owner's rows
// and keeps one running fp32 sum: the owners' partial sums are combined in owner
// order inside registers and the pooled vector is stored once.  No atomics, no
// zero-filled output, and the result does not depend on timing.
template <int LANES, int DT>
__device__ __forceinline__ void rowwise_run(const BlsParams &p, int slot, int run, int R, int runs_per_chunk, int lane, int g)
{
    constexpr int U = LANES < 8 ? LANES : 8;
    const unsigned gmask = LANES == 32 ? 0xffffffffu : (((1u << LANES) - 1u) << (g * LANES));
    const int chunk = run / runs_per_chunk;    // (table, requester), table-major
    const int s0 = (run - chunk * runs_per_chunk) * R;
    const int t = chunk / p.P, src = chunk - t * p.P;
    const int nb = min(R, p.b - s0);
    const BlsTableDesc tb = p.tab[t];
    const uint4 *rowbase = reinterpret_cast<const uint4 *>(tb.weight) + lane;
    const unsigned rows_m1 = (unsigned)tb.rows - 1u;
    const int *sb = p.sendbuf + ((size_t)slot * p.P + src) * (size_t)p.cap;
    const int *ss = p.sub_start + ((size_t)slot * p.P + src) * (size_t)p.sub_stride +
                    ((size_t)t * p.b + s0) * p.P;
    float *o = p.out + (size_t)slot * p.out_slot_elems +
               (((size_t)src * p.b + s0) * p.T + t) * p.D + lane * Acc<DT>::N;
    if (p.P <= LANES) {
        // All owners fit in one lane group (lane d = owner d).  Three bags are in
        // flight: while the rows of bag k are loaded and added, the IDs of bag k+1
        // are already on their way and the bounds of bags k+2, k+3 are being fetched,
        // so only the row loads are ever waited for.
        const int d = lane;
        const bool own_lane = d < p.P;
        auto bound = [&](int k) { return own_lane ? min(max(ss[(size_t)k * p.P + d], 0), p.cap) : 0; };
        struct Pre { int idv, own, total, st, excl; };
        auto prepare = [&](int st, int en_raw) {        // scan the owners' counts, fetch this lane's ID
            Pre q;
            const int n = max(en_raw - st, 0);
            int incl = n;
            #pragma unroll
            for (int w = 1; w < LANES; w <<= 1) {
                const int y = __shfl_up_sync(gmask, incl, w, LANES);
                if (lane >= w) incl += y;
            }
            q.st = st;
            q.excl = incl - n;
            q.total = __shfl_sync(gmask, incl, LANES - 1, LANES);
            int own = 0;                                // last lane whose first row is <= lane
            #pragma unroll
            for (int step = LANES / 2; step >= 1; step >>= 1) {
                const int ex = __shfl_sync(gmask, q.excl, own + step, LANES);
                if (ex <= lane) own += step;
            }
            const int pos = __shfl_sync(gmask, st, own, LANES) + lane - __shfl_sync(gmask, q.excl, own, LANES);
            q.own = own;
            q.idv = lane < q.total ? __ldcs(sb + min(pos, p.cap - 1)) : 0;
            return q;
        };
        int r0v = bound(0), r1v = bound(1);
        int r2v = nb >= 2 ? bound(2) : 0;
        Pre cur = prepare(r0v, r1v);
        int st_n = r1v, en_n = r2v;                     // bounds of bag 1
        for (int bag = 0; bag < nb; bag++, o += (size_t)p.T * p.D) {
            const int r3v = bag + 3 <= nb ? bound(bag + 3) : 0;            // bounds two bags ahead
            Pre nxt = cur;
            if (bag + 1 < nb) nxt = prepare(st_n, en_n);                   // IDs one bag ahead
            Acc<DT> acc;
            acc.zero();
            const unsigned grow = min((unsigned)cur.own * (unsigned)tb.blk + (unsigned)cur.idv, rows_m1);
            const int m = min(LANES, cur.total);
            #pragma unroll 1
            for (int u0 = 0; u0 < m; u0 += U) {
                uint4 v[U];
                #pragma unroll
                for (int u = 0; u < U; u++) {
                    const unsigned row = __shfl_sync(gmask, grow, u0 + u, LANES);
                    v[u] = (u0 + u < m) ? __ldg(rowbase + (size_t)row * LANES) : make_uint4(0u, 0u, 0u, 0u);
                }
                #pragma unroll
                for (int u = 0; u < U; u++)
                    if (u0 + u < m) acc.add(v[u]);
            }
            for (int r0 = LANES; r0 < cur.total; r0 += LANES) {           // rare: more rows than lanes
                const int r = r0 + lane;
                int own = 0;
                #pragma unroll
                for (int step = LANES / 2; step >= 1; step >>= 1) {
                    const int ex = __shfl_sync(gmask, cur.excl, own + step, LANES);
                    if (ex <= r) own += step;
                }
                const int pos = __shfl_sync(gmask, cur.st, own, LANES) + r - __shfl_sync(gmask, cur.excl, own, LANES);
                unsigned g2 = 0;
                if (r < cur.total) g2 = min((unsigned)own * (unsigned)tb.blk + (unsigned)__ldcs(sb + min(pos, p.cap - 1)), rows_m1);
                const int m2 = min(LANES, cur.total - r0);
                for (int u = 0; u < m2; u++) {
                    const unsigned row = __shfl_sync(gmask, g2, u, LANES);
                    acc.add(__ldg(rowbase + (size_t)row * LANES));
                }
            }
            flush<DT>(o, acc);
            cur = nxt;
            st_n = en_n;
            en_n = r3v;
        }
    } else {
        for (int bag = 0; bag < nb; bag++, ss += p.P, o += (size_t)p.T * p.D) {
            Acc<DT> acc;
            acc.zero();
            for (int c0 = 0; c0 < p.P; c0 += LANES) {      // owners c0 .. c0+LANES-1, one per lane
                const int d = c0 + lane;
                int st = 0, en = 0;
                if (d < p.P) {
                    st = min(max(ss[d], 0), p.cap);
                    en = min(max(ss[p.P + d], st), p.cap);
                }
                const int n = en - st;
                int incl = n;                               // inclusive scan over the group's lanes
                #pragma unroll
                for (int w = 1; w < LANES; w <<= 1) {
                    const int y = __shfl_up_sync(gmask, incl, w, LANES);
                    if (lane >= w) incl += y;
                }
                const int excl = incl - n;
                const int total = __shfl_sync(gmask, incl, LANES - 1, LANES);
                for (int r0 = 0; r0 < total; r0 += LANES) {
                    const int r = r0 + lane;                // this lane fetches the ID of row r
                    int own = 0;                            // last lane whose first row is <= r
                    #pragma unroll
                    for (int step = LANES / 2; step >= 1; step >>= 1) {
                        const int ex = __shfl_sync(gmask, excl, own + step, LANES);
                        if (ex <= r) own += step;
                    }
                    const int pos = __shfl_sync(gmask, st, own, LANES) + r - __shfl_sync(gmask, excl, own, LANES);
                    unsigned grow = 0;
                    if (r < total) {
                        const unsigned id = (unsigned)__ldcs(sb + pos);
                        grow = min((unsigned)(c0 + own) * (unsigned)tb.blk + id, rows_m1);
                    }
                    const int m = min(LANES, total - r0);
                    #pragma unroll 1
                    for (int u0 = 0; u0 < m; u0 += U) {
                        uint4 v[U];
                        #pragma unroll
                        for (int u = 0; u < U; u++) {
                            const unsigned row = __shfl_sync(gmask, grow, u0 + u, LANES);
                            v[u] = (u0 + u < m) ? __ldg(rowbase + (size_t)row * LANES) : make_uint4(0u, 0u, 0u, 0u);
                        }
                        #pragma unroll
                        for (int u = 0; u < U; u++)
                            if (u0 + u < m) acc.add(v[u]);
                    }
                }
            }
            flush<DT>(o, acc);
        }
    }
}
