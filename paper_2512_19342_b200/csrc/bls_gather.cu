// Steps 2 and 3 fused: the owner-side embedding-bag lookup (gather rows, sum-pool
// per bag with fp32 accumulation; Listing 1's apply_emb) writes each pooled vector
// straight into the requester's output slot out[src][s][t][:], so the pooled
// vectors never make a round trip through memory.
//
// HBM-bound random row reads: a group of LANES = row_bytes/16 lanes owns one
// sub-bag; every lane keeps one 16-byte piece of the row, loads of up to 8 rows
// are issued back to back before the first add (memory-level parallelism), IDs
// are read coalesced and broadcast with shuffles.  Sub-bags are visited
// table-major, so the SMs work on one table at a time and the Zipf-hot rows of
// that table stay in L1/L2.  IDs and outputs use streaming loads/stores so they
// do not evict table rows.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "bls_internal.h"

template <int DT> struct Acc;
template <> struct Acc<BLS_F32> {
    float v[4];
    __device__ __forceinline__ void zero() { v[0] = v[1] = v[2] = v[3] = 0.f; }
    __device__ __forceinline__ void add(const uint4 &u)
    {
        v[0] += __uint_as_float(u.x); v[1] += __uint_as_float(u.y);
        v[2] += __uint_as_float(u.z); v[3] += __uint_as_float(u.w);
    }
    static constexpr int N = 4;
};
template <> struct Acc<BLS_BF16> {
    float v[8];
    __device__ __forceinline__ void zero() { for (int i = 0; i < 8; i++) v[i] = 0.f; }
    __device__ __forceinline__ void add(const uint4 &u)
    {   // a bf16 is the upper half of an fp32: widening is exact
        v[0] += __uint_as_float(u.x << 16); v[1] += __uint_as_float(u.x & 0xffff0000u);
        v[2] += __uint_as_float(u.y << 16); v[3] += __uint_as_float(u.y & 0xffff0000u);
        v[4] += __uint_as_float(u.z << 16); v[5] += __uint_as_float(u.z & 0xffff0000u);
        v[6] += __uint_as_float(u.w << 16); v[7] += __uint_as_float(u.w & 0xffff0000u);
    }
    static constexpr int N = 8;
};
template <> struct Acc<BLS_F16> {
    float v[8];
    __device__ __forceinline__ void zero() { for (int i = 0; i < 8; i++) v[i] = 0.f; }
    __device__ __forceinline__ void add(const uint4 &u)
    {
        const unsigned w[4] = {u.x, u.y, u.z, u.w};
        #pragma unroll
        for (int i = 0; i < 4; i++) {
            float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            v[2 * i] += f.x; v[2 * i + 1] += f.y;
        }
    }
    static constexpr int N = 8;
};

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

template <int LANES, int DT, bool ROWWISE>
__global__ void __launch_bounds__(256) bls_gather_pool_kernel(BlsParams p, long long n_work)
{
    constexpr int U = LANES < 8 ? LANES : 8;           // rows in flight per group and batch
    constexpr int GROUPS = 256 / LANES;
    const int lane = threadIdx.x % LANES;
    const int gidx = threadIdx.x / LANES;
    const unsigned gmask = LANES == 32 ? 0xffffffffu
                                       : (((1u << LANES) - 1u) << ((threadIdx.x & 31) / LANES * LANES));
    const long long Pb = (long long)p.P * p.b;
    const BlsDev *dev = p.dev;

    for (long long w = (long long)blockIdx.x * GROUPS + gidx; w < n_work; w += (long long)gridDim.x * GROUPS) {
        const int i = (int)(w / Pb);                   // (owner, table) pair, owner-major
        const int rem = (int)(w - (long long)i * Pb);
        const int src = rem / p.b, s = rem - src * p.b;
        const BlsPairDesc pr = p.pair[i];
        const long long j = dev->serve_iter[pr.dst];
        if (j < 0) continue;                           // this owner does not serve in this wave
        const int slot = (int)(j % p.S);
        const int *ss = p.sub_start + ((size_t)slot * p.P + src) * (size_t)p.sub_stride + (size_t)i * p.b + s;
        int st = ss[0], en = ss[1];
        st = min(max(st, 0), p.cap);
        en = min(max(en, st), p.cap);
        if (ROWWISE && en == st) continue;             // nothing to add
        const int *sb = p.sendbuf + ((size_t)slot * p.P + src) * (size_t)p.cap;
        const uint4 *base = reinterpret_cast<const uint4 *>(pr.base);
        const unsigned nrows_m1 = (unsigned)pr.nrows - 1u;

        Acc<DT> acc;
        acc.zero();
        for (int c0 = st; c0 < en; c0 += LANES) {
            const int n = min(LANES, en - c0);
            int my = (lane < n) ? __ldcs(sb + c0 + lane) : 0;
            #pragma unroll 1
            for (int u0 = 0; u0 < n; u0 += U) {
                uint4 v[U];
                #pragma unroll
                for (int u = 0; u < U; u++) {
                    unsigned row = (unsigned)__shfl_sync(gmask, my, u0 + u, LANES);
                    row = min(row, nrows_m1);
                    if (u0 + u < n) v[u] = __ldg(base + (size_t)row * LANES + lane);
                    else v[u] = make_uint4(0u, 0u, 0u, 0u);
                }
                #pragma unroll
                for (int u = 0; u < U; u++) acc.add(v[u]);
            }
        }
        float *o = p.out + (size_t)slot * p.out_slot_elems +
                   (((size_t)src * p.b + s) * p.T + pr.t) * p.D + lane * Acc<DT>::N;
        if (ROWWISE) {
            red_add_v4(o, acc.v[0], acc.v[1], acc.v[2], acc.v[3]);
            if (Acc<DT>::N == 8) red_add_v4(o + 4, acc.v[4], acc.v[5], acc.v[6], acc.v[7]);
        } else {
            __stcs(reinterpret_cast<float4 *>(o), make_float4(acc.v[0], acc.v[1], acc.v[2], acc.v[3]));
            if (Acc<DT>::N == 8)
                __stcs(reinterpret_cast<float4 *>(o) + 1, make_float4(acc.v[4], acc.v[5], acc.v[6], acc.v[7]));
        }
    }
}

template <int LANES, int DT>
static void launch_gather(const bls_plan_t *pl)
{
    const BlsParams &p = pl->prm;
    const long long n_work = (long long)p.NI * p.P * p.b;
    const int groups = 256 / LANES;
    long long blocks = (n_work + groups - 1) / groups;
    const long long cap_blocks = (long long)pl->sm_count * 64;
    if (blocks > cap_blocks) blocks = cap_blocks;
    if (blocks < 1) blocks = 1;
    if (p.part == BLS_PART_ROW_BLOCK)
        bls_gather_pool_kernel<LANES, DT, true><<<(unsigned)blocks, 256, 0, pl->stream>>>(p, n_work);
    else
        bls_gather_pool_kernel<LANES, DT, false><<<(unsigned)blocks, 256, 0, pl->stream>>>(p, n_work);
}

template <int DT>
static void launch_gather_dt(const bls_plan_t *pl)
{
    switch (pl->prm.lanes) {
    case 1: launch_gather<1, DT>(pl); break;
    case 2: launch_gather<2, DT>(pl); break;
    case 4: launch_gather<4, DT>(pl); break;
    case 8: launch_gather<8, DT>(pl); break;
    case 16: launch_gather<16, DT>(pl); break;
    default: launch_gather<32, DT>(pl); break;
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
