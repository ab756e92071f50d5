// BLS alltoallv of raw bytes between the P logical ranks (Section III-C), the
// collective on its own, without the lookup around it.
//
// Initiation (bls_a2a_post): for request j every rank puts its P segments into the
// receivers' buffers R(dst, j mod S), S = k_max + 1, and the arrivals are counted per
// (slot, receiver) - the counterpart of the tagged messages the paper counts on the
// NIC.  No rank waits for another.  Completion (bls_a2a_wait): the oldest outstanding
// request is complete when its slot has counted one message from each of the P
// sources; requests complete in issue order and a slot is reused S requests later,
// so at most S requests may be outstanding (k = 0: one, i.e. a plain alltoallv).
//
// On one GPU a post is one kernel over all (src, dst) pairs; the segment of src for
// dst lands at rdispls[dst][src] = sum of the counts of lower-ranked sources, which
// every block derives from the count matrix itself.
#include <stdlib.h>
#include "bls_device.cuh"

struct bls_a2a {
    int P, S;
    long long cap;                 // receive capacity per rank and slot, bytes (multiple of 16)
    char *recv;                    // [S][P][cap]
    long long *recvcounts;         // [S][P][P] indexed [dst][src]
    long long *rdispls;            // [S][P][P]
    int *arrived;                  // [S][P] messages counted per slot and receiver
    int *status;                   // device status word (BLS_ST_* bits)
    int *blocks_done;              // last-block detection of the post kernel
    cudaStream_t stream;
    long long posted, completed;   // host-side request counters
    int sm_count;
};

namespace {

size_t a256(size_t x) { return (x + 255) / 256 * 256; }

struct A2aLayout { size_t recv, recvcounts, rdispls, arrived, status, blocks_done, total; };

A2aLayout a2a_layout(int P, int S, long long cap)
{
    A2aLayout L;
    size_t o = 0;
    auto take = [&](size_t b) { size_t at = o; o = a256(o + b); return at; };
    L.recv = take((size_t)S * P * cap);
    L.recvcounts = take(sizeof(long long) * S * P * P);
    L.rdispls = take(sizeof(long long) * S * P * P);
    L.arrived = take(sizeof(int) * S * P);
    L.status = take(sizeof(int));
    L.blocks_done = take(sizeof(int));
    L.total = o;
    return L;
}

struct A2aArgs {
    int P, slot;
    long long cap, send_stride;
    const char *send;
    const long long *sendcounts, *sdispls;   // [P][P] indexed [src][dst], bytes
    char *recv;                              // slot base: [P][cap]
    long long *recvcounts, *rdispls;         // slot base: [P][P]
    int *arrived;                            // slot base: [P]
    int *status, *blocks_done;
};

// Whether the segment src -> dst is accepted, and where it lands.  Receiver dst takes the
// segments of sources 0, 1, ... in rank order: a segment is accepted when its count and
// displacement lie inside the sender's stride and it still fits behind the accepted
// segments of the lower-ranked sources; a rejected one counts as empty, so the reported
// counts and displacements always agree with each other.
__device__ __forceinline__ bool a2a_accept(const A2aArgs &a, int src, int dst, long long &n, long long &rd, int &why)
{
    rd = 0;
    bool ok = false;
    for (int s2 = 0; s2 <= src; s2++) {
        n = a.sendcounts[s2 * a.P + dst];
        const long long sd = a.sdispls[s2 * a.P + dst];
        const bool inside = n >= 0 && sd >= 0 && sd + n <= a.send_stride;
        ok = inside && rd + n <= a.cap;
        why = inside ? BLS_ST_ENOSPC : BLS_ST_EINVAL;
        if (s2 < src && ok) rd += n;
    }
    return ok;
}

// grid (chunks, P*P): the blocks (*, src*P+dst) copy the segment src -> dst, chunk by chunk
// with stride gridDim.x, so a segment of any length is covered whatever the host's size hint was.
__global__ void __launch_bounds__(256) bls_a2a_put_kernel(A2aArgs a, long long chunk_bytes)
{
    stream_order_enter();
    const int src = blockIdx.y / a.P, dst = blockIdx.y % a.P;
    long long n, rd;
    int why;
    const bool ok = a2a_accept(a, src, dst, n, rd, why);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (!ok) atomicOr(a.status, why);
        a.recvcounts[dst * a.P + src] = ok ? n : 0;
        a.rdispls[dst * a.P + src] = rd;
    }
    if (ok) {
        const char *from = a.send + (size_t)src * a.send_stride + a.sdispls[src * a.P + dst];
        char *to = a.recv + (size_t)dst * a.cap + rd;
        const bool aligned = ((reinterpret_cast<uintptr_t>(from) | reinterpret_cast<uintptr_t>(to)) & 15) == 0;
        for (long long lo = (long long)blockIdx.x * chunk_bytes; lo < n; lo += (long long)gridDim.x * chunk_bytes) {
            const long long hi = min(n, lo + chunk_bytes);
            if (aligned) {
                const long long v_hi = lo + ((hi - lo) & ~15LL);          // 16 bytes per thread while both sides are aligned
                long long i = lo + (long long)threadIdx.x * 16;
                for (; i + 3 * 256 * 16 < v_hi; i += 4 * 256 * 16) {       // four loads in flight per thread
                    uint4 v[4];
                    #pragma unroll
                    for (int q = 0; q < 4; q++) v[q] = __ldcs(reinterpret_cast<const uint4 *>(from + i + q * 256 * 16));
                    #pragma unroll
                    for (int q = 0; q < 4; q++) __stcs(reinterpret_cast<uint4 *>(to + i + q * 256 * 16), v[q]);
                }
                for (; i < v_hi; i += 256 * 16)
                    *reinterpret_cast<uint4 *>(to + i) = __ldcs(reinterpret_cast<const uint4 *>(from + i));
                for (long long i2 = v_hi + threadIdx.x; i2 < hi; i2 += 256) to[i2] = from[i2];
            } else {
                for (long long i = lo + threadIdx.x; i < hi; i += 256) to[i] = from[i];
            }
        }
    }
    // the last block to finish counts the arrivals: at every receiver one message per source
    // whose segment was accepted (all copies are complete by then)
    __shared__ int s_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(a.blocks_done, 1) == (int)(gridDim.x * gridDim.y) - 1;
    }
    __syncthreads();
    if (s_last) {
        if ((int)threadIdx.x < a.P) {
            int got = 0;
            for (int s2 = 0; s2 < a.P; s2++) {
                long long n2, rd2;
                int why2;
                got += a2a_accept(a, s2, threadIdx.x, n2, rd2, why2) ? 1 : 0;
            }
            atomicAdd(&a.arrived[threadIdx.x], got);
        }
        if (threadIdx.x == 0) *a.blocks_done = 0;
    }
}

// Completion check of the oldest request: every receiver of the slot has counted P messages
// (fewer means a segment was rejected, which the post has already reported, or that the
// slot was completed before its request had run).
__global__ void bls_a2a_complete_kernel(int *arrived, int P, int *status)
{
    stream_order_enter();
    const int r = threadIdx.x;
    if (r < P) {
        if (arrived[r] != P) atomicOr(status, BLS_ST_ESTATE);
        arrived[r] = 0;                                   // the slot is free for request j + S
    }
}

}  // namespace

extern "C" {

bls_status_t bls_a2a_bytes(int P, int k_max, int64_t max_bytes_per_rank, size_t *bytes)
{
    if (!bytes || P < 1 || P > BLS_MAX_RANKS || k_max < 0 || k_max + 1 > BLS_MAX_SLOTS || max_bytes_per_rank < 0)
        return BLS_EINVAL;
    *bytes = a2a_layout(P, k_max + 1, (long long)a256((size_t)max_bytes_per_rank)).total;
    return BLS_OK;
}

bls_status_t bls_a2a_create(int P, int k_max, int64_t max_bytes_per_rank, void *workspace, size_t bytes,
                            void *cuda_stream, bls_a2a_t **handle)
{
    if (!handle || !workspace || ((uintptr_t)workspace & 255) || P < 1 || P > BLS_MAX_RANKS || k_max < 0 ||
        k_max + 1 > BLS_MAX_SLOTS || max_bytes_per_rank < 0)
        return BLS_EINVAL;
    const long long cap = (long long)a256((size_t)max_bytes_per_rank);
    A2aLayout L = a2a_layout(P, k_max + 1, cap);
    if (bytes < L.total) return BLS_ENOSPC;
    bls_a2a *h = (bls_a2a *)calloc(1, sizeof(bls_a2a));
    if (!h) return BLS_ENOSPC;
    char *ws = (char *)workspace;
    h->P = P; h->S = k_max + 1; h->cap = cap;
    h->recv = ws + L.recv;
    h->recvcounts = (long long *)(ws + L.recvcounts);
    h->rdispls = (long long *)(ws + L.rdispls);
    h->arrived = (int *)(ws + L.arrived);
    h->status = (int *)(ws + L.status);
    h->blocks_done = (int *)(ws + L.blocks_done);
    h->stream = (cudaStream_t)cuda_stream;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaMemsetAsync(ws + L.recvcounts, 0, L.total - L.recvcounts, h->stream) != cudaSuccess) {
        free(h);
        return BLS_ECUDA;
    }
    *handle = h;
    return BLS_OK;
}

void bls_a2a_destroy(bls_a2a_t *h) { free(h); }

bls_status_t bls_a2a_post(bls_a2a_t *h, const void *sendbuf, int64_t send_stride, const int64_t *sendcounts,
                          const int64_t *sdispls, int64_t max_segment_bytes)
{
    if (!h || !sendbuf || !sendcounts || !sdispls || send_stride < 0 || max_segment_bytes < 0) return BLS_EINVAL;
    if (h->posted - h->completed >= h->S) return BLS_ESTATE;          // all slots hold unread data: wait first
    const int slot = (int)(h->posted % h->S);
    A2aArgs a;
    a.P = h->P; a.slot = slot; a.cap = h->cap; a.send_stride = send_stride;
    a.send = (const char *)sendbuf;
    a.sendcounts = (const long long *)sendcounts;
    a.sdispls = (const long long *)sdispls;
    a.recv = h->recv + (size_t)slot * h->P * h->cap;
    a.recvcounts = h->recvcounts + (size_t)slot * h->P * h->P;
    a.rdispls = h->rdispls + (size_t)slot * h->P * h->P;
    a.arrived = h->arrived + (size_t)slot * h->P;
    a.status = h->status; a.blocks_done = h->blocks_done;
    // four times as many chunks as fill the machine (measured: evens out the tail on large messages), at least 16 KiB each
    long long chunks = ((long long)h->sm_count * 32 + h->P * h->P - 1) / (h->P * h->P);
    long long chunk_bytes = (max_segment_bytes + chunks - 1) / (chunks > 0 ? chunks : 1);
    if (chunk_bytes < 16384) chunk_bytes = 16384;
    chunk_bytes = (chunk_bytes + 15) / 16 * 16;
    chunks = max_segment_bytes > 0 ? (max_segment_bytes + chunk_bytes - 1) / chunk_bytes : 1;
    if (chunks > 65535) return BLS_EINVAL;
    // (small messages are bound by the latency between dependent launches: see stream_order_enter)
    launch_serialised(bls_a2a_put_kernel, dim3((unsigned)chunks, h->P * h->P), dim3(256), h->stream, a, chunk_bytes);
    h->posted++;
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}

bls_status_t bls_a2a_wait(bls_a2a_t *h, const void **recv, int64_t *recv_stride, const int64_t **recvcounts,
                          const int64_t **rdispls, int64_t *request)
{
    if (!h) return BLS_EINVAL;
    if (h->completed == h->posted) return BLS_ESTATE;                 // nothing outstanding
    const int slot = (int)(h->completed % h->S);
    launch_serialised(bls_a2a_complete_kernel, dim3(1), dim3(32), h->stream, h->arrived + (size_t)slot * h->P, h->P, h->status);
    if (recv) *recv = h->recv + (size_t)slot * h->P * h->cap;
    if (recv_stride) *recv_stride = h->cap;
    if (recvcounts) *recvcounts = (const int64_t *)(h->recvcounts + (size_t)slot * h->P * h->P);
    if (rdispls) *rdispls = (const int64_t *)(h->rdispls + (size_t)slot * h->P * h->P);
    if (request) *request = h->completed;
    h->completed++;
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}

bls_status_t bls_a2a_status(bls_a2a_t *h)
{
    if (!h) return BLS_EINVAL;
    int st = 0;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess ||
        cudaMemcpy(&st, h->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return BLS_ECUDA;
    if (st & BLS_ST_EINVAL) return BLS_EINVAL;
    if (st & BLS_ST_ENOSPC) return BLS_ENOSPC;
    if (st & BLS_ST_ESTATE) return BLS_ESTATE;
    return BLS_OK;
}

}  // extern "C"
