// bls_route_table_rr_static: the table-wise router (step 1) for callers that
// cannot allocate device memory.
//
// Who that is: code that runs inside a process whose device memory is owned by
// someone else - an inference server or framework that has reserved the whole
// GPU for its own pool, a plugin that is handed fixed input and output buffers
// and nothing else, a latency-critical loop in which cudaMalloc is unacceptable
// because it synchronises the device and can fail once the pool holds all the
// memory.  Such a caller cannot provide the workspace a plan needs and cannot
// let the library allocate one.
//
// What it does: the same two kernels as the plan-based table-wise router (chunk
// lengths -> exclusive scan -> send counts, displacements and chunk bases; then
// the coalesced copy of every chunk to its place in the packed send buffer and
// the sub-bag starts), except that the chunk-base scratch, which the plan-based
// router keeps in the caller's workspace, lives in a file-scope __device__ array
// of fixed size.  Every GPU that loads the library holds that array (128 KiB)
// until the process exits.  Inputs and outputs are the caller's.
//
// The array is shared by every call on the device and keeps the contents of the
// last call.  The part a call uses is cleared at the start of the call; calls
// whose GPU work overlaps (different streams, or different host threads) race on
// it and must be serialised by the caller.
#include <mutex>
#include "bls_internal.h"

#define BLS_STATIC_MAX_INTS 32768            // capacity of the static scratch: P * (T + 1) must fit

static __device__ __align__(256) int bls_static_scratch[BLS_STATIC_MAX_INTS];

namespace {

// The symbol above is a host-side stand-in, not a device address.  Its device
// address is looked up once per device, with that device current.
std::mutex g_setup_mutex;
int *g_scratch_ptr[64] = {nullptr};

bls_status_t scratch_for_current_device(int **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return BLS_ECUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        int *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, bls_static_scratch) != cudaSuccess || !p) return BLS_ECUDA;
        g_scratch_ptr[dev] = p;
    }
    *ptr = g_scratch_ptr[dev];
    return BLS_OK;
}

// Position of table t in (owner, table) order for round-robin placement over P ranks.
__device__ __forceinline__ int pair_index(int t, int T, int P)
{
    const int d = t % P;
    // owners 0..d-1 hold ceil((T - o) / P) tables each
    int before = 0;
    for (int o = 0; o < d; o++) before += (T - o + P - 1) / P;
    return before + t / P;
}

struct StaticArgs {
    const long long *rows;        // [T] table heights (device)
    const int *ids, *off;         // inputs (device)
    long long n_ids;
    int *sendcounts, *sdispls;    // [P][P]
    int *sendbuf;                 // [P][cap]
    int *sub_start;               // [P][T*b + 1]
    int *status;                  // one int, OR of BLS_ST_* bits
    int *chunk_base;              // static scratch: [P][T + 1]
    long long cap;
    int T, P, b;
};

// One block per requester: chunk lengths from the offsets, exclusive scan in
// (owner, table) order, send counts, displacements, chunk bases.
__global__ void __launch_bounds__(128) bls_static_meta_kernel(StaticArgs a)
{
    const int src = blockIdx.x;
    int *cb = a.chunk_base + (size_t)src * (a.T + 1);
    const long long g_rank = (long long)src * a.T * a.b;
    // chunk lengths, stored at their (owner, table) position
    for (int t = threadIdx.x; t < a.T; t += blockDim.x) {
        const long long g0 = g_rank + (long long)t * a.b;
        long long lo = a.off[g0], hi = a.off[g0 + a.b], n = hi - lo;
        if (lo < 0 || n < 0 || hi > a.n_ids) { n = 0; atomicOr(a.status, BLS_ST_EINVAL); }
        cb[pair_index(t, a.T, a.P)] = (int)n;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long run = 0;
        int i = 0;
        for (int d = 0; d < a.P; d++) {
            const int nt = d < a.T ? (a.T - d + a.P - 1) / a.P : 0;
            // totals beyond the 32-bit range are clamped (and reported below as exceeding cap), so
            // that no chunk base can wrap to a negative position
            a.sdispls[src * a.P + d] = (int)min(run, (long long)0x7fffffff);
            const long long before = run;
            for (int q = 0; q < nt; q++, i++) {
                const int n = cb[i];
                cb[i] = (int)min(run, (long long)0x7fffffff);
                run += n;
            }
            a.sendcounts[src * a.P + d] = (int)min(run - before, (long long)0x7fffffff);
        }
        cb[a.T] = (int)min(run, (long long)0x7fffffff);
        if (run > a.cap) atomicOr(a.status, BLS_ST_ENOSPC);
        a.sub_start[(size_t)src * ((size_t)a.T * a.b + 1) + (size_t)a.T * a.b] = (int)(run > a.cap ? a.cap : run);
    }
}

// grid (T * ceil(b / 128), P): copies one tile of a (requester, table) chunk.
__global__ void __launch_bounds__(256) bls_static_copy_kernel(StaticArgs a, int tiles_per_table)
{
    const int src = blockIdx.y;
    const int t = blockIdx.x / tiles_per_table;
    const int s0 = (blockIdx.x % tiles_per_table) * BLS_ROUTE_TB;
    const int nb = min(BLS_ROUTE_TB, a.b - s0);
    const int i = pair_index(t, a.T, a.P);
    const int *cbp = a.chunk_base + (size_t)src * (a.T + 1);
    const int cb = cbp[i], cn = cbp[i + 1] - cb;
    const long long g0 = ((long long)src * a.T + t) * a.b;
    const long long off0 = a.off[g0];
    int *sub = a.sub_start + (size_t)src * ((size_t)a.T * a.b + 1) + (size_t)i * a.b + s0;
    __shared__ int s_lo, s_hi;
    if (threadIdx.x < nb) {
        long long st = (long long)a.off[g0 + s0 + threadIdx.x] - off0, en = (long long)a.off[g0 + s0 + threadIdx.x + 1] - off0;
        if (!(st >= 0 && st <= en && en <= cn)) { st = en = 0; atomicOr(a.status, BLS_ST_EINVAL); }
        const long long pos = cb + st;
        sub[threadIdx.x] = (int)(pos > a.cap ? a.cap : pos);
        if (threadIdx.x == 0) s_lo = (int)st;
        if (threadIdx.x == nb - 1) s_hi = (int)en;
    }
    __syncthreads();
    // a table height below 1 is malformed input: reported, and every ID of the table is then out of range
    const long long rows_in = a.rows[t];
    if (rows_in < 1 && threadIdx.x == 0) atomicOr(a.status, BLS_ST_EINVAL);
    const unsigned long long rows = rows_in < 1 ? 0ull : (unsigned long long)rows_in;
    const int lo = s_lo, hi = max(s_lo, s_hi);
    int *dst = a.sendbuf + (size_t)src * a.cap;
    for (int l = lo + threadIdx.x; l < hi; l += blockDim.x) {
        int id = a.ids[off0 + l];
        if ((unsigned long long)(unsigned)id >= rows) { id = 0; atomicOr(a.status, BLS_ST_ERANGE); }
        const long long pos = (long long)cb + l;
        if (pos >= 0 && pos < a.cap) dst[pos] = id;
    }
}

}  // namespace

extern "C" bls_status_t bls_route_table_rr_static(const int64_t *table_rows, int T, int P, int local_batch,
                                                  const int32_t *ids, const int32_t *offsets, int64_t n_ids,
                                                  int32_t *sendcounts, int32_t *sdispls, int32_t *sendbuf,
                                                  int64_t cap, int32_t *sub_start, int32_t *status,
                                                  void *cuda_stream)
{
    if (!table_rows || !offsets || (!ids && n_ids > 0) || !sendcounts || !sdispls || !sendbuf || !sub_start ||
        !status || T < 1 || P < 1 || P > BLS_MAX_RANKS || local_batch < 1 || n_ids < 0 || cap < 1 ||
        cap > 0x7ffffff0LL || (long long)P * T * local_batch > 0x7ffffff0LL)
        return BLS_EINVAL;
    if ((long long)P * (T + 1) > BLS_STATIC_MAX_INTS) return BLS_ENOSPC;   // beyond the static scratch
    int *scratch = nullptr;
    bls_status_t st = scratch_for_current_device(&scratch);
    if (st != BLS_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the array keeps the previous call's contents: clear the part this call uses, and the status word
    if (cudaMemsetAsync(scratch, 0, sizeof(int) * (size_t)P * (T + 1), s) != cudaSuccess ||
        cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess)
        return BLS_ECUDA;
    StaticArgs a;
    a.rows = (const long long *)table_rows;
    a.ids = ids; a.off = offsets; a.n_ids = n_ids;
    a.sendcounts = sendcounts; a.sdispls = sdispls; a.sendbuf = sendbuf; a.sub_start = sub_start;
    a.status = status; a.chunk_base = scratch; a.cap = cap; a.T = T; a.P = P; a.b = local_batch;
    const int tpt = (local_batch + BLS_ROUTE_TB - 1) / BLS_ROUTE_TB;
    bls_static_meta_kernel<<<P, 128, 0, s>>>(a);
    bls_static_copy_kernel<<<dim3(T * tpt, P), 256, 0, s>>>(a, tpt);
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}
