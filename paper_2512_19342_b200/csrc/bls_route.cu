// Step 1, the router: every requester rank sorts the rows it needs by owner rank
// (Section I: every rank works out which vector IDs it needs from which other rank and
// fetches them with an alltoallv).  Output per requester:
// sendcounts / sdispls, the stably packed send buffer of owner-local rows, and
// the start of every sub-bag inside it (the owner rebuilds bag boundaries from
// consecutive differences).
//
// Positions never depend on the order in which atomics land: counts come from
// histograms, positions from exclusive scans, so the packed buffer is the unique
// stable counting sort by destination.
//
// Table-wise placement: the owner depends on the table only, so a requester's
// (table) chunks move as a whole; counts follow from the offsets alone.
// Row-wise placement: a real multisplit, done per tile of 128 bags of one table.
#include "bls_route.cuh"

// Blocks of 128 threads and at most 32 registers, 16 to an SM.  In overlapped mode the kernel sits on
// a second stream behind the gather kernel (3 x 256 threads x 80 registers per SM); measured, its
// blocks come in as the gather kernel's retire (kernels whose L1 / shared-memory splits differ are
// not made resident together) and the small blocks fill that tail quickly.
__global__ void __launch_bounds__(128, 16) bls_tw_copy_kernel(BlsParams p) { tw_copy_tile<8>(p, TileFromGrid()); }

__global__ void __launch_bounds__(BLS_ROUTE_TB, 8) bls_rw_count_kernel(BlsParams p) { rw_count_tile(p, TileFromGrid()); }

__global__ void __launch_bounds__(128, 16) bls_rw_scan_kernel(BlsParams p) { rw_scan_tile(p, TileFromGrid()); }

__global__ void __launch_bounds__(BLS_ROUTE_TB, 8) bls_rw_scatter_kernel(BlsParams p) { rw_scatter_tile(p, TileFromGrid()); }

void bls_launch_route_beside(const bls_plan_t *pl, cudaStream_t stream)
{
    const BlsParams &p = pl->prm;
    bls_tw_copy_kernel<<<dim3(p.NT, p.P), 128, 0, stream>>>(p);
}

int bls_route_kernels(const bls_plan_t *pl) { return pl->prm.part == BLS_PART_TABLE_RR ? 1 : 3; }

void bls_launch_route(const bls_plan_t *pl)
{
    const BlsParams &p = pl->prm;
    dim3 grid(p.NT, p.P);
    if (p.part == BLS_PART_TABLE_RR) {
        bls_tw_copy_kernel<<<grid, 128, 0, pl->stream>>>(p);
    } else {
        bls_rw_count_kernel<<<grid, BLS_ROUTE_TB, 0, pl->stream>>>(p);
        bls_rw_scan_kernel<<<dim3(p.P, p.P), 128, 0, pl->stream>>>(p);
        bls_rw_scatter_kernel<<<grid, BLS_ROUTE_TB, rw_scatter_smem(p), pl->stream>>>(p);
    }
}
