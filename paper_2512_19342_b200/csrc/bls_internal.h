// Internal structures shared by the kernels and the host API of libbls.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "bls.h"

#define BLS_MAX_RANKS 32
#define BLS_MAX_SLOTS 16
#define BLS_ROUTE_TB 128          // smallest routing tile in bags; threads per block of the row-wise router

// step modes understood by the gate kernel
enum { BLS_MODE_STEP = 0, BLS_MODE_DRAIN = 1, BLS_MODE_ROUTE_ONLY = 2, BLS_MODE_LOOKUP_ONLY = 3 };

// bits of the device status word
enum { BLS_ST_EINVAL = 1, BLS_ST_ENOSPC = 2, BLS_ST_ERANGE = 4, BLS_ST_ETIMEOUT = 8, BLS_ST_ESTATE = 16 };

// ---- persistent ring kernel (bls_event.cu): a queue of actions that a scheduler warp
// publishes and worker blocks execute tile by tile, all inside one launch ----
#define BLS_Q_CAP 4096            // actions one launch can publish: at most (k_max + 1) iterations x 4 P
enum { BLS_ACT_TW_META = 0, BLS_ACT_TW_COPY, BLS_ACT_RW_COUNT, BLS_ACT_RW_SCAN, BLS_ACT_RW_SCATTER,
       BLS_ACT_GATHER_TW, BLS_ACT_GATHER_RW };
struct BlsAct {
    int kind;           // BLS_ACT_*
    int rank;           // requester (router actions) or owner (table-wise gather)
    int slot;           // ring slot of the iteration
    int n_tiles;        // tiles of BLS_ROUTE_TB threads' work
    int next;           // next tile to hand out (atomic)
    int finished;       // tiles completed (atomic)
    int aux;            // gather actions: number of runs
    int first;          // table-wise gather: the owner's first (owner, table) pair
};
struct BlsQueue {
    unsigned tail;      // actions published so far in this launch (release / acquire)
    int exit;           // set by the scheduler when the launch is over
    int exited;         // blocks that have left; the last one clears this header for the next launch
    int pad;
    BlsAct act[BLS_Q_CAP];
};
// what a logical rank is doing between two posts (event-driven mode)
enum { BLS_RS_IDLE = 0,        // previous iteration dealt with; the delay of the next one has not started
       BLS_RS_DELAY = 1,       // inside its injected delay (until ready_ns)
       BLS_RS_WANT_POST = 2,   // ready to post as soon as the slot is free and the inputs are there
       BLS_RS_POSTING = 3,     // router actions in flight
       BLS_RS_AFTER_POST = 4 };// posted; completes what has arrived, blocks while more than k are outstanding
#define BLS_TL_ITERS 1024         // iterations whose time stamps are kept (a ring indexed by iteration mod this)

// Device-resident state of the slot ring.  Counters are monotone: posted[r] =
// iterations whose requests rank r has put into the owners' slots, served[o] =
// iterations owner o has answered, done[r] = iterations rank r has completed.
struct BlsDev {
    long long posted[BLS_MAX_RANKS];
    long long served[BLS_MAX_RANKS];
    long long done[BLS_MAX_RANKS];
    unsigned long long ready_ns[BLS_MAX_RANKS];   // rank may act again at this globaltimer value
    unsigned long long stall_ns[BLS_MAX_RANKS];   // injected delay before each iteration
    unsigned long long stall_rand_ns[BLS_MAX_RANKS];  // plus a uniform random part in [0, this]
    unsigned long long stall_seed;                // seed of the counter-based generator for the random part
    // plan of the current wave: iteration each rank routes / serves / completes, or -1
    long long route_iter[BLS_MAX_RANKS];
    long long serve_iter[BLS_MAX_RANKS];
    long long consume_iter[BLS_MAX_RANKS];
    // inputs of the iterations that are still in the ring, by slot
    const int *in_ids[BLS_MAX_SLOTS];
    const int *in_off[BLS_MAX_SLOTS];
    long long in_n[BLS_MAX_SLOTS];
    int rstate[BLS_MAX_RANKS];                    // BLS_RS_*: event-driven mode only
    unsigned long long wait_limit_ns;
    long long max_lag;                            // max over time of newest posted - oldest incomplete
    int status;                                   // OR of BLS_ST_* bits
    int work_ctr;                                 // next run of the gather kernel (reset by the gate)
    int done_ctr;                                 // blocks of the wave's last kernel that have finished
    int small_ctr;                                // blocks of the fused small-iteration kernel that have finished (its last block resets it)
};

struct BlsTableDesc {
    const void *weight;
    long long rows;
    int blk;            // ceil(rows / P) for row-block placement, else 0
    unsigned magic;     // floor(2^32 / blk) (2^32 - 1 for blk = 1): division by blk as a multiply
};

// A (owner, table) pair in owner-major order.  Table-wise: one pair per table.
// Row-wise: P pairs per table.
struct BlsPairDesc {
    const void *base;   // first row this owner holds of the table
    int t;              // table number
    int dst;            // owner rank
    int nrows;          // rows the owner holds (for clamping); >= 1
    int pad;
};

// Hot-row staging (optional, table-wise placement): per table the K most frequently
// requested rows, found from observed ID batches, are copied into shared memory by
// the gather kernel; the router marks every lookup with its slot in that copy.
struct BlsHot {
    int enabled;                 // lists built: the router marks lookups, the gather kernel stages rows
    int K;                       // slots per table
    unsigned *counts;            // [sum rows]    observed request counts
    unsigned *bitmap;            // [sum words]   bit r of table t set: row r is hot
    unsigned *prefix;            // [sum words]   hot rows of the table before this word
    const long long *row_base;   // [T+1] first counter of table t
    const long long *word_base;  // [T+1] first bitmap word of table t
    int *rows;                   // [T][K] hot row numbers, slot order
    int *count;                  // [T]    hot rows of table t (<= K)
    unsigned short *hotslot;     // [S][P][cap] slot of every packed lookup, 0xFFFF = not staged
    int *pair_ctr;               // [NI]   next run of each (owner, table) pair (reset by the gate)
};

struct BlsParams {
    int P, T, b, part, S, D, dtype, lanes;
    int NI;                 // number of (owner, table) pairs
    int NQ;                 // sub-bags per requester = NI * b
    int cap;                // IDs per rank per iteration (send buffer capacity)
    int NT;                 // routing tiles per requester = T * tiles_per_table
    int tiles_per_table;    // ceil(b / tile_bags)
    int tile_bags;          // bags per routing tile: BLS_ROUTE_TB or a power-of-two multiple of it
    int row_bytes;
    BlsDev *dev;
    const BlsTableDesc *tab;     // [T]
    const BlsPairDesc *pair;     // [NI]
    const int *pair_of_table;    // [T] index of table t's (first) pair; row-wise: unused
    const int *pair_first;       // [P+1] first pair of owner d (pairs are owner-major); [P] = NI
    int *counts;                 // [S][4][P][P]: sendcounts, sdispls, recvcounts, rdispls
    int *sendbuf;                // [S][P][cap]
    int *sub_start;              // [S][P][sub_stride]
    float *out;                  // [S][P][b][T][D]
    int *chunk_base;             // [P][NI+1]   table-wise: start of each (src, table) chunk
    int *tile_cnt;               // [P][NT][P]  row-wise: per tile, per destination counts / bases
    int *rw_total;               // [P][P]      row-wise: lookups of requester src that go to d (zeroed by the gate)
    BlsQueue *queue;             // action queue of the persistent ring kernel
    unsigned long long *stamps;  // [BLS_TL_ITERS][P][3] globaltimer at post / serve / completion of (iteration, rank)
    int *stage_ids;              // [S][P*cap]  staging for host inputs
    int *stage_off;              // [S][G+1]
    long long sub_stride;        // NQ + 1 rounded up to a multiple of 4
    long long out_slot_elems;    // P*b*T*D
    BlsHot hot;
};

struct bls_plan {
    BlsParams prm;
    cudaStream_t stream;
    int k_max;
    int k_cur;              // bound in use, -1 when nothing is outstanding
    long long t_next;       // next iteration to issue
    long long t_handed;     // iterations handed back so far
    long long routed_only;  // iteration routed by bls_route and not yet looked up, or -1
    size_t bytes;
    int sm_count;
    // optional stage timing (events are created on first use, 4 per recorded call)
    int prof_on;
    int prof_n;
    cudaEvent_t *prof_ev;
    // host-buffer entry points: copy streams and events, created on first use
    cudaStream_t s_in, s_out;
    cudaEvent_t e_in, e_comp, e_out;
    int host_path;
    long long comp_iter;          // value of t_next when e_comp was last recorded (it then marks the end of iteration t_next - 1)
    long long kernels_launched;   // total kernels enqueued through this plan
    int any_stall;                // a delay was injected at some point: ranks may be out of lockstep
    int bags_per_run;             // gather kernel: consecutive sub-bags streamed by one lane group
    int rows_in_flight;           // gather kernel: row loads per batch (4 or 8)
    long long *h_rows;            // host copy of the table heights
    int ring_used;                // the loop in progress has used the ring kernel: its drain does too (ranks may be behind)
    int ring_mode;                // persistent ring kernel: -1 only with injected delays, 0 also for small iterations, 1 always
    int ring_blocks_per_sm;       // resident blocks of the ring kernel per SM (0 = not queried yet)
    int poison;                   // debug: fill an output slot with NaN patterns before an iteration is issued into it
    int hot_attached;             // a hot-row buffer has been attached
    // overlapped mode (bound >= 1, table-wise, no injected delays): the router of iteration t
    // runs on a stream of its own beside the gather kernel of iteration t - 1
    cudaStream_t s_side;
    cudaEvent_t e_fork, e_join;
    int side_ready;
    int unserved;                 // iterations posted whose answer has not been enqueued yet (0 or 1)
    int overlap_mode;             // -1 never, 0 chosen by the size of an iteration, 1 whenever the mode applies
    int fused_mode;               // one-launch kernel for small table-wise iterations: -1 never, 0 chosen by size, 1 whenever it applies
};
#define BLS_PROF_MAX 1024

// kernel launchers (defined in the .cu files)
void bls_launch_gate(const bls_plan_t *pl, int mode, long long t_last, long long forced_floor, int k,
                     const int *ids, const int *off, long long n_ids, int overlapped = 0);
// one launch of the persistent ring kernel (event-driven mode); returns a cudaError_t as int
int bls_launch_ring(bls_plan_t *pl, int mode, long long t_last, long long floor_, int k,
                    const int *ids, const int *off, long long n_ids);
void bls_gather_tiling(const bls_plan_t *pl, int *R, int *runs_per_chunk);   // run length the gather kernels use
void bls_launch_commit(const bls_plan_t *pl);
void bls_launch_meta(const bls_plan_t *pl, cudaStream_t stream);   // table-wise router, first half, as a kernel of its own
void bls_launch_route(const bls_plan_t *pl);
void bls_launch_route_beside(const bls_plan_t *pl, cudaStream_t stream);   // table-wise router sized to run beside the gather kernel
void bls_launch_gather(const bls_plan_t *pl);
// the whole of iteration t (route, gather, return, ring bookkeeping) in one launch: small table-wise iterations, ranks in lockstep
void bls_launch_small(const bls_plan_t *pl, long long t, const int *ids, const int *off, long long n_ids);
int bls_route_kernels(const bls_plan_t *pl);   // kernels bls_launch_route enqueues
