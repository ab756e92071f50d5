// The dense stages either side of the lookup (Listing 1 / Listing 2): bottom MLP on the
// dense features, feature interaction with the pooled embedding vectors, top MLP.
//
// A linear layer Y = act(X W^T + bias) is a dense contraction, so it runs on the tensor
// cores: one CTA computes a 128 x BN tile of Y.  One thread feeds a ring of shared-memory
// stages with TMA tile loads (cp.async.bulk.tensor, 128-byte swizzle, never multicast),
// one thread issues tcgen05.mma (bf16 x bf16 -> fp32, M = 128, N = BN, K = 16 per
// instruction) with the accumulator in tensor memory, and four warps read the
// accumulator back with tcgen05.ld, add the bias, apply the activation and store.
// X [M][K] and W [N][K] are both K-major, which is what an nn.Linear-style weight and a
// row-major activation matrix are.  Ragged M, N and K are handled by the zero fill of
// out-of-bounds TMA boxes and by guarded stores.
//
// Every wait is bounded by the clock; a wait that gives up latches BLS_ST_ETIMEOUT in the
// handle's status word, the roles wind down, and tensor memory is always released.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <stdlib.h>
#include <string.h>
#include <new>
#include <vector>
#include "bls_internal.h"

namespace {

constexpr int MLP_BM = 128;          // rows of Y per CTA (= TMEM lanes)
constexpr int MLP_BK = 64;           // K per stage: 64 bf16 = 128 bytes = one swizzle span
constexpr int MLP_STAGES = 3;          // 3 x 32 KiB of tiles at BN = 128: two CTAs per SM, one computes while the other stores
constexpr int MLP_THREADS = 192;     // warp 0: TMA, warp 1: MMA + TMEM allocation, warps 2-5: epilogue

__device__ __forceinline__ unsigned long long mlp_clock()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned s_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mb_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mb_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity: false (and the status bit) after two seconds.
__device__ __forceinline__ bool mb_wait(unsigned bar, unsigned parity, int *status)
{
    unsigned tries = 0;
    unsigned long long t0 = 0;
    for (;;) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((++tries & 255u) == 0) {
            const unsigned long long now = mlp_clock();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 2000000000ull) { atomicOr(status, BLS_ST_ETIMEOUT); return false; }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap *map, unsigned bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// Shared-memory matrix descriptor of a K-major tile stored with the 128-byte swizzle:
// rows of 128 bytes, groups of 8 rows 1024 bytes apart (stride byte offset), descriptor
// version 1, layout type 2 (128-byte swizzle).  The leading byte offset is not used by
// this layout.  `addr` is the byte address of the first row (a multiple of 1024) plus
// the byte offset of the K slice inside the 128-byte row.
__device__ __forceinline__ unsigned long long umma_desc(unsigned addr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3FFFu);          // start address, 16-byte units
    d |= (unsigned long long)1u << 16;                         // leading byte offset (unused), 16-byte units
    d |= (unsigned long long)(1024u >> 4) << 32;               // stride byte offset: 8 rows x 128 bytes
    d |= (unsigned long long)1u << 46;                         // descriptor version of this architecture
    d |= (unsigned long long)2u << 61;                         // 128-byte swizzle
    return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n.
__device__ __forceinline__ unsigned umma_idesc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(MLP_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(unsigned d_tmem, unsigned long long da, unsigned long long db, unsigned idesc, unsigned acc)
{
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(unsigned bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct LinArgs {
    int M, N, K;
    const float *bias;      // [N]
    void *Y;                // [M][ldy] bf16, or fp32 when y_fp32
    int ldy;
    int act;                // 0 none, 1 ReLU, 2 logistic function
    int y_fp32;
    int *status;
};

// grid (ceil(N / BN), ceil(M / 128)); dynamic shared memory: 1024 bytes of slack for
// alignment + MLP_STAGES * (128 + BN) * 128 bytes of tiles; barriers are static.
template <int BN>
__global__ void __launch_bounds__(MLP_THREADS, 1)
bls_linear_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, LinArgs a)
{
    extern __shared__ unsigned char mlp_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * MLP_STAGES + 1];
    __shared__ unsigned tmem_slot;
    constexpr unsigned A_BYTES = MLP_BM * MLP_BK * 2, B_BYTES = BN * MLP_BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    const unsigned tiles = (s_addr(mlp_smem) + 1023u) & ~1023u;          // the swizzle pattern repeats every 1024 bytes
    const unsigned full0 = s_addr(&bars[0]), empty0 = s_addr(&bars[MLP_STAGES]), done_bar = s_addr(&bars[2 * MLP_STAGES]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * MLP_BM;
    const int nkb = (a.K + MLP_BK - 1) / MLP_BK;

    if (threadIdx.x == 0) {
        // fetch the two tensor maps now: the first tile loads would otherwise wait for them
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        for (int s = 0; s < MLP_STAGES; s++) { mb_init(full0 + 8 * s, 1); mb_init(empty0 + 8 * s, 1); }
        mb_init(done_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                                      // BN fp32 accumulator columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_addr(&tmem_slot)), "r"((unsigned)BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = *(volatile unsigned *)&tmem_slot;

    if (warp == 0 && lane == 0) {
        // producer: one K block of X and of W per stage
        for (int kb = 0; kb < nkb; kb++) {
            const int s = kb % MLP_STAGES;
            if (!mb_wait(empty0 + 8 * s, ((kb / MLP_STAGES) & 1) ^ 1, a.status)) break;
            mb_expect_tx(full0 + 8 * s, STAGE_BYTES);
            tma_load_2d(tiles + s * STAGE_BYTES, &map_x, full0 + 8 * s, kb * MLP_BK, m0);
            tma_load_2d(tiles + s * STAGE_BYTES + A_BYTES, &map_w, full0 + 8 * s, kb * MLP_BK, n0);
        }
    } else if (warp == 1 && lane == 0) {
        // MMA issuer: four K = 16 steps per stage, then the stage is handed back
        const unsigned idesc = umma_idesc(BN);
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; kb++) {
            const int s = kb % MLP_STAGES;
            ok = mb_wait(full0 + 8 * s, (kb / MLP_STAGES) & 1, a.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned sa = tiles + s * STAGE_BYTES, sb = sa + A_BYTES;
            #pragma unroll
            for (int k = 0; k < MLP_BK / 16; k++)
                umma_f16(tmem, umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (kb | k) ? 1u : 0u);
            umma_commit(empty0 + 8 * s);
        }
        umma_commit(done_bar);                                            // the accumulator is complete
    } else if (warp >= 2) {
        // epilogue: warp w reads TMEM lanes 32 (w mod 4) .. +31, one row of the tile per thread
        const int q = warp & 3;
        const int row = m0 + q * 32 + lane;
        if (mb_wait(done_bar, 0, a.status)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // bf16 output with whole 16-byte pieces: the warp's 32 x BN block goes through shared memory (the
            // tile ring is free: every MMA that read it has completed) and leaves as coalesced row pieces
            const bool staged = !a.y_fp32 && (a.ldy & 7) == 0 && (a.N & 7) == 0;
            constexpr int ROWB = BN * 2;                                      // bytes of one staged row
            const unsigned stage = tiles + (unsigned)q * 32u * ROWB;
            #pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                unsigned r[32];
                tmem_ld32(tmem + ((unsigned)(q * 32) << 16) + (unsigned)c0, r);   // sync.aligned: the whole warp, also rows past M
                if (staged) {
                    #pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        unsigned pk[4];
                        #pragma unroll
                        for (int e = 0; e < 8; e += 2) {
                            const int col = n0 + c0 + j + e;
                            float v0 = __uint_as_float(r[j + e]) + (col < a.N ? a.bias[col] : 0.f);
                            float v1 = __uint_as_float(r[j + e + 1]) + (col + 1 < a.N ? a.bias[col + 1] : 0.f);
                            if (a.act == 1) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
                            else if (a.act == 2) { v0 = 1.f / (1.f + expf(-v0)); v1 = 1.f / (1.f + expf(-v1)); }
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                            pk[e >> 1] = *reinterpret_cast<unsigned *>(&h2);
                        }
                        // 16-byte piece number (c0 + j) / 8 of the row, rotated by the row number so that the
                        // lanes of a warp (32 different rows, same piece) hit different banks
                        const unsigned piece = ((unsigned)((c0 + j) >> 3) + (unsigned)lane) % (unsigned)(BN / 8);
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(stage + (unsigned)lane * ROWB + piece * 16u), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    }
                } else if (row < a.M) {
                    #pragma unroll
                    for (int j = 0; j < 32; j++) {
                        const int col = n0 + c0 + j;
                        if (col < a.N) {
                            float v = __uint_as_float(r[j]) + a.bias[col];
                            if (a.act == 1) v = fmaxf(v, 0.f);
                            else if (a.act == 2) v = 1.f / (1.f + expf(-v));
                            if (a.y_fp32) ((float *)a.Y)[(size_t)row * a.ldy + col] = v;
                            else ((__nv_bfloat16 *)a.Y)[(size_t)row * a.ldy + col] = __float2bfloat16_rn(v);
                        }
                    }
                }
            }
            if (staged) {
                __syncwarp();
                constexpr int PPR = BN / 8;                                   // 16-byte pieces per row
                for (int e = lane; e < 32 * PPR; e += 32) {
                    const int rr = e / PPR, pc = e % PPR;                     // row of the block, piece of the row
                    const int grow = m0 + q * 32 + rr, col = n0 + pc * 8;
                    if (grow < a.M && col < a.N) {                            // N and ldy are multiples of 8: a piece is inside or outside
                        const unsigned piece = ((unsigned)pc + (unsigned)rr) % (unsigned)PPR;
                        uint4 v;
                        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stage + (unsigned)rr * ROWB + piece * 16u));
                        *reinterpret_cast<uint4 *>((__nv_bfloat16 *)a.Y + (size_t)grow * a.ldy + col) = v;
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((unsigned)BN) : "memory");
    }
}

// Feature interaction, one block of 64 threads per sample: v_0 = the bottom MLP's output (bf16),
// v_1..v_T = the pooled vectors (fp32); R = [v_0, <v_i, v_j> for i = 1..T, j < i], bf16, zero-padded
// to ldr.  The vectors are staged in shared memory; a thread computes a 3 x 3 block of the matrix of
// dot products (only blocks on or below the diagonal exist), so every value read from shared
// memory is used three times.
__global__ void __launch_bounds__(64) bls_interact_kernel(const __nv_bfloat16 *x, int ldx, const float *pooled, int B, int T, int D,
                                                          __nv_bfloat16 *r, int ldr)
{
    extern __shared__ float iv[];                      // [3 * nb][D + 1]: rows padded so that vectors start in different banks
    const int b = blockIdx.x;
    const int W = D + 1;
    const int nb = (T + 1 + 2) / 3;                    // blocks of three vectors
    for (int c = threadIdx.x; c < D; c += blockDim.x) iv[c] = __bfloat162float(x[(size_t)b * ldx + c]);
    for (int e = (T + 1) * D + threadIdx.x; e < 3 * nb * D; e += blockDim.x) iv[(e / D) * W + e % D] = 0.f;   // rows that pad the last block
    if ((D & 3) == 0) {
        // the sample's T pooled vectors are one contiguous piece of T * D floats: 16-byte loads, four in flight per thread
        const float4 *src = reinterpret_cast<const float4 *>(pooled + (size_t)b * T * D);
        const int n4 = T * D / 4;
        for (int e0 = threadIdx.x; e0 < n4; e0 += 4 * blockDim.x) {
            float4 v[4];
            #pragma unroll
            for (int u = 0; u < 4; u++) {
                const int e = e0 + u * blockDim.x;
                if (e < n4) v[u] = __ldcs(src + e);
            }
            #pragma unroll
            for (int u = 0; u < 4; u++) {
                const int e = e0 + u * blockDim.x;
                if (e < n4) {
                    const int i = 1 + (e * 4) / D, c = (e * 4) % D;
                    float *dst = iv + i * W + c;
                    dst[0] = v[u].x; dst[1] = v[u].y; dst[2] = v[u].z; dst[3] = v[u].w;
                }
            }
        }
    } else {
        for (int e = threadIdx.x; e < T * D; e += blockDim.x) iv[(1 + e / D) * W + e % D] = pooled[(size_t)b * T * D + e];
    }
    __syncthreads();
    __nv_bfloat16 *out = r + (size_t)b * ldr;
    for (int c = threadIdx.x; c < D; c += blockDim.x) out[c] = x[(size_t)b * ldx + c];
    const int npairs = T * (T + 1) / 2;
    for (int q = threadIdx.x; q < nb * (nb + 1) / 2; q += blockDim.x) {
        // block pair number q -> (bi, bj), bj <= bi, row-major over the lower triangle including the diagonal
        int bi = (int)((sqrtf(1.f + 8.f * (float)q) - 1.f) * 0.5f);
        while (bi * (bi + 1) / 2 > q) bi--;
        while ((bi + 1) * (bi + 2) / 2 <= q) bi++;
        const int bj = q - bi * (bi + 1) / 2;
        const float *pa = iv + 3 * bi * W, *pb = iv + 3 * bj * W;
        float acc[3][3] = {};
        for (int c = 0; c < D; c++) {
            const float a0 = pa[c], a1 = pa[W + c], a2 = pa[2 * W + c];
            const float b0 = pb[c], b1 = pb[W + c], b2 = pb[2 * W + c];
            acc[0][0] = fmaf(a0, b0, acc[0][0]); acc[0][1] = fmaf(a0, b1, acc[0][1]); acc[0][2] = fmaf(a0, b2, acc[0][2]);
            acc[1][0] = fmaf(a1, b0, acc[1][0]); acc[1][1] = fmaf(a1, b1, acc[1][1]); acc[1][2] = fmaf(a1, b2, acc[1][2]);
            acc[2][0] = fmaf(a2, b0, acc[2][0]); acc[2][1] = fmaf(a2, b1, acc[2][1]); acc[2][2] = fmaf(a2, b2, acc[2][2]);
        }
        #pragma unroll
        for (int u = 0; u < 3; u++)
            #pragma unroll
            for (int v = 0; v < 3; v++) {
                const int i = 3 * bi + u, j = 3 * bj + v;
                if (i <= T && j < i) out[D + i * (i - 1) / 2 + j] = __float2bfloat16_rn(acc[u][v]);
            }
    }
    for (int c = D + npairs + threadIdx.x; c < ldr; c += blockDim.x) out[c] = __float2bfloat16_rn(0.f);
}

PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

bool encode_ready()
{
    if (g_encode) return true;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return false;
    g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    return true;
}

// Tensor map of a row-major bf16 matrix [rows][cols] with row pitch ld elements: boxes of 64 columns x box_rows rows,
// 128-byte swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap *map, const void *base, long long rows, long long cols, long long ld, int box_rows)
{
    if (!encode_ready()) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)MLP_BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pick_bn(int N) { return N > 64 ? 128 : (N > 32 ? 64 : 32); }

template <int BN>
cudaError_t launch_linear_bn(const CUtensorMap &mx, const CUtensorMap &mw, const LinArgs &a, cudaStream_t s)
{
    const size_t smem = 1024 + (size_t)MLP_STAGES * (MLP_BM + BN) * MLP_BK * 2;
    // set on every launch: the attribute belongs to the current device, and the call costs about a microsecond
    cudaError_t e = cudaFuncSetAttribute(bls_linear_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((a.N + BN - 1) / BN, (a.M + MLP_BM - 1) / MLP_BM);
    bls_linear_kernel<BN><<<grid, MLP_THREADS, smem, s>>>(mx, mw, a);
    return cudaGetLastError();
}

cudaError_t launch_linear(const CUtensorMap &mx, const CUtensorMap &mw, const LinArgs &a, cudaStream_t s)
{
    switch (pick_bn(a.N)) {
    case 128: return launch_linear_bn<128>(mx, mw, a, s);
    case 64: return launch_linear_bn<64>(mx, mw, a, s);
    default: return launch_linear_bn<32>(mx, mw, a, s);
    }
}

}  // namespace

struct bls_mlp {
    int n_layers, max_rows, last_act;
    std::vector<int> dims;
    std::vector<const void *> weights;
    std::vector<const float *> bias;
    std::vector<CUtensorMap> map_w;        // per layer
    std::vector<CUtensorMap> map_h;        // per hidden activation buffer (input of layer i + 1)
    std::vector<void *> hidden;            // bf16 [max_rows][dims[i + 1]] for i < n_layers - 1
    int *status;
};

extern "C" {

bls_status_t bls_mlp_bytes(int n_layers, const int *dims, int max_rows, size_t *bytes)
{
    if (!bytes || !dims || n_layers < 1 || n_layers > 16 || max_rows < 1) return BLS_EINVAL;
    size_t o = 256;                                                   // the status word
    for (int i = 0; i <= n_layers; i++)
        if (dims[i] < 1 || (i < n_layers && dims[i] % 8) || dims[i] > 65536) return BLS_EINVAL;
    for (int i = 1; i < n_layers; i++) o += ((size_t)max_rows * dims[i] * 2 + 255) / 256 * 256;
    *bytes = o;
    return BLS_OK;
}

bls_status_t bls_mlp_create(int n_layers, const int *dims, const void *const *weights, const float *const *bias,
                            int last_act, int max_rows, void *workspace, size_t bytes, void *cuda_stream, bls_mlp_t **handle)
{
    size_t need = 0;
    if (!handle || !weights || !bias || !workspace || ((uintptr_t)workspace & 255) || last_act < 0 || last_act > 2) return BLS_EINVAL;
    bls_status_t st = bls_mlp_bytes(n_layers, dims, max_rows, &need);
    if (st != BLS_OK) return st;
    if (bytes < need) return BLS_ENOSPC;
    bls_mlp *h = new (std::nothrow) bls_mlp();
    if (!h) return BLS_ENOSPC;
    h->n_layers = n_layers; h->max_rows = max_rows; h->last_act = last_act;
    h->dims.assign(dims, dims + n_layers + 1);
    char *ws = (char *)workspace;
    h->status = (int *)ws;
    size_t o = 256;
    h->map_w.resize(n_layers);
    h->map_h.resize(n_layers > 1 ? n_layers - 1 : 0);
    for (int i = 0; i < n_layers; i++) {
        if (!weights[i] || !bias[i] || ((uintptr_t)weights[i] & 15)) { delete h; return BLS_EINVAL; }
        h->weights.push_back(weights[i]);
        h->bias.push_back(bias[i]);
        if (!make_map(&h->map_w[i], weights[i], dims[i + 1], dims[i], dims[i], pick_bn(dims[i + 1]))) { delete h; return BLS_ECUDA; }
        if (i + 1 < n_layers) {
            h->hidden.push_back(ws + o);
            if (!make_map(&h->map_h[i], ws + o, max_rows, dims[i + 1], dims[i + 1], MLP_BM)) { delete h; return BLS_ECUDA; }
            o += ((size_t)max_rows * dims[i + 1] * 2 + 255) / 256 * 256;
        }
    }
    if (cudaMemsetAsync(h->status, 0, sizeof(int), (cudaStream_t)cuda_stream) != cudaSuccess) { delete h; return BLS_ECUDA; }
    *handle = h;
    return BLS_OK;
}

void bls_mlp_destroy(bls_mlp_t *h) { delete h; }

bls_status_t bls_mlp_forward(bls_mlp_t *h, const void *x, int ldx, int rows, void *y, int ldy, int y_fp32, void *cuda_stream)
{
    if (!h || !x || !y || rows < 1 || rows > h->max_rows || ldx < h->dims[0] || (ldx % 8) || ((uintptr_t)x & 15) ||
        ldy < h->dims[h->n_layers])
        return BLS_EINVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    CUtensorMap map_x;
    if (!make_map(&map_x, x, rows, h->dims[0], ldx, MLP_BM)) return BLS_ECUDA;
    for (int i = 0; i < h->n_layers; i++) {
        const bool last = i + 1 == h->n_layers;
        LinArgs a;
        a.M = rows; a.N = h->dims[i + 1]; a.K = h->dims[i];
        a.bias = h->bias[i];
        a.Y = last ? y : h->hidden[i];
        a.ldy = last ? ldy : h->dims[i + 1];
        a.act = last ? h->last_act : 1;
        a.y_fp32 = last ? y_fp32 : 0;
        a.status = h->status;
        if (launch_linear(i == 0 ? map_x : h->map_h[i - 1], h->map_w[i], a, s) != cudaSuccess) return BLS_ECUDA;
    }
    return BLS_OK;
}

bls_status_t bls_interact(const void *x, int ldx, const float *pooled, int rows, int T, int D, void *r, int ldr,
                          void *cuda_stream)
{
    if (!x || !pooled || !r || rows < 1 || T < 1 || D < 1 || ldx < D || ldr < D + T * (T + 1) / 2) return BLS_EINVAL;
    const size_t smem = sizeof(float) * (size_t)(3 * ((T + 3) / 3)) * (D + 1);
    if (smem > 48 * 1024) return BLS_ENOSPC;
    bls_interact_kernel<<<rows, 64, smem, (cudaStream_t)cuda_stream>>>((const __nv_bfloat16 *)x, ldx, pooled, rows, T, D,
                                                                         (__nv_bfloat16 *)r, ldr);
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}

bls_status_t bls_mlp_status(bls_mlp_t *h, void *cuda_stream)
{
    if (!h) return BLS_EINVAL;
    int st = 0;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess ||
        cudaMemcpy(&st, h->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return BLS_ECUDA;
    return (st & BLS_ST_ETIMEOUT) ? BLS_ETIMEOUT : BLS_OK;
}

}  // extern "C"
