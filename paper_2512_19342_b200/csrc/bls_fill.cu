// Input-generation helper (not part of the method): fills a table with the
// counter-hash values of the synthetic workloads, so that tables of tens of GB
// never have to exist on the host.  Element (row, c) of table t: SplitMix64
// (Steele, Lea, Flood 2014) output number counter + 1 for the given seed, with
// counter = t << 48 | row << 16 | c; the four 16-bit fields are summed, centred
// (-131070) and scaled once in fp32 to about unit variance, then rounded to
// nearest even into the storage type.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "bls_internal.h"

__device__ __forceinline__ float hash_value(unsigned long long seed, int t, long long row, int c)
{
    unsigned long long counter = ((unsigned long long)t << 48) | ((unsigned long long)row << 16) | (unsigned long long)c;
    unsigned long long z = seed + (counter + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    int s = (int)(z & 0xFFFF) + (int)((z >> 16) & 0xFFFF) + (int)((z >> 32) & 0xFFFF) + (int)(z >> 48) - 131070;
    return __fmul_rn((float)s, __uint_as_float(0x37ddb3d7u));   // 1/sqrt((65536^2-1)/3) in fp32
}

template <int DT>
__global__ void __launch_bounds__(256) bls_fill_kernel(void *w, long long rows, int dim, unsigned long long seed, int t)
{
    const long long n = rows * dim;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        float v = hash_value(seed, t, e / dim, (int)(e % dim));
        if (DT == BLS_F32) ((float *)w)[e] = v;
        else if (DT == BLS_BF16) ((__nv_bfloat16 *)w)[e] = __float2bfloat16_rn(v);
        else ((__half *)w)[e] = __float2half_rn(v);
    }
}

extern "C" bls_status_t bls_fill_hash_table(void *weight, int64_t rows, int32_t dim, int32_t dtype,
                                            uint64_t seed, int32_t t, void *cuda_stream)
{
    if (!weight || rows < 1 || dim < 1 || dim > 65536 || t < 0 || t > 65535 || rows > 0xffffffffLL) return BLS_EINVAL;
    long long n = (long long)rows * dim;
    long long blocks = (n + 255) / 256;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return BLS_ECUDA;
    if (blocks > (long long)sms * 32) blocks = (long long)sms * 32;   // grid-stride loop: 32 blocks per SM at most
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == BLS_F32) bls_fill_kernel<BLS_F32><<<(unsigned)blocks, 256, 0, s>>>(weight, rows, dim, seed, t);
    else if (dtype == BLS_BF16) bls_fill_kernel<BLS_BF16><<<(unsigned)blocks, 256, 0, s>>>(weight, rows, dim, seed, t);
    else if (dtype == BLS_F16) bls_fill_kernel<BLS_F16><<<(unsigned)blocks, 256, 0, s>>>(weight, rows, dim, seed, t);
    else return BLS_EINVAL;
    return cudaGetLastError() == cudaSuccess ? BLS_OK : BLS_ECUDA;
}
