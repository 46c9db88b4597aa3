// Plain CUDA-core kernels: sign packing / unpacking and a diagnostic GEMM.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "gemm_tc.h"

namespace bd {

// One thread per output word: reads 32 consecutive int8 (two 16-byte loads, so
// a warp reads 1 KiB contiguously) and sets bit j when element j is positive.
__global__ void pack_kernel(const int8_t* __restrict__ S, uint32_t* __restrict__ bits, long long words) {
    const long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= words) return;
    const uint4* src = reinterpret_cast<const uint4*>(S + w * 32);
    uint32_t word = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint4 v = __ldg(src + h);
        const uint32_t q[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int byte = 0; byte < 4; ++byte) {
                const int8_t s = (int8_t)((q[i] >> (8 * byte)) & 0xFF);
                if (s > 0) word |= 1u << (h * 16 + i * 4 + byte);
            }
        }
    }
    bits[w] = word;
}

__global__ void unpack_kernel(const uint32_t* __restrict__ bits, int8_t* __restrict__ S, long long words) {
    const long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= words) return;
    const uint32_t word = __ldg(bits + w);
    uint4* dst = reinterpret_cast<uint4*>(S + w * 32);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t q[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t v = 0;
#pragma unroll
            for (int byte = 0; byte < 4; ++byte) {
                const uint32_t bit = (word >> (h * 16 + i * 4 + byte)) & 1u;
                v |= (bit ? 0x01u : 0xFFu) << (8 * byte);
            }
            q[i] = v;
        }
        dst[h] = make_uint4(q[0], q[1], q[2], q[3]);
    }
}

// One warp per (tenant, weight row); lanes stride over the sign words, so lane l
// owns k = 32w .. 32w+31 for w = l, l+32, ...  fp32 accumulation, shuffle reduce.
__global__ void gemm_simt_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ W,
                                 const uint32_t* __restrict__ bits, const float* __restrict__ alpha,
                                 __nv_bfloat16* __restrict__ Y, int B, int m, int N, int K) {
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= (long long)B * N) return;
    const int b = (int)(gw / N);
    const int n = (int)(gw % N);
    const int words = K >> 5;
    const uint32_t* brow = bits + ((size_t)b * N + n) * words;
    const __nv_bfloat16* wrow = W + (size_t)n * K;
    const float al = alpha[b];
    for (int t = 0; t < m; ++t) {
        const __nv_bfloat16* xrow = X + ((size_t)b * m + t) * K;
        float base = 0.f, delta = 0.f;
        for (int w = lane; w < words; w += 32) {
            const uint32_t word = brow[w];
#pragma unroll 8
            for (int j = 0; j < 32; ++j) {
                const float x = __bfloat162float(xrow[w * 32 + j]);
                base = fmaf(x, __bfloat162float(wrow[w * 32 + j]), base);
                delta += ((word >> j) & 1u) ? x : -x;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            base += __shfl_xor_sync(0xFFFFFFFFu, base, o);
            delta += __shfl_xor_sync(0xFFFFFFFFu, delta, o);
        }
        if (lane == 0) Y[((size_t)b * m + t) * N + n] = __float2bfloat16_rn(fmaf(al, delta, base));
    }
}

cudaError_t launch_pack(const int8_t* S, uint32_t* bits, long long words, cudaStream_t stream) {
    const int threads = 256;
    const long long blocks = (words + threads - 1) / threads;
    pack_kernel<<<(unsigned)blocks, threads, 0, stream>>>(S, bits, words);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const uint32_t* bits, int8_t* S, long long words, cudaStream_t stream) {
    const int threads = 256;
    const long long blocks = (words + threads - 1) / threads;
    unpack_kernel<<<(unsigned)blocks, threads, 0, stream>>>(bits, S, words);
    return cudaGetLastError();
}

cudaError_t launch_gemm_simt(const void* X, const void* W, const uint32_t* bits, const float* alpha, void* Y,
                             int B, int m, int N, int K, cudaStream_t stream) {
    const int threads = 256;
    const long long warps = (long long)B * N;
    const long long blocks = (warps * 32 + threads - 1) / threads;
    gemm_simt_kernel<<<(unsigned)blocks, threads, 0, stream>>>(
        reinterpret_cast<const __nv_bfloat16*>(X), reinterpret_cast<const __nv_bfloat16*>(W), bits, alpha,
        reinterpret_cast<__nv_bfloat16*>(Y), B, m, N, K);
    return cudaGetLastError();
}

}  // namespace bd
