// Plain CUDA-core kernels: sign packing / unpacking and a diagnostic GEMM.
#include <cuda_bf16.h>
#include <cuda_fp8.h>
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

// ---------------------------------------------------------------------------------------------
// Activation split for the decode schedule.  The delta contraction there runs on the 8-bit float
// tensor path (K = 32 per instruction, signs decoded four per register), so each bf16 activation
// is rewritten, once per call, as a chain of four e5m2 pieces: p0 = rn(x), p1 = rn(x - p0), ...
// Each piece removes three more bits, so x = p0 + p1 + p2 + p3 up to 2^-12 |x| (e5m2 has the
// exponent range of fp16: magnitudes above 57344 saturate, below 2^-16 vanish).  Elementwise; one
// thread per group of 32 k.  Inside a group the pieces are stored in the order the sign decode
// produces: byte slot 4c+i holds k = c + 8i.  Output rows: X8[(b*4 + q)*m + t, :] for piece q.
__device__ __forceinline__ float e5m2_value(uint8_t v) {
    return __half2float(__half(__nv_cvt_fp8_to_halfraw(v, __NV_E5M2)));
}
__device__ __forceinline__ uint8_t e5m2_round(float v) {
    return (uint8_t)__nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E5M2);
}

__global__ void __launch_bounds__(128) x_split_kernel(const __nv_bfloat16* __restrict__ X, uint8_t* __restrict__ X8,
                                                      int m, int K, long long total_groups) {
    // Let the GEMM kernel queued behind this one start its weight prefetch right away.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= total_groups) return;
    const int groups = K >> 5;
    const int row = (int)(gid / groups);
    const int g = (int)(gid - (long long)row * groups);
    const int b = row / m, t = row - b * m;
    const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)row * K + g * 32);
    float y[32];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const uint4 v = __ldg(src + h);
        const uint32_t q[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[h * 8 + 2 * i] = __uint_as_float(q[i] << 16);
            y[h * 8 + 2 * i + 1] = __uint_as_float(q[i] & 0xFFFF0000u);
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint32_t acc = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint8_t pc = e5m2_round(y[c + 8 * i]);
                y[c + 8 * i] -= e5m2_value(pc);
                acc |= (uint32_t)pc << (8 * i);
            }
            w[c] = acc;
        }
        uint4* dst = reinterpret_cast<uint4*>(X8 + ((size_t)(b * 4 + q) * m + t) * K + g * 32);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

cudaError_t launch_x_split(const void* X, uint8_t* X8, int B, int m, int K, cudaStream_t stream) {
    const long long total = (long long)B * m * (K >> 5);
    const int threads = 128;
    const long long blocks = (total + threads - 1) / threads;
    x_split_kernel<<<(unsigned)blocks, threads, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(X), X8, m, K,
                                                             total);
    return cudaGetLastError();
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
