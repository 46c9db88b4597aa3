// Plain CUDA-core kernels: sign packing / unpacking and a diagnostic GEMM.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include "gemm_tc.h"
#include "ptx.cuh"

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
// 16-bit values of the I/O type (bf16, or IEEE binary16 when `f16`) <-> fp32.
__device__ __forceinline__ float io16_to_float(uint16_t h, int f16) {
    return f16 ? __half2float(__ushort_as_half(h)) : __uint_as_float((uint32_t)h << 16);
}
__device__ __forceinline__ uint16_t float_to_io16(float v, int f16) {
    return f16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

__global__ void gemm_simt_kernel(const uint16_t* __restrict__ X, const uint16_t* __restrict__ W,
                                 const uint32_t* __restrict__ bits, const float* __restrict__ alpha,
                                 const uint16_t* __restrict__ bias, uint16_t* __restrict__ Y, int B, int m, int N,
                                 int K, int f16, int act) {
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= (long long)B * N) return;
    const int b = (int)(gw / N);
    const int n = (int)(gw % N);
    const int words = K >> 5;
    const float al = alpha[b];
    if (act == 2) {
        // SiLU gate over interleaved (gate, up) rows: the warp of the gate row computes both rows of its pair
        if (n & 1) return;
        for (int t = 0; t < m; ++t) {
            const uint16_t* xrow = X + ((size_t)b * m + t) * K;
            float z[2];
            for (int r = 0; r < 2; ++r) {
                const uint32_t* brow2 = bits + ((size_t)b * N + n + r) * words;
                const uint16_t* wrow2 = W + (size_t)(n + r) * K;
                float base = 0.f, delta = 0.f;
                for (int w = lane; w < words; w += 32) {
                    const uint32_t word = brow2[w];
#pragma unroll 8
                    for (int j = 0; j < 32; ++j) {
                        const float x = io16_to_float(xrow[w * 32 + j], f16);
                        base = fmaf(x, io16_to_float(wrow2[w * 32 + j], f16), base);
                        delta += ((word >> j) & 1u) ? x : -x;
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    base += __shfl_xor_sync(0xFFFFFFFFu, base, o);
                    delta += __shfl_xor_sync(0xFFFFFFFFu, delta, o);
                }
                z[r] = fmaf(al, delta, base) + (bias ? io16_to_float(bias[n + r], f16) : 0.f);
            }
            if (lane == 0) Y[((size_t)b * m + t) * (N >> 1) + (n >> 1)] = float_to_io16(z[0] / (1.f + __expf(-z[0])) * z[1], f16);
        }
        return;
    }
    const uint32_t* brow = bits + ((size_t)b * N + n) * words;
    const uint16_t* wrow = W + (size_t)n * K;
    const float bias_n = bias ? io16_to_float(bias[n], f16) : 0.f;
    for (int t = 0; t < m; ++t) {
        const uint16_t* xrow = X + ((size_t)b * m + t) * K;
        float base = 0.f, delta = 0.f;
        for (int w = lane; w < words; w += 32) {
            const uint32_t word = brow[w];
#pragma unroll 8
            for (int j = 0; j < 32; ++j) {
                const float x = io16_to_float(xrow[w * 32 + j], f16);
                base = fmaf(x, io16_to_float(wrow[w * 32 + j], f16), base);
                delta += ((word >> j) & 1u) ? x : -x;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            base += __shfl_xor_sync(0xFFFFFFFFu, base, o);
            delta += __shfl_xor_sync(0xFFFFFFFFu, delta, o);
        }
        if (lane == 0) {
            float v = fmaf(al, delta, base) + bias_n;
            if (act == 1) v = v / (1.f + __expf(-v));   // SiLU
            Y[((size_t)b * m + t) * N + n] = float_to_io16(v, f16);
        }
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

// Status word of this translation unit: [0] = 9 (BITDELTA_ERR_RANGE) once the split has met a magnitude of
// 2^16 or more (it is clamped to 65504, the largest binary16 number, exactly as the GEMM kernels' own split does).
static __device__ unsigned int g_simple_status[2];

__global__ void __launch_bounds__(128) x_split_kernel(const uint16_t* __restrict__ X, uint8_t* __restrict__ X8,
                                                      int m, int K, long long total_groups, int f16) {
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
    bool out_of_range = false;
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const uint4 v = __ldg(src + h);
        const uint32_t q[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[h * 8 + 2 * i] = io16_to_float((uint16_t)(q[i] & 0xFFFFu), f16);
            y[h * 8 + 2 * i + 1] = io16_to_float((uint16_t)(q[i] >> 16), f16);
            if (!f16 && (((q[i] & 0x7FFFu) >= 0x4780u) || (((q[i] >> 16) & 0x7FFFu) >= 0x4780u))) out_of_range = true;
        }
    }
    if (out_of_range) {
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = fminf(fmaxf(y[i], -65504.f), 65504.f);
        atomicCAS(&g_simple_status[0], 0u, 9u);
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

cudaError_t read_simple_status(unsigned int out[2]) {
    cudaError_t e = cudaMemcpyFromSymbol(out, g_simple_status, sizeof(unsigned int) * 2);
    if (e != cudaSuccess) return e;
    if (out[0] != 0) {
        unsigned int zero[2] = {0, 0};
        e = cudaMemcpyToSymbol(g_simple_status, zero, sizeof(zero));
    }
    return e;
}

cudaError_t launch_x_split(const void* X, uint8_t* X8, int B, int m, int K, int f16, cudaStream_t stream) {
    const long long total = (long long)B * m * (K >> 5);
    const int threads = 128;
    const long long blocks = (total + threads - 1) / threads;
    x_split_kernel<<<(unsigned)blocks, threads, 0, stream>>>(reinterpret_cast<const uint16_t*>(X), X8, m, K, total, f16);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------- compress
// The step before the product: bits = [W_fine - W_base > 0], alpha[b] = mean |W_fine - W_base|.
// A warp takes tiles of one weight row x 1024 consecutive k (one sign word per lane), a fixed stride apart; for each
// it keeps its piece of W_base in registers (as floats) and walks the tenants, so W_base is read once for all of
// them.  Per thread and tenant: 64 bytes of W_fine in (two 32-byte loads), one word out.  The comparison is taken on
// the exact bf16 values (as fp32), through the sign of (base - fine); |delta| is formed in fp32, four at a time, and
// summed in double: per thread, then across the warp (shuffles), over the warp's tiles and the block (fixed order)
// into one partial per block and tenant; a second kernel adds the partials of a tenant in a fixed order.  Nothing
// depends on the order in which blocks run, nor on the device (the grid is a fixed number of blocks).
// Measured on 8 x 4096 x 4096: 61.4 us per call (0.79 of the HBM roofline), the main kernel alone 60 us: bound by memory
// latency at half occupancy (eight warps waiting on loads per issued instruction, issue slots 54 % busy).  Tried
// without gain: 512 contiguous bytes per load instruction across the warp with the sign bytes put together by
// shuffles (82-96 us), the next tenant's loads issued one iteration ahead (65 us at 80 registers).
constexpr int kCompressWarps = 8;
constexpr int kCompressTenantChunk = 32;   // tenants whose warp sums are staged in shared memory at once

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
// 32 bytes (32-byte aligned) through the read-only path in one load.
__device__ __forceinline__ void ld_nc_256(const uint4* p, uint4& a, uint4& b) {
    asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
                 : "l"(p));
}

__global__ void __launch_bounds__(kCompressWarps * 32)
compress_kernel(const uint4* __restrict__ Wf, const uint4* __restrict__ Wb, uint32_t* __restrict__ bits,
                double* __restrict__ partial, int B, int N, int K, int kchunks, long long tiles) {
    __shared__ double warp_sum[kCompressTenantChunk][kCompressWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int words = K >> 5;
    if (threadIdx.x == 0) grid_launch_dependents();   // (the finishing kernel may become resident; it waits for this grid's end)
    for (int b0 = 0; b0 < B; b0 += kCompressTenantChunk) {
        const int nb = min(kCompressTenantChunk, B - b0);
        for (int bb = lane; bb < nb; bb += 32) warp_sum[bb][warp] = 0.0;
        __syncwarp();
        // this warp's tiles (weight row, 1024 k), a fixed stride apart: the grid is a fixed number of blocks (see
        // compress_blocks), every multiprocessor holds its share of them from the start to the end of the kernel
        for (long long tile = (long long)blockIdx.x * kCompressWarps + warp; tile < tiles; tile += (long long)gridDim.x * kCompressWarps) {
            const int n = (int)(tile / kchunks);
            const int w = (int)(tile - (long long)n * kchunks) * 32 + lane;   // this lane's sign word
            const bool ok = w < words;
            // This lane's 32 base weights as floats, once for all tenants of the chunk; x + 0 turns a -0 into +0 (see the
            // sign rule below).
            float gf[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) gf[i] = 0.f;
            if (ok) {
                const uint4* src = Wb + ((size_t)n * K + (size_t)w * 32) / 8;
                uint4 wb[4];
                ld_nc_256(src, wb[0], wb[1]);
                ld_nc_256(src + 2, wb[2], wb[3]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t g[4] = {wb[i].x, wb[i].y, wb[i].z, wb[i].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        gf[i * 8 + q * 2] = __fadd_rn(bf16lo(g[q]), 0.f);
                        gf[i * 8 + q * 2 + 1] = __fadd_rn(bf16hi(g[q]), 0.f);
                    }
                }
            }
            for (int bb = 0; bb < nb; ++bb) {
                const int b = b0 + bb;
                double acc = 0.0;
                if (ok) {
                    const uint4* src = Wf + (((size_t)b * N + n) * K + (size_t)w * 32) / 8;
                    uint4 wf[4];
                    ld_nc_256(src, wf[0], wf[1]);       // (32 bytes per lane and load)
                    ld_nc_256(src + 2, wf[2], wf[3]);
                    // Sign bit k of the word = (fine > base) for element k = the sign of (base - fine), which is +0 when
                    // the two are equal (a base of -0 was made +0 above): the elements are taken from the last to the
                    // first and each difference's sign bit is shifted in from the right (one funnel shift per element
                    // instead of a compare and a predicated OR).
                    uint32_t word = 0;
#pragma unroll
                    for (int i = 3; i >= 0; --i) {
                        const uint32_t f[4] = {wf[i].x, wf[i].y, wf[i].z, wf[i].w};
                        float s4[2] = {0.f, 0.f};
#pragma unroll
                        for (int q = 3; q >= 0; --q) {
                            const float d1 = gf[i * 8 + q * 2 + 1] - bf16hi(f[q]);
                            word = __funnelshift_l(__float_as_uint(d1), word, 1);
                            const float d0 = gf[i * 8 + q * 2] - bf16lo(f[q]);
                            word = __funnelshift_l(__float_as_uint(d0), word, 1);
                            s4[q >> 1] += fabsf(d0) + fabsf(d1);
                        }
                        acc += (double)s4[0] + (double)s4[1];
                    }
                    bits[((size_t)b * N + n) * words + w] = word;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (lane == 0) warp_sum[bb][warp] += acc;
            }
        }
        __syncthreads();
        for (int bb = threadIdx.x; bb < nb; bb += blockDim.x) {
            double t = 0.0;
#pragma unroll
            for (int i = 0; i < kCompressWarps; ++i) t += warp_sum[bb][i];
            partial[(size_t)(b0 + bb) * gridDim.x + blockIdx.x] = t;
        }
        __syncthreads();
    }
}

// alpha[b] = (sum of the tenant's block partials, in a fixed order) / (N K), rounded to fp32.
__global__ void compress_finish_kernel(const double* __restrict__ partial, float* __restrict__ alpha, int nblocks,
                                       double inv_count) {
    // Launched with an early start behind compress_kernel (which releases it at once): resident and waiting when the
    // partials are complete, instead of a launch gap later.
    grid_dependency_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    double t = 0.0;
    for (int i = lane; i < nblocks; i += 32) t += partial[(size_t)b * nblocks + i];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    if (lane == 0) alpha[b] = (float)(t * inv_count);
}

// Blocks of the compress kernel: one per eight tiles, but never more than a B200 holds at once (148 multiprocessors x 4
// blocks of 256 threads and 64 registers): a fixed number, so that the order of the sums does not depend on the device.
constexpr long long kCompressMaxBlocks = 148 * 4;
long long compress_blocks(int N, int K) {
    const long long kchunks = (K / 32 + 31) / 32;
    const long long tiles = (long long)N * kchunks;
    const long long blocks = (tiles + kCompressWarps - 1) / kCompressWarps;
    return blocks < kCompressMaxBlocks ? blocks : kCompressMaxBlocks;
}

cudaError_t launch_compress(const void* Wf, const void* Wb, uint32_t* bits, float* alpha, double* partial, int B, int N,
                            int K, cudaStream_t stream) {
    const int kchunks = (K / 32 + 31) / 32;
    const long long tiles = (long long)N * kchunks;
    const long long blocks = compress_blocks(N, K);
    compress_kernel<<<(unsigned)blocks, kCompressWarps * 32, 0, stream>>>(
        reinterpret_cast<const uint4*>(Wf), reinterpret_cast<const uint4*>(Wb), bits, partial, B, N, K, kchunks, tiles);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)B);
    cfg.blockDim = dim3(32u);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, compress_finish_kernel, const_cast<const double*>(partial), alpha, (int)blocks,
                              1.0 / ((double)N * (double)K));
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

cudaError_t launch_gemm_simt(const void* X, const void* W, const uint32_t* bits, const float* alpha, const void* bias,
                             void* Y, int B, int m, int N, int K, int f16, int act, cudaStream_t stream) {
    const int threads = 256;
    const long long warps = (long long)B * N;
    const long long blocks = (warps * 32 + threads - 1) / threads;
    gemm_simt_kernel<<<(unsigned)blocks, threads, 0, stream>>>(
        reinterpret_cast<const uint16_t*>(X), reinterpret_cast<const uint16_t*>(W), bits, alpha,
        reinterpret_cast<const uint16_t*>(bias), reinterpret_cast<uint16_t*>(Y), B, m, N, K, f16, act);
    return cudaGetLastError();
}

}  // namespace bd
