// Element-wise pre- and post-operations of the GSA layer (Sec. 3.3): the Swish feature map of
// q, k, v (with its derivative for the backward) and the output path Swish -> RMSNorm over all
// heads of a token (forward, and backward with the gradient of the norm's weight).  All of them
// stream their tensors once with 16-byte accesses: HBM-bound.
//
// Why these are kernels of their own and not part of the chunk kernels: a d-sized tile of the
// tensor-core kernels goes from the copy engine straight into the matrix unit; passing it through
// registers for a Swish costs two special-function operations per element -- 2 k cycles per 128 x 128
// tile at 16 per clock and SM, as much as a whole chunk of the scan takes -- and every tile is read by
// three of the eight scans.  Applied once, in a kernel that runs at memory speed on all SMs, the same
// work costs one pass over q, k, v.  The decode kernel, which touches d values per (sequence, head)
// against 2 m d of memory, applies the feature map as it loads.
#include "common.cuh"

namespace gsa {
namespace {

__device__ __forceinline__ float swishf(float x) { return x / (1.f + __expf(-x)); }
__device__ __forceinline__ float swish_gradf(float x) {
    const float s = 1.f / (1.f + __expf(-x));
    return s * (1.f + x * (1.f - s));
}

template <typename IO>
__global__ void __launch_bounds__(256) swish_fwd_kernel(const IO* __restrict__ in, IO* __restrict__ out, size_t nvec) {
    constexpr int V = IoTraits<IO>::kVec;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
        float x[V];
        load_vec(in + i * V, x);
#pragma unroll
        for (int e = 0; e < V; ++e) x[e] = swishf(x[e]);
        store_vec(out + i * V, x);
    }
}
// d <- d * Swish'(x), in place on the gradient
template <typename IO>
__global__ void __launch_bounds__(256) swish_bwd_kernel(const IO* __restrict__ x_in, IO* __restrict__ d, size_t nvec) {
    constexpr int V = IoTraits<IO>::kVec;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
        float x[V], g[V];
        load_vec(x_in + i * V, x);
        load_vec(d + i * V, g);
#pragma unroll
        for (int e = 0; e < V; ++e) g[e] *= swish_gradf(x[e]);
        store_vec(d + i * V, g);
    }
}

__device__ __forceinline__ float block_sum(float v, float* scratch) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();                      // scratch may still be read from a previous call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += scratch[w];     // same order in every thread: deterministic
    return t;
}

// One CTA per token: y = w * Swish(o) / sqrt(mean(Swish(o)^2) + eps) over the N = H d_v values of the token.
// A thread keeps up to kMaxVecPerThread vectors of the row in registers (N <= 256 threads * that * V).
constexpr int kMaxVecPerThread = 2;
template <typename IO>
__global__ void __launch_bounds__(256) out_norm_fwd_kernel(const IO* __restrict__ o, const float* __restrict__ weight,
                                                           float eps, IO* __restrict__ y, int N) {
    constexpr int V = IoTraits<IO>::kVec;
    __shared__ float scratch[8];
    const size_t row = blockIdx.x;
    const int nvec = N / V;
    float x[kMaxVecPerThread][V];
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxVecPerThread; ++j) {
        const int c = threadIdx.x + j * 256;
        if (c < nvec) {
            load_vec(o + row * N + (size_t)c * V, x[j]);
#pragma unroll
            for (int e = 0; e < V; ++e) { x[j][e] = swishf(x[j][e]); ss += x[j][e] * x[j][e]; }
        }
    }
    const float inv = rsqrtf(block_sum(ss, scratch) / (float)N + eps);
#pragma unroll
    for (int j = 0; j < kMaxVecPerThread; ++j) {
        const int c = threadIdx.x + j * 256;
        if (c < nvec) {
#pragma unroll
            for (int e = 0; e < V; ++e) x[j][e] *= inv * (weight ? weight[c * V + e] : 1.f);
            store_vec(y + row * N + (size_t)c * V, x[j]);
        }
    }
}

// Backward: a CTA takes kRowsPerCta consecutive tokens (so that the weight gradient can be summed
// over them in registers, one partial row per CTA; a second kernel adds the partial rows in order).
constexpr int kRowsPerCta = 16;
template <typename IO>
__global__ void __launch_bounds__(256) out_norm_bwd_kernel(const IO* __restrict__ o, const IO* __restrict__ dy,
                                                           const float* __restrict__ weight, float eps, IO* __restrict__ d_o,
                                                           float* __restrict__ dw_part, int N, size_t rows) {
    constexpr int V = IoTraits<IO>::kVec;
    __shared__ float scratch[8];
    const int nvec = N / V;
    float dw[kMaxVecPerThread][V];
#pragma unroll
    for (int j = 0; j < kMaxVecPerThread; ++j)
#pragma unroll
        for (int e = 0; e < V; ++e) dw[j][e] = 0.f;
    for (int r = 0; r < kRowsPerCta; ++r) {
        const size_t row = (size_t)blockIdx.x * kRowsPerCta + r;
        if (row >= rows) break;
        float ov[kMaxVecPerThread][V], x[kMaxVecPerThread][V], g[kMaxVecPerThread][V];
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxVecPerThread; ++j) {
            const int c = threadIdx.x + j * 256;
            if (c < nvec) {
                load_vec(o + row * N + (size_t)c * V, ov[j]);
                load_vec(dy + row * N + (size_t)c * V, g[j]);
#pragma unroll
                for (int e = 0; e < V; ++e) { x[j][e] = swishf(ov[j][e]); ss += x[j][e] * x[j][e]; }
            }
        }
        const float inv = rsqrtf(block_sum(ss, scratch) / (float)N + eps);
        float dot = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxVecPerThread; ++j) {
            const int c = threadIdx.x + j * 256;
            if (c < nvec) {
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    x[j][e] *= inv;                                         // xhat
                    dw[j][e] += g[j][e] * x[j][e];
                    g[j][e] *= weight ? weight[c * V + e] : 1.f;           // gradient w.r.t. xhat
                    dot += g[j][e] * x[j][e];
                }
            }
        }
        const float mean = block_sum(dot, scratch) / (float)N;
#pragma unroll
        for (int j = 0; j < kMaxVecPerThread; ++j) {
            const int c = threadIdx.x + j * 256;
            if (c < nvec) {
#pragma unroll
                for (int e = 0; e < V; ++e) g[j][e] = (g[j][e] - x[j][e] * mean) * inv * swish_gradf(ov[j][e]);
                store_vec(d_o + row * N + (size_t)c * V, g[j]);
            }
        }
    }
    if (dw_part != nullptr) {
#pragma unroll
        for (int j = 0; j < kMaxVecPerThread; ++j) {
            const int c = threadIdx.x + j * 256;
            if (c < nvec) {
#pragma unroll
                for (int e = 0; e < V; ++e) dw_part[(size_t)blockIdx.x * N + c * V + e] = dw[j][e];
            }
        }
    }
}
__global__ void out_norm_dw_kernel(const float* __restrict__ dw_part, float* __restrict__ dweight, int N, int nparts) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= N) return;
    double acc = 0.0;
    for (int p = 0; p < nparts; ++p) acc += (double)dw_part[(size_t)p * N + c];
    dweight[c] = (float)acc;
}

unsigned stream_blocks(size_t nvec) {
    const size_t want = (nvec + 255) / 256;
    return (unsigned)(want < 148 * 16 ? (want ? want : 1) : 148 * 16);
}

}  // namespace

// n elements (a multiple of the 16-byte vector) of io type
cudaError_t launch_swish_fwd(const void* in, void* out, size_t n, int io, cudaStream_t st) {
    if (io == GSA_BF16) {
        const size_t nv = n / 8;
        swish_fwd_kernel<__nv_bfloat16><<<stream_blocks(nv), 256, 0, st>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, nv);
    } else {
        const size_t nv = n / 4;
        swish_fwd_kernel<float><<<stream_blocks(nv), 256, 0, st>>>((const float*)in, (float*)out, nv);
    }
    return cudaGetLastError();
}
cudaError_t launch_swish_bwd(const void* x, void* d, size_t n, int io, cudaStream_t st) {
    if (io == GSA_BF16) {
        const size_t nv = n / 8;
        swish_bwd_kernel<__nv_bfloat16><<<stream_blocks(nv), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)d, nv);
    } else {
        const size_t nv = n / 4;
        swish_bwd_kernel<float><<<stream_blocks(nv), 256, 0, st>>>((const float*)x, (float*)d, nv);
    }
    return cudaGetLastError();
}
int out_norm_max_width(int io) { return 256 * kMaxVecPerThread * (io == GSA_BF16 ? 8 : 4); }
size_t out_norm_bwd_parts(size_t rows) { return (rows + kRowsPerCta - 1) / kRowsPerCta; }
cudaError_t launch_out_norm_fwd(const void* o, const float* weight, float eps, void* y, size_t rows, int N, int io,
                                cudaStream_t st) {
    if (io == GSA_BF16) out_norm_fwd_kernel<__nv_bfloat16><<<(unsigned)rows, 256, 0, st>>>((const __nv_bfloat16*)o, weight, eps, (__nv_bfloat16*)y, N);
    else out_norm_fwd_kernel<float><<<(unsigned)rows, 256, 0, st>>>((const float*)o, weight, eps, (float*)y, N);
    return cudaGetLastError();
}
cudaError_t launch_out_norm_bwd(const void* o, const void* dy, const float* weight, float eps, void* d_o, float* dw_part,
                                float* dweight, size_t rows, int N, int io, cudaStream_t st) {
    const unsigned parts = (unsigned)out_norm_bwd_parts(rows);
    if (io == GSA_BF16)
        out_norm_bwd_kernel<__nv_bfloat16><<<parts, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)dy, weight, eps,
                                                                (__nv_bfloat16*)d_o, dweight ? dw_part : nullptr, N, rows);
    else
        out_norm_bwd_kernel<float><<<parts, 256, 0, st>>>((const float*)o, (const float*)dy, weight, eps, (float*)d_o,
                                                        dweight ? dw_part : nullptr, N, rows);
    if (dweight != nullptr) out_norm_dw_kernel<<<(N + 255) / 256, 256, 0, st>>>(dw_part, dweight, N, (int)parts);
    return cudaGetLastError();
}

}  // namespace gsa
