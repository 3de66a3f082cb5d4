// Slot-axis (m-sized) kernels of the GSA layer: the chunk-local log-gate cumulative sum
// (chunk_cumsum of Algorithm 1), the slot softmax between the two passes and its
// backward, and the forget-gate gradient (reversed cumulative sum, App. B).
// All of them stream [B,T,H,m] fp32 tensors once: they are HBM-bound.
#include "common.cuh"

namespace gsa {

// ------------------------------------------------------------------ chunk_cumsum
// One thread per (chunk, slot); a block covers 256/M consecutive chunks of one (b,h).
// `chunk` is the chunk length of the kernels that will consume G (64 or 128).
// Rows of one chunk are read 8 at a time so that several loads are in flight.
template <int M>
__global__ void __launch_bounds__(256) gate_cumsum_kernel(const float* __restrict__ gate,
                                                          int gate_is_log,
                                                          float* __restrict__ G,
                                                          float* __restrict__ I, int T, int H,
                                                          int chunk, int nchunks) {
    const int s = threadIdx.x;
    const int n = blockIdx.y * blockDim.y + threadIdx.y;
    if (n >= nchunks) return;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * chunk;
    const int rows = min(chunk, T - t0);
    const size_t stride = (size_t)H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    float run = 0.f;
    for (int i0 = 0; i0 < rows; i0 += 8) {
        float x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            x[u] = (i0 + u < rows) ? gate[base + (size_t)(i0 + u) * stride] : (gate_is_log ? 0.f : 1.f);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (i0 + u < rows) {
                float g, inp;
                if (gate_is_log) {
                    g = x[u];
                    inp = -expm1f(g);
                } else {
                    g = logf(x[u]);
                    inp = 1.f - x[u];
                }
                g = fmaxf(g, kLogGateMin);
                run += g;
                G[base + (size_t)(i0 + u) * stride] = run;
                I[base + (size_t)(i0 + u) * stride] = inp;
            }
        }
    }
}

cudaError_t launch_gate_cumsum(const float* gate, int gate_is_log, float* G, float* I, int B,
                               int T, int H, int M, int chunk, cudaStream_t st) {
    const int nchunks = (T + chunk - 1) / chunk;
    dim3 block(M, 256 / M);
    dim3 grid(B * H, (nchunks + block.y - 1) / block.y);
    if (M == 64)
        gate_cumsum_kernel<64><<<grid, block, 0, st>>>(gate, gate_is_log, G, I, T, H, chunk, nchunks);
    else
        gate_cumsum_kernel<32><<<grid, block, 0, st>>>(gate, gate_is_log, G, I, T, H, chunk, nchunks);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ slot softmax
// One warp per token-head row of M slots (M/32 values per lane).
template <int M>
__global__ void __launch_bounds__(256) slot_softmax_fwd_kernel(const float* __restrict__ part,
                                                               int nslice, float scale,
                                                               float* __restrict__ ok,
                                                               float* __restrict__ p,
                                                               size_t rows) {
    constexpr int R = M / 32;
    const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const size_t total = rows * M;
    float z[R];
    float zmax = -INFINITY;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const size_t idx = row * M + lane + 32 * r;
        float acc = 0.f;
        for (int sl = 0; sl < nslice; ++sl) acc += part[idx + (size_t)sl * total];
        z[r] = acc * scale;
        zmax = fmaxf(zmax, z[r]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
    float e[R], den = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) { e[r] = __expf(z[r] - zmax); den += e[r]; }
#pragma unroll
    for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    const float inv = 1.f / den;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const size_t idx = row * M + lane + 32 * r;
        ok[idx] = z[r];
        p[idx] = e[r] * inv;
    }
}

cudaError_t launch_slot_softmax_fwd(const float* part, int nslice, float scale, float* ok,
                                    float* p, size_t rows, int M, cudaStream_t st) {
    const unsigned grid = (unsigned)((rows + 7) / 8);
    if (M == 64)
        slot_softmax_fwd_kernel<64><<<grid, 256, 0, st>>>(part, nslice, scale, ok, p, rows);
    else
        slot_softmax_fwd_kernel<32><<<grid, 256, 0, st>>>(part, nslice, scale, ok, p, rows);
    return cudaGetLastError();
}

// Softmax backward (dsoftmax of Algorithm 1): from the scaled logits ok and the gradient dp
// w.r.t. the softmax output (summed over the d_v slices that produced it):
//   p = softmax(ok); dok = p * (dp - <p,dp>); dz = scale * dok (gradient w.r.t. the unscaled
//   pass-1 output); u = p*dp + ok*dok (the two "query x query-gradient" terms of the
//   forget-gate gradient).
template <int M>
__global__ void __launch_bounds__(256) slot_softmax_bwd_kernel(const float* __restrict__ ok,
                                                               const float* __restrict__ dp_part,
                                                               int nslice, float scale,
                                                               float* __restrict__ p,
                                                               float* __restrict__ dz,
                                                               float* __restrict__ u,
                                                               size_t rows) {
    constexpr int R = M / 32;
    const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const size_t total = rows * M;
    float z[R], dpv[R];
    float zmax = -INFINITY;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const size_t idx = row * M + lane + 32 * r;
        z[r] = ok[idx];
        zmax = fmaxf(zmax, z[r]);
        float acc = 0.f;
        for (int sl = 0; sl < nslice; ++sl) acc += dp_part[idx + (size_t)sl * total];
        dpv[r] = acc;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
    float e[R], den = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) { e[r] = __expf(z[r] - zmax); den += e[r]; }
#pragma unroll
    for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    const float inv = 1.f / den;
    float pdp = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) { e[r] *= inv; pdp += e[r] * dpv[r]; }
#pragma unroll
    for (int o = 16; o; o >>= 1) pdp += __shfl_xor_sync(0xffffffffu, pdp, o);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const size_t idx = row * M + lane + 32 * r;
        const float dok = e[r] * (dpv[r] - pdp);
        p[idx] = e[r];
        dz[idx] = scale * dok;
        u[idx] = e[r] * dpv[r] + z[r] * dok;
    }
}

cudaError_t launch_slot_softmax_bwd(const float* ok, const float* dp_part, int nslice,
                                    float scale, float* p, float* dz, float* u, size_t rows,
                                    int M, cudaStream_t st) {
    const unsigned grid = (unsigned)((rows + 7) / 8);
    if (M == 64)
        slot_softmax_bwd_kernel<64><<<grid, 256, 0, st>>>(ok, dp_part, nslice, scale, p, dz, u, rows);
    else
        slot_softmax_bwd_kernel<32><<<grid, 256, 0, st>>>(ok, dp_part, nslice, scale, p, dz, u, rows);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ forget-gate gradient
// d(log a_t)|decay = sum_{i>=t} (u_i - I_i * dI_i) + <dKT, K_T>_rows + <dVT, V_T>_rows
// (the reversed cumulative sum of App. B, taken over the whole sequence), then
//   gate holds a     : dgate = d(log a)|decay / a - dI
//   gate holds log a : dgate = d(log a)|decay - a * dI
// Three steps: per-chunk totals, an exclusive suffix scan over the chunk totals (fp64),
// and the chunk-local reversed sums started from that carry.
template <int M>
__device__ __forceinline__ float sum_parts(const float* part, int nslice, size_t idx, size_t total) {
    float acc = 0.f;
    for (int sl = 0; sl < nslice; ++sl) acc += part[idx + (size_t)sl * total];
    return acc;
}

template <int M>
__global__ void __launch_bounds__(256) gate_grad_totals_kernel(
    const float* __restrict__ u, const float* __restrict__ I, const float* __restrict__ dIk, int nsk,
    const float* __restrict__ dIv, int nsv, float* __restrict__ chunk_tot, int B, int T, int H,
    int nchunks) {
    const int s = threadIdx.x;
    const int n = blockIdx.y * blockDim.y + threadIdx.y;
    if (n >= nchunks) return;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * kChunk;
    const int rows = min(kChunk, T - t0);
    const size_t stride = (size_t)H * M, total = (size_t)B * T * H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    float tot = 0.f;
    for (int i = 0; i < rows; ++i) {
        const size_t idx = base + (size_t)i * stride;
        const float dI = sum_parts<M>(dIk, nsk, idx, total) + sum_parts<M>(dIv, nsv, idx, total);
        tot += u[idx] - I[idx] * dI;
    }
    chunk_tot[((size_t)bh * nchunks + n) * M + s] = tot;
}

// chunk_tot[bh][n][s] <- sum over chunks n' > n of the totals, plus the final-memory term.
template <int M>
__global__ void gate_grad_scan_kernel(float* __restrict__ chunk_tot, const float* __restrict__ dKT,
                                      const float* __restrict__ KT, const float* __restrict__ dVT,
                                      const float* __restrict__ VT, int d_k, int d_v, int nchunks) {
    const int s = threadIdx.x, bh = blockIdx.x;
    double carry = 0.0;
    if (dKT != nullptr) {
        const float* a = dKT + ((size_t)bh * M + s) * d_k;
        const float* bb = KT + ((size_t)bh * M + s) * d_k;
        for (int c = 0; c < d_k; ++c) carry += (double)a[c] * (double)bb[c];
    }
    if (dVT != nullptr) {
        const float* a = dVT + ((size_t)bh * M + s) * d_v;
        const float* bb = VT + ((size_t)bh * M + s) * d_v;
        for (int c = 0; c < d_v; ++c) carry += (double)a[c] * (double)bb[c];
    }
    for (int n = nchunks - 1; n >= 0; --n) {
        const size_t idx = ((size_t)bh * nchunks + n) * M + s;
        const float t = chunk_tot[idx];
        chunk_tot[idx] = (float)carry;
        carry += (double)t;
    }
}

template <int M>
__global__ void __launch_bounds__(256) gate_grad_final_kernel(
    const float* __restrict__ u, const float* __restrict__ I, const float* __restrict__ dIk, int nsk,
    const float* __restrict__ dIv, int nsv, const float* __restrict__ gate, int gate_is_log,
    const float* __restrict__ chunk_carry, float* __restrict__ dgate, int B, int T, int H,
    int nchunks) {
    const int s = threadIdx.x;
    const int n = blockIdx.y * blockDim.y + threadIdx.y;
    if (n >= nchunks) return;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * kChunk;
    const int rows = min(kChunk, T - t0);
    const size_t stride = (size_t)H * M, total = (size_t)B * T * H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    float run = chunk_carry[((size_t)bh * nchunks + n) * M + s];
    for (int i = rows - 1; i >= 0; --i) {
        const size_t idx = base + (size_t)i * stride;
        const float dI = sum_parts<M>(dIk, nsk, idx, total) + sum_parts<M>(dIv, nsv, idx, total);
        run += u[idx] - I[idx] * dI;
        const float gt = gate[idx];
        float out;
        if (gate_is_log) {
            out = run - __expf(fmaxf(gt, kLogGateMin)) * dI;
        } else {
            // a == 0 leaves no way back from d(log a) to da: only the input-gate part is kept
            out = (gt > 0.f) ? run / gt - dI : -dI;
        }
        dgate[idx] = out;
    }
}

cudaError_t launch_gate_grad(const float* u, const float* I, const float* dIk_part, int nsk,
                             const float* dIv_part, int nsv, const float* gate,
                             int gate_is_log, const float* dKT, const float* KT,
                             const float* dVT, const float* VT, int d_k, int d_v,
                             float* chunk_tot, float* dgate, int B, int T, int H, int M,
                             cudaStream_t st) {
    const int nchunks = (T + kChunk - 1) / kChunk;
    dim3 block(M, 256 / M);
    dim3 grid(B * H, (nchunks + block.y - 1) / block.y);
    if (M == 64) {
        gate_grad_totals_kernel<64><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv,
                                                            chunk_tot, B, T, H, nchunks);
        gate_grad_scan_kernel<64><<<B * H, 64, 0, st>>>(chunk_tot, dKT, KT, dVT, VT, d_k, d_v, nchunks);
        gate_grad_final_kernel<64><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv, gate,
                                                           gate_is_log, chunk_tot, dgate, B, T, H,
                                                           nchunks);
    } else {
        gate_grad_totals_kernel<32><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv,
                                                            chunk_tot, B, T, H, nchunks);
        gate_grad_scan_kernel<32><<<B * H, 32, 0, st>>>(chunk_tot, dKT, KT, dVT, VT, d_k, d_v, nchunks);
        gate_grad_final_kernel<32><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv, gate,
                                                           gate_is_log, chunk_tot, dgate, B, T, H,
                                                           nchunks);
    }
    return cudaGetLastError();
}

}  // namespace gsa
