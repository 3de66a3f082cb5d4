// Slot-axis (m-sized) kernels of the GSA layer: the chunk-local log-gate cumulative sum
// (chunk_cumsum of Algorithm 1), the slot softmax between the two passes and its
// backward, and the forget-gate gradient (reversed cumulative sum, App. B).
// All of them stream [B,T,H,m] fp32 tensors once: they are HBM-bound.
#include "common.cuh"
#include "tc_common.cuh"

namespace gsa {

// ------------------------------------------------------------------ chunk_cumsum
// One CTA per (b,h, chunk): M/2 slot pairs x (chunk / 8) row groups.  A thread takes the logs
// of its 8 rows x 2 slots (8 independent 8-byte loads in flight), sums them, the group sums
// are scanned through shared memory, and the thread writes its running sums.  `chunk` is the
// chunk length of the kernels that will consume G (64 or 128).
constexpr int kCumRows = 8;

// (x0, x1) as a packed bf16 pair and the packed rounding residuals: two packed conversions
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
    lo = *reinterpret_cast<const uint32_t*>(&l);
}
template <int M>
__device__ __forceinline__ void store_split2(__nv_bfloat16* row, int c, float x0, float x1) {
    uint32_t hi, lo;
    split_bf16x2(x0, x1, hi, lo);
    *reinterpret_cast<uint32_t*>(row + c) = hi;
    *reinterpret_cast<uint32_t*>(row + M + c) = lo;
}

// Packed sequences: is token t the first token of a sequence other than the first?  cu holds the
// nseq + 1 ascending sequence offsets along T (cu[0] = 0, cu[nseq] = T).
__device__ __forceinline__ bool sequence_starts_at(const int* __restrict__ cu, int nseq, int t) {
    if (cu == nullptr || t == 0) return false;
    int lo = 1, hi = nseq - 1;
    while (lo <= hi) {
        const int mid = (lo + hi) >> 1, v = cu[mid];
        if (v == t) return true;
        if (v < t) lo = mid + 1; else hi = mid - 1;
    }
    return false;
}

template <int M>
__global__ void __launch_bounds__(M * 8 > 1024 ? 1024 : M * 8, M > 64 ? 1 : 2) gate_cumsum_kernel(const float* __restrict__ gate,
                                                            int gate_kind, float inv_tau,
                                                            float* __restrict__ G,
                                                            float* __restrict__ I, int T, int H,
                                                            int chunk, int* __restrict__ strong_flag, int nseg,
                                                            __nv_bfloat16* __restrict__ decayed, int fast_log,
                                                            const int* __restrict__ cu_seqlens, int nseq) {
    __shared__ double group_sum[16][M];
    const int s = 2 * threadIdx.x, grp = threadIdx.y;          // blockDim.y = chunk / 8 <= 16
    const int n = blockIdx.y;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * chunk + grp * kCumRows;
    const int rows = max(0, min(kCumRows, min(T, (n + 1) * chunk) - t0));
    const size_t stride = (size_t)H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    float2 g[kCumRows], inps[kCumRows];
#pragma unroll
    for (int i = 0; i < kCumRows; ++i) {
        // (rows past the end: a = 1, log a = 0)
        const float neutral = gate_kind == GSA_GATE_LOG_A ? 0.f : (gate_kind == GSA_GATE_LOGITS ? 80.f : 1.f);
        float2 x = make_float2(neutral, neutral);
        if (i < rows) x = *reinterpret_cast<const float2*>(gate + base + (size_t)i * stride);
        if (gate_kind == GSA_GATE_LOGITS) x = make_float2(log_gate_from_logit(x.x, inv_tau), log_gate_from_logit(x.y, inv_tau));
        if (gate_kind != GSA_GATE_A) {
            g[i] = x;
            inps[i] = make_float2(-expm1f(x.x), -expm1f(x.y));
        } else {
            g[i] = fast_log ? make_float2(__logf(x.x), __logf(x.y)) : make_float2(logf(x.x), logf(x.y));
            inps[i] = make_float2(1.f - x.x, 1.f - x.y);
        }
        g[i].x = fmaxf(g[i].x, kLogGateMin);
        g[i].y = fmaxf(g[i].y, kLogGateMin);
        // the first token of a packed sequence drops what the memories carried (its decay is exp(-100) = 0 in
        // fp32); its own write, 1 - a, is untouched.  The chunk is then flagged for the strong-decay kernels.
        if (sequence_starts_at(cu_seqlens, nseq, t0 + i)) g[i] = make_float2(kLogGateMin, kLogGateMin);
        if (i < rows) *reinterpret_cast<float2*>(I + base + (size_t)i * stride) = inps[i];
    }
    // running sums: fp32 inside the thread's 8 rows (g becomes the running sum), fp64 across the
    // row groups -- G stays within an ulp of the exact cumulative sum also where strong decay
    // makes |G| reach the hundreds, without a conversion per element
#pragma unroll
    for (int i = 1; i < kCumRows; ++i) {
        g[i].x = (i < rows) ? g[i - 1].x + g[i].x : g[i - 1].x;
        g[i].y = (i < rows) ? g[i - 1].y + g[i].y : g[i - 1].y;
    }
    const double acc0 = rows > 0 ? (double)g[kCumRows - 1].x : 0.0, acc1 = rows > 0 ? (double)g[kCumRows - 1].y : 0.0;
    group_sum[grp][s] = acc0;
    group_sum[grp][s + 1] = acc1;
    __syncthreads();
    double before0 = 0.0, before1 = 0.0;
    for (int q = 0; q < grp; ++q) {
        before0 += group_sum[q][s];
        before1 += group_sum[q][s + 1];
    }
    // the chunk's total log-decay decides which of the chunk kernels takes this (b,h)
    // (with segment-parallel scheduling the flags are per (batch, segment, head))
    if (strong_flag != nullptr && grp == (int)blockDim.y - 1 &&
        fmin(before0 + acc0, before1 + acc1) < (double)kFactorisedDecayMin) {
        const int seg = (int)(((long long)n * chunk) / (T / nseg));
        strong_flag[(b * nseg + seg) * H + h] = 1;
    }
    // second pass over the same rows: the sums of the groups before as a float pair (value, rest)
    const float b0h = (float)before0, b0l = (float)(before0 - (double)b0h);
    const float b1h = (float)before1, b1l = (float)(before1 - (double)b1h);
#pragma unroll
    for (int i = 0; i < kCumRows; ++i)
        if (i < rows) {
            const float G0 = b0h + (b0l + g[i].x), G1 = b1h + (b1l + g[i].y);
            *reinterpret_cast<float2*>(G + base + (size_t)i * stride) = make_float2(G0, G1);
            if (decayed != nullptr) {
                // (meaningful for moderate decay only; pairs with a strong-decay chunk do not read it)
                store_split2<M>(decayed + 2 * (base + (size_t)i * stride - s), s, inps[i].x * __expf(-G0),
                                inps[i].y * __expf(-G1));
            }
        }
}

cudaError_t launch_gate_cumsum(const float* gate, int gate_kind, float inv_tau, float* G, float* I, int B,
                               int T, int H, int M, int chunk, int* strong_flag, int nseg, void* decayed, int fast_log,
                               cudaStream_t st, const int* cu_seqlens, int nseq) {
    if (chunk % kCumRows != 0 || chunk / kCumRows > 16 || (M / 2) * (chunk / kCumRows) > 1024) return cudaErrorInvalidValue;
    const int nchunks = (T + chunk - 1) / chunk;
    dim3 block(M / 2, chunk / kCumRows);
    dim3 grid(B * H, nchunks);
    if (M == 128)
        gate_cumsum_kernel<128><<<grid, block, 0, st>>>(gate, gate_kind, inv_tau, G, I, T, H, chunk, strong_flag, nseg < 1 ? 1 : nseg,
                                                        static_cast<__nv_bfloat16*>(decayed), fast_log, cu_seqlens, nseq);
    else if (M == 64)
        gate_cumsum_kernel<64><<<grid, block, 0, st>>>(gate, gate_kind, inv_tau, G, I, T, H, chunk, strong_flag, nseg < 1 ? 1 : nseg,
                                                       static_cast<__nv_bfloat16*>(decayed), fast_log, cu_seqlens, nseq);
    else
        gate_cumsum_kernel<32><<<grid, block, 0, st>>>(gate, gate_kind, inv_tau, G, I, T, H, chunk, strong_flag, nseg < 1 ? 1 : nseg,
                                                       static_cast<__nv_bfloat16*>(decayed), fast_log, cu_seqlens, nseq);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ slot softmax
// M/4 lanes per token-head row of M slots, four adjacent slots per lane (one 16-byte access per
// tensor and lane), 128/M rows per warp; reductions run over the lanes of a row.
constexpr int kSmR = 4;                                  // slots per lane
__device__ __forceinline__ void ld_vec(const float* p, float (&x)[kSmR]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
}
__device__ __forceinline__ void st_vec(float* p, const float (&x)[kSmR]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
// the lane's slots of a decayed-operand row [hi(M) | lo(M)]
template <int M>
__device__ __forceinline__ void st_split(__nv_bfloat16* row, int c, const float (&x)[kSmR]) {
    uint32_t h0, h1, l0, l1;
    split_bf16x2(x[0], x[1], h0, l0);
    split_bf16x2(x[2], x[3], h1, l1);
    *reinterpret_cast<uint2*>(row + c) = make_uint2(h0, h1);
    *reinterpret_cast<uint2*>(row + M + c) = make_uint2(l0, l1);
}
template <int LPR>
__device__ __forceinline__ float row_max(float x) {
#pragma unroll
    for (int o = LPR / 2; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
template <int LPR>
__device__ __forceinline__ float row_sum(float x) {
#pragma unroll
    for (int o = LPR / 2; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <int M>
__global__ void __launch_bounds__(256) slot_softmax_fwd_kernel(const float* __restrict__ part,
                                                               int nslice, float scale, int act,
                                                               float* __restrict__ ok,
                                                               float* __restrict__ p,
                                                               int rows_per_batch, const float* __restrict__ G,
                                                               __nv_bfloat16* __restrict__ p_decayed,
                                                               PendingDecay pend, int m_active) {
    constexpr int R = kSmR, LPR = M / R, RPW = 32 / LPR;       // lanes per row, rows per warp
    const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
    const int r_in_b = (blockIdx.x * 8 + (threadIdx.x >> 5)) * RPW + sub, b = blockIdx.y;
    const bool live = r_in_b < rows_per_batch;       // a row past the end repeats the last one (full-warp shuffles)
    const int rr = live ? r_in_b : rows_per_batch - 1;
    const size_t row = (size_t)b * rows_per_batch + rr;
    const size_t total = (size_t)gridDim.y * rows_per_batch * M;
    const size_t idx = row * M + l * R;
    const bool pending = pend.pending(b, rr);
    // slots from m_active on are padding (a layer with fewer slots than the kernels' tile): they take no part
    const bool padded = l * R >= m_active;
    // serving the flagged pairs only: a warp none of whose rows is flagged has nothing to do
    const bool skip = pend.strong_only != 0 && pending;
    if (__all_sync(0xffffffffu, skip)) return;
    float z[R], eg[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { z[r] = 0.f; eg[r] = 1.f; }
#pragma unroll 4
    for (int sl = 0; sl < nslice; ++sl) {
        float t[R];
        ld_vec(part + idx + (size_t)sl * total, t);
#pragma unroll
        for (int r = 0; r < R; ++r) z[r] += t[r];
    }
    if (G != nullptr) {
        ld_vec(G + idx, eg);
#pragma unroll
        for (int r = 0; r < R; ++r) eg[r] = __expf(eg[r]);
    }
    float zmax = -INFINITY;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (pending) z[r] *= eg[r];
        z[r] *= scale;
        if (!padded) zmax = fmaxf(zmax, z[r]);
    }
    float e[R];
    if (act == GSA_ACT_SOFTMAX) {
        zmax = row_max<LPR>(zmax);
        float den = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) { e[r] = padded ? 0.f : __expf(z[r] - zmax); den += e[r]; }
        den = row_sum<LPR>(den);
        const float inv = 1.f / den;
#pragma unroll
        for (int r = 0; r < R; ++r) e[r] *= inv;
    } else {               // element-wise replacement of the softmax (uniform over the launch)
#pragma unroll
        for (int r = 0; r < R; ++r) e[r] = padded ? 0.f : slot_act_value(z[r], act);
    }
    if (!live || skip) return;
    if (ok != nullptr) st_vec(ok + idx, z);
    // fp32 p is read by the general chunk kernels and the CUDA-core kernels only: rows of a pair
    // that the pipelined kernels serve (pending) get the decayed bf16 rows alone
    if (!pending) st_vec(p + idx, e);
    if (p_decayed != nullptr) {
#pragma unroll
        for (int r = 0; r < R; ++r) e[r] *= eg[r];
        st_split<M>(p_decayed + row * 2 * M, l * R, e);
    }
}

cudaError_t launch_slot_softmax_fwd(const float* part, int nslice, float scale, int act, float* ok,
                                    float* p, int B, int rows_per_batch, int M, const float* G, void* p_decayed,
                                    PendingDecay pend, cudaStream_t st, int m_active) {
    if (m_active <= 0 || m_active > M) m_active = M;
    const int rpb = 8 * (128 / M);       // rows per block: 8 warps x 128/M rows
    const dim3 grid((unsigned)((rows_per_batch + rpb - 1) / rpb), (unsigned)B);
    const int rows = rows_per_batch;
    if (M == 128)
        slot_softmax_fwd_kernel<128><<<grid, 256, 0, st>>>(part, nslice, scale, act, ok, p, rows, G,
                                                           static_cast<__nv_bfloat16*>(p_decayed), pend, m_active);
    else if (M == 64)
        slot_softmax_fwd_kernel<64><<<grid, 256, 0, st>>>(part, nslice, scale, act, ok, p, rows, G,
                                                          static_cast<__nv_bfloat16*>(p_decayed), pend, m_active);
    else
        slot_softmax_fwd_kernel<32><<<grid, 256, 0, st>>>(part, nslice, scale, act, ok, p, rows, G,
                                                          static_cast<__nv_bfloat16*>(p_decayed), pend, m_active);
    return cudaGetLastError();
}

// Softmax backward (dsoftmax of Algorithm 1; f'(ok) dp for an element-wise replacement f): from the scaled logits ok and the gradient dp
// w.r.t. the softmax output (summed over the d_v slices that produced it):
//   p = softmax(ok); dok = p * (dp - <p,dp>); dz = scale * dok (gradient w.r.t. the unscaled
//   pass-1 output); u = p*dp + ok*dok (the two "query x query-gradient" terms of the
//   forget-gate gradient).
template <int M>
__global__ void __launch_bounds__(256) slot_softmax_bwd_kernel(const float* __restrict__ ok,
                                                               const float* __restrict__ dp_part,
                                                               int nslice, float scale, int act,
                                                               float* __restrict__ p,
                                                               float* __restrict__ dz,
                                                               float* __restrict__ u,
                                                               int rows_per_batch, const float* __restrict__ G,
                                                               __nv_bfloat16* __restrict__ p_decayed,
                                                               __nv_bfloat16* __restrict__ dz_decayed,
                                                               PendingDecay pend, int m_active) {
    constexpr int R = kSmR, LPR = M / R, RPW = 32 / LPR;       // lanes per row, rows per warp
    const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
    const int r_in_b = (blockIdx.x * 8 + (threadIdx.x >> 5)) * RPW + sub, b = blockIdx.y;
    const bool live = r_in_b < rows_per_batch;       // a row past the end repeats the last one (full-warp shuffles)
    const int rr = live ? r_in_b : rows_per_batch - 1;
    const size_t row = (size_t)b * rows_per_batch + rr;
    const size_t total = (size_t)gridDim.y * rows_per_batch * M;
    const size_t idx = row * M + l * R;
    const bool pending = pend.pending(b, rr);
    const bool skip = pend.strong_only != 0 && pending;      // (as in the forward kernel)
    const bool padded = l * R >= m_active;                   // (likewise)
    if (__all_sync(0xffffffffu, skip)) return;
    float z[R], dpv[R], eg[R];
    ld_vec(ok + idx, z);
#pragma unroll
    for (int r = 0; r < R; ++r) { dpv[r] = 0.f; eg[r] = 1.f; }
#pragma unroll 4
    for (int sl = 0; sl < nslice; ++sl) {
        float t[R];
        ld_vec(dp_part + idx + (size_t)sl * total, t);
#pragma unroll
        for (int r = 0; r < R; ++r) dpv[r] += t[r];
    }
    if (G != nullptr) {
        ld_vec(G + idx, eg);
#pragma unroll
        for (int r = 0; r < R; ++r) eg[r] = __expf(eg[r]);
    }
    float zmax = -INFINITY;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (pending) dpv[r] *= eg[r];
        if (padded) { z[r] = 0.f; dpv[r] = 0.f; }
        else zmax = fmaxf(zmax, z[r]);
    }
    float e[R], dzv[R], uv[R];
    if (act == GSA_ACT_SOFTMAX) {
        zmax = row_max<LPR>(zmax);
        float den = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) { e[r] = padded ? 0.f : __expf(z[r] - zmax); den += e[r]; }
        den = row_sum<LPR>(den);
        const float inv = 1.f / den;
        float pdp = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) { e[r] *= inv; pdp += e[r] * dpv[r]; }
        pdp = row_sum<LPR>(pdp);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float dok = e[r] * (dpv[r] - pdp);
            dzv[r] = scale * dok;
            uv[r] = e[r] * dpv[r] + z[r] * dok;
        }
    } else {               // element-wise replacement f of the softmax: dok = f'(ok) dp
#pragma unroll
        for (int r = 0; r < R; ++r) {
            e[r] = padded ? 0.f : slot_act_value(z[r], act);
            const float dok = slot_act_slope(z[r], act) * dpv[r];
            dzv[r] = scale * dok;
            uv[r] = e[r] * dpv[r] + z[r] * dok;
        }
    }
    if (!live || skip) return;
    if (!pending) {       // (as in the forward: fp32 p and dz only where a non-pipelined kernel reads them)
        if (p != nullptr) st_vec(p + idx, e);      // (p == NULL: the forward's p is kept and in use)
        st_vec(dz + idx, dzv);
    }
    st_vec(u + idx, uv);
    if (dz_decayed != nullptr) {
#pragma unroll
        for (int r = 0; r < R; ++r) { e[r] *= eg[r]; dzv[r] *= eg[r]; }
        if (p_decayed != nullptr) st_split<M>(p_decayed + row * 2 * M, l * R, e);
        st_split<M>(dz_decayed + row * 2 * M, l * R, dzv);
    }
}

cudaError_t launch_slot_softmax_bwd(const float* ok, const float* dp_part, int nslice,
                                    float scale, int act, float* p, float* dz, float* u, int B, int rows_per_batch,
                                    int M, const float* G, void* p_decayed, void* dz_decayed,
                                    PendingDecay pend, cudaStream_t st, int m_active) {
    if (m_active <= 0 || m_active > M) m_active = M;
    const int rpb = 8 * (128 / M);       // rows per block: 8 warps x 128/M rows
    const dim3 grid((unsigned)((rows_per_batch + rpb - 1) / rpb), (unsigned)B);
    const int rows = rows_per_batch;
    if (M == 128)
        slot_softmax_bwd_kernel<128><<<grid, 256, 0, st>>>(ok, dp_part, nslice, scale, act, p, dz, u, rows, G,
                                                           static_cast<__nv_bfloat16*>(p_decayed),
                                                           static_cast<__nv_bfloat16*>(dz_decayed), pend, m_active);
    else if (M == 64)
        slot_softmax_bwd_kernel<64><<<grid, 256, 0, st>>>(ok, dp_part, nslice, scale, act, p, dz, u, rows, G,
                                                          static_cast<__nv_bfloat16*>(p_decayed),
                                                          static_cast<__nv_bfloat16*>(dz_decayed), pend, m_active);
    else
        slot_softmax_bwd_kernel<32><<<grid, 256, 0, st>>>(ok, dp_part, nslice, scale, act, p, dz, u, rows, G,
                                                          static_cast<__nv_bfloat16*>(p_decayed),
                                                          static_cast<__nv_bfloat16*>(dz_decayed), pend, m_active);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ forget-gate gradient
// d(log a_t)|decay = sum_{i>=t} (u_i - I_i * dI_i) + <dKT, K_T>_rows + <dVT, V_T>_rows
// (the reversed cumulative sum of App. B, taken over the whole sequence), then
//   gate holds a     : dgate = d(log a)|decay / a - dI
//   gate holds log a : dgate = d(log a)|decay - a * dI
// Three steps: block-local reversed sums of 16-row blocks (the only pass over the inputs), an
// exclusive suffix scan over the block totals (fp64), and the addition of each block's carry.

constexpr int kGG = 16;   // rows per thread of the gate-gradient kernels

// From the decay-path gradient d(log a) (`run`: what this block knows of it) and the input-gate
// gradient dI to the gradient with respect to the gate tensor as passed (`gt`):
//   a       : run / a - dI            (a == 0 leaves no way back from d(log a): only -dI is kept)
//   log a   : run - a dI
//   logits  : (run - a dI) sigmoid(-x) / tau
__device__ __forceinline__ float gate_grad_out(float run, float dI, float gt, int gate_kind, float inv_tau) {
    if (gate_kind == GSA_GATE_A) return (gt > 0.f) ? run / gt - dI : -dI;
    if (gate_kind == GSA_GATE_LOG_A) return run - __expf(fmaxf(gt, kLogGateMin)) * dI;
    const float a = __expf(fmaxf(log_gate_from_logit(gt, inv_tau), kLogGateMin));
    return (run - a * dI) * dlog_gate_dlogit(gt, inv_tau);
}
// the carry of the blocks after this one, in the same units
__device__ __forceinline__ float gate_grad_carry(float carry, float gt, int gate_kind, float inv_tau) {
    if (gate_kind == GSA_GATE_A) return (gt > 0.f) ? carry / gt : 0.f;
    if (gate_kind == GSA_GATE_LOG_A) return carry;
    return carry * dlog_gate_dlogit(gt, inv_tau);
}

// dI[i] = sum over the d_k and d_v slices of the input-gate gradient partial sums, for the
// kGG rows x 2 slots of this thread; the rows of one slice are loaded together (16 loads of 8
// bytes in flight).
__device__ __forceinline__ void load_dI(const float* __restrict__ dIk, int nsk, const float* __restrict__ dIv,
                                        int nsv, size_t base, size_t stride, size_t total, int rows,
                                        float2 (&dI)[kGG]) {
#pragma unroll
    for (int i = 0; i < kGG; ++i) dI[i] = make_float2(0.f, 0.f);
    for (int sl = 0; sl < nsk + nsv; ++sl) {
        const float* src = sl < nsk ? dIk + (size_t)sl * total : dIv + (size_t)(sl - nsk) * total;
        float2 t[kGG];
#pragma unroll
        for (int i = 0; i < kGG; ++i)
            t[i] = (i < rows) ? *reinterpret_cast<const float2*>(src + base + (size_t)i * stride) : make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kGG; ++i) { dI[i].x += t[i].x; dI[i].y += t[i].y; }
    }
}

// blk_tot[bh][n][s] <- sum over blocks n' > n of the totals, plus the final-memory term.
// One CTA per (b,h): M slots x 16 segments of consecutive blocks; fp64 running sums.
template <int M>
__global__ void __launch_bounds__(M * (M > 64 ? 8 : 16)) gate_grad_scan_kernel(
    float* __restrict__ blk_tot, const float* __restrict__ dKT, const float* __restrict__ KT,
    const float* __restrict__ dVT, const float* __restrict__ VT, int d_k, int d_v, int nblk) {
    constexpr int kSeg = M > 64 ? 8 : 16;       // segments of consecutive blocks (threads: M slots x kSeg)
    __shared__ double seg_sum[kSeg][M];
    const int s = threadIdx.x, seg = threadIdx.y, bh = blockIdx.x;
    const int per = (nblk + kSeg - 1) / kSeg;
    const int lo = seg * per, hi = min(nblk, lo + per);
    double sum = 0.0;
    for (int n = lo; n < hi; ++n) sum += (double)blk_tot[((size_t)bh * nblk + n) * M + s];
    seg_sum[seg][s] = sum;
    // final-memory term <dK~_T[s], K~_T[s]> + <dV~_T[s], V~_T[s]>: a warp per slot, lanes along the row
    __shared__ double final_term[M];
    const int warp = (seg * M + s) >> 5, lane = (seg * M + s) & 31, nwarp = (M * kSeg) >> 5;
    for (int slot = warp; slot < M; slot += nwarp) {
        double dot = 0.0;
        if (dKT != nullptr) {
            const float* a = dKT + ((size_t)bh * M + slot) * d_k;
            const float* bb = KT + ((size_t)bh * M + slot) * d_k;
            for (int c = lane; c < d_k; c += 32) dot += (double)a[c] * (double)bb[c];
        }
        if (dVT != nullptr) {
            const float* a = dVT + ((size_t)bh * M + slot) * d_v;
            const float* bb = VT + ((size_t)bh * M + slot) * d_v;
            for (int c = lane; c < d_v; c += 32) dot += (double)a[c] * (double)bb[c];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        if (lane == 0) final_term[slot] = dot;
    }
    __syncthreads();
    double carry = final_term[s];
    for (int g = seg + 1; g < kSeg; ++g) carry += seg_sum[g][s];
    for (int n = hi - 1; n >= lo; --n) {
        const size_t idx = ((size_t)bh * nblk + n) * M + s;
        const float t = blk_tot[idx];
        blk_tot[idx] = (float)carry;
        carry += (double)t;
    }
}

// Block-local pass: for each 16-row block, the reversed running sums of x = u - I dI that start
// at the block's end, turned into the gate gradient as if nothing followed the block, plus
// the block total for the scan.  One read of every input.
template <int M>
__global__ void __launch_bounds__(128) gate_grad_local_kernel(
    const float* __restrict__ u, const float* __restrict__ I, const float* __restrict__ dIk, int nsk,
    const float* __restrict__ dIv, int nsv, const float* __restrict__ gate, int gate_kind, float inv_tau,
    float* __restrict__ blk_tot, float* __restrict__ dgate, int B, int T, int H, int nblk, PendingDecay pend) {
    const int s = 2 * threadIdx.x;                       // this thread's two slots
    const int n = blockIdx.y * blockDim.y + threadIdx.y;
    if (n >= nblk) return;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * kGG;
    const int rows = min(kGG, T - t0);
    const size_t stride = (size_t)H * M, total = (size_t)B * T * H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    auto ld2 = [&](const float* p, int i, float fill) {
        return (i < rows) ? *reinterpret_cast<const float2*>(p + base + (size_t)i * stride) : make_float2(fill, fill);
    };
    float2 x[kGG], dI[kGG], gt[kGG];
    load_dI(dIk, nsk, dIv, nsv, base, stride, total, rows, dI);
    if (pend.G != nullptr && pend.strong[(b * pend.nseg + t0 / (T / pend.nseg)) * H + h] == 0) {
        // the time-reversed value_side runs left their row factor exp(-G_i) to this kernel
#pragma unroll
        for (int i = 0; i < kGG; ++i) gt[i] = ld2(pend.G, i, 0.f);
#pragma unroll
        for (int i = 0; i < kGG; ++i) { dI[i].x *= __expf(-gt[i].x); dI[i].y *= __expf(-gt[i].y); }
    }
#pragma unroll
    for (int i = 0; i < kGG; ++i) gt[i] = ld2(I, i, 0.f);
#pragma unroll
    for (int i = 0; i < kGG; ++i) x[i] = make_float2(-gt[i].x * dI[i].x, -gt[i].y * dI[i].y);
#pragma unroll
    for (int i = 0; i < kGG; ++i) gt[i] = ld2(u, i, 0.f);
#pragma unroll
    for (int i = 0; i < kGG; ++i) { x[i].x += gt[i].x; x[i].y += gt[i].y; }
#pragma unroll
    for (int i = 0; i < kGG; ++i) gt[i] = ld2(gate, i, 1.f);
    float run0 = 0.f, run1 = 0.f;
#pragma unroll
    for (int i = kGG - 1; i >= 0; --i) {
        run0 += x[i].x;
        run1 += x[i].y;
        if (i < rows) {
            const float2 out = make_float2(gate_grad_out(run0, dI[i].x, gt[i].x, gate_kind, inv_tau),
                                           gate_grad_out(run1, dI[i].y, gt[i].y, gate_kind, inv_tau));
            *reinterpret_cast<float2*>(dgate + base + (size_t)i * stride) = out;
        }
    }
    *reinterpret_cast<float2*>(blk_tot + ((size_t)bh * nblk + n) * M + s) = make_float2(run0, run1);
}

// The same block-local pass with its inputs staged through shared memory by TMA (M = 64): one
// CTA per (b,h) and 32 rows, every tile of every input stream (u, I, gate, G and the n_k + n_v
// slices of the input-gate gradient: 12 x 8 KB at d = 512) requested at once by one thread --
// 96 KB in flight per CTA, two CTAs per SM, several times what registers can hold as landing
// space.  Thread = (slot, 16-row group, early or late half of the group).
constexpr int kGGTmaRows = 32;
constexpr int kGGTmaMaxSlices = 8;
constexpr int kGGTileB = kGGTmaRows * 64 * 4;      // bytes of one [32 x 64] fp32 tile (two swizzled panels)

__global__ void __launch_bounds__(256) gate_grad_local_tma_kernel(
    const __grid_constant__ CUtensorMap mapU, const __grid_constant__ CUtensorMap mapI,
    const __grid_constant__ CUtensorMap mapGate, const __grid_constant__ CUtensorMap mapG,
    const __grid_constant__ CUtensorMap mapDIk, const __grid_constant__ CUtensorMap mapDIv, int nsk, int nsv,
    int gate_kind, float inv_tau, float* __restrict__ blk_tot, float* __restrict__ dgate, int T, int H, int nblk,
    const int* __restrict__ strong, int nseg, int32_t* dev_status) {
    using namespace tc;
    constexpr int M = 64;
    extern __shared__ unsigned char gg_smem_raw[];
    unsigned char* smem = gg_smem_raw + ((1024u - (smem_u32(gg_smem_raw) & 1023u)) & 1023u);
    __shared__ uint64_t bar;
    __shared__ float late_half[kGGTmaRows / kGG][M];
    // slot, 16-row group, early (0) or late (1) 8 rows of the group
    const int tx = threadIdx.x & 63, ty = (threadIdx.x >> 6) & 1, hh = threadIdx.x >> 7;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = blockIdx.y * kGGTmaRows;
    const int nslices = nsk + nsv;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // tiles 0..3 = u, I, gate, G; I is not read when the gate tensor holds a itself (1 - a is one
        // subtraction), G only when a row factor is pending
        const bool need[4] = {true, gate_kind != GSA_GATE_A, true, strong != nullptr};
        int ntiles = nslices;
        for (int i = 0; i < 4; ++i) ntiles += need[i] ? 1 : 0;
        mbar_expect_tx(&bar, (uint32_t)(ntiles * kGGTileB));
        const CUtensorMap* maps[4] = {&mapU, &mapI, &mapGate, &mapG};
        for (int i = 0; i < 4; ++i) {
            if (!need[i]) continue;
            tma_load_4d(smem + i * kGGTileB, maps[i], &bar, 0, h, t0, b);
            tma_load_4d(smem + i * kGGTileB + kGGTileB / 2, maps[i], &bar, 32, h, t0, b);
        }
        for (int sl = 0; sl < nslices; ++sl) {
            const CUtensorMap* m = sl < nsk ? &mapDIk : &mapDIv;
            const int z = sl < nsk ? sl : sl - nsk;
            tma_load_5d(smem + (4 + sl) * kGGTileB, m, &bar, 0, h, t0, b, z);
            tma_load_5d(smem + (4 + sl) * kGGTileB + kGGTileB / 2, m, &bar, 32, h, t0, b, z);
        }
    }
    __syncthreads();
    const bool landed = mbar_wait(&bar, 0);
    if (!landed && threadIdx.x == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
    if (__syncthreads_or(!landed)) return;

    constexpr int kHalf = kGG / 2;
    const int n = blockIdx.y * (kGGTmaRows / kGG) + ty;           // 16-row block of the sequence
    const int rows = n < nblk ? min(kGG, T - n * kGG) : 0;
    // row r (of this thread's 16), this thread's slot, of tile `tile`
    auto at = [&](int tile, int r) {
        const int row = ty * kGG + hh * kHalf + r, c = tx;
        const unsigned char* p = smem + tile * kGGTileB + (c >> 5) * (kGGTileB / 2) + swz128(row, (c & 31) >> 2) + (c & 3) * 4;
        return *reinterpret_cast<const float*>(p);
    };
    float x[kHalf], dI[kHalf];
#pragma unroll
    for (int i = 0; i < kHalf; ++i) dI[i] = 0.f;
    for (int sl = 0; sl < nslices; ++sl) {
#pragma unroll
        for (int i = 0; i < kHalf; ++i) dI[i] += at(4 + sl, i);
    }
    if (strong != nullptr && strong[(b * nseg + t0 / (T / nseg)) * H + h] == 0) {
        // the time-reversed value_side runs left their row factor exp(-G_i) to this kernel
#pragma unroll
        for (int i = 0; i < kHalf; ++i) dI[i] *= __expf(-at(3, i));
    }
#pragma unroll
    for (int i = 0; i < kHalf; ++i) {
        const float ii = gate_kind == GSA_GATE_A ? 1.f - at(2, i) : at(1, i);      // 1 - a as the gate kernel formed it
        x[i] = at(0, i) - ii * dI[i];                                              // rows past the end: u = dI = 0
    }
    const size_t stride = (size_t)H * M;
    const size_t base = (((size_t)b * T + n * kGG + hh * kHalf) * H + h) * M + tx;
    // the early half starts from the total of the late half of its group
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < kHalf; ++i) tot += x[i];
    if (hh == 1) late_half[ty][tx] = tot;
    __syncthreads();
    float run = hh == 0 ? late_half[ty][tx] : 0.f;
#pragma unroll
    for (int i = kHalf - 1; i >= 0; --i) {
        run += x[i];
        if (hh * kHalf + i < rows)
            dgate[base + (size_t)i * stride] = gate_grad_out(run, dI[i], at(2, i), gate_kind, inv_tau);
    }
    if (hh == 0 && n < nblk) blk_tot[((size_t)bh * nblk + n) * M + tx] = run;
}

// The TMA-staged pass as a ring, for wide heads (n_k + n_v >= 6: a CTA per tile then keeps
// only two tiles per SM in flight and the copies pause while it computes, leaves and the next
// one starts).  A tile is 32 rows of one (b,h) with every input stream (u, I, gate, G and the n_k + n_v slices of the
// input-gate gradient: 12 x 8 KB at d = 512).  One persistent CTA per SM walks the tiles
// blockIdx.x, blockIdx.x + gridDim.x, ... through a ring of 2-4 stages: a ninth warp requests the
// tiles of the stages ahead while the eight compute warps work on the current one, so copies
// are in flight all the time.  Compute thread = (slot, 16-row group, early or late half of it).
constexpr int kGGMaxStages = 4;
constexpr int kGGRingMinSlices = 6;
constexpr int kGGComputeThreads = 256;

__global__ void __launch_bounds__(kGGComputeThreads + 32) gate_grad_local_ring_kernel(
    const __grid_constant__ CUtensorMap mapU, const __grid_constant__ CUtensorMap mapI,
    const __grid_constant__ CUtensorMap mapGate, const __grid_constant__ CUtensorMap mapG,
    const __grid_constant__ CUtensorMap mapDIk, const __grid_constant__ CUtensorMap mapDIv, int nsk, int nsv,
    int gate_kind, float inv_tau, float* __restrict__ blk_tot, float* __restrict__ dgate, int T, int H, int BH,
    int ntile, int nstage, int nblk, const int* __restrict__ strong, int nseg, int32_t* dev_status) {
    using namespace tc;
    constexpr int M = 64;
    extern __shared__ unsigned char gg_smem_raw[];
    unsigned char* smem0 = gg_smem_raw + ((1024u - (smem_u32(gg_smem_raw) & 1023u)) & 1023u);
    __shared__ uint64_t bar_full[kGGMaxStages], bar_empty[kGGMaxStages];
    __shared__ float late_half[kGGTmaRows / kGG][M];
    __shared__ volatile int failed_s, stop_s;
    const int nslices = nsk + nsv;
    const int stage_bytes = (4 + nslices) * kGGTileB;
    const int total = BH * ntile;
    if (threadIdx.x == 0) {
        failed_s = 0;
        for (int s = 0; s < nstage; ++s) {
            mbar_init(&bar_full[s], 1);
            mbar_init(&bar_empty[s], 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (threadIdx.x == kGGComputeThreads) {
        // =============================== copy lane
        // tiles 0..3 = u, I, gate, G; I is not read when the gate tensor holds a itself (1 - a is one
        // subtraction), G only when a row factor is pending
        const bool need[4] = {true, gate_kind != GSA_GATE_A, true, strong != nullptr};
        int ntiles = nslices;
        for (int i = 0; i < 4; ++i) ntiles += need[i] ? 1 : 0;
        const CUtensorMap* maps[4] = {&mapU, &mapI, &mapGate, &mapG};
        int it = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
            const int s = it % nstage;
            if (it >= nstage && !mbar_wait(&bar_empty[s], ((it / nstage) - 1) & 1)) {
                failed_s = 1;
                break;
            }
            const int bh = t % BH, b = bh / H, h = bh % H, t0 = (t / BH) * kGGTmaRows;
            unsigned char* smem = smem0 + (size_t)s * stage_bytes;
            mbar_expect_tx(&bar_full[s], (uint32_t)(ntiles * kGGTileB));
            for (int i = 0; i < 4; ++i) {
                if (!need[i]) continue;
                tma_load_4d(smem + i * kGGTileB, maps[i], &bar_full[s], 0, h, t0, b);
                tma_load_4d(smem + i * kGGTileB + kGGTileB / 2, maps[i], &bar_full[s], 32, h, t0, b);
            }
            for (int sl = 0; sl < nslices; ++sl) {
                const CUtensorMap* m = sl < nsk ? &mapDIk : &mapDIv;
                const int z = sl < nsk ? sl : sl - nsk;
                tma_load_5d(smem + (4 + sl) * kGGTileB, m, &bar_full[s], 0, h, t0, b, z);
                tma_load_5d(smem + (4 + sl) * kGGTileB + kGGTileB / 2, m, &bar_full[s], 32, h, t0, b, z);
            }
        }
    } else if (threadIdx.x < kGGComputeThreads) {
        // =============================== compute warps
        // slot, 16-row group, early (0) or late (1) 8 rows of the group
        const int tx = threadIdx.x & 63, ty = (threadIdx.x >> 6) & 1, hh = threadIdx.x >> 7;
        constexpr int kHalf = kGG / 2;
        const size_t stride = (size_t)H * M;
        auto csync = [] { asm volatile("bar.sync 1, 256;" ::: "memory"); };
        int it = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
            const int s = it % nstage;
            const int bh = t % BH, b = bh / H, h = bh % H, ty0 = t / BH, t0 = ty0 * kGGTmaRows;
            const unsigned char* smem = smem0 + (size_t)s * stage_bytes;
            const bool landed = mbar_wait(&bar_full[s], (it / nstage) & 1);
            if (!landed) failed_s = 1;
            const int n = ty0 * (kGGTmaRows / kGG) + ty;           // 16-row block of the sequence
            const int rows = n < nblk ? min(kGG, T - n * kGG) : 0;
            // row r (of this thread's 8), this thread's slot, of tile `tile`
            auto at = [&](int tile, int r) {
                const int row = ty * kGG + hh * kHalf + r, c = tx;
                const unsigned char* p = smem + tile * kGGTileB + (c >> 5) * (kGGTileB / 2) + swz128(row, (c & 31) >> 2) + (c & 3) * 4;
                return *reinterpret_cast<const float*>(p);
            };
            float x[kHalf], dI[kHalf], gt[kHalf];
#pragma unroll
            for (int i = 0; i < kHalf; ++i) { dI[i] = 0.f; x[i] = 0.f; gt[i] = 1.f; }
            if (landed) {
                for (int sl = 0; sl < nslices; ++sl) {
#pragma unroll
                    for (int i = 0; i < kHalf; ++i) dI[i] += at(4 + sl, i);
                }
                if (strong != nullptr && strong[(b * nseg + t0 / (T / nseg)) * H + h] == 0) {
                    // the time-reversed value_side runs left their row factor exp(-G_i) to this kernel
#pragma unroll
                    for (int i = 0; i < kHalf; ++i) dI[i] *= __expf(-at(3, i));
                }
#pragma unroll
                for (int i = 0; i < kHalf; ++i) {
                    gt[i] = at(2, i);
                    const float ii = gate_kind == GSA_GATE_A ? 1.f - gt[i] : at(1, i);      // 1 - a as the gate kernel formed it
                    x[i] = at(0, i) - ii * dI[i];                                          // rows past the end: u = dI = 0
                }
            }
            // the early half starts from the total of the late half of its group
            float tot = 0.f;
#pragma unroll
            for (int i = 0; i < kHalf; ++i) tot += x[i];
            if (hh == 1) late_half[ty][tx] = tot;
            csync();                              // (also: every thread has read its part of the stage)
            if (threadIdx.x == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_empty[s])) : "memory");
            float run = hh == 0 ? late_half[ty][tx] : 0.f;
            const size_t base = (((size_t)b * T + n * kGG + hh * kHalf) * H + h) * M + tx;
#pragma unroll
            for (int i = kHalf - 1; i >= 0; --i) {
                run += x[i];
                if (hh * kHalf + i < rows)
                    dgate[base + (size_t)i * stride] = gate_grad_out(run, dI[i], gt[i], gate_kind, inv_tau);
            }
            if (hh == 0 && n < nblk) blk_tot[((size_t)bh * nblk + n) * M + tx] = run;
            // (one thread reads the flag that the copy lane may raise at any time, so that all leave together)
            if (threadIdx.x == 0) stop_s = failed_s;
            csync();                              // late_half may be rewritten
            if (stop_s) break;
        }
    }
    __syncthreads();
    if (failed_s) {
        if (threadIdx.x == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        // bounded grace period for tile copies still in flight before shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
}

// Adds what follows the block: dgate += carry (log gate) or carry / a (linear gate).  A thread
// takes two slots of eight rows (half a block): threadIdx = (slot pair, block, half).
template <int M>
__global__ void __launch_bounds__(256) gate_grad_carry_kernel(
    const float* __restrict__ gate, int gate_kind, float inv_tau, const float* __restrict__ blk_carry,
    float* __restrict__ dgate, int T, int H, int nblk) {
    constexpr int kRows = kGG / 2;
    const int s = 2 * threadIdx.x;
    const int n = blockIdx.y * blockDim.y + threadIdx.y;
    if (n >= nblk) return;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;
    const int t0 = n * kGG + threadIdx.z * kRows;
    const int rows = max(0, min(kRows, T - t0));
    const size_t stride = (size_t)H * M;
    const size_t base = (((size_t)b * T + t0) * H + h) * M + s;
    const float2 carry = *reinterpret_cast<const float2*>(blk_carry + ((size_t)bh * nblk + n) * M + s);
    float2 d[kRows], gt[kRows];
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
        d[i] = (i < rows) ? *reinterpret_cast<const float2*>(dgate + base + (size_t)i * stride) : make_float2(0.f, 0.f);
        gt[i] = (i < rows && gate_kind != GSA_GATE_LOG_A) ? *reinterpret_cast<const float2*>(gate + base + (size_t)i * stride)
                                                          : make_float2(1.f, 1.f);
    }
#pragma unroll
    for (int i = 0; i < kRows; ++i)
        if (i < rows) {
            float2 out;
            out.x = d[i].x + gate_grad_carry(carry.x, gt[i].x, gate_kind, inv_tau);
            out.y = d[i].y + gate_grad_carry(carry.y, gt[i].y, gate_kind, inv_tau);
            *reinterpret_cast<float2*>(dgate + base + (size_t)i * stride) = out;
        }
}

int gate_grad_blocks(int T) { return (T + kGG - 1) / kGG; }

cudaError_t launch_gate_grad(const float* u, const float* I, const float* dIk_part, int nsk,
                             const float* dIv_part, int nsv, const float* gate,
                             int gate_kind, float inv_tau, const float* dKT, const float* KT,
                             const float* dVT, const float* VT, int d_k, int d_v,
                             float* blk_tot, float* dgate, int B, int T, int H, int M,
                             PendingDecay pend, cudaStream_t st, int32_t* dev_status) {
    const int nblk = gate_grad_blocks(T);
    dim3 block(M / 2, 256 / M);      // 128 threads: M/2 slot pairs x 16-row blocks
    dim3 grid(B * H, (nblk + block.y - 1) / block.y);
    if (M == 64) {
        const int nsl = nsk + nsv;
        bool staged = nsl <= kGGTmaMaxSlices;
        CUtensorMap mu, mi, mg, mG, mk, mv;
        if (staged) {
            const float* Gp = pend.G != nullptr ? pend.G : u;      // (unused without a pending factor)
            cudaError_t e = make_tensor_map_bthd(&mu, u, B, T, H, M, kGGTmaRows, 4);
            if (e == cudaSuccess) e = make_tensor_map_bthd(&mi, I, B, T, H, M, kGGTmaRows, 4);
            if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, gate, B, T, H, M, kGGTmaRows, 4);
            if (e == cudaSuccess) e = make_tensor_map_bthd(&mG, Gp, B, T, H, M, kGGTmaRows, 4);
            if (e == cudaSuccess) e = make_tensor_map_sliced(&mk, dIk_part, nsk, B, T, H, M, kGGTmaRows, 4);
            if (e == cudaSuccess) e = make_tensor_map_sliced(&mv, dIv_part, nsv, B, T, H, M, kGGTmaRows, 4);
            staged = e == cudaSuccess;
        }
        if (staged && nsl >= kGGRingMinSlices) {
            const int stage_bytes = (4 + nsl) * kGGTileB;
            const int nstage = 2;
            const size_t smem = 1024 + (size_t)nstage * stage_bytes;
            cudaError_t e = cudaFuncSetAttribute(gate_grad_local_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return e;
            static int sm_count = 0;
            if (sm_count == 0) {
                int dev = 0;
                if (cudaGetDevice(&dev) != cudaSuccess ||
                    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
                    return cudaErrorUnknown;
            }
            const int BH = B * H, ntile = (T + kGGTmaRows - 1) / kGGTmaRows;
            const long long total = (long long)BH * ntile;
            const int ctas = (int)(total < sm_count ? total : sm_count);      // one persistent CTA per SM
            gate_grad_local_ring_kernel<<<ctas, kGGComputeThreads + 32, smem, st>>>(
                mu, mi, mg, mG, mk, mv, nsk, nsv, gate_kind, inv_tau, blk_tot, dgate, T, H, BH, ntile, nstage, nblk,
                pend.G != nullptr ? pend.strong : nullptr, pend.nseg, dev_status);
        } else if (staged) {
            const size_t smem = 1024 + (size_t)(4 + nsl) * kGGTileB;
            cudaError_t e = cudaFuncSetAttribute(gate_grad_local_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return e;
            dim3 tgrid(B * H, (T + kGGTmaRows - 1) / kGGTmaRows);
            gate_grad_local_tma_kernel<<<tgrid, 256, smem, st>>>(mu, mi, mg, mG, mk, mv, nsk, nsv, gate_kind, inv_tau, blk_tot,
                                                                dgate, T, H, nblk, pend.G != nullptr ? pend.strong : nullptr,
                                                                pend.nseg, dev_status);
        } else {
            gate_grad_local_kernel<64><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv, gate, gate_kind, inv_tau,
                                                               blk_tot, dgate, B, T, H, nblk, pend);
        }
        gate_grad_scan_kernel<64><<<B * H, dim3(64, 16), 0, st>>>(blk_tot, dKT, KT, dVT, VT, d_k, d_v, nblk);
        gate_grad_carry_kernel<64><<<grid, dim3(block.x, block.y, 2), 0, st>>>(gate, gate_kind, inv_tau, blk_tot, dgate, T, H, nblk);
    } else if (M == 128) {
        gate_grad_local_kernel<128><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv, gate, gate_kind, inv_tau,
                                                            blk_tot, dgate, B, T, H, nblk, pend);
        gate_grad_scan_kernel<128><<<B * H, dim3(128, 8), 0, st>>>(blk_tot, dKT, KT, dVT, VT, d_k, d_v, nblk);
        gate_grad_carry_kernel<128><<<grid, dim3(block.x, block.y, 2), 0, st>>>(gate, gate_kind, inv_tau, blk_tot, dgate, T, H, nblk);
    } else {
        gate_grad_local_kernel<32><<<grid, block, 0, st>>>(u, I, dIk_part, nsk, dIv_part, nsv, gate, gate_kind, inv_tau,
                                                           blk_tot, dgate, B, T, H, nblk, pend);
        gate_grad_scan_kernel<32><<<B * H, dim3(32, 16), 0, st>>>(blk_tot, dKT, KT, dVT, VT, d_k, d_v, nblk);
        gate_grad_carry_kernel<32><<<grid, dim3(block.x, block.y, 2), 0, st>>>(gate, gate_kind, inv_tau, blk_tot, dgate, T, H, nblk);
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------ ABC: no decay, cumulative-softmax write weights
// Eq. 3-4 (the ungated ancestor of GSA, the "no decay" row of the ablations): the memories only
// accumulate, K~_t = K~_{t-1} + phi_t (x) k_t, with write weights phi_t = exp(s_t) / sum_{j<=t} exp(s_j)
// per slot.  In the layer's terms: log a = 0 everywhere and the input gate is phi.  The cumulative
// softmax over time is a scan per (batch, head, slot): one thread each, the rows of eight time steps
// requested together so that the loads overlap; running maximum and rescaled running sum as in any
// streaming softmax.  The decayed bf16 rows of the tensor-core kernels are phi itself (exp(-G) = 1).
constexpr int kAbcBatch = 8;

template <int M>
__global__ void __launch_bounds__(M) abc_write_kernel(const float* __restrict__ s_in, float* __restrict__ G,
                                                      float* __restrict__ I, __nv_bfloat16* __restrict__ decayed, int T,
                                                      int H) {
    const int bh = blockIdx.x, b = bh / H, h = bh % H, s = threadIdx.x;
    const size_t stride = (size_t)H * M;
    size_t idx = ((size_t)b * T * H + h) * M + s;
    float mx = -INFINITY, z = 0.f;
    for (int t0 = 0; t0 < T; t0 += kAbcBatch) {
        float x[kAbcBatch];
#pragma unroll
        for (int i = 0; i < kAbcBatch; ++i) x[i] = (t0 + i < T) ? s_in[idx + (size_t)i * stride] : 0.f;
#pragma unroll
        for (int i = 0; i < kAbcBatch; ++i) {
            if (t0 + i >= T) break;
            const float nm = fmaxf(mx, x[i]);
            const float e = __expf(x[i] - nm);
            z = z * __expf(mx - nm) + e;
            mx = nm;
            const float phi = e / z;
            const size_t at = idx + (size_t)i * stride;
            G[at] = 0.f;
            I[at] = phi;
            if (decayed != nullptr) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(phi);
                __nv_bfloat16* row = decayed + 2 * (at - s);
                row[s] = hi;
                row[M + s] = __float2bfloat16_rn(phi - __bfloat162float(hi));
            }
        }
        idx += (size_t)kAbcBatch * stride;
    }
}

// Gradient w.r.t. the scores: with dphi_t the gradient w.r.t. the write weights (the sum of the input-gate
// gradient partial sums of both passes),
//     ds_j = phi_j (dphi_j - R_j),   R_j = dphi_j phi_j + (1 - phi_{j+1}) R_{j+1}
// (Z_j / Z_t = prod_{r=j+1..t} (1 - phi_r): nothing but phi is needed).  A reverse scan, same thread layout.
template <int M>
__global__ void __launch_bounds__(M) abc_grad_kernel(const float* __restrict__ phi_in, const float* __restrict__ dIk, int nsk,
                                                     const float* __restrict__ dIv, int nsv, float* __restrict__ ds, int T,
                                                     int H, size_t total) {
    const int bh = blockIdx.x, b = bh / H, h = bh % H, s = threadIdx.x;
    const size_t stride = (size_t)H * M;
    const size_t base = ((size_t)b * T * H + h) * M + s;
    float R = 0.f, phi_next = 0.f;          // (1 - phi_{T}) R_{T} = 0
    for (int t1 = T; t1 > 0; t1 -= kAbcBatch) {
        float phi[kAbcBatch], dphi[kAbcBatch];
#pragma unroll
        for (int i = 0; i < kAbcBatch; ++i) {
            const int t = t1 - 1 - i;
            phi[i] = 0.f; dphi[i] = 0.f;
            if (t >= 0) {
                const size_t at = base + (size_t)t * stride;
                phi[i] = phi_in[at];
                for (int sl = 0; sl < nsk; ++sl) dphi[i] += dIk[at + (size_t)sl * total];
                for (int sl = 0; sl < nsv; ++sl) dphi[i] += dIv[at + (size_t)sl * total];
            }
        }
#pragma unroll
        for (int i = 0; i < kAbcBatch; ++i) {
            const int t = t1 - 1 - i;
            if (t < 0) break;
            R = dphi[i] * phi[i] + (1.f - phi_next) * R;
            ds[base + (size_t)t * stride] = phi[i] * (dphi[i] - R);
            phi_next = phi[i];
        }
    }
}

cudaError_t launch_abc_write(const float* s_in, float* G, float* I, void* decayed, int B, int T, int H, int M, cudaStream_t st) {
    if (M == 128) abc_write_kernel<128><<<B * H, 128, 0, st>>>(s_in, G, I, static_cast<__nv_bfloat16*>(decayed), T, H);
    else if (M == 64) abc_write_kernel<64><<<B * H, 64, 0, st>>>(s_in, G, I, static_cast<__nv_bfloat16*>(decayed), T, H);
    else abc_write_kernel<32><<<B * H, 32, 0, st>>>(s_in, G, I, static_cast<__nv_bfloat16*>(decayed), T, H);
    return cudaGetLastError();
}
cudaError_t launch_abc_grad(const float* phi, const float* dIk, int nsk, const float* dIv, int nsv, float* ds, int B, int T,
                            int H, int M, cudaStream_t st) {
    const size_t total = (size_t)B * T * H * M;
    if (M == 128) abc_grad_kernel<128><<<B * H, 128, 0, st>>>(phi, dIk, nsk, dIv, nsv, ds, T, H, total);
    else if (M == 64) abc_grad_kernel<64><<<B * H, 64, 0, st>>>(phi, dIk, nsk, dIv, nsv, ds, T, H, total);
    else abc_grad_kernel<32><<<B * H, 32, 0, st>>>(phi, dIk, nsk, dIv, nsv, ds, T, H, total);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ data-independent decay
// A gate that does not depend on the input (the "data-independent decay" row of the ablations) is one
// row [H, M] for all tokens: it is spread over [B,T,H,M] on the way in, and the gate gradient is
// summed over the tokens on the way out (partial sums per block of rows, added in order).
__global__ void broadcast_rows_kernel(const float* __restrict__ row, float* __restrict__ out, size_t rows, int n) {
    const size_t total = rows * (size_t)n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
        out[i] = row[i % n];
}
constexpr int kColSumRows = 256;
__global__ void column_partial_kernel(const float* __restrict__ in, float* __restrict__ part, size_t rows, int n) {
    const int c = blockIdx.y * blockDim.x + threadIdx.x;
    if (c >= n) return;
    const size_t r0 = (size_t)blockIdx.x * kColSumRows;
    const size_t r1 = r0 + kColSumRows < rows ? r0 + kColSumRows : rows;
    float acc = 0.f;
    for (size_t r = r0; r < r1; ++r) acc += in[r * n + c];
    part[(size_t)blockIdx.x * n + c] = acc;
}
__global__ void column_final_kernel(const float* __restrict__ part, float* __restrict__ out, int nparts, int n) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n) return;
    double acc = 0.0;
    for (int p = 0; p < nparts; ++p) acc += (double)part[(size_t)p * n + c];
    out[c] = (float)acc;
}
cudaError_t launch_broadcast_rows(const float* row, float* out, size_t rows, int n, cudaStream_t st) {
    const size_t total = rows * (size_t)n;
    const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
    broadcast_rows_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(row, out, rows, n);
    return cudaGetLastError();
}
size_t column_sum_parts(size_t rows) { return (rows + kColSumRows - 1) / kColSumRows; }
// out[c] = sum over rows of in[r][c]; part: column_sum_parts(rows) * n floats of scratch
cudaError_t launch_column_sum(const float* in, float* part, float* out, size_t rows, int n, cudaStream_t st) {
    const unsigned parts = (unsigned)column_sum_parts(rows);
    column_partial_kernel<<<dim3(parts, (n + 127) / 128), 128, 0, st>>>(in, part, rows, n);
    column_final_kernel<<<(n + 127) / 128, 128, 0, st>>>(part, out, (int)parts, n);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ gate tensor in bfloat16
__global__ void widen_bf16_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out, size_t n) {
    for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; i < n; i += (size_t)gridDim.x * blockDim.x * 2) {
        if (i + 1 < n) {
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(in + i));
            *reinterpret_cast<float2*>(out + i) = f;
        } else {
            out[i] = __bfloat162float(in[i]);
        }
    }
}
cudaError_t launch_widen_bf16(const void* in, float* out, size_t n, cudaStream_t st) {
    const size_t pairs = (n + 1) / 2;
    const unsigned blocks = (unsigned)((pairs + 255) / 256 < 148 * 32 ? (pairs + 255) / 256 : 148 * 32);
    widen_bf16_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(in), out, n);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ slot padding
// Rows of n_in floats copied into rows of n_out floats: widened rows get `fill` in their tail,
// narrowed rows lose theirs.  Used when a layer with 32 slots runs on the 64-slot tiles of the
// tensor-core kernels: gate rows are widened with a neutral gate, memories with empty slots.
__global__ void resize_rows_kernel(const float* __restrict__ in, float* __restrict__ out, size_t rows, int n_in, int n_out,
                                   float fill) {
    const size_t total = rows * (size_t)n_out;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / n_out;
        const int c = (int)(i - r * n_out);
        out[i] = c < n_in ? in[r * n_in + c] : fill;
    }
}
cudaError_t launch_resize_rows(const float* in, float* out, size_t rows, int n_in, int n_out, float fill, cudaStream_t st) {
    const size_t total = rows * (size_t)n_out;
    const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
    resize_rows_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(in, out, rows, n_in, n_out, fill);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ segment-parallel scheduling
// The memories are linear in (k, v): K~ after a segment = D * K~ before + (K~ of the segment run
// from empty memories), D = product of the gates over the segment.  A sequence cut into nseg
// segments can therefore run as nseg independent sequences once every segment's start
// memories are known.
//
// seg_logdecay[b][r][h][s] = sum over the chunks of segment r of G at the chunk's last row.
template <int M>
__global__ void segment_logdecay_kernel(const float* __restrict__ G, float* __restrict__ seg_logdecay, int T, int H,
                                        int nseg, int chunk) {
    const int s = threadIdx.x, h = blockIdx.y;
    const int b = blockIdx.x / nseg, r = blockIdx.x % nseg;
    const int Tseg = T / nseg;
    double acc = 0.0;
    for (int t = r * Tseg + chunk - 1; t < (r + 1) * Tseg; t += chunk)
        acc += (double)G[(((size_t)b * T + t) * H + h) * M + s];
    // (a ragged last chunk, possible only when the whole sequence is one segment)
    if (((r + 1) * Tseg) % chunk != 0) acc += (double)G[(((size_t)b * T + (r + 1) * Tseg - 1) * H + h) * M + s];
    seg_logdecay[(((size_t)b * nseg + r) * H + h) * M + s] = (float)acc;
}

// start[b][r] = D[r-1] start[b][r-1] + local_end[b][r-1], start[b][0] = S0[b] (or 0); the memory
// after the last segment goes to final (nullable).  Memories [.., H, M, D]; one thread per (s, c).
// reverse: the same from the last segment down (time-reversed scans: start[r] is the state that
// enters segment r from the right, S0 the one after the last token, final the one before the first).
template <int M>
__global__ void segment_combine_kernel(const float* __restrict__ seg_logdecay, const float* __restrict__ local_end,
                                       const float* __restrict__ S0, float* __restrict__ start,
                                       float* __restrict__ final_state, int H, int D, int nseg, int reverse) {
    const int b = blockIdx.x / H, h = blockIdx.x % H;
    const int idx = blockIdx.y * blockDim.x + threadIdx.x;
    if (idx < M * D) {
        const int s = idx / D;
        float cur = S0 ? S0[((size_t)(b * H + h)) * M * D + idx] : 0.f;
        for (int i = 0; i < nseg; ++i) {
            const int r = reverse ? nseg - 1 - i : i;
            const size_t pair = ((size_t)b * nseg + r) * H + h;
            start[pair * M * D + idx] = cur;
            cur = fmaf(cur, __expf(seg_logdecay[pair * M + s]), local_end[pair * M * D + idx]);
        }
        if (final_state) final_state[((size_t)(b * H + h)) * M * D + idx] = cur;
    }
}

// Sequence sharding across GPUs (same linearity): the gathered per-shard log-decays [R,B,H,M] and
// local end memories [R,B,H,M,D] of all R shards -> the memories entering shard `rank` (from the left;
// reverse: from the right, for the reversed scans of the backward) and, optionally, the memories after
// the last shard (reverse: before the first).  S0: what enters the first shard (reverse: the last).
__global__ void shard_combine_kernel(const float* __restrict__ logdecay_all, const float* __restrict__ local_all,
                                     const float* __restrict__ S0, float* __restrict__ start, float* __restrict__ final_state,
                                     int BH, int M, int D, int nshard, int rank, int reverse) {
    const int bh = blockIdx.x;
    const int idx = blockIdx.y * blockDim.x + threadIdx.x;
    if (idx >= M * D) return;
    const int s = idx / D;
    float cur = S0 ? S0[(size_t)bh * M * D + idx] : 0.f;
    for (int i = 0; i < nshard; ++i) {
        const int r = reverse ? nshard - 1 - i : i;
        if (r == rank && start != nullptr) start[(size_t)bh * M * D + idx] = cur;
        const size_t pair = (size_t)r * BH + bh;
        cur = fmaf(cur, __expf(logdecay_all[pair * M + s]), local_all[pair * M * D + idx]);
    }
    if (final_state != nullptr) final_state[(size_t)bh * M * D + idx] = cur;
}
cudaError_t launch_shard_combine(const float* logdecay_all, const float* local_all, const float* S0, float* start,
                                 float* final_state, int B, int H, int M, int D, int nshard, int rank, int reverse,
                                 cudaStream_t st) {
    dim3 grid(B * H, (M * D + 255) / 256);
    shard_combine_kernel<<<grid, 256, 0, st>>>(logdecay_all, local_all, S0, start, final_state, B * H, M, D, nshard, rank, reverse);
    return cudaGetLastError();
}

cudaError_t launch_segment_logdecay(const float* G, float* seg_logdecay, int B, int T, int H, int M, int nseg,
                                    int chunk, cudaStream_t st) {
    dim3 grid(B * nseg, H);
    if (M == 128) segment_logdecay_kernel<128><<<grid, 128, 0, st>>>(G, seg_logdecay, T, H, nseg, chunk);
    else if (M == 64) segment_logdecay_kernel<64><<<grid, 64, 0, st>>>(G, seg_logdecay, T, H, nseg, chunk);
    else segment_logdecay_kernel<32><<<grid, 32, 0, st>>>(G, seg_logdecay, T, H, nseg, chunk);
    return cudaGetLastError();
}

cudaError_t launch_segment_combine(const float* seg_logdecay, const float* local_end, const float* S0, float* start,
                                   float* final_state, int B, int H, int M, int D, int nseg, int reverse, cudaStream_t st) {
    dim3 grid(B * H, (M * D + 255) / 256);
    if (M == 64)
        segment_combine_kernel<64><<<grid, 256, 0, st>>>(seg_logdecay, local_end, S0, start, final_state, H, D, nseg, reverse);
    else
        segment_combine_kernel<32><<<grid, 256, 0, st>>>(seg_logdecay, local_end, S0, start, final_state, H, D, nseg, reverse);
    return cudaGetLastError();
}

}  // namespace gsa
