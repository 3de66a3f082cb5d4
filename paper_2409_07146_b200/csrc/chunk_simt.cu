// fp32 CUDA-core versions of the two chunk primitives of Algorithm 1 (see common.cuh).
//
// They are the kernels of the fp32 io type (whose tolerance bf16 or tf32 tensor-core
// operands cannot meet) and run either io type when asked for (GSA_IMPL_SIMT).  One CTA of
// 256 threads owns one (batch, head) and one 64-wide slice of the head dimension, walks the
// chunks in order with the slice of the state in shared memory, and does every contraction
// of a chunk as a 64 x N x 64 register-tiled product out of shared memory.
//
// Decay handling inside a chunk.  With G the chunk-local cumulative log gate, the decay
// between rows j <= i is exp(G_i - G_j).  When the chunk's total decay is moderate
// (min_s G_C[s] >= kFactorisedDecayMin) it is factorised as exp(G_i) * exp(-G_j) and folded
// into the operands of a plain product; otherwise the differences are formed explicitly
// (all exponents <= 0, nothing can overflow).
#include "common.cuh"

namespace gsa {
namespace {

constexpr int kC = kChunk;      // rows per chunk
constexpr int kDS = 64;         // head-dimension slice per CTA
constexpr int kLd = 68;         // shared-memory pitch of a 64-wide fp32 tile (16-byte aligned rows)

// ---- 64-row register-tiled products out of shared memory; thread (ty, tx) of a 16 x 16 grid.
// NN: acc[ii][jj] += sum_k A[(4 ty + ii)][k] * B[k][NJ tx + jj]
template <int NJ>
__device__ __forceinline__ void mm_nn(const float* A, int lda, const float* B, int ldb, int K,
                                      int ty, int tx, float (&acc)[4][NJ]) {
    for (int k = 0; k < K; k += 4) {
        float a[4][4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) {
            const float4 t = *reinterpret_cast<const float4*>(A + (4 * ty + ii) * lda + k);
            a[ii][0] = t.x; a[ii][1] = t.y; a[ii][2] = t.z; a[ii][3] = t.w;
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            float b[NJ];
            if constexpr (NJ == 8) {
                const float4 t = *reinterpret_cast<const float4*>(B + (k + kk) * ldb + 8 * tx);
                const float4 t2 = *reinterpret_cast<const float4*>(B + (k + kk) * ldb + 8 * tx + 4);
                b[0] = t.x; b[1] = t.y; b[2] = t.z; b[3] = t.w; b[4] = t2.x; b[5] = t2.y; b[6] = t2.z; b[7] = t2.w;
            } else if constexpr (NJ == 4) {
                const float4 t = *reinterpret_cast<const float4*>(B + (k + kk) * ldb + 4 * tx);
                b[0] = t.x; b[1] = t.y; b[2] = t.z; b[3] = t.w;
            } else {
                const float2 t = *reinterpret_cast<const float2*>(B + (k + kk) * ldb + 2 * tx);
                b[0] = t.x; b[1] = t.y;
            }
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < NJ; ++jj) acc[ii][jj] = fmaf(a[ii][kk], b[jj], acc[ii][jj]);
        }
    }
}
// TN: acc[ii][jj] += sum_k A[k][4 ty + ii] * B[k][NJ tx + jj]
template <int NJ>
__device__ __forceinline__ void mm_tn(const float* A, int lda, const float* B, int ldb, int K,
                                      int ty, int tx, float (&acc)[4][NJ]) {
#pragma unroll 4
    for (int k = 0; k < K; ++k) {
        const float4 t = *reinterpret_cast<const float4*>(A + k * lda + 4 * ty);
        const float a[4] = {t.x, t.y, t.z, t.w};
        float b[NJ];
        if constexpr (NJ == 8) {
            const float4 u = *reinterpret_cast<const float4*>(B + k * ldb + 8 * tx);
            const float4 u2 = *reinterpret_cast<const float4*>(B + k * ldb + 8 * tx + 4);
            b[0] = u.x; b[1] = u.y; b[2] = u.z; b[3] = u.w; b[4] = u2.x; b[5] = u2.y; b[6] = u2.z; b[7] = u2.w;
        } else if constexpr (NJ == 4) {
            const float4 u = *reinterpret_cast<const float4*>(B + k * ldb + 4 * tx);
            b[0] = u.x; b[1] = u.y; b[2] = u.z; b[3] = u.w;
        } else {
            const float2 u = *reinterpret_cast<const float2*>(B + k * ldb + 2 * tx);
            b[0] = u.x; b[1] = u.y;
        }
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < NJ; ++jj) acc[ii][jj] = fmaf(a[ii], b[jj], acc[ii][jj]);
    }
}
// NT: acc[ii][jj] += sum_k A[4 ty + ii][k] * B[tx + 16 jj][k]      (64 columns: jj < 4)
__device__ __forceinline__ void mm_nt(const float* A, int lda, const float* B, int ldb, int K,
                                      int ty, int tx, float (&acc)[4][4]) {
    for (int k = 0; k < K; k += 4) {
        float4 a[4], b[4];
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) a[ii] = *reinterpret_cast<const float4*>(A + (4 * ty + ii) * lda + k);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) b[jj] = *reinterpret_cast<const float4*>(B + (tx + 16 * jj) * ldb + k);
#pragma unroll
        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                acc[ii][jj] = fmaf(a[ii].x, b[jj].x, acc[ii][jj]);
                acc[ii][jj] = fmaf(a[ii].y, b[jj].y, acc[ii][jj]);
                acc[ii][jj] = fmaf(a[ii].z, b[jj].z, acc[ii][jj]);
                acc[ii][jj] = fmaf(a[ii].w, b[jj].w, acc[ii][jj]);
            }
    }
}

// ---- tile loads: 64 rows x 64 columns of io type -> fp32 shared (rows >= valid are zero)
template <typename IO>
__device__ __forceinline__ void load_io_tile(float* dst, const IO* src, size_t row_stride, int valid) {
    constexpr int V = IoTraits<IO>::kVec;
    constexpr int PER_ROW = kDS / V;
    for (int idx = threadIdx.x; idx < kC * PER_ROW; idx += 256) {
        const int r = idx / PER_ROW, c = (idx % PER_ROW) * V;
        float x[V];
        if (r < valid) {
            load_vec(src + (size_t)r * row_stride + c, x);
        } else {
#pragma unroll
            for (int e = 0; e < V; ++e) x[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < V; e += 4)
            *reinterpret_cast<float4*>(dst + r * kLd + c + e) = make_float4(x[e], x[e + 1], x[e + 2], x[e + 3]);
    }
}
// 64 rows x M fp32; rows >= valid get `fill` (0 for weights) or replicate the last valid row (G)
template <int M, bool REPLICATE_LAST>
__device__ __forceinline__ void load_slot_tile(float* dst, const float* src, size_t row_stride, int valid) {
    constexpr int PER_ROW = M / 4;
    for (int idx = threadIdx.x; idx < kC * PER_ROW; idx += 256) {
        const int r = idx / PER_ROW, c = (idx % PER_ROW) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < valid) x = *reinterpret_cast<const float4*>(src + (size_t)r * row_stride + c);
        else if (REPLICATE_LAST) x = *reinterpret_cast<const float4*>(src + (size_t)(valid - 1) * row_stride + c);
        *reinterpret_cast<float4*>(dst + r * (M + 4) + c) = x;
    }
}

// Decide, for the whole CTA, whether this chunk may use the factorised decay.
template <int M>
__device__ __forceinline__ bool chunk_is_moderate(const float* sG, int* flag) {
    if (threadIdx.x == 0) *flag = 1;
    __syncthreads();
    if (threadIdx.x < M && sG[(kC - 1) * (M + 4) + threadIdx.x] < kFactorisedDecayMin) *flag = 0;
    __syncthreads();
    return *flag != 0;
}

// =============================================================== value_side (pass-1 form)
template <typename IO, int M, bool REV>
__global__ void __launch_bounds__(256) value_side_simt_kernel(ValueSideArgs a) {
    constexpr int NJ = M / 16;
    constexpr int LM = M + 4;
    extern __shared__ __align__(16) float smem[];
    float* sXq = smem;                 // [64][68]
    float* sXk = sXq + kC * kLd;       // [64][68]
    float* sP = sXk + kC * kLd;        // [64][68]
    float* sS = sP + kC * kLd;         // [64 (channel)][LM]
    float* sW = sS + kDS * LM;         // [64][LM]
    float* sG = sW + kC * LM;          // [64][LM]
    __shared__ int s_flag;

    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int slice = blockIdx.y, bh = blockIdx.x, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDS;
    const size_t strideD = (size_t)a.H * a.D, strideM = (size_t)a.H * M;
    const IO* xq = (const IO*)a.xq + ((size_t)b * a.T * a.H + h) * a.D + d0;
    const IO* xk = (const IO*)a.xk + ((size_t)b * a.T * a.H + h) * a.D + d0;
    const float* w = a.w + ((size_t)b * a.T * a.H + h) * M;
    const float* G = a.G + ((size_t)b * a.T * a.H + h) * M;
    float* out = a.out + (size_t)slice * a.B * a.T * a.H * M + ((size_t)b * a.T * a.H + h) * M;

    // state slice S[c][s] <- S0[bh][s][d0 + c]
    for (int idx = tid; idx < kDS * M; idx += 256) {
        const int s = idx / kDS, c = idx % kDS;
        sS[c * LM + s] = a.S0 ? a.S0[((size_t)bh * M + s) * a.D + d0 + c] : 0.f;
    }
    const int nchunks = (a.T + kC - 1) / kC;
    for (int it = 0; it < nchunks; ++it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int t0 = n * kC;
        const int valid = min(kC, a.T - t0);
        __syncthreads();
        load_io_tile<IO>(sXq, xq + (size_t)t0 * strideD, strideD, valid);
        load_io_tile<IO>(sXk, xk + (size_t)t0 * strideD, strideD, valid);
        load_slot_tile<M, false>(sW, w + (size_t)t0 * strideM, strideM, valid);
        load_slot_tile<M, true>(sG, G + (size_t)t0 * strideM, strideM, valid);
        __syncthreads();
        const bool moderate = chunk_is_moderate<M>(sG, &s_flag);
        if (moderate) {
            // W' = W * exp(-G) (forward) or W * exp(G) (reverse)
            for (int idx = tid; idx < kC * M; idx += 256) {
                const int r = idx / M, s = idx % M;
                const float g = sG[r * LM + s];
                sW[r * LM + s] *= __expf(REV ? g : -g);
            }
        }
        // P = Xq Xk^T, masked to the causal (forward) or anti-causal (reverse) triangle
        {
            float acc[4][4] = {};
            mm_nt(sXq, kLd, sXk, kLd, kDS, ty, tx, acc);
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int i = 4 * ty + ii, j = tx + 16 * jj;
                    const bool keep = REV ? (j >= i) : (j <= i);
                    sP[i * kLd + j] = keep ? acc[ii][jj] : 0.f;
                }
        }
        __syncthreads();
        // out = rowscale * ( colscale * (Xq S) + P W' )
        {
            float acc[4][NJ] = {};
            mm_nn<NJ>(sXq, kLd, sS, LM, kDS, ty, tx, acc);
            if (moderate) {
                if (REV) {
#pragma unroll
                    for (int jj = 0; jj < NJ; ++jj) {
                        const float e = __expf(sG[(kC - 1) * LM + NJ * tx + jj]);
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii) acc[ii][jj] *= e;
                    }
                }
                mm_nn<NJ>(sP, kLd, sW, LM, kC, ty, tx, acc);
#pragma unroll
                for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                    for (int jj = 0; jj < NJ; ++jj) {
                        const float g = sG[(4 * ty + ii) * LM + NJ * tx + jj];
                        acc[ii][jj] *= __expf(REV ? -g : g);
                    }
            } else {
                float gi[4][NJ];
#pragma unroll
                for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                    for (int jj = 0; jj < NJ; ++jj) {
                        gi[ii][jj] = sG[(4 * ty + ii) * LM + NJ * tx + jj];
                        const float gc = sG[(kC - 1) * LM + NJ * tx + jj];
                        acc[ii][jj] *= __expf(REV ? gc - gi[ii][jj] : gi[ii][jj]);
                    }
                for (int j = 0; j < kC; ++j) {
#pragma unroll
                    for (int jj = 0; jj < NJ; ++jj) {
                        const float gj = sG[j * LM + NJ * tx + jj];
                        const float wj = sW[j * LM + NJ * tx + jj];
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii) {
                            const float pij = sP[(4 * ty + ii) * kLd + j];
                            const float ex = REV ? gj - gi[ii][jj] : gi[ii][jj] - gj;
                            acc[ii][jj] = fmaf(pij * wj, __expf(fminf(ex, 0.f)), acc[ii][jj]);
                        }
                    }
                }
            }
#pragma unroll
            for (int ii = 0; ii < 4; ++ii) {
                const int i = 4 * ty + ii;
                if (i < valid) {
#pragma unroll
                    for (int jj = 0; jj < NJ; ++jj) out[(size_t)(t0 + i) * strideM + NJ * tx + jj] = acc[ii][jj];
                }
            }
        }
        __syncthreads();
        // W~ for the state update: forward W exp(G_C - G), reverse W exp(G)
        for (int idx = tid; idx < kC * M; idx += 256) {
            const int r = idx / M, s = idx % M;
            const float gc = sG[(kC - 1) * LM + s];
            float f;
            if (moderate) f = REV ? 1.f : __expf(gc);
            else f = __expf(REV ? sG[r * LM + s] : gc - sG[r * LM + s]);
            sW[r * LM + s] *= f;
        }
        __syncthreads();
        // S <- S * exp(G_C) + Xk^T W~
        {
            float acc[4][NJ] = {};
            mm_tn<NJ>(sXk, kLd, sW, LM, kC, ty, tx, acc);
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < NJ; ++jj) {
                    const int c = 4 * ty + ii, s = NJ * tx + jj;
                    sS[c * LM + s] = fmaf(sS[c * LM + s], __expf(sG[(kC - 1) * LM + s]), acc[ii][jj]);
                }
        }
    }
    __syncthreads();
    if (a.Send) {
        for (int idx = tid; idx < kDS * M; idx += 256) {
            const int s = idx / kDS, c = idx % kDS;
            a.Send[((size_t)bh * M + s) * a.D + d0 + c] = sS[c * LM + s];
        }
    }
}

// =============================================================== key_side (pass-2 form)
template <typename IO, int M, bool REV>
__global__ void __launch_bounds__(256) key_side_simt_kernel(KeySideArgs a) {
    constexpr int LM = M + 4;
    extern __shared__ __align__(16) float smem[];
    float* sQ = smem;                  // [64][LM]  uq (scaled in place)
    float* sK = sQ + kC * LM;          // [64][LM]  uk (scaled in place)
    float* sG = sK + kC * LM;          // [64][LM]
    float* sV = sG + kC * LM;          // [64][68]
    float* sA = sV + kC * kLd;         // [64][68]
    float* sS = sA + kC * kLd;         // [M][68]
    __shared__ int s_flag;

    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int slice = blockIdx.y, bh = blockIdx.x, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDS;
    const size_t strideD = (size_t)a.H * a.D, strideM = (size_t)a.H * M;
    const float* uq = a.uq + ((size_t)b * a.T * a.H + h) * M;
    const float* uk = a.uk + ((size_t)b * a.T * a.H + h) * M;
    const float* G = a.G + ((size_t)b * a.T * a.H + h) * M;
    const IO* xv = (const IO*)a.xv + ((size_t)b * a.T * a.H + h) * a.D + d0;
    IO* out = (IO*)a.out + ((size_t)b * a.T * a.H + h) * a.D + d0;

    for (int idx = tid; idx < M * kDS; idx += 256) {
        const int s = idx / kDS, c = idx % kDS;
        sS[s * kLd + c] = a.S0 ? a.S0[((size_t)bh * M + s) * a.D + d0 + c] : 0.f;
    }
    const int nchunks = (a.T + kC - 1) / kC;
    for (int it = 0; it < nchunks; ++it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int t0 = n * kC;
        const int valid = min(kC, a.T - t0);
        __syncthreads();
        load_slot_tile<M, false>(sQ, uq + (size_t)t0 * strideM, strideM, valid);
        load_slot_tile<M, false>(sK, uk + (size_t)t0 * strideM, strideM, valid);
        load_slot_tile<M, true>(sG, G + (size_t)t0 * strideM, strideM, valid);
        load_io_tile<IO>(sV, xv + (size_t)t0 * strideD, strideD, valid);
        __syncthreads();
        const bool moderate = chunk_is_moderate<M>(sG, &s_flag);
        // A_ij = sum_s uq_i[s] uk_j[s] exp(+-(G_i[s] - G_j[s])) on the kept triangle
        if (moderate) {
            for (int idx = tid; idx < kC * M; idx += 256) {
                const int r = idx / M, s = idx % M;
                const float e = __expf(sG[r * LM + s]);
                const float einv = __expf(-sG[r * LM + s]);
                sQ[r * LM + s] *= REV ? einv : e;
                sK[r * LM + s] *= REV ? e : einv;
            }
            __syncthreads();
            float acc[4][4] = {};
            mm_nt(sQ, LM, sK, LM, M, ty, tx, acc);
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int i = 4 * ty + ii, j = tx + 16 * jj;
                    const bool keep = REV ? (j >= i) : (j <= i);
                    sA[i * kLd + j] = keep ? acc[ii][jj] : 0.f;
                }
        } else {
            float acc[4][4] = {};
            for (int s = 0; s < M; ++s) {
                float qi[4], gi[4], kj[4], gj[4];
#pragma unroll
                for (int ii = 0; ii < 4; ++ii) { qi[ii] = sQ[(4 * ty + ii) * LM + s]; gi[ii] = sG[(4 * ty + ii) * LM + s]; }
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) { kj[jj] = sK[(tx + 16 * jj) * LM + s]; gj[jj] = sG[(tx + 16 * jj) * LM + s]; }
#pragma unroll
                for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const float ex = REV ? gj[jj] - gi[ii] : gi[ii] - gj[jj];
                        acc[ii][jj] = fmaf(qi[ii] * kj[jj], __expf(fminf(ex, 0.f)), acc[ii][jj]);
                    }
            }
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int i = 4 * ty + ii, j = tx + 16 * jj;
                    const bool keep = REV ? (j >= i) : (j <= i);
                    sA[i * kLd + j] = keep ? acc[ii][jj] : 0.f;
                }
        }
        __syncthreads();
        // bring uq, uk to the scalings of the state terms:
        //   forward: Q- = uq exp(G),        K- = uk exp(G_C - G)
        //   reverse: Q- = uq exp(G_C - G),  K- = uk exp(G)
        for (int idx = tid; idx < kC * M; idx += 256) {
            const int r = idx / M, s = idx % M;
            const float g = sG[r * LM + s], gc = sG[(kC - 1) * LM + s];
            float fq, fk;
            if (moderate) {
                fq = REV ? __expf(gc) : 1.f;
                fk = REV ? 1.f : __expf(gc);
            } else {
                fq = __expf(REV ? gc - g : g);
                fk = __expf(REV ? g : gc - g);
            }
            sQ[r * LM + s] *= fq;
            sK[r * LM + s] *= fk;
        }
        __syncthreads();
        // out = Q- S + A Xv
        {
            float acc[4][4] = {};
            mm_nn<4>(sQ, LM, sS, kLd, M, ty, tx, acc);
            mm_nn<4>(sA, kLd, sV, kLd, kC, ty, tx, acc);
#pragma unroll
            for (int ii = 0; ii < 4; ++ii) {
                const int i = 4 * ty + ii;
                if (i < valid) store_vec4(out + (size_t)(t0 + i) * strideD + 4 * tx, acc[ii]);
            }
        }
        __syncthreads();
        // S <- exp(G_C)[:,None] S + K-^T Xv   (thread (ty,tx): slots 4ty.., channels 4tx..)
        // (64 slots per sweep of the 16 x 16 thread grid)
        for (int s0 = 0; s0 < M; s0 += 64) {
            if (s0 + 4 * ty >= M) break;
            float acc[4][4] = {};
            mm_tn<4>(sK + s0, LM, sV, kLd, kC, ty, tx, acc);
#pragma unroll
            for (int ii = 0; ii < 4; ++ii) {
                const int s = s0 + 4 * ty + ii;
                const float e = __expf(sG[(kC - 1) * LM + s]);
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    sS[s * kLd + 4 * tx + jj] = fmaf(sS[s * kLd + 4 * tx + jj], e, acc[ii][jj]);
            }
        }
    }
    __syncthreads();
    if (a.Send) {
        for (int idx = tid; idx < M * kDS; idx += 256) {
            const int s = idx / kDS, c = idx % kDS;
            a.Send[((size_t)bh * M + s) * a.D + d0 + c] = sS[s * kLd + c];
        }
    }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename IO, int M, bool REV>
cudaError_t launch_vs(const ValueSideArgs& a, cudaStream_t st) {
    const size_t smem = sizeof(float) * (3 * kC * kLd + (kDS + 2 * kC) * (M + 4));
    cudaError_t e = set_smem(value_side_simt_kernel<IO, M, REV>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDS);
    value_side_simt_kernel<IO, M, REV><<<grid, 256, smem, st>>>(a);
    return cudaGetLastError();
}
template <typename IO, int M, bool REV>
cudaError_t launch_ks(const KeySideArgs& a, cudaStream_t st) {
    const size_t smem = sizeof(float) * (3 * kC * (M + 4) + 2 * kC * kLd + M * kLd);
    cudaError_t e = set_smem(key_side_simt_kernel<IO, M, REV>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDS);
    key_side_simt_kernel<IO, M, REV><<<grid, 256, smem, st>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_value_side_simt(const ValueSideArgs& a, int io, int M, int reverse, cudaStream_t st) {
#define GSA_VS(IO, MM)                                                                   \
    return reverse ? launch_vs<IO, MM, true>(a, st) : launch_vs<IO, MM, false>(a, st)
    if (io == GSA_BF16) {
        if (M == 128) { GSA_VS(__nv_bfloat16, 128); } else if (M == 64) { GSA_VS(__nv_bfloat16, 64); } else { GSA_VS(__nv_bfloat16, 32); }
    } else {
        if (M == 128) { GSA_VS(float, 128); } else if (M == 64) { GSA_VS(float, 64); } else { GSA_VS(float, 32); }
    }
#undef GSA_VS
}

cudaError_t launch_key_side_simt(const KeySideArgs& a, int io, int M, int reverse, cudaStream_t st) {
#define GSA_KS(IO, MM)                                                                   \
    return reverse ? launch_ks<IO, MM, true>(a, st) : launch_ks<IO, MM, false>(a, st)
    if (io == GSA_BF16) {
        if (M == 128) { GSA_KS(__nv_bfloat16, 128); } else if (M == 64) { GSA_KS(__nv_bfloat16, 64); } else { GSA_KS(__nv_bfloat16, 32); }
    } else {
        if (M == 128) { GSA_KS(float, 128); } else if (M == 64) { GSA_KS(float, 64); } else { GSA_KS(float, 32); }
    }
#undef GSA_KS
}

}  // namespace gsa
