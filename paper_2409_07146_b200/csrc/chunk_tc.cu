// tcgen05 (bf16 tensor-core) versions of the two chunk primitives of Algorithm 1.
//
// One CTA of 128 threads owns one (batch, head) and one 128-wide slice of the head
// dimension and walks the chunks (128 tokens each) in order.  Thread i is row i of the
// chunk and channel i of the state slice, which is also TMEM lane i of every accumulator.
// Per chunk:
//   * the d-sized tiles (xq, xk / xv) arrive by TMA (128-byte swizzle), double buffered:
//     the tiles of chunk n+1 are requested before chunk n is computed;
//   * the slot-sized rows (weights, cumulative log gate G) are read by their thread,
//     scaled by the decay factors and written as bf16 operand panels;
//   * all contractions run as tcgen05.mma (M = 128) with fp32 accumulators in tensor
//     memory; thread 0 issues them and commits to an mbarrier that everybody waits on;
//   * the fp32 master copy of the state slice stays in registers (64 per thread); its bf16
//     copy for the next chunk's state product is rewritten every chunk.
// Decay inside a chunk is factorised as exp(G_i) * exp(-G_j) while the chunk's total
// log-decay stays above kFactorisedDecayMin; a chunk that forgets harder computes its
// intra-chunk term with explicit exponent differences on the CUDA cores instead.
// Every wait is bounded: on expiry the CTA flags dev_status, frees its tensor memory and
// returns.
#include "common.cuh"
#include "tc_common.cuh"

namespace gsa {
namespace {
using namespace tc;

constexpr int kCT = 128;               // chunk length of the tensor-core kernels
constexpr int kDST = 128;              // head-dimension slice per CTA
constexpr int kM = 64;                 // slots
constexpr int kPanelB = 128 * 128;     // bytes of a 128-row operand panel
constexpr uint32_t kTmemCols = 512;

// accumulator columns
constexpr int kColP = 0;       // P / A           [128 x 128]
constexpr int kColO = 128;     // inter (+ intra for key_side) output
constexpr int kColU = 256;     // state update    [128 x 64]
constexpr int kColO2 = 320;    // value_side intra output [128 x 64]

struct Ctl {
    uint64_t bar_load[2];
    uint64_t bar_mma1;
    uint64_t bar_mma2;
    uint32_t tmem_slot;
    volatile int abort;
    int moderate;
    float gc[kM];        // G of the chunk's last row
    float egc[kM];       // exp(gc)
};

__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
    const float4 t0 = __ldg(reinterpret_cast<const float4*>(p));
    const float4 t1 = __ldg(reinterpret_cast<const float4*>(p) + 1);
    x[0] = t0.x; x[1] = t0.y; x[2] = t0.z; x[3] = t0.w;
    x[4] = t1.x; x[5] = t1.y; x[6] = t1.z; x[7] = t1.w;
}

// bf16 copy of this thread's state row (64 values) as row `row` of a one-panel operand
__device__ __forceinline__ void store_state_row(unsigned char* panel, int row, const float (&S)[kM]) {
#pragma unroll
    for (int c = 0; c < kM / 8; ++c) {
        const float x[8] = {S[8 * c], S[8 * c + 1], S[8 * c + 2], S[8 * c + 3],
                            S[8 * c + 4], S[8 * c + 5], S[8 * c + 6], S[8 * c + 7]};
        store_chunk(panel, row, c, x);
    }
}

// The last thread publishes the G row of the chunk's last valid token, its exponential and
// the "moderate decay" decision.  Ends with a __syncthreads.
__device__ __forceinline__ void publish_chunk_decay(Ctl* ctl, int tid, const float* g_last_row) {
    if (tid >= kCT - kM / 4) {           // 16 threads, one float4 each
        const int c = tid - (kCT - kM / 4);
        const float4 t = __ldg(reinterpret_cast<const float4*>(g_last_row) + c);
        ctl->gc[4 * c] = t.x; ctl->gc[4 * c + 1] = t.y; ctl->gc[4 * c + 2] = t.z; ctl->gc[4 * c + 3] = t.w;
        ctl->egc[4 * c] = __expf(t.x); ctl->egc[4 * c + 1] = __expf(t.y);
        ctl->egc[4 * c + 2] = __expf(t.z); ctl->egc[4 * c + 3] = __expf(t.w);
    }
    __syncthreads();
    if (tid == 0) {
        float gmin = 0.f;
#pragma unroll
        for (int s = 0; s < kM; ++s) gmin = fminf(gmin, ctl->gc[s]);
        ctl->moderate = gmin >= kFactorisedDecayMin;
    }
    __syncthreads();
}

__device__ __forceinline__ void ctl_init(Ctl* ctl, int tid, int warp) {
    if (tid == 0) {
        mbar_init(&ctl->bar_load[0], 1);
        mbar_init(&ctl->bar_load[1], 1);
        mbar_init(&ctl->bar_mma1, 1);
        mbar_init(&ctl->bar_mma2, 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&ctl->tmem_slot, kTmemCols);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}

// ======================================================================================
// value_side: out_i[s] = rs_inter * (xq_i S)[s] + sum_j P_ij w_j[s] decay_ij[s]
// ======================================================================================
template <bool REV>
__global__ void __launch_bounds__(128, 1)
value_side_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                     ValueSideArgs a, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sXq = smem;                       // [2 stages][2 panels]
    unsigned char* sXk = sXq + 4 * kPanelB;          // [2 stages][2 panels]
    unsigned char* sPm = sXk + 4 * kPanelB;          // masked P, K-major A, 2 panels      (32 KB)
    unsigned char* sWp = sPm + 2 * kPanelB;          // W'^T  K-major B [64][128]: 2 panels of 64 rows (16 KB)
    unsigned char* sWt = sWp + kPanelB;              // W~^T  same shape                   (16 KB)
    unsigned char* sSb = sWt + kPanelB;              // state copy, MN-major B [128][64]   (16 KB)
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + kPanelB);
    float* sStageW = reinterpret_cast<float*>(sPm);               // fp32 [128][64] (strong-decay path)
    float* sStageG = reinterpret_cast<float*>(sPm + 2 * kPanelB); // fp32 [128][64] over sWp + sWt

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;
    const size_t strideM = (size_t)a.H * kM;
    const float* wbase = a.w + ((size_t)b * a.T * a.H + h) * kM;
    const float* gbase = a.G + ((size_t)b * a.T * a.H + h) * kM;
    float* obase = a.out + (size_t)slice * a.B * a.T * a.H * kM + ((size_t)b * a.T * a.H + h) * kM;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;

    const int nchunks = (a.T + kCT - 1) / kCT;
    auto issue_loads = [&](int it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int st = it & 1;
        mbar_expect_tx(&ctl->bar_load[st], 4 * kPanelB);
        tma_load_4d(sXq + (2 * st) * kPanelB, &mapQ, &ctl->bar_load[st], d0, h, n * kCT, b);
        tma_load_4d(sXq + (2 * st + 1) * kPanelB, &mapQ, &ctl->bar_load[st], d0 + 64, h, n * kCT, b);
        tma_load_4d(sXk + (2 * st) * kPanelB, &mapK, &ctl->bar_load[st], d0, h, n * kCT, b);
        tma_load_4d(sXk + (2 * st + 1) * kPanelB, &mapK, &ctl->bar_load[st], d0 + 64, h, n * kCT, b);
    };
    if (tid == 0) {
        prefetch_tmap(&mapQ);
        prefetch_tmap(&mapK);
        issue_loads(0);
    }

    // state slice: S[c = tid][s]
    float S[kM];
#pragma unroll
    for (int s = 0; s < kM; ++s) S[s] = a.S0 ? a.S0[((size_t)bh * kM + s) * a.D + d0 + tid] : 0.f;

    constexpr uint32_t idescP = make_idesc(128, 128, false, false);
    constexpr uint32_t idescO = make_idesc(128, kM, false, true);    // B = state copy, MN-major
    constexpr uint32_t idescU = make_idesc(128, kM, true, false);    // A = xk^T, MN-major
    constexpr uint32_t idescI = make_idesc(128, kM, false, false);   // intra: Pm x W'^T

    int it = 0;
    int n_mma2 = 0;    // completed phases of bar_mma2 (only moderate chunks use it)
    for (; it < nchunks; ++it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int st = it & 1;
        const int t0 = n * kCT;
        const int valid = min(kCT, a.T - t0);
        if (tid == 0 && it + 1 < nchunks) issue_loads(it + 1);

        publish_chunk_decay(ctl, tid, gbase + (size_t)(t0 + valid - 1) * strideM);
        const bool moderate = ctl->moderate != 0;
        // ---- slot-sized rows of this thread's token -> operand panels
        const float* grow = gbase + (size_t)(t0 + min(tid, valid - 1)) * strideM;
        const float* wrow = wbase + (size_t)(t0 + min(tid, valid - 1)) * strideM;
        {
            unsigned char* pWp = sWp + (tid >> 6) * (kM * 128);
            unsigned char* pWt = sWt + (tid >> 6) * (kM * 128);
            const int col = tid & 63;
            const float live = tid < valid ? 1.f : 0.f;
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 8) {
                float g[8], w[8];
                load8(grow + s0, g);
                load8(wrow + s0, w);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int s = s0 + e;
                    // state-update weights: forward w exp(G_C - G), reverse w exp(G)  (exponent <= 0)
                    const float wt = live * w[e] * __expf(REV ? g[e] : ctl->gc[s] - g[e]);
                    store_elem(pWt, s, col, wt);
                    if (moderate) {
                        // intra weights: forward w exp(-G), reverse w exp(G)
                        const float wp = REV ? wt : live * w[e] * __expf(-g[e]);
                        store_elem(pWp, s, col, wp);
                    }
                }
            }
        }
        store_state_row(sSb, tid, S);
        fence_async_smem();
        if (!mbar_wait(&ctl->bar_load[st], (it >> 1) & 1)) ctl->abort = 1;
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;

        // ---- P = xq xk^T, inter = xq S, U = xk^T W~
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t aQ = smem_u32(sXq + 2 * st * kPanelB), aK = smem_u32(sXk + 2 * st * kPanelB);
            const uint32_t aS = smem_u32(sSb), aWt = smem_u32(sWt);
#pragma unroll
            for (int kk = 0; kk < kDST / 16; ++kk)
                mma_bf16(tmem + kColP, desc_kmajor(aQ + (kk >> 2) * kPanelB, kk),
                         desc_kmajor(aK + (kk >> 2) * kPanelB, kk), idescP, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kDST / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aQ + (kk >> 2) * kPanelB, kk),
                         desc_mnmajor(aS, kk, kPanelB), idescO, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColU, desc_mnmajor(aK, kk, kPanelB),
                         desc_kmajor(aWt + (kk >> 2) * (kM * 128), kk), idescU, kk > 0);
            mma_commit(&ctl->bar_mma1);
        }
        if (!mbar_wait(&ctl->bar_mma1, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();

        if (moderate) {
            // masked P -> bf16 operand rows
#pragma unroll
            for (int c0 = 0; c0 < kCT; c0 += 16) {
                float v[16];
                tmem_ld16(tmem_row_addr(tmem, warp, kColP + c0), v);
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int j = c0 + e;
                    const bool keep = REV ? (j >= tid) : (j <= tid);
                    v[e] = keep ? v[e] : 0.f;
                }
                const float x0[8] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]};
                const float x1[8] = {v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]};
                unsigned char* panel = sPm + (c0 >> 6) * kPanelB;
                store_chunk(panel, tid, (c0 & 63) >> 3, x0);
                store_chunk(panel, tid, ((c0 & 63) >> 3) + 1, x1);
            }
            fence_async_smem();
        }
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
        if (moderate) {
            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t aP = smem_u32(sPm), aWp = smem_u32(sWp);
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kColO2, desc_kmajor(aP + (kk >> 2) * kPanelB, kk),
                             desc_kmajor(aWp + (kk >> 2) * (kM * 128), kk), idescI, kk > 0);
                mma_commit(&ctl->bar_mma2);
            }
        } else {
            // Strong decay: explicit exponent differences on the CUDA cores.  The W and G rows
            // are staged in fp32 over operand buffers that the finished products no longer need.
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 8) {
                float g[8], w[8];
                load8(grow + s0, g);
                load8(wrow + s0, w);
                const float live = tid < valid ? 1.f : 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    sStageW[tid * kM + s0 + e] = live * w[e];
                    sStageG[tid * kM + s0 + e] = g[e];
                }
            }
            __syncthreads();
            const int jlo = REV ? tid : 0, jhi = REV ? kCT - 1 : tid;
            // the accumulator loads are warp-collective: loop bounds are those of the whole warp
            const int wlo = REV ? warp * 32 : 0, whi = REV ? kCT - 1 : warp * 32 + 31;
            for (int s0 = 0; s0 < kM; s0 += 16) {
                float gi[16], acc[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) { gi[e] = sStageG[tid * kM + s0 + e]; acc[e] = 0.f; }
                for (int c0 = wlo; c0 <= whi; c0 += 16) {
                    float v[16];
                    tmem_ld16(tmem_row_addr(tmem, warp, kColP + c0), v);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int j = c0 + e;
                        if (j < jlo || j > jhi) continue;
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            const float gj = sStageG[j * kM + s0 + u];
                            const float ex = REV ? gj - gi[u] : gi[u] - gj;
                            acc[u] = fmaf(v[e] * sStageW[j * kM + s0 + u], __expf(fminf(ex, 0.f)), acc[u]);
                        }
                    }
                }
                float vi[16];
                tmem_ld16(tmem_row_addr(tmem, warp, kColO + s0), vi);
                if (tid < valid) {
                    float* dst = obase + (size_t)(t0 + tid) * strideM + s0;
#pragma unroll
                    for (int e = 0; e < 16; e += 4) {
                        float r[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            r[u] = fmaf(vi[e + u], __expf(REV ? ctl->gc[s0 + e + u] - gi[e + u] : gi[e + u]), acc[e + u]);
                        *reinterpret_cast<float4*>(dst + e) = make_float4(r[0], r[1], r[2], r[3]);
                    }
                }
            }
        }

        // ---- state update from U (complete since bar_mma1): S <- S exp(G_C) + U
#pragma unroll
        for (int c0 = 0; c0 < kM; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, warp, kColU + c0), v);
#pragma unroll
            for (int e = 0; e < 16; ++e) S[c0 + e] = fmaf(S[c0 + e], ctl->egc[c0 + e], v[e]);
        }

        // ---- output rows of a moderate chunk: rowscale * (inter + intra)
        if (moderate) {
            if (!mbar_wait(&ctl->bar_mma2, n_mma2 & 1)) ctl->abort = 1;
            ++n_mma2;
            tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < kM; c0 += 16) {
                float vi[16], vo[16], g0[8], g1[8];
                tmem_ld16(tmem_row_addr(tmem, warp, kColO + c0), vi);
                tmem_ld16(tmem_row_addr(tmem, warp, kColO2 + c0), vo);
                load8(grow + c0, g0);
                load8(grow + c0 + 8, g1);
                if (tid < valid) {
                    float* dst = obase + (size_t)(t0 + tid) * strideM + c0;
#pragma unroll
                    for (int e = 0; e < 16; e += 4) {
                        float r[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float g = (e + u < 8) ? g0[(e + u) & 7] : g1[(e + u) & 7];
                            if (REV) {
                                const float einv = __expf(-g);
                                r[u] = einv * fmaf(vi[e + u], ctl->egc[c0 + e + u], vo[e + u]);
                            } else {
                                r[u] = __expf(g) * (vi[e + u] + vo[e + u]);
                            }
                        }
                        *reinterpret_cast<float4*>(dst + e) = make_float4(r[0], r[1], r[2], r[3]);
                    }
                }
            }
        }
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        // give an outstanding prefetch a bounded chance to land before shared memory goes away
        if (it + 1 < nchunks) mbar_wait(&ctl->bar_load[(it + 1) & 1], ((it + 1) >> 1) & 1);
    } else if (a.Send) {
#pragma unroll
        for (int s = 0; s < kM; ++s) a.Send[((size_t)bh * kM + s) * a.D + d0 + tid] = S[s];
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ======================================================================================
// key_side: out_i = (uq_i * qscale_i) S + sum_j A_ij xv_j,  A_ij = sum_s uq_i[s] uk_j[s] decay_ij[s]
// ======================================================================================
template <bool REV>
__global__ void __launch_bounds__(128, 1)
key_side_tc_kernel(const __grid_constant__ CUtensorMap mapV, KeySideArgs a, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sXv = smem;                       // [2 stages][2 panels]
    unsigned char* sQt = sXv + 4 * kPanelB;          // uq with the intra scaling, K-major A [128][64]
    unsigned char* sKt = sQt + kPanelB;              // uk with the intra scaling, K-major B [128][64]
    unsigned char* sQb = sKt + kPanelB;              // uq with the state scaling, K-major A [128][64]
    unsigned char* sKb = sQb + kPanelB;              // (uk with the state scaling)^T, K-major B [64][128]
    unsigned char* sAm = sKb + kPanelB;              // masked A, K-major A, 2 panels
    unsigned char* sSb = sAm + 2 * kPanelB;          // state copy, K-major B [128 (channel)][64]
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + kPanelB);
    float* sStageK = reinterpret_cast<float*>(sQt);               // fp32 [128][64] over sQt + sKt
    float* sStageG = reinterpret_cast<float*>(sQb);               // fp32 [128][64] over sQb + sKb

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;
    const size_t strideM = (size_t)a.H * kM, strideD = (size_t)a.H * a.D;
    const float* qbase = a.uq + ((size_t)b * a.T * a.H + h) * kM;
    const float* kbase = a.uk + ((size_t)b * a.T * a.H + h) * kM;
    const float* gbase = a.G + ((size_t)b * a.T * a.H + h) * kM;
    __nv_bfloat16* obase = (__nv_bfloat16*)a.out + ((size_t)b * a.T * a.H + h) * a.D + d0;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;

    const int nchunks = (a.T + kCT - 1) / kCT;
    auto issue_loads = [&](int it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int st = it & 1;
        mbar_expect_tx(&ctl->bar_load[st], 2 * kPanelB);
        tma_load_4d(sXv + (2 * st) * kPanelB, &mapV, &ctl->bar_load[st], d0, h, n * kCT, b);
        tma_load_4d(sXv + (2 * st + 1) * kPanelB, &mapV, &ctl->bar_load[st], d0 + 64, h, n * kCT, b);
    };
    if (tid == 0) {
        prefetch_tmap(&mapV);
        issue_loads(0);
    }

    // state slice, transposed: S[c = tid][s]
    float S[kM];
#pragma unroll
    for (int s = 0; s < kM; ++s) S[s] = a.S0 ? a.S0[((size_t)bh * kM + s) * a.D + d0 + tid] : 0.f;

    constexpr uint32_t idescA = make_idesc(128, 128, false, false);   // Q~ K~^T
    constexpr uint32_t idescO = make_idesc(128, kDST, false, false);  // Q- x state copy (K-major B)
    constexpr uint32_t idescU = make_idesc(128, kM, true, false);     // xv^T (MN-major A) x K-^T
    constexpr uint32_t idescV = make_idesc(128, kDST, false, true);   // A x xv (MN-major B)

    int it = 0;
    for (; it < nchunks; ++it) {
        const int n = REV ? nchunks - 1 - it : it;
        const int st = it & 1;
        const int t0 = n * kCT;
        const int valid = min(kCT, a.T - t0);
        if (tid == 0 && it + 1 < nchunks) issue_loads(it + 1);

        publish_chunk_decay(ctl, tid, gbase + (size_t)(t0 + valid - 1) * strideM);
        const bool moderate = ctl->moderate != 0;
        const size_t rowoff = (size_t)(t0 + min(tid, valid - 1)) * strideM;
        const float live = tid < valid ? 1.f : 0.f;
        {
            unsigned char* pKb = sKb + (tid >> 6) * (kM * 128);
            const int col = tid & 63;
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 8) {
                float g[8], uq[8], uk[8], qb[8], qt[8], kt[8];
                load8(gbase + rowoff + s0, g);
                load8(qbase + rowoff + s0, uq);
                load8(kbase + rowoff + s0, uk);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int s = s0 + e;
                    const float eg = __expf(g[e]);
                    const float egc_g = __expf(ctl->gc[s] - g[e]);
                    // state terms: forward Q- = uq exp(G), K- = uk exp(G_C - G); reverse swapped
                    qb[e] = live * uq[e] * (REV ? egc_g : eg);
                    store_elem(pKb, s, col, live * uk[e] * (REV ? eg : egc_g));
                    if (moderate) {
                        const float einv = __expf(-g[e]);
                        qt[e] = live * uq[e] * (REV ? einv : eg);
                        kt[e] = live * uk[e] * (REV ? eg : einv);
                    }
                }
                store_chunk(sQb, tid, s0 >> 3, qb);
                if (moderate) {
                    store_chunk(sQt, tid, s0 >> 3, qt);
                    store_chunk(sKt, tid, s0 >> 3, kt);
                }
            }
        }
        store_state_row(sSb, tid, S);
        fence_async_smem();
        if (!mbar_wait(&ctl->bar_load[st], (it >> 1) & 1)) ctl->abort = 1;
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;

        const uint32_t aV = smem_u32(sXv + 2 * st * kPanelB);
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t aQt = smem_u32(sQt), aKt = smem_u32(sKt), aQb = smem_u32(sQb);
            const uint32_t aKb = smem_u32(sKb), aS = smem_u32(sSb);
            if (moderate) {
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kColP, desc_kmajor(aQt, kk), desc_kmajor(aKt, kk), idescA, kk > 0);
            }
#pragma unroll
            for (int kk = 0; kk < kM / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aQb, kk), desc_kmajor(aS, kk), idescO, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColU, desc_mnmajor(aV, kk, kPanelB),
                         desc_kmajor(aKb + (kk >> 2) * (kM * 128), kk), idescU, kk > 0);
            mma_commit(&ctl->bar_mma1);
        }
        if (!mbar_wait(&ctl->bar_mma1, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();

        if (moderate) {
#pragma unroll
            for (int c0 = 0; c0 < kCT; c0 += 16) {
                float v[16];
                tmem_ld16(tmem_row_addr(tmem, warp, kColP + c0), v);
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int j = c0 + e;
                    const bool keep = REV ? (j >= tid) : (j <= tid);
                    v[e] = keep ? v[e] : 0.f;
                }
                const float x0[8] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]};
                const float x1[8] = {v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]};
                unsigned char* panel = sAm + (c0 >> 6) * kPanelB;
                store_chunk(panel, tid, (c0 & 63) >> 3, x0);
                store_chunk(panel, tid, ((c0 & 63) >> 3) + 1, x1);
            }
        } else {
            // Strong decay: A_ij with explicit exponent differences.  uk and G rows of all tokens
            // are staged in fp32 over operand buffers whose products have completed.
            __syncthreads();
            float gi[kM], qi[kM];
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 8) {
                float g[8], uq[8], uk[8];
                load8(gbase + rowoff + s0, g);
                load8(qbase + rowoff + s0, uq);
                load8(kbase + rowoff + s0, uk);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    gi[s0 + e] = g[e];
                    qi[s0 + e] = live * uq[e];
                    sStageK[tid * kM + s0 + e] = live * uk[e];
                    sStageG[tid * kM + s0 + e] = g[e];
                }
            }
            __syncthreads();
            for (int c0 = 0; c0 < kCT; c0 += 8) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = c0 + e;
                    const bool keep = REV ? (j >= tid) : (j <= tid);
                    float acc = 0.f;
                    if (keep) {
#pragma unroll
                        for (int s = 0; s < kM; ++s) {
                            const float gj = sStageG[j * kM + s];
                            const float ex = REV ? gj - gi[s] : gi[s] - gj;
                            acc = fmaf(qi[s] * sStageK[j * kM + s], __expf(fminf(ex, 0.f)), acc);
                        }
                    }
                    x[e] = acc;
                }
                store_chunk(sAm + (c0 >> 6) * kPanelB, tid, (c0 & 63) >> 3, x);
            }
        }
        fence_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t aA = smem_u32(sAm);
#pragma unroll
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aA + (kk >> 2) * kPanelB, kk),
                         desc_mnmajor(aV, kk, kPanelB), idescV, true);
            mma_commit(&ctl->bar_mma2);
        }

        // ---- state update from U^T (complete since bar_mma1): S <- exp(G_C) S + U^T
#pragma unroll
        for (int c0 = 0; c0 < kM; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, warp, kColU + c0), v);
#pragma unroll
            for (int e = 0; e < 16; ++e) S[c0 + e] = fmaf(S[c0 + e], ctl->egc[c0 + e], v[e]);
        }

        // ---- output rows
        if (!mbar_wait(&ctl->bar_mma2, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();
#pragma unroll
        for (int c0 = 0; c0 < kDST; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, warp, kColO + c0), v);
            if (tid < valid) {
                __nv_bfloat16* dst = obase + (size_t)(t0 + tid) * strideD + c0;
                const uint4 lo = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
                const uint4 hi = make_uint4(pack_bf16(v[8], v[9]), pack_bf16(v[10], v[11]), pack_bf16(v[12], v[13]), pack_bf16(v[14], v[15]));
                *reinterpret_cast<uint4*>(dst) = lo;
                *reinterpret_cast<uint4*>(dst + 8) = hi;
            }
        }
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        if (it + 1 < nchunks) mbar_wait(&ctl->bar_load[(it + 1) & 1], ((it + 1) >> 1) & 1);
    } else if (a.Send) {
#pragma unroll
        for (int s = 0; s < kM; ++s) a.Send[((size_t)bh * kM + s) * a.D + d0 + tid] = S[s];
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

constexpr size_t kSmemValueSide = 1024 + 8 * kPanelB + 2 * kPanelB + 3 * kPanelB + sizeof(Ctl);
constexpr size_t kSmemKeySide = 1024 + 4 * kPanelB + 4 * kPanelB + 2 * kPanelB + kPanelB + sizeof(Ctl);

template <typename K>
cudaError_t prepare(K kernel, size_t smem) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // each CTA takes the whole tensor memory of its SM: make sure no second CTA can be co-resident
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 128, smem);
    if (e != cudaSuccess) return e;
    return per_sm == 1 ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

}  // namespace

bool tc_supported(int d_k, int d_v, int M) {
    return M == kM && d_k % kDST == 0 && d_v % kDST == 0;
}
int tc_value_side_slices(int D) { return D / kDST; }
int tc_chunk() { return kCT; }

cudaError_t launch_value_side_tc(const ValueSideArgs& a, int M, int reverse, cudaStream_t st, int32_t* dev_status) {
    if (M != kM || a.D % kDST != 0) return cudaErrorNotSupported;
    CUtensorMap mq, mk;
    cudaError_t e = make_tensor_map_bthd(&mq, a.xq, a.B, a.T, a.H, a.D, kCT);
    if (e != cudaSuccess) return e;
    e = make_tensor_map_bthd(&mk, a.xk, a.B, a.T, a.H, a.D, kCT);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDST);
    if (reverse) {
        e = prepare(value_side_tc_kernel<true>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<true><<<grid, 128, kSmemValueSide, st>>>(mq, mk, a, dev_status);
    } else {
        e = prepare(value_side_tc_kernel<false>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<false><<<grid, 128, kSmemValueSide, st>>>(mq, mk, a, dev_status);
    }
    return cudaGetLastError();
}

cudaError_t launch_key_side_tc(const KeySideArgs& a, int M, int reverse, cudaStream_t st, int32_t* dev_status) {
    if (M != kM || a.D % kDST != 0) return cudaErrorNotSupported;
    CUtensorMap mv;
    cudaError_t e = make_tensor_map_bthd(&mv, a.xv, a.B, a.T, a.H, a.D, kCT);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDST);
    if (reverse) {
        e = prepare(key_side_tc_kernel<true>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<true><<<grid, 128, kSmemKeySide, st>>>(mv, a, dev_status);
    } else {
        e = prepare(key_side_tc_kernel<false>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<false><<<grid, 128, kSmemKeySide, st>>>(mv, a, dev_status);
    }
    return cudaGetLastError();
}

}  // namespace gsa
