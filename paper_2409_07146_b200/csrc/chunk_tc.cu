// tcgen05 (bf16 tensor-core) versions of the two chunk primitives of Algorithm 1.
//
// One CTA of 128 threads owns one (batch, head) and one 128-wide slice of the head
// dimension and walks the chunks (128 tokens each) in order.  Thread i is row i of the
// chunk and channel i of the state slice, which is also TMEM lane i of every accumulator.
// Per chunk:
//   * every tile -- the d-sized ones (xq, xk / xv, bf16) and the slot-sized ones (weights,
//     cumulative log gate G, fp32) -- arrives by TMA with the 128-byte swizzle, requested as
//     soon as the buffer it lands in has been consumed by the previous chunk, so the copy of
//     chunk n+1 runs under the computation of chunk n;
//   * each thread reads its own row of the slot-sized tiles (conflict-free under the
//     swizzle), scales it by the decay factors and writes bf16 operand rows;
//   * all contractions run as tcgen05.mma (M = 128) with fp32 accumulators in tensor
//     memory; thread 0 issues them and commits to an mbarrier that everybody waits on;
//   * the fp32 master copy of the state slice stays in registers (64 per thread); its bf16
//     copy for the next chunk's state product is rewritten every chunk.
// Decay inside a chunk is factorised as exp(G_i) * exp(-G_j) while the chunk's total
// log-decay stays above kFactorisedDecayMin; a chunk that forgets harder computes its
// intra-chunk term with explicit exponent differences on the CUDA cores instead.
// Every wait is bounded: on expiry the CTA flags dev_status, frees its tensor memory and
// returns.
#include <stdio.h>

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

// Optional phase timing for development builds (-DGSA_TC_PROF): CTA 0 prints, for its fifth
// chunk, the SM clock at each phase boundary.
#ifdef GSA_TC_PROF
#define PROF_DECL long long prof_t[12]; int prof_n = 0;
#define PROF_MARK() do { if (prof_n < 12) prof_t[prof_n++] = clock64(); } while (0)
#define PROF_DUMP(name) do { if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0 && it == 4) { \
    printf("%s:", name); for (int i_ = 1; i_ < prof_n; ++i_) printf(" %lld", prof_t[i_] - prof_t[i_ - 1]); printf("\n"); } prof_n = 0; } while (0)
#else
#define PROF_DECL
#define PROF_MARK() do {} while (0)
#define PROF_DUMP(name) do {} while (0)
#endif

struct Ctl {
    uint64_t bar_x;        // d-sized tiles of the current chunk
    uint64_t bar_g[2];     // value_side: G tile, two stages; key_side: [0] = uk + G tiles
    uint64_t bar_w;        // value_side: weight tile; key_side: uq tile
    uint64_t bar_mma1;
    uint64_t bar_mma2;
    uint32_t tmem_slot;
    volatile int abort;
    float gc[kM];        // G of the chunk's last valid row
    float egc[kM];       // exp(gc)
};

// 8 consecutive fp32 values (columns s0 .. s0+7, s0 % 8 == 0) of row `row` of a slot-sized
// fp32 tile: two panels of 32 columns, 128-byte swizzle.
__device__ __forceinline__ void tile_row8(const unsigned char* tile, int row, int s0, float (&x)[8]) {
    const unsigned char* panel = tile + (s0 >> 5) * kPanelB;
    const int c = (s0 & 31) >> 2;
    const float4 t0 = *reinterpret_cast<const float4*>(panel + swz128(row, c));
    const float4 t1 = *reinterpret_cast<const float4*>(panel + swz128(row, c + 1));
    x[0] = t0.x; x[1] = t0.y; x[2] = t0.z; x[3] = t0.w;
    x[4] = t1.x; x[5] = t1.y; x[6] = t1.z; x[7] = t1.w;
}
__device__ __forceinline__ float tile_elem(const unsigned char* tile, int row, int s) {
    return *reinterpret_cast<const float*>(tile + (s >> 5) * kPanelB + swz128(row, (s & 31) >> 2) + (s & 3) * 4);
}

// bf16 copy of this thread's state row (64 values, optionally scaled per slot) as row `row`
// of a one-panel operand
template <bool SCALE>
__device__ __forceinline__ void store_state_row(unsigned char* panel, int row, const float (&S)[kM], const float* scale) {
#pragma unroll
    for (int c = 0; c < kM / 8; ++c) {
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = SCALE ? S[8 * c + e] * scale[8 * c + e] : S[8 * c + e];
        store_chunk(panel, row, c, x);
    }
}

// Publish the G row of the chunk's last valid token, its exponential and decide whether the
// chunk's decay is moderate.  One __syncthreads inside; the result is uniform.
__device__ __forceinline__ bool publish_chunk_decay(Ctl* ctl, int tid, const unsigned char* gtile, int last_row) {
    bool fine = true;
    if (tid < kM) {
        const float g = tile_elem(gtile, last_row, tid);
        ctl->gc[tid] = g;
        ctl->egc[tid] = __expf(g);
        fine = g >= kFactorisedDecayMin;
    }
    return __syncthreads_and(fine) != 0;
}

__device__ __forceinline__ void ctl_init(Ctl* ctl, int tid, int warp) {
    if (tid == 0) {
        mbar_init(&ctl->bar_x, 1);
        mbar_init(&ctl->bar_g[0], 1);
        mbar_init(&ctl->bar_g[1], 1);
        mbar_init(&ctl->bar_w, 1);
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

// masked accumulator row -> bf16 K-major operand row (two 64-column panels)
template <bool REV>
__device__ __forceinline__ void store_masked_row(uint32_t tmem, int warp, int tid, unsigned char* dst) {
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
        unsigned char* panel = dst + (c0 >> 6) * kPanelB;
        store_chunk(panel, tid, (c0 & 63) >> 3, x0);
        store_chunk(panel, tid, ((c0 & 63) >> 3) + 1, x1);
    }
}

// ======================================================================================
// value_side: out_i[s] = sum_{j<=i} <xq_i, xk_j> w_j[s] decay_ij[s]  + decayed (xq_i S)[s]
// ======================================================================================
template <bool REV>
__global__ void __launch_bounds__(128, 1)
value_side_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                     const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapG,
                     ValueSideArgs a, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sXq = smem;                       // 2 panels                                  (32 KB)
    unsigned char* sXk = sXq + 2 * kPanelB;          // 2 panels                                  (32 KB)
    unsigned char* sG = sXk + 2 * kPanelB;           // G tile fp32, [2 stages][2 panels]         (64 KB)
    unsigned char* sPm = sG + 4 * kPanelB;           // masked P, K-major A, 2 panels             (32 KB)
    unsigned char* sW = sPm;                         //   ... shared with the weight tile fp32, 2 panels
    unsigned char* sWp = sPm + 2 * kPanelB;          // intra weights, MN-major B [128][64]       (16 KB)
    unsigned char* sWt = sWp + kPanelB;              // state-update weights, MN-major B [128][64] (16 KB)
    unsigned char* sSb = sWt + kPanelB;              // state copy, MN-major B [128][64]          (16 KB)
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;
    const size_t strideM = (size_t)a.H * kM;
    float* obase = a.out + (size_t)slice * a.B * a.T * a.H * kM + ((size_t)b * a.T * a.H + h) * kM;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;

    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int it) { return (REV ? nchunks - 1 - it : it) * kCT; };
    auto load_x = [&](int it) {
        const int t = chunk_t0(it);
        mbar_expect_tx(&ctl->bar_x, 4 * kPanelB);
        tma_load_4d(sXq, &mapQ, &ctl->bar_x, d0, h, t, b);
        tma_load_4d(sXq + kPanelB, &mapQ, &ctl->bar_x, d0 + 64, h, t, b);
        tma_load_4d(sXk, &mapK, &ctl->bar_x, d0, h, t, b);
        tma_load_4d(sXk + kPanelB, &mapK, &ctl->bar_x, d0 + 64, h, t, b);
    };
    auto load_g = [&](int it) {
        const int t = chunk_t0(it), st = it & 1;
        mbar_expect_tx(&ctl->bar_g[st], 2 * kPanelB);
        tma_load_4d(sG + (2 * st) * kPanelB, &mapG, &ctl->bar_g[st], 0, h, t, b);
        tma_load_4d(sG + (2 * st + 1) * kPanelB, &mapG, &ctl->bar_g[st], 32, h, t, b);
    };
    auto load_w = [&](int it) {
        const int t = chunk_t0(it);
        mbar_expect_tx(&ctl->bar_w, 2 * kPanelB);
        tma_load_4d(sW, &mapW, &ctl->bar_w, 0, h, t, b);
        tma_load_4d(sW + kPanelB, &mapW, &ctl->bar_w, 32, h, t, b);
    };
    if (tid == 0) {
        prefetch_tmap(&mapQ); prefetch_tmap(&mapK); prefetch_tmap(&mapW); prefetch_tmap(&mapG);
        load_g(0);
        load_w(0);
        load_x(0);
    }

    // state slice: S[c = tid][s]
    float S[kM];
#pragma unroll
    for (int s = 0; s < kM; ++s) S[s] = a.S0 ? a.S0[((size_t)bh * kM + s) * a.D + d0 + tid] : 0.f;

    constexpr uint32_t idescP = make_idesc(128, 128, false, false);  // xq xk^T
    constexpr uint32_t idescO = make_idesc(128, kM, false, true);    // xq x state copy (MN-major B)
    constexpr uint32_t idescU = make_idesc(128, kM, true, true);     // xk^T (MN-major A) x W~ (MN-major B)
    constexpr uint32_t idescI = make_idesc(128, kM, false, true);    // Pm x W' (MN-major B)

    int it = 0;
    int n_mma2 = 0;    // completed phases of bar_mma2 (only moderate chunks use it)
    PROF_DECL
    for (; it < nchunks; ++it) {
        const int t0 = chunk_t0(it);
        const int valid = min(kCT, a.T - t0);
        const unsigned char* gt = sG + (2 * (it & 1)) * kPanelB;
        PROF_MARK();
        if (tid == 0 && it + 1 < nchunks) load_g(it + 1);
        if (!mbar_wait(&ctl->bar_g[it & 1], (it >> 1) & 1)) ctl->abort = 1;
        if (!mbar_wait(&ctl->bar_w, it & 1)) ctl->abort = 1;
        const bool moderate = publish_chunk_decay(ctl, tid, gt, valid - 1);
        if (ctl->abort) break;
        PROF_MARK();

        // ---- this token's slot rows -> operand rows (rows past the end: zero weights)
        const int grow = min(tid, valid - 1);
#pragma unroll
        for (int s0 = 0; s0 < kM; s0 += 8) {
            float g[8], w[8], wp[8], wt[8];
            tile_row8(gt, grow, s0, g);
            tile_row8(sW, tid, s0, w);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (REV) {
                    // reverse: both the intra and the state-update weights are w exp(G)
                    wt[e] = w[e] * __expf(g[e]);
                    wp[e] = wt[e];
                } else if (moderate) {
                    // forward: intra w exp(-G), state update w exp(G_C - G) = intra * exp(G_C)
                    wp[e] = w[e] * __expf(-g[e]);
                    wt[e] = wp[e] * ctl->egc[s0 + e];
                } else {
                    wp[e] = 0.f;
                    wt[e] = w[e] * __expf(ctl->gc[s0 + e] - g[e]);
                }
            }
            store_chunk(sWt, tid, s0 >> 3, wt);
            if (moderate) store_chunk(sWp, tid, s0 >> 3, wp);
        }
        // state copy for the inter-chunk product; a moderate reverse chunk folds exp(G_C) in
        if (REV && moderate) store_state_row<true>(sSb, tid, S, ctl->egc);
        else store_state_row<false>(sSb, tid, S, nullptr);
        fence_async_smem();
        if (!mbar_wait(&ctl->bar_x, it & 1)) ctl->abort = 1;
        PROF_MARK();
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
        PROF_MARK();

        // ---- P = xq xk^T, O = xq S, U = xk^T W~
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t aQ = smem_u32(sXq), aK = smem_u32(sXk);
            const uint32_t aS = smem_u32(sSb), aWt = smem_u32(sWt);
#pragma unroll
            for (int kk = 0; kk < kDST / 16; ++kk)
                mma_bf16(tmem + kColP, desc_kmajor(aQ + (kk >> 2) * kPanelB, kk),
                         desc_kmajor(aK + (kk >> 2) * kPanelB, kk), idescP, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColU, desc_mnmajor(aK, kk, kPanelB), desc_mnmajor(aWt, kk, kPanelB), idescU, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kDST / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aQ + (kk >> 2) * kPanelB, kk),
                         desc_mnmajor(aS, kk, kPanelB), idescO, kk > 0);
            mma_commit(&ctl->bar_mma1);
        }
        PROF_MARK();
        if (!mbar_wait(&ctl->bar_mma1, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();
        PROF_MARK();
        // the d-sized tiles are consumed: request the next chunk's
        if (tid == 0 && it + 1 < nchunks) load_x(it + 1);

        if (moderate) {
            store_masked_row<REV>(tmem, warp, tid, sPm);    // overwrites the weight tile: all rows were read
            fence_async_smem();
        }
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
        PROF_MARK();
        if (moderate) {
            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t aP = smem_u32(sPm), aWp = smem_u32(sWp);
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kColO, desc_kmajor(aP + (kk >> 2) * kPanelB, kk),
                             desc_mnmajor(aWp, kk, kPanelB), idescI, true);
                mma_commit(&ctl->bar_mma2);
            }
        } else {
            // Strong decay: the intra-chunk term with explicit exponent differences on the CUDA
            // cores, straight from the fp32 weight and G tiles.
            const int jlo = REV ? tid : 0, jhi = REV ? kCT - 1 : tid;
            // the accumulator loads are warp-collective: loop bounds are those of the whole warp
            const int wlo = REV ? warp * 32 : 0, whi = REV ? kCT - 1 : warp * 32 + 31;
            for (int s0 = 0; s0 < kM; s0 += 16) {
                float gi[16], acc[16], tmp[8];
                tile_row8(gt, grow, s0, tmp);
#pragma unroll
                for (int e = 0; e < 8; ++e) gi[e] = tmp[e];
                tile_row8(gt, grow, s0 + 8, tmp);
#pragma unroll
                for (int e = 0; e < 8; ++e) gi[8 + e] = tmp[e];
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] = 0.f;
                for (int c0 = wlo; c0 <= whi; c0 += 16) {
                    float v[16];
                    tmem_ld16(tmem_row_addr(tmem, warp, kColP + c0), v);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int j = c0 + e;
                        if (j < jlo || j > jhi) continue;
                        const int jg = min(j, valid - 1);
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            const float gj = tile_elem(gt, jg, s0 + u);
                            const float ex = REV ? gj - gi[u] : gi[u] - gj;
                            acc[u] = fmaf(v[e] * tile_elem(sW, j, s0 + u), __expf(fminf(ex, 0.f)), acc[u]);
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
        PROF_MARK();

        // ---- output rows of a moderate chunk: exp(+-G_i) * (inter + intra)
        if (moderate) {
            if (!mbar_wait(&ctl->bar_mma2, n_mma2 & 1)) ctl->abort = 1;
            ++n_mma2;
            tc_fence_after_sync();
            PROF_MARK();
#pragma unroll
            for (int c0 = 0; c0 < kM; c0 += 16) {
                float vo[16], g0[8], g1[8];
                tmem_ld16(tmem_row_addr(tmem, warp, kColO + c0), vo);
                tile_row8(gt, grow, c0, g0);
                tile_row8(gt, grow, c0 + 8, g1);
                if (tid < valid) {
                    float* dst = obase + (size_t)(t0 + tid) * strideM + c0;
#pragma unroll
                    for (int e = 0; e < 16; e += 4) {
                        float r[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float g = (e + u < 8) ? g0[(e + u) & 7] : g1[(e + u) & 7];
                            r[u] = vo[e + u] * __expf(REV ? -g : g);
                        }
                        *reinterpret_cast<float4*>(dst + e) = make_float4(r[0], r[1], r[2], r[3]);
                    }
                }
            }
        }
        tc_fence_before_sync();
        __syncthreads();
        // the weight tile's buffer (masked P) is free again: request the next chunk's weights
        if (tid == 0 && it + 1 < nchunks && !ctl->abort) load_w(it + 1);
        PROF_MARK();
        PROF_DUMP("value_side");
        if (ctl->abort) break;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        // bounded grace period for tile copies still in flight before shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
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
key_side_tc_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapUq,
                   const __grid_constant__ CUtensorMap mapUk, const __grid_constant__ CUtensorMap mapG,
                   KeySideArgs a, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* sXv = smem;                       // 2 panels                                   (32 KB)
    unsigned char* sUk = sXv + 2 * kPanelB;          // uk tile fp32, 2 panels                     (32 KB)
    unsigned char* sG = sUk + 2 * kPanelB;           // G tile fp32, 2 panels                      (32 KB)
    unsigned char* sAm = sG + 2 * kPanelB;           // masked A, K-major A, 2 panels              (32 KB)
    unsigned char* sUq = sAm;                        //   ... shared with the uq tile fp32, 2 panels
    unsigned char* sQt = sAm + 2 * kPanelB;          // uq, intra scaling, K-major A [128][64]     (16 KB)
    unsigned char* sKt = sQt + kPanelB;              // uk, intra scaling, K-major B [128][64]     (16 KB)
    unsigned char* sQb = sKt + kPanelB;              // uq, state scaling, K-major A [128][64]     (16 KB)
    unsigned char* sKb = sQb + kPanelB;              // uk, state scaling, MN-major B [128][64]    (16 KB)
    unsigned char* sSb = sKb + kPanelB;              // state copy, K-major B [128 (channel)][64]  (16 KB)
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;
    const size_t strideD = (size_t)a.H * a.D;
    __nv_bfloat16* obase = (__nv_bfloat16*)a.out + ((size_t)b * a.T * a.H + h) * a.D + d0;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;

    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int it) { return (REV ? nchunks - 1 - it : it) * kCT; };
    auto load_v = [&](int it) {
        const int t = chunk_t0(it);
        mbar_expect_tx(&ctl->bar_x, 2 * kPanelB);
        tma_load_4d(sXv, &mapV, &ctl->bar_x, d0, h, t, b);
        tma_load_4d(sXv + kPanelB, &mapV, &ctl->bar_x, d0 + 64, h, t, b);
    };
    auto load_kg = [&](int it) {
        const int t = chunk_t0(it);
        mbar_expect_tx(&ctl->bar_g[0], 4 * kPanelB);
        tma_load_4d(sUk, &mapUk, &ctl->bar_g[0], 0, h, t, b);
        tma_load_4d(sUk + kPanelB, &mapUk, &ctl->bar_g[0], 32, h, t, b);
        tma_load_4d(sG, &mapG, &ctl->bar_g[0], 0, h, t, b);
        tma_load_4d(sG + kPanelB, &mapG, &ctl->bar_g[0], 32, h, t, b);
    };
    auto load_q = [&](int it) {
        const int t = chunk_t0(it);
        mbar_expect_tx(&ctl->bar_w, 2 * kPanelB);
        tma_load_4d(sUq, &mapUq, &ctl->bar_w, 0, h, t, b);
        tma_load_4d(sUq + kPanelB, &mapUq, &ctl->bar_w, 32, h, t, b);
    };
    if (tid == 0) {
        prefetch_tmap(&mapV); prefetch_tmap(&mapUq); prefetch_tmap(&mapUk); prefetch_tmap(&mapG);
        load_kg(0);
        load_q(0);
        load_v(0);
    }

    // state slice, transposed: S[c = tid][s]
    float S[kM];
#pragma unroll
    for (int s = 0; s < kM; ++s) S[s] = a.S0 ? a.S0[((size_t)bh * kM + s) * a.D + d0 + tid] : 0.f;

    constexpr uint32_t idescA = make_idesc(128, 128, false, false);   // Q~ K~^T
    constexpr uint32_t idescO = make_idesc(128, kDST, false, false);  // Q- x state copy (K-major B)
    constexpr uint32_t idescU = make_idesc(128, kM, true, true);      // xv^T (MN-major A) x K- (MN-major B)
    constexpr uint32_t idescV = make_idesc(128, kDST, false, true);   // A x xv (MN-major B)

    int it = 0;
    PROF_DECL
    for (; it < nchunks; ++it) {
        const int t0 = chunk_t0(it);
        const int valid = min(kCT, a.T - t0);
        PROF_MARK();
        if (!mbar_wait(&ctl->bar_g[0], it & 1)) ctl->abort = 1;
        if (!mbar_wait(&ctl->bar_w, it & 1)) ctl->abort = 1;
        const bool moderate = publish_chunk_decay(ctl, tid, sG, valid - 1);
        if (ctl->abort) break;
        PROF_MARK();

        const int grow = min(tid, valid - 1);
#pragma unroll
        for (int s0 = 0; s0 < kM; s0 += 8) {
            float g[8], uq[8], uk[8], qb[8], kb[8], qt[8], kt[8];
            tile_row8(sG, grow, s0, g);
            tile_row8(sUq, tid, s0, uq);
            tile_row8(sUk, tid, s0, uk);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float eg = __expf(g[e]);
                const float egc_g = __expf(ctl->gc[s0 + e] - g[e]);
                // state terms: forward Q- = uq exp(G), K- = uk exp(G_C - G); reverse swapped
                qb[e] = uq[e] * (REV ? egc_g : eg);
                kb[e] = uk[e] * (REV ? eg : egc_g);
                if (moderate) {
                    const float einv = __expf(-g[e]);
                    qt[e] = uq[e] * (REV ? einv : eg);
                    kt[e] = uk[e] * (REV ? eg : einv);
                }
            }
            store_chunk(sQb, tid, s0 >> 3, qb);
            store_chunk(sKb, tid, s0 >> 3, kb);
            if (moderate) {
                store_chunk(sQt, tid, s0 >> 3, qt);
                store_chunk(sKt, tid, s0 >> 3, kt);
            }
        }
        store_state_row<false>(sSb, tid, S, nullptr);
        fence_async_smem();
        if (!mbar_wait(&ctl->bar_x, it & 1)) ctl->abort = 1;
        PROF_MARK();
        tc_fence_before_sync();
        __syncthreads();
        if (ctl->abort) break;
        PROF_MARK();

        const uint32_t aV = smem_u32(sXv);
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
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColU, desc_mnmajor(aV, kk, kPanelB), desc_mnmajor(aKb, kk, kPanelB), idescU, kk > 0);
#pragma unroll
            for (int kk = 0; kk < kM / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aQb, kk), desc_kmajor(aS, kk), idescO, kk > 0);
            mma_commit(&ctl->bar_mma1);
            // a moderate chunk is done with the uk and G tiles: request the next chunk's
            if (moderate && it + 1 < nchunks) load_kg(it + 1);
        }
        PROF_MARK();
        if (!mbar_wait(&ctl->bar_mma1, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();
        PROF_MARK();

        if (moderate) {
            store_masked_row<REV>(tmem, warp, tid, sAm);    // overwrites the uq tile: all rows were read
        } else {
            // Strong decay: A_ij with explicit exponent differences, from the fp32 uk and G tiles.
            float gi[kM], qi[kM];
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 8) {
                float g[8], uq[8];
                tile_row8(sG, grow, s0, g);
                tile_row8(sUq, tid, s0, uq);
#pragma unroll
                for (int e = 0; e < 8; ++e) { gi[s0 + e] = g[e]; qi[s0 + e] = uq[e]; }
            }
            __syncthreads();          // every thread has its uq row in registers before sAm is written
            for (int c0 = 0; c0 < kCT; c0 += 8) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = c0 + e;
                    const bool keep = REV ? (j >= tid) : (j <= tid);
                    float acc = 0.f;
                    if (keep) {
                        const int jg = min(j, valid - 1);
#pragma unroll
                        for (int s = 0; s < kM; ++s) {
                            const float gj = tile_elem(sG, jg, s);
                            const float ex = REV ? gj - gi[s] : gi[s] - gj;
                            acc = fmaf(qi[s] * tile_elem(sUk, j, s), __expf(fminf(ex, 0.f)), acc);
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
        PROF_MARK();
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t aA = smem_u32(sAm);
#pragma unroll
            for (int kk = 0; kk < kCT / 16; ++kk)
                mma_bf16(tmem + kColO, desc_kmajor(aA + (kk >> 2) * kPanelB, kk),
                         desc_mnmajor(aV, kk, kPanelB), idescV, true);
            mma_commit(&ctl->bar_mma2);
            if (!moderate && it + 1 < nchunks) load_kg(it + 1);
        }

        // ---- state update from U^T (complete since bar_mma1): S <- exp(G_C) S + U^T
#pragma unroll
        for (int c0 = 0; c0 < kM; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, warp, kColU + c0), v);
#pragma unroll
            for (int e = 0; e < 16; ++e) S[c0 + e] = fmaf(S[c0 + e], ctl->egc[c0 + e], v[e]);
        }
        PROF_MARK();

        // ---- output rows
        if (!mbar_wait(&ctl->bar_mma2, it & 1)) ctl->abort = 1;
        tc_fence_after_sync();
        PROF_MARK();
        // xv and the masked A are consumed: request the next chunk's xv and uq tiles
        if (tid == 0 && it + 1 < nchunks && !ctl->abort) {
            load_v(it + 1);
            load_q(it + 1);
        }
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
        PROF_MARK();
        PROF_DUMP("key_side");
        if (ctl->abort) break;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        // bounded grace period for tile copies still in flight before shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
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

constexpr size_t kSmemValueSide = 1024 + 13 * kPanelB + sizeof(Ctl);
constexpr size_t kSmemKeySide = 1024 + 13 * kPanelB + sizeof(Ctl);

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
    CUtensorMap mq, mk, mw, mg;
    cudaError_t e = make_tensor_map_bthd(&mq, a.xq, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mk, a.xk, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, a.w, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDST);
    if (reverse) {
        e = prepare(value_side_tc_kernel<true>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<true><<<grid, 128, kSmemValueSide, st>>>(mq, mk, mw, mg, a, dev_status);
    } else {
        e = prepare(value_side_tc_kernel<false>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<false><<<grid, 128, kSmemValueSide, st>>>(mq, mk, mw, mg, a, dev_status);
    }
    return cudaGetLastError();
}

cudaError_t launch_key_side_tc(const KeySideArgs& a, int M, int reverse, cudaStream_t st, int32_t* dev_status) {
    if (M != kM || a.D % kDST != 0) return cudaErrorNotSupported;
    CUtensorMap mv, muq, muk, mg;
    cudaError_t e = make_tensor_map_bthd(&mv, a.xv, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muq, a.uq, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muk, a.uk, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, a.D / kDST);
    if (reverse) {
        e = prepare(key_side_tc_kernel<true>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<true><<<grid, 128, kSmemKeySide, st>>>(mv, muq, muk, mg, a, dev_status);
    } else {
        e = prepare(key_side_tc_kernel<false>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<false><<<grid, 128, kSmemKeySide, st>>>(mv, muq, muk, mg, a, dev_status);
    }
    return cudaGetLastError();
}

}  // namespace gsa
