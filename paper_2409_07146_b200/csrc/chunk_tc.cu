// tcgen05 (bf16 tensor-core) versions of the two chunk primitives of Algorithm 1.
//
// One CTA owns one (batch, head) and one 128-wide slice of the head dimension and walks the
// chunks (128 tokens each) in order.  It has 256 compute threads and one issuing warp.
// Compute threads r and r + 128 share row r of the chunk, which is channel r of the state
// slice and TMEM lane r of every accumulator; the first works on slots (or columns) 0..31
// (0..63), the second on the rest.  One lane of the issuing warp requests every tile copy
// and issues every MMA, running ahead of the compute threads; the two sides meet on
// mbarriers only.
// Per chunk:
//   * every tile -- the d-sized ones (xq, xk / xv, bf16) and the slot-sized ones (weights,
//     cumulative log gate G, fp32) -- arrives by TMA with the 128-byte swizzle, requested as
//     soon as the buffer it lands in has been consumed by the previous chunk, so the copy of
//     chunk n+1 runs under the computation of chunk n;
//   * each thread reads its own row of the slot-sized tiles (conflict-free under the
//     swizzle), scales it by the decay factors and writes bf16 operand rows;
//   * all contractions run as tcgen05.mma (M = 128) with fp32 accumulators in tensor
//     memory, committed to mbarriers that the compute threads wait on;
//   * the fp32 master copy of the state slice stays in registers (32 per thread); its bf16
//     copy for the next chunk's state product is rewritten every chunk.
// Decay inside a chunk is factorised as exp(G_i) * exp(-G_j) while the chunk's total
// log-decay stays above kFactorisedDecayMin; a chunk that forgets harder computes its
// intra-chunk term with explicit exponent differences on the CUDA cores instead.
// Every wait is bounded: on expiry the CTA flags dev_status, frees its tensor memory and
// returns.
#include "chunk_tc_shared.cuh"

namespace gsa {
namespace {
using namespace tc;
using namespace tcchunk;

struct Ctl {
    // filled by TMA
    uint64_t bar_x;        // d-sized tiles of the current chunk
    uint64_t bar_g[2];     // value_side: G tile, two stages; key_side: [0] = uk + G tiles
    uint64_t bar_w;        // value_side: weight tile; key_side: uq tile
    // signalled by tcgen05.commit
    uint64_t bar_p;        // first product of the chunk (P or A) complete
    uint64_t bar_mma1;     // state and inter-chunk products complete
    uint64_t bar_mma2;     // intra-chunk product complete
    // signalled by the compute threads (one arrival after their barrier)
    uint64_t bar_ops;      // operand rows of the chunk are in shared memory
    uint64_t bar_pm;       // masked P / A rows are in shared memory
    uint64_t bar_out;      // output rows are staged (or the chunk is otherwise done)
    uint64_t bar_sb;       // value_side: the state copy for the next chunk is written
                           // key_side: (issuing warp ->) the output staging buffer is free again
    uint32_t tmem_slot;
    volatile int abort;
    volatile int moderate[2];   // decision of the chunk, by chunk parity
    alignas(16) float gc[kM];    // G of the chunk's last valid row
    alignas(16) float egc[kM];   // exp(gc)
};

// Publish the G row of the chunk's last valid token, its exponential and decide whether the
// chunk's decay is moderate.  One compute-thread barrier inside; the result is uniform.
__device__ __forceinline__ bool publish_chunk_decay(Ctl* ctl, int tid, const unsigned char* gtile, int last_row) {
    bool fine = true;
    if (tid < kM) {
        const float g = tile_elem(gtile, last_row, tid);
        ctl->gc[tid] = g;
        ctl->egc[tid] = __expf(g);
        fine = g >= kFactorisedDecayMin;
    }
    return compute_sync_and(fine);
}

__device__ __forceinline__ void ctl_init(Ctl* ctl, int tid, int warp) {
    if (tid == 0) {
        mbar_init(&ctl->bar_x, 1);
        mbar_init(&ctl->bar_g[0], 1);
        mbar_init(&ctl->bar_g[1], 1);
        mbar_init(&ctl->bar_w, 1);
        mbar_init(&ctl->bar_p, 1);
        mbar_init(&ctl->bar_mma1, 1);
        mbar_init(&ctl->bar_mma2, 1);
        mbar_init(&ctl->bar_ops, 1);
        mbar_init(&ctl->bar_pm, 1);
        mbar_init(&ctl->bar_out, 1);
        mbar_init(&ctl->bar_sb, 1);
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

// Strong-decay chunks (App. A: a decay too strong for one reference point per chunk).  The decay
// between two rows of a chunk is a product of per-step gates, prod_{r=j+1..i} a_r[s], every factor
// <= 1: walking j away from the target row i, the product is carried along by ONE multiplication
// per step and slot -- no exponential in the loop, nothing can overflow -- and the walk stops as
// soon as the product has fallen below 2^-40 for all slots of the thread (what is left of the sum is
// then below 1e-12 of its leading terms).  With strong forgetting that is after a dozen steps.
// The per-step gates a_j = exp(G_j - G_{j-1}) are formed once per chunk, in place of the G tile.
constexpr float kDecayFloor = 9.094947e-13f;      // 2^-40

// Replace the G tile by the per-step gates (rows past the end: 1).  gi receives this thread's own
// G row (slots sb .. sb+31) first.  Two compute-thread barriers inside.
__device__ __forceinline__ void gates_in_place(unsigned char* gt, int row, int half, int sb, int valid, float (&gi)[kHS]) {
    const int grow = min(row, valid - 1);
    float aj[kHS];
#pragma unroll
    for (int c = 0; c < kHS / 8; ++c) {
        float g[8], gp[8];
        tile_row8(gt, grow, sb + 8 * c, g);
        if (row > 0 && row < valid) tile_row8(gt, row - 1, sb + 8 * c, gp);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            gi[8 * c + e] = g[e];
            aj[8 * c + e] = row >= valid ? 1.f : __expf(row > 0 ? g[e] - gp[e] : g[e]);
        }
    }
    compute_sync();           // every thread has read what it needs of G
    unsigned char* panel = gt + half * kPanelB;
#pragma unroll
    for (int c = 0; c < kHS / 4; ++c)
        *reinterpret_cast<float4*>(panel + swz128(row, c)) = make_float4(aj[4 * c], aj[4 * c + 1], aj[4 * c + 2], aj[4 * c + 3]);
    compute_sync();
}

// 16 consecutive fp32 values (s0 % 16 == 0) of row `row` of a slot-sized fp32 tile
__device__ __forceinline__ void tile_row16(const unsigned char* tile, int row, int s0, float (&x)[16]) {
    const unsigned char* panel = tile + (s0 >> 5) * kPanelB;
    const int c = (s0 & 31) >> 2;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 t = *reinterpret_cast<const float4*>(panel + swz128(row, c + q));
        x[4 * q] = t.x; x[4 * q + 1] = t.y; x[4 * q + 2] = t.z; x[4 * q + 3] = t.w;
    }
}

// Strong-decay chunk of value_side: this thread's 32 output slots of row `row`,
//   out[s] = exp(+-..) * inter[s] + sum_j P_ij w_j[s] prod a_r[s]   (j <= i forward, j >= i reverse),
// P and the inter-chunk product are read from the accumulators; the row goes straight to global
// memory.  `gt` holds the per-step gates (gates_in_place), gi this thread's G row.
template <bool REV>
__device__ __forceinline__ void value_side_explicit_rows(const unsigned char* gt, const unsigned char* sW,
                                                      const float* gc, const float (&gi)[kHS], uint32_t tmem, int wq,
                                                      int row, int sb, int valid, float* out_row) {
    // the accumulator loads are warp-collective: the 16-column segments are those of the whole warp,
    // walked away from the diagonal
    const int first = REV ? wq * 32 : wq * 32 + 16, last = REV ? kCT - 16 : 0, step = REV ? 16 : -16;
#pragma unroll 1
    for (int s0 = sb; s0 < sb + kHS; s0 += 16) {
        float acc[16], dec[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) { acc[e] = 0.f; dec[e] = 1.f; }
        bool live = true;
#pragma unroll 1
        for (int c0 = first; REV ? c0 <= last : c0 >= last; c0 += step) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, wq, kColP + c0), v);
            if (live) {
#pragma unroll
                for (int ee = 0; ee < 16; ++ee) {
                    const int e = REV ? ee : 15 - ee;
                    const int j = c0 + e;
                    if ((REV ? j < row : j > row) || !live) continue;
                    float aj[16], wj[16];
                    tile_row16(gt, j, s0, aj);
                    tile_row16(sW, j, s0, wj);
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        if (REV && j > row) dec[u] *= aj[u];            // prod_{r=i+1..j}
                        acc[u] = fmaf(v[e] * wj[u], dec[u], acc[u]);
                        if (!REV) dec[u] *= aj[u];                      // prod_{r=j..i} for the next (earlier) row
                    }
                    if ((ee & 3) == 3) {
                        float top = 0.f;
#pragma unroll
                        for (int u = 0; u < 16; ++u) top = fmaxf(top, dec[u]);
                        live = top >= kDecayFloor;
                    }
                }
            }
            if (!__any_sync(0xffffffffu, live)) break;
        }
        float vi[16], vj[16];
        tmem_ld16(tmem_row_addr(tmem, wq, kColO + s0), vi);
        tmem_ld16(tmem_row_addr(tmem, wq, kColO + kM + s0), vj);       // (the state copy is a high/low pair)
#pragma unroll
        for (int e = 0; e < 16; ++e) vi[e] += vj[e];
        if (row < valid) {
#pragma unroll
            for (int e = 0; e < 16; e += 4) {
                float r[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    r[u] = fmaf(vi[e + u], __expf(REV ? gc[s0 + e + u] - gi[s0 - sb + e + u] : gi[s0 - sb + e + u]), acc[e + u]);
                *reinterpret_cast<float4*>(out_row + s0 + e) = make_float4(r[0], r[1], r[2], r[3]);
            }
        }
    }
}

// ======================================================================================
// value_side: out_i[s] = sum_{j<=i} <xq_i, xk_j> w_j[s] decay_ij[s]  + decayed (xq_i S)[s]
// ======================================================================================
template <bool REV, bool GENERAL>
__global__ void __launch_bounds__(kThreads, 1)
value_side_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                     const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapG,
                     const __grid_constant__ CUtensorMap mapO, ValueSideArgs a, const int* __restrict__ strong_flag,
                     int32_t* dev_status) {
    // Two kernels are launched back to back: this general one (with the strong-decay path) takes
    // the (batch, head) pairs flagged as having a strong-decay chunk, the pipelined one the others.
    if (strong_flag[blockIdx.x] == 0) return;
    extern __shared__ unsigned char smem_raw[];
    // align by pointer arithmetic (not an integer round trip) so accesses stay in the shared window
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sXq = smem;                       // 2 panels                                  (32 KB)
    unsigned char* sXk = sXq + 2 * kPanelB;          // 2 panels                                  (32 KB)
    unsigned char* sG = sXk + 2 * kPanelB;           // G tile fp32, [2 stages][2 panels]         (64 KB)
    unsigned char* sW = sG + 4 * kPanelB;            // weight tile fp32, 2 panels                (32 KB)
    unsigned char* sWa = sW + 2 * kPanelB;           // decayed weights, bf16 high part, MN-major B [128][64] (16 KB)
    unsigned char* sWb = sWa + kPanelB;              // ... their bf16 rounding residual (low part)           (16 KB)
    unsigned char* sSb = sWb + kPanelB;              // state copy, MN-major B [128][hi 64 | lo 64]  (32 KB)
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + 2 * kPanelB);
    // (the masked P never goes through shared memory: it is rewritten in place in tensor memory as a bf16
    // high/low pair and read from there as the A operand of the intra-chunk product)

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;
    const size_t strideM = (size_t)a.H * kM;
    float* obase = a.out + (size_t)slice * a.B * a.T * a.H * kM + ((size_t)b * a.T * a.H + h) * kM;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int it) { return (REV ? nchunks - 1 - it : it) * kCT; };

    if (warp == kComputeThreads / 32) {
        // =============================== issuing warp: TMA loads / stores and all MMAs
        if (elect_one()) {
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
            prefetch_tmap(&mapQ); prefetch_tmap(&mapK); prefetch_tmap(&mapW); prefetch_tmap(&mapG); prefetch_tmap(&mapO);
            load_g(0);
            load_w(0);
            load_x(0);
            constexpr uint32_t idescP = make_idesc(128, 128, false, false);  // xq xk^T
            constexpr uint32_t idescO = make_idesc(128, 2 * kM, false, true);  // xq x state copy [S_hi | S_lo] (MN-major B)
            // the high and the low part of the weights are two adjacent 64-column panels of ONE
            // MN-major B operand (N = 128): one product yields [.. W_hi | .. W_lo]
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);   // xk^T (MN-major A) x [W_hi | W_lo]
            constexpr uint32_t idescI = make_idesc(128, 2 * kM, false, true);  // masked P (tensor memory) x [W_hi | W_lo]
            // base descriptors of every operand (K step 0); advancing along K is one add each
            const uint64_t dQk = desc_kmajor(smem_u32(sXq), 0), dKk = desc_kmajor(smem_u32(sXk), 0);
            const uint64_t dKm = desc_mnmajor(smem_u32(sXk), 0, kPanelB), dWa = desc_mnmajor(smem_u32(sWa), 0, kPanelB);
            const uint64_t dS = desc_mnmajor(smem_u32(sSb), 0, kPanelB);
            // byte offset of K step kk: K-major operands walk 32 bytes inside a 64-column panel,
            // MN-major operands walk 16 rows (2048 bytes)
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            int n_mod = 0;      // moderate chunks so far (phases of bar_pm / bar_mma2)
            PROF_DECL
            for (int it = 0; it < nchunks && !ctl->abort; ++it) {
                const int t0 = chunk_t0(it);
                PROF_MARK();
                const unsigned char* gt = sG + (2 * (it & 1)) * kPanelB;
                // P = xq xk^T needs nothing but the d-sized tiles: it runs under the operand build
                WAIT_OR_ABORT(&ctl->bar_x, it & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kColP, desc_advance(dQk, kmaj(kk)), desc_advance(dKk, kmaj(kk)), idescP, kk > 0);
                mma_commit(&ctl->bar_p);
                // so does the inter-chunk product O = xq S: the state copy was written at the end
                // of the previous chunk
                WAIT_OR_ABORT(&ctl->bar_sb, it & 1);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kColO, desc_advance(dQk, kmaj(kk)), desc_advance(dS, mnmaj(kk)), idescO, kk > 0);
                PROF_MARK();
                if (it + 1 < nchunks) {
                    bulk_wait_read();     // the output rows staged in that G buffer one chunk ago have left
                    load_g(it + 1);
                }
                // U = xk^T W (high + low part of the weights) once the operand rows are there
                PROF_MARK();
                WAIT_OR_ABORT(&ctl->bar_ops, it & 1);
                tc_fence_after_sync();
                PROF_MARK();
                const bool moderate = !GENERAL || ctl->moderate[it & 1] != 0;
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kColU, desc_advance(dKm, mnmaj(kk)), desc_advance(dWa, mnmaj(kk)), idescU, kk > 0);
                mma_commit(&ctl->bar_mma1);
                PROF_MARK();
                if (moderate) {
                    WAIT_OR_ABORT(&ctl->bar_pm, n_mod & 1);
                    tc_fence_after_sync();
                    PROF_MARK();
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16_ta(tmem + kColO2, tmem + kColP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dWa, mnmaj(kk)),
                                    idescI, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)      // ... and the rounding residual of the masked P
                        mma_bf16_ta(tmem + kColO2, tmem + kColP + 64 * (kk >> 2) + 32 + 8 * (kk & 3),
                                    desc_advance(dWa, mnmaj(kk)), idescI, true);
                    mma_commit(&ctl->bar_mma2);
                    PROF_MARK();
                }
                // the d-sized tiles are consumed once U and O are done: request the next chunk's
                WAIT_OR_ABORT(&ctl->bar_mma1, it & 1);
                PROF_MARK();
                if (it + 1 < nchunks) load_x(it + 1);
                if (moderate) {
                    // the masked P is consumed: its buffer takes the next chunk's weight tile
                    WAIT_OR_ABORT(&ctl->bar_mma2, n_mod & 1);
                    ++n_mod;
                    if (it + 1 < nchunks) load_w(it + 1);
                }
                PROF_MARK();
                WAIT_OR_ABORT(&ctl->bar_out, it & 1);
                PROF_MARK();
                PROF_DUMP("value_side issue");
                if (ctl->abort) break;
                if (moderate) {
                    tma_store_5d(&mapO, gt, 0, h, t0, b, slice);
                    tma_store_5d(&mapO, gt + kPanelB, 32, h, t0, b, slice);
                    bulk_commit();
                } else if (it + 1 < nchunks) {
                    load_w(it + 1);       // a strong-decay chunk read the weight tile until now
                }
            }
            bulk_wait_read();      // staged output rows must have left before shared memory goes away
        }
    } else {
        // =============================== compute threads
        // state slice: S[c = row][s], slots sb .. sb+31
        float S[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) S[s] = (a.S0 && d0 + row < a.D) ? a.S0[((size_t)bh * kM + sb + s) * a.D + d0 + row] : 0.f;

        // bf16 copy of the state (value + rounding residual) for the first chunk's inter-chunk product
        store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);
        fence_async_smem();
        compute_sync();
        if (tid == 0) mbar_arrive(&ctl->bar_sb);

        int n_mod = 0;
        PROF_DECL
        for (int it = 0; it < nchunks; ++it) {
            const int t0 = chunk_t0(it);
            const int valid = min(kCT, a.T - t0);
            PROF_MARK();
            const unsigned char* gt = sG + (2 * (it & 1)) * kPanelB;
            WAIT_OR_ABORT(&ctl->bar_g[it & 1], (it >> 1) & 1);
            WAIT_OR_ABORT(&ctl->bar_w, it & 1);
            PROF_MARK();
            const bool moderate = publish_chunk_decay(ctl, tid, gt, valid - 1) || !GENERAL;
            if (ctl->abort) break;
            PROF_MARK();

            // ---- this token's slot rows -> operand rows (rows past the end: zero weights)
            const int grow = min(row, valid - 1);
            const float strong = moderate ? 0.f : 1.f;      // adds G_C to the exponent of a strong-decay chunk
#pragma unroll
            for (int s0 = sb; s0 < sb + kHS; s0 += 8) {
                float g[8], w[8], wd[8];
                tile_row8(gt, grow, s0, g);
                tile_row8(sW, row, s0, w);
                // ONE set of decayed weights serves the intra-chunk product and the state update,
                // branch-free over the elements (a branch per element would serialise the exps):
                //   reverse           : w exp(G)
                //   forward, moderate : w exp(-G); the state update gets its exp(G_C) afterwards,
                //                       S <- exp(G_C) (S + xk^T W)
                //   forward, strong   : w exp(G_C - G) (state update only; no intra product)
                // They are stored as a bf16 pair (value + rounding residual): the weights multiply
                // sums that cancel in the gate gradient, where a plain bf16 rounding is too coarse.
                const float4 gc0 = *reinterpret_cast<const float4*>(&ctl->gc[s0]);
                const float4 gc1 = *reinterpret_cast<const float4*>(&ctl->gc[s0 + 4]);
                const float gcv[8] = {gc0.x, gc0.y, gc0.z, gc0.w, gc1.x, gc1.y, gc1.z, gc1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) wd[e] = w[e] * __expf(REV ? g[e] : fmaf(strong, gcv[e], -g[e]));
                store_chunk_split(sWa, sWb, row, s0 >> 3, wd);
            }
            fence_async_smem();
            if (tid == 0) ctl->moderate[it & 1] = moderate;
            compute_sync();                     // every row is written and the weight tile is read
            if (tid == 0) mbar_arrive(&ctl->bar_ops);
            PROF_MARK();

            WAIT_OR_ABORT(&ctl->bar_p, it & 1);
            tc_fence_after_sync();
            PROF_MARK();
            if (moderate) {
                mask_row_in_tmem<REV, true>(tmem, wq, row, half, kColP);
                tc_fence_before_sync();
                compute_sync();
                if (tid == 0) mbar_arrive(&ctl->bar_pm);
            } else if constexpr (GENERAL) {
                // Strong decay: the intra-chunk term with explicit exponent differences on the CUDA
                // cores (only the general variant of the kernel carries this path).
                WAIT_OR_ABORT(&ctl->bar_mma1, it & 1);    // the inter-chunk product
                tc_fence_after_sync();
                if (!a.state_only) {
                    float gi[kHS];
                    gates_in_place(const_cast<unsigned char*>(gt), row, half, sb, valid, gi);
                    value_side_explicit_rows<REV>(gt, sW, ctl->gc, gi, tmem, wq, row, sb, valid,
                                                  obase + (size_t)(t0 + row) * strideM);
                }
            }

            // ---- state update from U: S <- S exp(G_C) + U  (forward moderate chunk: exp(G_C) (S + U))
            PROF_MARK();
            WAIT_OR_ABORT(&ctl->bar_mma1, it & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kColU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, kColU + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&ctl->egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float u = v[e + t] + vl[e + t];
                        S[e + t] = (!REV && moderate) ? (S[e + t] + u) * ecv[t] : fmaf(S[e + t], ecv[t], u);
                    }
                }
            }
            // its bf16 copy feeds the next chunk's inter-chunk product (issued as soon as the next
            // tiles are there); the product of this chunk that read the old copy is complete
            store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);

            // ---- output rows of a moderate chunk: exp(+-G_i) * (inter + intra)
            PROF_MARK();
            if (moderate) {
                WAIT_OR_ABORT(&ctl->bar_mma2, n_mod & 1);
                ++n_mod;
                tc_fence_after_sync();
                PROF_MARK();
                // the scaled rows replace this chunk's G rows in place (each thread reads and rewrites
                // only its own 32 slots) and leave as one tiled store, clipped at the sequence end
                float vo[kHS], vi[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kColO2 + sb), vo);
                tmem_ld32(tmem_row_addr(tmem, wq, kColO2 + kM + sb), vi);
#pragma unroll
                for (int e = 0; e < kHS; ++e) vo[e] += vi[e];          // high + low weight parts
                {
                    float vj[kHS];
                    tmem_ld32(tmem_row_addr(tmem, wq, kColO + sb), vi);
                    tmem_ld32(tmem_row_addr(tmem, wq, kColO + kM + sb), vj);
#pragma unroll
                    for (int e = 0; e < kHS; ++e) vi[e] += vj[e];      // high + low state parts
                }
                // forward: exp(G) (inter + intra); reverse: exp(-G) (exp(G_C) inter + intra)
#pragma unroll
                for (int e = 0; e < kHS; ++e) vo[e] = REV ? fmaf(vi[e], ctl->egc[sb + e], vo[e]) : vo[e] + vi[e];
                if (row < valid) {
                    unsigned char* panel = const_cast<unsigned char*>(gt) + half * kPanelB;
#pragma unroll
                    for (int c = 0; c < kHS / 4; ++c) {
                        float4* cell = reinterpret_cast<float4*>(panel + swz128(row, c));
                        const float4 g = *cell;
                        *cell = make_float4(vo[4 * c] * __expf(REV ? -g.x : g.x), vo[4 * c + 1] * __expf(REV ? -g.y : g.y),
                                            vo[4 * c + 2] * __expf(REV ? -g.z : g.z), vo[4 * c + 3] * __expf(REV ? -g.w : g.w));
                    }
                }
            }
            fence_async_smem();
            tc_fence_before_sync();
            compute_sync();                 // rows staged; gc / egc and the accumulators may be reused
            if (tid == 0) {
                mbar_arrive(&ctl->bar_sb);
                mbar_arrive(&ctl->bar_out);
            }
            PROF_MARK();
            PROF_DUMP("value_side compute");
            if (ctl->abort) break;
        }
        if (!ctl->abort && a.Send && d0 + row < a.D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) a.Send[((size_t)bh * kM + sb + s) * a.D + d0 + row] = S[s];
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        // bounded grace period for tile copies still in flight before shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// Strong-decay chunk of key_side: A_ij = sum_s uq_i[s] uk_j[s] prod a_r[s] on the kept triangle, by
// the same walk: the thread carries uq_i[s] times the running decay product for its 64 slots, one
// multiplication per step and slot, and stops once every product is below 2^-40.  Written into tensor
// memory as the bf16 high/low operand rows of the masked matrix, in the layout mask_row_in_tmem leaves
// (this thread's 64 columns: 32 packed high parts, then 32 packed residuals).  `sG` is replaced by the
// per-step gates on the way.
template <bool REV>
__device__ __forceinline__ void key_side_explicit_rows(unsigned char* sG, const unsigned char* sUq,
                                                    const unsigned char* sUk, uint32_t tmem, int wq, int row, int half,
                                                    int sb, int grow, int valid) {
    // thread (row, half) fills columns j in [64 half, 64 half + 63]; its walk starts at the column nearest to
    // the diagonal: j0 = min(row, 64 half + 63) forward, max(row, 64 half) reverse
    const int jlo = 64 * half, jhi = jlo + 63;
    const bool any = REV ? row <= jhi : row >= jlo;
    const int j0 = REV ? max(row, jlo) : min(row, jhi);
    float qd[kM];
    {
        // uq_i[s] exp(G_i[s] - G_j0[s]) (reverse: G_j0 - G_i): the product of the gates between the row and the
        // start of the walk, 64 exponentials once (zero exponent when the walk starts on the diagonal)
        const int g0 = min(j0, valid - 1);
#pragma unroll
        for (int s0 = 0; s0 < kM; s0 += 8) {
            float g[8], gj[8], uq[8];
            tile_row8(sG, grow, s0, g);
            tile_row8(sG, g0, s0, gj);
            tile_row8(sUq, row, s0, uq);
#pragma unroll
            for (int e = 0; e < 8; ++e) qd[s0 + e] = uq[e] * __expf(fminf(REV ? gj[e] - g[e] : g[e] - gj[e], 0.f));
        }
    }
    float gi[kHS];
    gates_in_place(sG, row, half, sb, valid, gi);       // (its barriers also cover: every uq row is in registers)
    (void)gi;
    float x[64];
#pragma unroll
    for (int e = 0; e < 64; ++e) x[e] = 0.f;
    if (any) {
        float start = 0.f;
#pragma unroll
        for (int s = 0; s < kM; ++s) start = fmaxf(start, fabsf(qd[s]));
        const float floor_ = start * kDecayFloor;
#pragma unroll 1
        for (int j = j0; REV ? j <= jhi : j >= jlo; j += REV ? 1 : -1) {
            // reverse: the product up to column j includes a_j (prod_{r=i+1..j}); j0 itself is already covered
            float acc = 0.f;
#pragma unroll
            for (int s0 = 0; s0 < kM; s0 += 16) {
                float aj[16], uk[16];
                tile_row16(sG, j, s0, aj);
                tile_row16(sUk, j, s0, uk);
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    if (REV && j > j0) qd[s0 + u] *= aj[u];
                    acc = fmaf(qd[s0 + u], uk[u], acc);
                    if (!REV) qd[s0 + u] *= aj[u];
                }
            }
            x[j - jlo] = acc;
            if (((j - j0) & 3) == 0) {        // every fourth step: has every product fallen below 2^-40 of the start?
                float top = 0.f;
#pragma unroll
                for (int s = 0; s < kM; ++s) top = fmaxf(top, fabsf(qd[s]));
                if (top <= floor_) break;
            }
        }
    }
    const int base = kColP + 64 * half;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float x0 = x[32 * q + 2 * e], x1 = x[32 * q + 2 * e + 1];
            hi[e] = pack_bf16(x0, x1);
            const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&hi[e]);
            lo[e] = pack_bf16(x0 - __bfloat162float(h.x), x1 - __bfloat162float(h.y));
        }
        tmem_st16(tmem_row_addr(tmem, wq, base + 16 * q), hi);
        tmem_st16(tmem_row_addr(tmem, wq, base + 32 + 16 * q), lo);
    }
    tmem_st_wait();
}

// ======================================================================================
// key_side: out_i = (uq_i * qscale_i) S + sum_j A_ij xv_j,  A_ij = sum_s uq_i[s] uk_j[s] decay_ij[s]
// ======================================================================================
template <bool REV, bool GENERAL>
__global__ void __launch_bounds__(kThreads, 1)
key_side_tc_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapUq,
                   const __grid_constant__ CUtensorMap mapUk, const __grid_constant__ CUtensorMap mapG,
                   const __grid_constant__ CUtensorMap mapO, KeySideArgs a, const int* __restrict__ strong_flag,
                   int32_t* dev_status) {
    // (see value_side_tc_kernel: the flagged (batch, head) pairs only)
    if (strong_flag[blockIdx.x] == 0) return;
    extern __shared__ unsigned char smem_raw[];
    // align by pointer arithmetic (not an integer round trip) so accesses stay in the shared window
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sXv = smem;                       // 2 panels                                   (32 KB)
    unsigned char* sUk = sXv + 2 * kPanelB;          // uk tile fp32, 2 panels                     (32 KB)
    unsigned char* sG = sUk + 2 * kPanelB;           // G tile fp32, 2 panels                      (32 KB)
    unsigned char* sUq = sG + 2 * kPanelB;           // uq tile fp32, 2 panels                     (32 KB)
    unsigned char* sQt = sUq + 2 * kPanelB;          // decayed uq, K-major A [128][64]: value, rounding residual (32 KB)
                                                     //   ... they also stage the output rows
    unsigned char* sKt = sQt + 2 * kPanelB;          // decayed uk, K-major / MN-major B [128][64]: value, residual (32 KB)
    unsigned char* sSb = sKt + 2 * kPanelB;          // state copy, K-major B [128 (channel)][64]: value, residual  (32 KB)
    Ctl* ctl = reinterpret_cast<Ctl*>(sSb + 2 * kPanelB);
    // (the masked A never goes through shared memory: it is rewritten in place in tensor memory as a bf16
    // high/low pair and read from there as the A operand of the intra-chunk product)

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;

    ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int it) { return (REV ? nchunks - 1 - it : it) * kCT; };

    if (warp == kComputeThreads / 32) {
        // =============================== issuing warp: TMA loads / stores and all MMAs
        if (elect_one()) {
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
            prefetch_tmap(&mapV); prefetch_tmap(&mapUq); prefetch_tmap(&mapUk); prefetch_tmap(&mapG); prefetch_tmap(&mapO);
            load_kg(0);
            load_q(0);
            load_v(0);
            constexpr uint32_t idescA = make_idesc(128, 128, false, false);   // Q~ K~^T
            constexpr uint32_t idescO = make_idesc(128, kDST, false, false);  // Q- x state copy (K-major B)
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);  // xv^T (MN-major A) x [K-_hi | K-_lo] (MN-major B)
            constexpr uint32_t idescV = make_idesc(128, kDST, false, true);   // masked A (tensor memory) x xv (MN-major B)
            // base descriptors of every operand (K step 0); advancing along K is one add each
            const uint64_t dV = desc_mnmajor(smem_u32(sXv), 0, kPanelB);
            const uint64_t dQt = desc_kmajor(smem_u32(sQt), 0), dKt = desc_kmajor(smem_u32(sKt), 0);
            const uint64_t dQl = desc_kmajor(smem_u32(sQt + kPanelB), 0), dKl = desc_kmajor(smem_u32(sKt + kPanelB), 0);
            const uint64_t dS = desc_kmajor(smem_u32(sSb), 0), dSl = desc_kmajor(smem_u32(sSb + kPanelB), 0);
            // the decayed uk read MN-major, its value and residual as one N = 128 operand
            const uint64_t dKtm = desc_mnmajor(smem_u32(sKt), 0, kPanelB);
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            for (int it = 0; it < nchunks && !ctl->abort; ++it) {
                const int t0 = chunk_t0(it);
                WAIT_OR_ABORT(&ctl->bar_ops, it & 1);
                WAIT_OR_ABORT(&ctl->bar_x, it & 1);
                tc_fence_after_sync();
                const bool moderate = !GENERAL || ctl->moderate[it & 1] != 0;
                if (moderate) {
                    // A = Q- K-^T with both factors as bf16 high/low pairs (the low x low term is dropped)
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kColP, desc_advance(dQt, kmaj(kk)), desc_advance(dKt, kmaj(kk)), idescA, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kColP, desc_advance(dQl, kmaj(kk)), desc_advance(dKt, kmaj(kk)), idescA, true);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kColP, desc_advance(dQt, kmaj(kk)), desc_advance(dKl, kmaj(kk)), idescA, true);
                    mma_commit(&ctl->bar_p);     // the state products below run under the read-out of A
                }
                // the decayed uk is read K-major by the intra product and MN-major by the state update
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kColU, desc_advance(dV, mnmaj(kk)), desc_advance(dKtm, mnmaj(kk)), idescU, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kColO, desc_advance(dQt, kmaj(kk)), desc_advance(dS, kmaj(kk)), idescO, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kColO, desc_advance(dQl, kmaj(kk)), desc_advance(dS, kmaj(kk)), idescO, true);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kColO, desc_advance(dQt, kmaj(kk)), desc_advance(dSl, kmaj(kk)), idescO, true);
                mma_commit(&ctl->bar_mma1);
                // a moderate chunk is done with the uk and G tiles: request the next chunk's
                if (moderate && it + 1 < nchunks) load_kg(it + 1);
                WAIT_OR_ABORT(&ctl->bar_pm, it & 1);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + kColO, tmem + kColP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)), idescV,
                                true);
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)      // ... and the rounding residual of A
                    mma_bf16_ta(tmem + kColO, tmem + kColP + 64 * (kk >> 2) + 32 + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)),
                                idescV, true);
                mma_commit(&ctl->bar_mma2);
                if (!moderate && it + 1 < nchunks) load_kg(it + 1);
                // every product of the chunk is done: the uq and xv tiles may be refilled
                WAIT_OR_ABORT(&ctl->bar_mma2, it & 1);
                if (it + 1 < nchunks) {
                    load_q(it + 1);
                    load_v(it + 1);
                }
                // the output rows are staged over the intra operands: store them, then tell the
                // compute threads that those buffers may be rewritten
                WAIT_OR_ABORT(&ctl->bar_out, it & 1);
                if (ctl->abort) break;
                tma_store_4d(&mapO, sQt, d0, h, t0, b);
                if (d0 + 64 < a.D) tma_store_4d(&mapO, sQt + kPanelB, d0 + 64, h, t0, b);
                bulk_commit();
                bulk_wait_read();
                mbar_arrive(&ctl->bar_sb);
            }
        }
    } else {
        // =============================== compute threads
        // state slice, transposed: S[c = row][s], slots sb .. sb+31
        float S[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) S[s] = (a.S0 && d0 + row < a.D) ? a.S0[((size_t)bh * kM + sb + s) * a.D + d0 + row] : 0.f;

        int n_mod = 0;     // moderate chunks so far (phases of bar_p)
        PROF_DECL
        for (int it = 0; it < nchunks; ++it) {
            const int t0 = chunk_t0(it);
            const int valid = min(kCT, a.T - t0);
            (void)t0;
            PROF_MARK();
            WAIT_OR_ABORT(&ctl->bar_g[0], it & 1);
            PROF_MARK();
            const bool moderate = publish_chunk_decay(ctl, tid, sG, valid - 1) || !GENERAL;
            if (ctl->abort) break;
            PROF_MARK();

            const int grow = min(row, valid - 1);
            // the previous chunk's output rows must have left sQt / sKt before they are rewritten
            if (it > 0) WAIT_OR_ABORT(&ctl->bar_sb, (it - 1) & 1);
            // key side first: it needs the uk and G tiles only; the uq tile (which shares its buffer
            // with the previous chunk's masked A) arrives last
#pragma unroll
            for (int s0 = sb; s0 < sb + kHS; s0 += 8) {
                float g[8], uk[8], kd[8], gcv[8];
                tile_row8(sG, grow, s0, g);
                tile_row8(sUk, row, s0, uk);
                // ONE decayed copy of uk serves the intra product and the state update, with one
                // exponential per element (the SFU is the scarce unit here) and no branch:
                //   reverse           : uk exp(G)
                //   forward, moderate : uk exp(-G); the state update gets its exp(G_C) afterwards,
                //                       S <- exp(G_C) (S + xv^T K)
                //   forward, strong   : uk exp(G_C - G) (state update only)
#pragma unroll
                for (int e = 0; e < 8; ++e) gcv[e] = 0.f;
                if (!REV && !moderate) tile_free_row8(&ctl->gc[s0], gcv);
#pragma unroll
                for (int e = 0; e < 8; ++e) kd[e] = uk[e] * __expf(REV ? g[e] : gcv[e] - g[e]);
                store_chunk_split(sKt, sKt + kPanelB, row, s0 >> 3, kd);
            }
            PROF_MARK();
            WAIT_OR_ABORT(&ctl->bar_w, it & 1);
            PROF_MARK();
#pragma unroll
            for (int s0 = sb; s0 < sb + kHS; s0 += 8) {
                float g[8], uq[8], qd[8], gcv[8];
                tile_row8(sG, grow, s0, g);
                tile_row8(sUq, row, s0, uq);
                // likewise ONE decayed copy of uq:
                //   forward           : uq exp(G)
                //   reverse, moderate : uq exp(-G); the inter-chunk product gets its exp(G_C) through
                //                       the state copy, which is scaled per slot
                //   reverse, strong   : uq exp(G_C - G)
#pragma unroll
                for (int e = 0; e < 8; ++e) gcv[e] = 0.f;
                if (REV && !moderate) tile_free_row8(&ctl->gc[s0], gcv);
#pragma unroll
                for (int e = 0; e < 8; ++e) qd[e] = uq[e] * __expf(REV ? gcv[e] - g[e] : g[e]);
                store_chunk_split(sQt, sQt + kPanelB, row, s0 >> 3, qd);
            }
            if (REV && moderate) store_state_row_split<true>(sSb, sSb + kPanelB, row, sb, S, ctl->egc);
            else store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);
            fence_async_smem();
            if (tid == 0) ctl->moderate[it & 1] = moderate;
            compute_sync();
            if (tid == 0) mbar_arrive(&ctl->bar_ops);
            PROF_MARK();

            if (moderate) {
                WAIT_OR_ABORT(&ctl->bar_p, n_mod & 1);
                ++n_mod;
                tc_fence_after_sync();
                PROF_MARK();
                mask_row_in_tmem<REV, true>(tmem, wq, row, half, kColP);
            } else if constexpr (GENERAL) {
                // Strong decay: A_ij by the walk over the per-step gates (only the general variant of the
                // kernel carries this path).
                if (!a.state_only) key_side_explicit_rows<REV>(sG, sUq, sUk, tmem, wq, row, half, sb, grow, valid);
            }
            tc_fence_before_sync();
            compute_sync();
            if (tid == 0) mbar_arrive(&ctl->bar_pm);
            PROF_MARK();

            // ---- state update from U^T: S <- exp(G_C) S + U^T  (forward moderate chunk: exp(G_C) (S + U^T))
            WAIT_OR_ABORT(&ctl->bar_mma1, it & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kColU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, kColU + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; ++e) v[e] += vl[e];          // value + residual of the decayed uk
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&ctl->egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        S[e + t] = (!REV && moderate) ? (S[e + t] + v[e + t]) * ecv[t] : fmaf(S[e + t], ecv[t], v[e + t]);
                }
            }

            // ---- output rows -> bf16, staged over the intra operands (consumed since bar_p), stored
            // by the issuing warp, clipped at the sequence end
            PROF_MARK();
            WAIT_OR_ABORT(&ctl->bar_mma2, it & 1);
            tc_fence_after_sync();
            PROF_MARK();
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                float v[32];
                tmem_ld32(tmem_row_addr(tmem, wq, kColO + 64 * half + c0), v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float x[8] = {v[8 * c], v[8 * c + 1], v[8 * c + 2], v[8 * c + 3],
                                        v[8 * c + 4], v[8 * c + 5], v[8 * c + 6], v[8 * c + 7]};
                    store_chunk(sQt + half * kPanelB, row, (c0 >> 3) + c, x);
                }
            }
            fence_async_smem();
            tc_fence_before_sync();
            compute_sync();
            if (tid == 0) mbar_arrive(&ctl->bar_out);
            PROF_MARK();
            PROF_DUMP("key_side compute");
            if (ctl->abort) break;
        }
        if (!ctl->abort && a.Send && d0 + row < a.D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) a.Send[((size_t)bh * kM + sb + s) * a.D + d0 + row] = S[s];
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

constexpr size_t kSmemValueSide = 1024 + 14 * kPanelB + sizeof(Ctl);
constexpr size_t kSmemKeySide = 1024 + 14 * kPanelB + sizeof(Ctl);

}  // namespace

// The general kernel of a scan runs on a side stream of the calling host thread, beside the
// pipelined kernel on the caller's stream (they write disjoint (batch, head) pairs): in the
// usual case that no pair is flagged, its launch and the exit of its CTAs then cost the
// caller's stream nothing.  fork: the side stream waits for what precedes on the caller's
// stream; join: the caller's stream waits for the general kernel.
namespace {
constexpr int kMaxLaneDevices = 64;
thread_local SideLane g_side_lanes[kMaxLaneDevices];
}  // namespace

cudaError_t side_lane(SideLane** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxLaneDevices) return cudaErrorInvalidDevice;
    SideLane& l = g_side_lanes[dev];
    if (l.stream == nullptr) {
        e = cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming);
        if (e != cudaSuccess) return e;
    }
    *out = &l;
    return cudaSuccess;
}

// destroys the calling thread's side stream and events on the current device (created again on demand)
cudaError_t side_lane_release() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxLaneDevices) return cudaErrorInvalidDevice;
    SideLane& l = g_side_lanes[dev];
    if (l.stream != nullptr) {
        cudaStreamDestroy(l.stream);
        if (l.fork != nullptr) cudaEventDestroy(l.fork);
        if (l.join != nullptr) cudaEventDestroy(l.join);
        l = SideLane{};
    }
    return cudaSuccess;
}

// Head dimensions the tensor-core kernels serve: multiples of the 128-wide slice, and 64 (half a
// slice: the tile copies zero-fill the channels beyond the head, stores are clipped).
bool tc_dim_ok(int D) { return D == 64 || (D > 0 && D % kDST == 0); }
bool tc_supported(int d_k, int d_v, int M) {
    return M == kM && tc_dim_ok(d_k) && tc_dim_ok(d_v);
}
int tc_value_side_slices(int D) { return (D + kDST - 1) / kDST; }
int tc_chunk() { return kCT; }

cudaError_t launch_value_side_tc(const ValueSideArgs& a, int M, int reverse, const int* strong_flag,
                                 cudaStream_t st, int32_t* dev_status) {
    if (M != kM || !tc_dim_ok(a.D) || strong_flag == nullptr) return cudaErrorNotSupported;
    CUtensorMap mq, mk, mw, mg, mo;
    cudaError_t e = make_tensor_map_bthd(&mq, a.xq, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_sliced(&mo, a.out, tc_value_side_slices(a.D), a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mk, a.xk, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, a.w, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
#define GSA_LAUNCH_VS(REVV, FLAGS)                                                                       \
    e = prepare(value_side_tc_kernel<REVV, true>, kSmemValueSide);                                       \
    if (e != cudaSuccess) return e;                                                                      \
    value_side_tc_kernel<REVV, true><<<grid, kThreads, kSmemValueSide, side->stream>>>(mq, mk, mw, mg, mo, a, FLAGS, dev_status)
    // the pipelined kernel for the (batch, head) pairs whose chunks all decay moderately, this
    // general one for the others; each CTA of the kernel that is not its own returns at once
    if (a.wd == nullptr) return cudaErrorInvalidValue;
    SideLane* side = nullptr;
    e = side_lane(&side);
    if (e == cudaSuccess) e = cudaEventRecord(side->fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (e == cudaSuccess) e = launch_value_side_lean(a, reverse, strong_flag, st, dev_status);
    if (e != cudaSuccess) return e;
    if (reverse) { GSA_LAUNCH_VS(true, strong_flag); }
    else { GSA_LAUNCH_VS(false, strong_flag); }
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaEventRecord(side->join, side->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
    if (e != cudaSuccess) return e;
#undef GSA_LAUNCH_VS
    return cudaGetLastError();
}

cudaError_t launch_value_side_general(const ValueSideArgs& a, int M, int reverse, const int* strong_flag,
                                      cudaStream_t st, int32_t* dev_status) {
    if (M != kM || !tc_dim_ok(a.D) || strong_flag == nullptr) return cudaErrorNotSupported;
    CUtensorMap mq, mk, mw, mg, mo;
    cudaError_t e = make_tensor_map_bthd(&mq, a.xq, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_sliced(&mo, a.out, tc_value_side_slices(a.D), a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mk, a.xk, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, a.w, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
    if (reverse) {
        e = prepare(value_side_tc_kernel<true, true>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<true, true><<<grid, kThreads, kSmemValueSide, st>>>(mq, mk, mw, mg, mo, a, strong_flag, dev_status);
    } else {
        e = prepare(value_side_tc_kernel<false, true>, kSmemValueSide);
        if (e != cudaSuccess) return e;
        value_side_tc_kernel<false, true><<<grid, kThreads, kSmemValueSide, st>>>(mq, mk, mw, mg, mo, a, strong_flag, dev_status);
    }
    return cudaGetLastError();
}

cudaError_t launch_key_side_general(const KeySideArgs& a, int M, int reverse, const int* strong_flag,
                                    cudaStream_t st, int32_t* dev_status) {
    if (M != kM || !tc_dim_ok(a.D) || strong_flag == nullptr) return cudaErrorNotSupported;
    CUtensorMap mv, muq, muk, mg, mo;
    cudaError_t e = make_tensor_map_bthd(&mv, a.xv, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mo, a.out, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muq, a.uq, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muk, a.uk, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
    if (reverse) {
        e = prepare(key_side_tc_kernel<true, true>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<true, true><<<grid, kThreads, kSmemKeySide, st>>>(mv, muq, muk, mg, mo, a, strong_flag, dev_status);
    } else {
        e = prepare(key_side_tc_kernel<false, true>, kSmemKeySide);
        if (e != cudaSuccess) return e;
        key_side_tc_kernel<false, true><<<grid, kThreads, kSmemKeySide, st>>>(mv, muq, muk, mg, mo, a, strong_flag, dev_status);
    }
    return cudaGetLastError();
}

cudaError_t launch_key_side_tc(const KeySideArgs& a, int M, int reverse, const int* strong_flag,
                               cudaStream_t st, int32_t* dev_status) {
    if (M != kM || !tc_dim_ok(a.D) || strong_flag == nullptr) return cudaErrorNotSupported;
    CUtensorMap mv, muq, muk, mg, mo;
    cudaError_t e = make_tensor_map_bthd(&mv, a.xv, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mo, a.out, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muq, a.uq, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muk, a.uk, a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mg, a.G, a.B, a.T, a.H, kM, kCT, 4);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
#define GSA_LAUNCH_KS(REVV, FLAGS)                                                                       \
    e = prepare(key_side_tc_kernel<REVV, true>, kSmemKeySide);                                           \
    if (e != cudaSuccess) return e;                                                                      \
    key_side_tc_kernel<REVV, true><<<grid, kThreads, kSmemKeySide, side->stream>>>(mv, muq, muk, mg, mo, a, FLAGS, dev_status)
    if (a.uq_d == nullptr || a.uk_d == nullptr) return cudaErrorInvalidValue;
    SideLane* side = nullptr;
    e = side_lane(&side);
    if (e == cudaSuccess) e = cudaEventRecord(side->fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (e == cudaSuccess) e = launch_key_side_lean(a, reverse, strong_flag, st, dev_status);
    if (e != cudaSuccess) return e;
    if (reverse) { GSA_LAUNCH_KS(true, strong_flag); }
    else { GSA_LAUNCH_KS(false, strong_flag); }
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaEventRecord(side->join, side->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
    if (e != cudaSuccess) return e;
#undef GSA_LAUNCH_KS
    return cudaGetLastError();
}

}  // namespace gsa
