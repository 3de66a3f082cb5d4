// The time-reversed scans of the backward come in pairs that share everything but their outputs
// (App. B: the gradients of a GLA pass w.r.t. its values and w.r.t. the weights that multiply them
// both carry the state gradient):
//     dv   = key_side(I, p, dO)  reversed      dI^v = value_side(v, dO, p)  reversed      state dV~
//     dk   = key_side(I, dz, q)  reversed      dI^k = value_side(k, q, dz)  reversed      state dK~
// Both members of a pair read the same d-sized tile X that enters the state (dO; q), the same decayed
// slot rows W (p exp(G); dz exp(G)) and run the same recurrence  S <- exp(G_C) S + X^T W.  This kernel
// runs a pair as ONE scan: X, W and the state are loaded / updated once, the second d-sized tile Y
// (v; k) and the decayed rows Q = I exp(-G) feed the two outputs
//     value-side:  out_v[i][s] = sum_{j>=i} <y_i, x_j> W_j[s]  +  exp(G_C)[s] (y_i S)[s]     (fp32 partial sums per slice)
//     key-side:    out_k[i]    = sum_{j>=i} <Q_i, W_j> x_j     +  Q_i (exp(G_C) S)           (io dtype)
// (row factors left out of out_v as in the single value_side kernel, see PendingDecay).  Per chunk
// that is seven products on one tensor pipe: while the compute threads mask one first product, the
// pipe works on the other member's.  Compared with two single scans the pair reads X, W and G once
// instead of twice (a scan is bound by the rate at which its SM pulls tiles) and does not repeat the
// state product.
//
// Only for (batch, head) pairs without a strong-decay chunk; the flagged ones take the two general
// kernels.  Geometry, operand pairs (bf16 value + rounding residual) and bounded waits are those
// of the pipelined single kernels.
#include "chunk_tc_shared.cuh"

namespace gsa {
namespace {
using namespace tc;
using namespace tcchunk;

constexpr int kPairThreads = kComputeThreads + 64;   // 8 compute warps, an MMA lane, a copy lane
constexpr int kMmaWarp = kComputeThreads / 32, kCopyWarp = kMmaWarp + 1;

struct PairCtl {
    // filled by TMA
    uint64_t bar_x[2];     // X tile, two stages
    uint64_t bar_w[2];     // decayed rows W [hi | lo], two stages
    uint64_t bar_yq;       // Y tile and decayed rows Q [hi | lo], one stage
    // signalled by tcgen05.commit
    uint64_t bar_p;        // P = Y X^T of a chunk
    uint64_t bar_a;        // A = Q W^T of a chunk
    uint64_t bar_yqfree;   // the two inter-chunk products (for the copy lane: Y and Q are consumed)
    uint64_t bar_mma1;     // state product U
    uint64_t bar_v4;       // value-side output accumulator complete
    uint64_t bar_k4;       // key-side output accumulator complete
    // signalled by the compute threads (one arrival after their barrier)
    uint64_t bar_pm;       // masked P rows are in tensor memory
    uint64_t bar_am;       // masked A rows are in tensor memory
    uint64_t bar_sb;       // state copy for the next chunk is written, the U accumulator is free
    uint64_t bar_outv[2];  // (by chunk parity) value-side rows staged, their accumulator free
    uint64_t bar_outk[2];  // (by chunk parity) key-side rows staged, their accumulator free
    uint32_t tmem_slot;
    volatile int abort;
    alignas(16) float egc[2][kM];   // exp(G of the chunk's last valid row), by chunk parity
};

// A wait that expires flags the CTA; once flagged, later waits return at once (see the single kernels).
#define PAIR_WAIT(bar, parity)                                              \
    do {                                                                    \
        if (!ctl->abort && !mbar_wait(bar, parity)) ctl->abort = 1;         \
    } while (0)

// accumulator columns: the two first products are masked in place; the state product and the
// value-side output accumulate their high and low operand parts into 64 columns each
constexpr int kPcP = 0, kPcA = 128, kPcO2 = 256, kPcU = 384, kPcOI = 448;

template <bool PAIRS>
__global__ void __launch_bounds__(kPairThreads, 1)
rev_pair_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapQ,
                const __grid_constant__ CUtensorMap mapOv, const __grid_constant__ CUtensorMap mapOk,
                const float* __restrict__ G, const float* __restrict__ S0, float* __restrict__ Send, int T, int H,
                int D, const int* __restrict__ strong_flag, int32_t* dev_status) {
    if (strong_flag[blockIdx.x] != 0) return;       // the general kernels take this (batch, head)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sX = smem;                        // X tile, 2 stages of 2 panels (64 KB); a stage also holds the
                                                     //   chunk's key-side rows once the tile is consumed
    unsigned char* sW = sX + 4 * kPanelB;            // W [hi 64 | lo 64], 2 stages of 2 panels (64 KB); a stage also
                                                     //   holds the chunk's value-side rows (fp32, 2 panels of 32 slots)
    unsigned char* sY = sW + 4 * kPanelB;            // Y tile, 2 panels (32 KB)
    unsigned char* sQ = sY + 2 * kPanelB;            // Q [hi | lo], 2 panels (32 KB)
    unsigned char* sSb = sQ + 2 * kPanelB;           // state copy exp(G_C) S as [128 (channel)][hi 64 | lo 64] (32 KB):
                                                     //   MN-major B of the value side, K-major B of the key side
    PairCtl* ctl = reinterpret_cast<PairCtl*>(sSb + 2 * kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / H, h = bh % H;
    const int d0 = slice * kDST;

    if (tid == 0) {
        mbar_init(&ctl->bar_x[0], 1); mbar_init(&ctl->bar_x[1], 1);
        mbar_init(&ctl->bar_w[0], 1); mbar_init(&ctl->bar_w[1], 1);
        mbar_init(&ctl->bar_yq, 1);
        mbar_init(&ctl->bar_p, 1); mbar_init(&ctl->bar_a, 1);
        mbar_init(&ctl->bar_mma1, 1); mbar_init(&ctl->bar_yqfree, 1);
        mbar_init(&ctl->bar_v4, 1); mbar_init(&ctl->bar_k4, 1);
        mbar_init(&ctl->bar_pm, 1); mbar_init(&ctl->bar_am, 1); mbar_init(&ctl->bar_sb, 1);
        mbar_init(&ctl->bar_outv[0], 1); mbar_init(&ctl->bar_outv[1], 1);
        mbar_init(&ctl->bar_outk[0], 1); mbar_init(&ctl->bar_outk[1], 1);
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
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int n) { return (nchunks - 1 - n) * kCT; };     // from the last chunk down

    if (warp == kCopyWarp) {
        if (elect_one()) {
            // =============================== copy lane: every tile load and store
            auto load_x = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                mbar_expect_tx(&ctl->bar_x[st], 2 * kPanelB);
                tma_load_4d(sX + (2 * st) * kPanelB, &mapX, &ctl->bar_x[st], d0, h, t, b);
                tma_load_4d(sX + (2 * st + 1) * kPanelB, &mapX, &ctl->bar_x[st], d0 + 64, h, t, b);
            };
            auto load_w = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                mbar_expect_tx(&ctl->bar_w[st], 2 * kPanelB);
                tma_load_4d(sW + (2 * st) * kPanelB, &mapW, &ctl->bar_w[st], 0, h, t, b);
                tma_load_4d(sW + (2 * st + 1) * kPanelB, &mapW, &ctl->bar_w[st], 64, h, t, b);
            };
            auto load_yq = [&](int n) {
                const int t = chunk_t0(n);
                mbar_expect_tx(&ctl->bar_yq, 4 * kPanelB);
                tma_load_4d(sY, &mapY, &ctl->bar_yq, d0, h, t, b);
                tma_load_4d(sY + kPanelB, &mapY, &ctl->bar_yq, d0 + 64, h, t, b);
                tma_load_4d(sQ, &mapQ, &ctl->bar_yq, 0, h, t, b);
                tma_load_4d(sQ + kPanelB, &mapQ, &ctl->bar_yq, 64, h, t, b);
            };
            prefetch_tmap(&mapX); prefetch_tmap(&mapY); prefetch_tmap(&mapW); prefetch_tmap(&mapQ);
            prefetch_tmap(&mapOv); prefetch_tmap(&mapOk);
            load_x(0);
            load_yq(0);
            load_w(0);
            if (nchunks > 1) {
                load_x(1);
                load_w(1);
            }
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int t = chunk_t0(n), st = n & 1;
                // Y and Q are consumed once the inter-chunk products of chunk n are done; their next tiles are
                // asked into L2 ahead of that, so that the copy itself is short
                if (n + 1 < nchunks) {
                    const int tn = chunk_t0(n + 1);
                    tma_prefetch_4d(&mapY, d0, h, tn, b);
                    if (d0 + 64 < D) tma_prefetch_4d(&mapY, d0 + 64, h, tn, b);
                    tma_prefetch_4d(&mapQ, 0, h, tn, b);
                    tma_prefetch_4d(&mapQ, 64, h, tn, b);
                }
                PAIR_WAIT(&ctl->bar_yqfree, n & 1);
                if (ctl->abort) break;
                if (n + 1 < nchunks) load_yq(n + 1);
                // W is consumed once the value-side output is complete; the compute threads then stage that
                // output in its place (a tiled store from shared memory costs less than the compute threads'
                // own stores to global memory: those were measured at 140 us a launch against 95).  Likewise X
                // and the key-side output.  When both have left, the buffers take the tiles of chunk n+2.
                PAIR_WAIT(&ctl->bar_outv[st], (n >> 1) & 1);
                if (ctl->abort) break;
                tma_store_5d(&mapOv, sW + (2 * st) * kPanelB, 0, h, t, b, slice);
                tma_store_5d(&mapOv, sW + (2 * st + 1) * kPanelB, 32, h, t, b, slice);
                bulk_commit();
                PAIR_WAIT(&ctl->bar_outk[st], (n >> 1) & 1);
                if (ctl->abort) break;
                tma_store_4d(&mapOk, sX + (2 * st) * kPanelB, d0, h, t, b);
                if (d0 + 64 < D) tma_store_4d(&mapOk, sX + (2 * st + 1) * kPanelB, d0 + 64, h, t, b);
                bulk_commit();
                bulk_wait_read();
                if (n + 2 < nchunks) {
                    load_x(n + 2);
                    load_w(n + 2);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        if (elect_one()) {
            // =============================== MMA lane
            constexpr uint32_t idescP = make_idesc(128, 128, false, false);    // Y X^T and Q W^T
            constexpr uint32_t idescU = make_idesc(128, kM, true, true);       // X^T (MN-major A) x W part (MN-major B)
            constexpr uint32_t idescYS = make_idesc(128, kM, false, true);     // Y x state-copy part (MN-major B); masked P x W part
            constexpr uint32_t idescQS = make_idesc(128, kDST, false, false);  // Q x state copy (K-major B)
            constexpr uint32_t idescAX = make_idesc(128, kDST, false, true);   // masked A x X (MN-major B)
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            const uint64_t dYk = desc_kmajor(smem_u32(sY), 0);
            const uint64_t dQh = desc_kmajor(smem_u32(sQ), 0), dQl = desc_kmajor(smem_u32(sQ + kPanelB), 0);
            const uint64_t dSh = desc_mnmajor(smem_u32(sSb), 0, kPanelB), dSl = desc_mnmajor(smem_u32(sSb + kPanelB), 0, kPanelB);
            const uint64_t dSkh = desc_kmajor(smem_u32(sSb), 0), dSkl = desc_kmajor(smem_u32(sSb + kPanelB), 0);
            auto issue_first = [&](int n) {
                const uint32_t xs = smem_u32(sX + 2 * (n & 1) * kPanelB), ws = smem_u32(sW + 2 * (n & 1) * kPanelB);
                const uint64_t dXk = desc_kmajor(xs, 0);
                const uint64_t dWh = desc_kmajor(ws, 0), dWl = desc_kmajor(ws + kPanelB, 0);
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kPcP, desc_advance(dYk, kmaj(kk)), desc_advance(dXk, kmaj(kk)), idescP, kk > 0);
                mma_commit(&ctl->bar_p);
                // A = Q W^T with both factors as bf16 high/low pairs (the low x low term is dropped)
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kPcA, desc_advance(dQh, kmaj(kk)), desc_advance(dWh, kmaj(kk)), idescP, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kPcA, desc_advance(dQl, kmaj(kk)), desc_advance(dWh, kmaj(kk)), idescP, true);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kPcA, desc_advance(dQh, kmaj(kk)), desc_advance(dWl, kmaj(kk)), idescP, true);
                }
                mma_commit(&ctl->bar_a);
            };
            PAIR_WAIT(&ctl->bar_x[0], 0);
            PAIR_WAIT(&ctl->bar_yq, 0);
            PAIR_WAIT(&ctl->bar_w[0], 0);
            tc_fence_after_sync();
            if (!ctl->abort) issue_first(0);
            PROF_DECL
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int it = n;
                (void)it;
                const uint32_t xs = smem_u32(sX + 2 * (n & 1) * kPanelB), ws = smem_u32(sW + 2 * (n & 1) * kPanelB);
                const uint64_t dXm = desc_mnmajor(xs, 0, kPanelB);
                const uint64_t dWh = desc_mnmajor(ws, 0, kPanelB), dWl = desc_mnmajor(ws + kPanelB, 0, kPanelB);
                PROF_MARK();
                // ---- inter-chunk products first (Y and Q, single-staged, are free for the next chunk's tiles behind
                // them): the state copy was written in chunk n-1, whose rows have been read out of the accumulators
                PAIR_WAIT(&ctl->bar_sb, n & 1);
                if (n >= 1) PAIR_WAIT(&ctl->bar_outv[(n - 1) & 1], ((n - 1) >> 1) & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kPcOI, desc_advance(dYk, kmaj(kk)), desc_advance(dSh, mnmaj(kk)), idescYS, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kDST / 16; ++kk)
                        mma_bf16(tmem + kPcOI, desc_advance(dYk, kmaj(kk)), desc_advance(dSl, mnmaj(kk)), idescYS, true);
                }
                PROF_MARK();
                if (n >= 1) {
                    PAIR_WAIT(&ctl->bar_outk[(n - 1) & 1], ((n - 1) >> 1) & 1);
                    tc_fence_after_sync();
                }
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kPcO2, desc_advance(dQh, kmaj(kk)), desc_advance(dSkh, kmaj(kk)), idescQS, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kPcO2, desc_advance(dQl, kmaj(kk)), desc_advance(dSkh, kmaj(kk)), idescQS, true);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kPcO2, desc_advance(dQh, kmaj(kk)), desc_advance(dSkl, kmaj(kk)), idescQS, true);
                }
                mma_commit(&ctl->bar_yqfree);
                PROF_MARK();
                // ---- state product U = X^T W (its accumulator was read in chunk n-1, before the state copy was written)
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kPcU, desc_advance(dXm, mnmaj(kk)), desc_advance(dWh, mnmaj(kk)), idescU, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16(tmem + kPcU, desc_advance(dXm, mnmaj(kk)), desc_advance(dWl, mnmaj(kk)), idescU, true);
                }
                mma_commit(&ctl->bar_mma1);
                PROF_MARK();
                // ---- value-side intra-chunk product: masked P (bf16 pair, in place in tensor memory) x W
                PAIR_WAIT(&ctl->bar_pm, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + kPcOI, tmem + kPcP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dWh, mnmaj(kk)), idescYS,
                                true);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16_ta(tmem + kPcOI, tmem + kPcP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dWl, mnmaj(kk)),
                                    idescYS, true);
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16_ta(tmem + kPcOI, tmem + kPcP + 64 * (kk >> 2) + 32 + 8 * (kk & 3),
                                    desc_advance(dWh, mnmaj(kk)), idescYS, true);
                }
                mma_commit(&ctl->bar_v4);
                PROF_MARK();
                // ---- key-side intra-chunk product: masked A x X on top of the inter-chunk one
                PAIR_WAIT(&ctl->bar_am, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + kPcO2, tmem + kPcA + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dXm, mnmaj(kk)), idescAX,
                                true);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16_ta(tmem + kPcO2, tmem + kPcA + 64 * (kk >> 2) + 32 + 8 * (kk & 3),
                                    desc_advance(dXm, mnmaj(kk)), idescAX, true);
                }
                mma_commit(&ctl->bar_k4);
                PROF_MARK();
                // ---- both first-product accumulators are free behind these: the next chunk's queue up
                if (n + 1 < nchunks) {
                    PAIR_WAIT(&ctl->bar_x[(n + 1) & 1], ((n + 1) >> 1) & 1);
                    PAIR_WAIT(&ctl->bar_yq, (n + 1) & 1);
                    PAIR_WAIT(&ctl->bar_w[(n + 1) & 1], ((n + 1) >> 1) & 1);
                    tc_fence_after_sync();
                    PROF_MARK();
                    if (!ctl->abort) issue_first(n + 1);
                }
                PROF_MARK();
                PROF_DUMP("rev_pair mma");
            }
        }
    } else if (tid < kComputeThreads) {
        // =============================== compute threads
        // state slice, transposed: S[c = row][s], slots sb .. sb+31
        float S[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) S[s] = (S0 && d0 + row < D) ? S0[((size_t)bh * kM + sb + s) * D + d0 + row] : 0.f;

        // G of the last valid row of chunk n (threads 0..63, one slot each), one chunk ahead
        auto chunk_gc = [&](int n) {
            const int last = min(chunk_t0(n) + kCT, T) - 1;
            return G[(((size_t)b * T + last) * H + h) * kM + tid];
        };
        float g_next = 0.f;
        if (tid < kM) {
            ctl->egc[0][tid] = __expf(chunk_gc(0));
            if (nchunks > 1) g_next = chunk_gc(1);
        }
        compute_sync();
        // the state copy carries the total decay of the chunk it is used in (the decayed rows leave it out)
        store_state_row_split<true>(sSb, sSb + kPanelB, row, sb, S, ctl->egc[0]);
        publish(&ctl->bar_sb, tid);

        PROF_DECL
        for (int n = 0; n < nchunks; ++n) {
            const int it = n;
            (void)it;
            const float* egc = ctl->egc[n & 1];
            if (tid < kM && n + 1 < nchunks) {
                ctl->egc[(n + 1) & 1][tid] = __expf(g_next);
                if (n + 2 < nchunks) g_next = chunk_gc(n + 2);
            }
            PROF_MARK();
            // ---- masked P rows, then masked A rows (the barriers inside also publish egc)
            PAIR_WAIT(&ctl->bar_p, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            mask_row_in_tmem<true, PAIRS>(tmem, wq, row, half, kPcP);
            publish(&ctl->bar_pm, tid);
            PROF_MARK();
            PAIR_WAIT(&ctl->bar_a, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            mask_row_in_tmem<true, PAIRS>(tmem, wq, row, half, kPcA);
            publish(&ctl->bar_am, tid);
            PROF_MARK();

            // ---- state update S <- exp(G_C) S + U, and its copy for the next chunk
            PAIR_WAIT(&ctl->bar_mma1, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kPcU + sb), v);
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) S[e + t] = fmaf(S[e + t], ecv[t], v[e + t]);
                }
            }
            store_state_row_split<true>(sSb, sSb + kPanelB, row, sb, S, ctl->egc[(n + 1) & 1]);
            publish(&ctl->bar_sb, tid);
            PROF_MARK();

            // ---- value-side rows (fp32, without their row factor), staged where W was
            PAIR_WAIT(&ctl->bar_v4, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float vo[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kPcOI + sb), vo);
                unsigned char* panel = sW + (2 * (n & 1) + half) * kPanelB;
#pragma unroll
                for (int c = 0; c < kHS / 4; ++c)
                    *reinterpret_cast<float4*>(panel + swz128(row, c)) =
                        make_float4(vo[4 * c], vo[4 * c + 1], vo[4 * c + 2], vo[4 * c + 3]);
            }
            publish(&ctl->bar_outv[n & 1], tid);
            PROF_MARK();

            // ---- key-side rows -> io dtype, staged where X was
            PAIR_WAIT(&ctl->bar_k4, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                float v[32];
                tmem_ld32(tmem_row_addr(tmem, wq, kPcO2 + 64 * half + c0), v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float x[8] = {v[8 * c], v[8 * c + 1], v[8 * c + 2], v[8 * c + 3],
                                        v[8 * c + 4], v[8 * c + 5], v[8 * c + 6], v[8 * c + 7]};
                    store_chunk(sX + (2 * (n & 1) + half) * kPanelB, row, (c0 >> 3) + c, x);
                }
            }
            const bool stop = publish_and_vote(&ctl->bar_outk[n & 1], tid, ctl->abort != 0);
            PROF_MARK();
            PROF_DUMP("rev_pair compute");
            if (stop) break;
        }
        if (!ctl->abort && Send && d0 + row < D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) Send[((size_t)bh * kM + sb + s) * D + d0 + row] = S[s];
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

constexpr size_t kSmemPair = 1024 + 14 * kPanelB + sizeof(PairCtl);

}  // namespace

bool rev_pair_supported(const ValueSideArgs& av, const KeySideArgs& ak, int M) {
    return M == kM && tc_dim_ok(av.D) && av.D == ak.D && av.B == ak.B && av.T == ak.T && av.H == ak.H &&
           av.xk == ak.xv && av.wd != nullptr && av.wd == ak.uk_d && ak.uq_d != nullptr && av.G == ak.G &&
           av.S0 == ak.S0 && av.Send == nullptr && !av.state_only && !ak.state_only && av.single == ak.single;
}

cudaError_t launch_rev_pair_tc(const ValueSideArgs& av, const KeySideArgs& ak, int M, const int* strong_flag,
                               cudaStream_t st, int32_t* dev_status) {
    if (!rev_pair_supported(av, ak, M) || strong_flag == nullptr) return cudaErrorNotSupported;
    CUtensorMap mx, my, mw, mq, mov, mok;
    cudaError_t e = make_tensor_map_bthd(&mx, ak.xv, ak.B, ak.T, ak.H, ak.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&my, av.xq, av.B, av.T, av.H, av.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, av.wd, av.B, av.T, av.H, 2 * kM, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mq, ak.uq_d, ak.B, ak.T, ak.H, 2 * kM, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_sliced(&mov, av.out, tc_value_side_slices(av.D), av.B, av.T, av.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mok, ak.out, ak.B, ak.T, ak.H, ak.D, kCT, 2);
    if (e != cudaSuccess) return e;
    // the flagged (batch, head) pairs: the two general kernels on the side stream, beside the pair kernel
    SideLane* side = nullptr;
    e = side_lane(&side);
    if (e == cudaSuccess) e = cudaEventRecord(side->fork, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (e != cudaSuccess) return e;
    const dim3 grid(av.B * av.H, tc_value_side_slices(av.D));
    auto launch = [&](auto kernel) {
        cudaError_t e2 = prepare(kernel, kSmemPair, kPairThreads);
        if (e2 != cudaSuccess) return e2;
        kernel<<<grid, kPairThreads, kSmemPair, st>>>(mx, my, mw, mq, mov, mok, ak.G, ak.S0, ak.Send, ak.T, ak.H, ak.D,
                                                      strong_flag, dev_status);
        return cudaGetLastError();
    };
    e = av.single ? launch(rev_pair_kernel<false>) : launch(rev_pair_kernel<true>);
    if (e == cudaSuccess) e = launch_value_side_general(av, M, 1, strong_flag, side->stream, dev_status);
    if (e == cudaSuccess) e = launch_key_side_general(ak, M, 1, strong_flag, side->stream, dev_status);
    if (e == cudaSuccess) e = cudaEventRecord(side->join, side->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
    return e;
}

}  // namespace gsa
