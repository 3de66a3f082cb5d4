// Pipelined ("lean") tcgen05 versions of the two chunk primitives of Algorithm 1, for the
// (batch, head) pairs whose chunks all decay moderately (total log-decay of every chunk above
// kFactorisedDecayMin), which is every pair of the paper's workloads except the strong-forgetting
// stress case.
//
// Differences from the general kernels (chunk_tc.cu):
//   * the slot-sized operands arrive by TMA already multiplied by their decay factor and already
//     in bfloat16 -- w exp(-G) or w exp(G) as a high/low pair, written once per (batch, head) by
//     the element-wise kernels that produce w (gate kernel, slot softmax forward / backward)
//     instead of being rebuilt by each of the D/128 slices of every scan;
//   * the per-chunk chain  product -> mask -> product -> read-out  is software-pipelined: the
//     issuing lane queues the first product of chunk n+1 behind the last product of chunk n and
//     requests every tile of chunk n+1 as soon as its buffer has been consumed, so the compute
//     threads find their next accumulator ready when they finish a chunk.
//   * tile copies and MMA issue are two lanes of two warps, so that a wait of one (for a store to
//     drain, for a tile to land) never delays the other.
// Tile geometry and the bounded waits are those of the general kernels.
// The file also holds the state-only scan that segment-parallel scheduling uses for the end
// memories of every segment (state_scan_kernel, below the two chunk kernels).
#include "chunk_tc_shared.cuh"

namespace gsa {
namespace {
using namespace tc;
using namespace tcchunk;

// 8 compute warps, one warp whose lane 0 issues every MMA, one warp whose lane 0 requests every
// tile copy (loads and stores)
constexpr int kLeanThreads = kComputeThreads + 64;
constexpr int kMmaWarp = kComputeThreads / 32, kCopyWarp = kMmaWarp + 1;   // (entered by one elected lane, see elect_one)

struct LeanCtl {
    // filled by TMA
    uint64_t bar_x;        // d-sized tiles of a chunk
    uint64_t bar_x2[2];    // key_side: d-sized tiles, two stages
    uint64_t bar_w[2];     // pre-decayed slot-sized operand tiles (value_side: two stages; key_side: [0] only)
    // signalled by tcgen05.commit
    uint64_t bar_p;        // first product of a chunk (P or A)
    uint64_t bar_mma1;     // state products (U and the inter-chunk product)
    uint64_t bar_mma2;     // intra-chunk product
    uint64_t bar_free1[2]; // = bar_mma1, for the copy lane (by chunk parity): tiles read by the state products
                           // may be overwritten
    // signalled by the compute threads (one arrival after their barrier)
    uint64_t bar_pm;       // masked P / A rows are in shared memory, the P / A accumulator is free
    uint64_t bar_sb;       // state copy for the next chunk is written, the U accumulator is free
    uint64_t bar_out[2];   // (by chunk parity) output rows are staged, the output accumulators are free
    uint32_t tmem_slot;
    volatile int abort;
    alignas(16) float egc[2][kM];   // exp(G of the chunk's last valid row), by chunk parity
};

// Every mbarrier below has one producer and waiters that its producer cannot run two phases ahead
// of: a barrier's next completion always needs something (a tile, a row, an accumulator) that a
// waiter supplies only after it has seen the previous one.  Where a resource has two stages, so
// has its barrier (indexed by chunk parity).
// A wait that expires flags the CTA; once flagged, later waits return at once.  The compute
// threads leave their loop only at the end-of-chunk barrier, on a vote, so that no thread is
// left waiting at a barrier that others have abandoned.
#define LEAN_WAIT(bar, parity)                                              \
    do {                                                                    \
        if (!ctl->abort && !mbar_wait(bar, parity)) ctl->abort = 1;         \
    } while (0)

__device__ __forceinline__ void lean_ctl_init(LeanCtl* ctl, int tid, int warp) {
    if (tid == 0) {
        mbar_init(&ctl->bar_x, 1);
        mbar_init(&ctl->bar_w[0], 1);
        mbar_init(&ctl->bar_w[1], 1);
        mbar_init(&ctl->bar_x2[0], 1);
        mbar_init(&ctl->bar_x2[1], 1);
        mbar_init(&ctl->bar_p, 1);
        mbar_init(&ctl->bar_mma1, 1);
        mbar_init(&ctl->bar_mma2, 1);
        mbar_init(&ctl->bar_free1[0], 1);
        mbar_init(&ctl->bar_free1[1], 1);
        mbar_init(&ctl->bar_pm, 1);
        mbar_init(&ctl->bar_sb, 1);
        mbar_init(&ctl->bar_out[0], 1);
        mbar_init(&ctl->bar_out[1], 1);
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

template <class Ctl>
__device__ __forceinline__ void lean_finish(Ctl* ctl, int tid, int warp, uint32_t tmem, int32_t* dev_status) {
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

// accumulator columns of the lean kernels
constexpr int kLvP = 0, kLvO = 128 /* high | low state part */, kLvU = 256, kLvI = 384;     // value_side
constexpr int kLkA = 0, kLkO = 128 /* two buffers of 128 */, kLkU = 384;                 // key_side

// ======================================================================================
// value_side: out_i[s] = sum_{j<=i} <xq_i, xk_j> w_j[s] decay_ij[s]  + decayed (xq_i S)[s]
//   wd holds w exp(-G) (forward) or w exp(G) (reverse) as [hi | lo] bf16 rows of 128.
//   The row factor -- exp(G_i) forward, exp(-G_i) reverse -- is NOT applied here: the kernel that
//   sums the slices of `out` multiplies it in (see PendingDecay), so this kernel needs no G tile.
// ======================================================================================
template <bool REV, bool PAIRS>
__global__ void __launch_bounds__(kLeanThreads, 1)
value_side_lean_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                       const __grid_constant__ CUtensorMap mapWd, const __grid_constant__ CUtensorMap mapO,
                       ValueSideArgs a, const int* __restrict__ strong_flag, int32_t* dev_status) {
    if (strong_flag[blockIdx.x] != 0) return;       // the general kernel takes this (batch, head)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sX = smem;                        // xq, xk tiles: 2 stages x (2 + 2 panels)  (128 KB)
    unsigned char* sWd = sX + 8 * kPanelB;           // decayed weights, MN-major B [128][hi 64 | lo 64], 2 stages (64 KB)
                                                     //   ... a stage also holds the chunk's output rows (fp32, 2
                                                     //   panels of 32 slots) once its weights are consumed
    unsigned char* sSb = sWd + 4 * kPanelB;          // state copy, MN-major B [128][hi 64 | lo 64] (32 KB)
    LeanCtl* ctl = reinterpret_cast<LeanCtl*>(sSb + 2 * kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;

    lean_ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int n) { return (REV ? nchunks - 1 - n : n) * kCT; };

    if (warp == kCopyWarp) {
        if (elect_one()) {
            // =============================== copy lane: every tile load and store
            auto load_x = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                unsigned char* sXq = sX + 4 * st * kPanelB;
                unsigned char* sXk = sXq + 2 * kPanelB;
                mbar_expect_tx(&ctl->bar_x2[st], 4 * kPanelB);
                tma_load_4d(sXq, &mapQ, &ctl->bar_x2[st], d0, h, t, b);
                tma_load_4d(sXq + kPanelB, &mapQ, &ctl->bar_x2[st], d0 + 64, h, t, b);
                tma_load_4d(sXk, &mapK, &ctl->bar_x2[st], d0, h, t, b);
                tma_load_4d(sXk + kPanelB, &mapK, &ctl->bar_x2[st], d0 + 64, h, t, b);
            };
            auto load_w = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                mbar_expect_tx(&ctl->bar_w[st], 2 * kPanelB);
                tma_load_4d(sWd + (2 * st) * kPanelB, &mapWd, &ctl->bar_w[st], 0, h, t, b);
                tma_load_4d(sWd + (2 * st + 1) * kPanelB, &mapWd, &ctl->bar_w[st], 64, h, t, b);
            };
            auto store_out = [&](int n) {
                const int t = chunk_t0(n);
                const unsigned char* sOut = sWd + 2 * (n & 1) * kPanelB;
                tma_store_5d(&mapO, sOut, 0, h, t, b, slice);
                tma_store_5d(&mapO, sOut + kPanelB, 32, h, t, b, slice);
                bulk_commit();
            };
            prefetch_tmap(&mapQ); prefetch_tmap(&mapK); prefetch_tmap(&mapWd); prefetch_tmap(&mapO);
            load_x(0);
            load_w(0);
            if (nchunks > 1) {
                load_x(1);
                load_w(1);
            }
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                // the d-sized tiles of chunk n are consumed once its state products are done: their
                // buffer takes the tiles of chunk n+2
                LEAN_WAIT(&ctl->bar_free1[n & 1], (n >> 1) & 1);
                if (n + 2 < nchunks) load_x(n + 2);
                // the weights are consumed once the intra-chunk product is done; the compute threads then
                // stage the output rows in their place, and when those have left the buffer takes the
                // weights of chunk n+2
                LEAN_WAIT(&ctl->bar_out[n & 1], (n >> 1) & 1);
                if (ctl->abort) break;
                store_out(n);
                bulk_wait_read();
                if (n + 2 < nchunks) load_w(n + 2);
            }
        }
    } else if (warp == kMmaWarp) {
        if (elect_one()) {
            // =============================== MMA lane
            constexpr uint32_t idescP = make_idesc(128, 128, false, false);    // xq xk^T
            constexpr uint32_t idescO = make_idesc(128, 2 * kM, false, true);  // xq x state copy [S_hi | S_lo] (MN-major B)
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);   // xk^T (MN-major A) x [W_hi | W_lo]
            constexpr uint32_t idescI = make_idesc(128, 2 * kM, false, true);  // masked P (tensor memory) x [W_hi | W_lo]
            const uint64_t dS = desc_mnmajor(smem_u32(sSb), 0, kPanelB);
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            auto issue_p = [&](int n) {
                const uint32_t xq = smem_u32(sX + 4 * (n & 1) * kPanelB);
                const uint64_t dQk = desc_kmajor(xq, 0), dKk = desc_kmajor(xq + 2 * kPanelB, 0);
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kLvP, desc_advance(dQk, kmaj(kk)), desc_advance(dKk, kmaj(kk)), idescP, kk > 0);
                mma_commit(&ctl->bar_p);
            };
            LEAN_WAIT(&ctl->bar_x2[0], 0);
            tc_fence_after_sync();
            issue_p(0);
            PROF_DECL
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int it = n;
                (void)it;
                const uint32_t xq = smem_u32(sX + 4 * (n & 1) * kPanelB);
                const uint64_t dQk = desc_kmajor(xq, 0), dKm = desc_mnmajor(xq + 2 * kPanelB, 0, kPanelB);
                const uint64_t dW = desc_mnmajor(smem_u32(sWd + 2 * (n & 1) * kPanelB), 0, kPanelB);
                PROF_MARK();
                // state products of chunk n: the state copy was written at the end of chunk n-1 (which also
                // says that the accumulators they overwrite have been read)
                LEAN_WAIT(&ctl->bar_w[n & 1], (n >> 1) & 1);
                PROF_MARK();
                LEAN_WAIT(&ctl->bar_sb, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kLvU, desc_advance(dKm, mnmaj(kk)), desc_advance(dW, mnmaj(kk)), idescU, kk > 0);
                // the inter-chunk output accumulator is single: the previous chunk's output rows must have
                // been read out (by now they almost always are: this is issued after that chunk's intra
                // product and the next first product)
                if (n >= 1) {
                    LEAN_WAIT(&ctl->bar_out[(n - 1) & 1], ((n - 1) >> 1) & 1);
                    tc_fence_after_sync();
                }
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + kLvO, desc_advance(dQk, kmaj(kk)), desc_advance(dS, mnmaj(kk)), idescO, kk > 0);
                mma_commit(&ctl->bar_mma1);
                mma_commit(&ctl->bar_free1[n & 1]);
                PROF_MARK();
                // intra-chunk product once the masked P rows are there (bf16, in place in tensor memory)
                LEAN_WAIT(&ctl->bar_pm, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + kLvI, tmem + kLvP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dW, mnmaj(kk)), idescI,
                                kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)      // ... and the rounding residual of the masked P
                        mma_bf16_ta(tmem + kLvI, tmem + kLvP + 64 * (kk >> 2) + 32 + 8 * (kk & 3),
                                    desc_advance(dW, mnmaj(kk)), idescI, true);
                }
                mma_commit(&ctl->bar_mma2);
                PROF_MARK();
                // the P accumulator is free: the next chunk's P queues right behind
                if (n + 1 < nchunks) {
                    LEAN_WAIT(&ctl->bar_x2[(n + 1) & 1], ((n + 1) >> 1) & 1);
                    tc_fence_after_sync();
                    PROF_MARK();
                    issue_p(n + 1);
                }
                PROF_MARK();
                PROF_DUMP("value_side lean mma");
            }
        }
    } else if (tid < kComputeThreads) {
        // =============================== compute threads
        // state slice: S[c = row][s], slots sb .. sb+31
        float S[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) S[s] = (a.S0 && d0 + row < a.D) ? a.S0[((size_t)bh * kM + sb + s) * a.D + d0 + row] : 0.f;
        store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);

        // G of the last valid row of chunk n (threads 0..63, one slot each), one chunk ahead
        auto chunk_gc = [&](int n) {
            const int last = min(chunk_t0(n) + kCT, a.T) - 1;
            return a.G[(((size_t)b * a.T + last) * a.H + h) * kM + tid];
        };
        float g_next = 0.f;
        if (tid < kM) {
            ctl->egc[0][tid] = __expf(chunk_gc(0));
            if (nchunks > 1) g_next = chunk_gc(1);
        }
        publish(&ctl->bar_sb, tid);

        PROF_DECL
        for (int n = 0; n < nchunks; ++n) {
            const int it = n;
            (void)it;
            PROF_MARK();
            const int valid = min(kCT, a.T - chunk_t0(n));
            const float* egc = ctl->egc[n & 1];
            if (tid < kM && n + 1 < nchunks) {
                ctl->egc[(n + 1) & 1][tid] = __expf(g_next);
                if (n + 2 < nchunks) g_next = chunk_gc(n + 2);
            }
            // ---- masked P rows (the barrier inside also publishes egc)
            LEAN_WAIT(&ctl->bar_p, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            mask_row_in_tmem<REV, PAIRS>(tmem, wq, row, half, kLvP);
            publish(&ctl->bar_pm, tid);
            PROF_MARK();

            // ---- state update from U: forward S <- exp(G_C) (S + U), reverse S <- exp(G_C) S + U
            LEAN_WAIT(&ctl->bar_mma1, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kLvU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, kLvU + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float u = v[e + t] + vl[e + t];
                        S[e + t] = REV ? fmaf(S[e + t], ecv[t], u) : (S[e + t] + u) * ecv[t];
                    }
                }
            }
            store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);
            publish(&ctl->bar_sb, tid);
            PROF_MARK();

            // ---- output rows without their row factor: inter + intra (reverse: exp(G_C) inter + intra),
            // staged for one tiled store, clipped at the sequence end
            LEAN_WAIT(&ctl->bar_mma2, n & 1);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float vo[kHS], vi[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kLvI + sb), vo);
                tmem_ld32(tmem_row_addr(tmem, wq, kLvI + kM + sb), vi);
#pragma unroll
                for (int e = 0; e < kHS; ++e) vo[e] += vi[e];          // high + low weight parts
                float vj[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kLvO + sb), vi);
                tmem_ld32(tmem_row_addr(tmem, wq, kLvO + kM + sb), vj);
#pragma unroll
                for (int e = 0; e < kHS; ++e) vi[e] += vj[e];          // high + low state parts
#pragma unroll
                for (int e = 0; e < kHS; ++e) vo[e] = REV ? fmaf(vi[e], egc[sb + e], vo[e]) : vo[e] + vi[e];
                unsigned char* panel = sWd + (2 * (n & 1) + half) * kPanelB;
#pragma unroll
                for (int c = 0; c < kHS / 4; ++c)
                    *reinterpret_cast<float4*>(panel + swz128(row, c)) =
                        make_float4(vo[4 * c], vo[4 * c + 1], vo[4 * c + 2], vo[4 * c + 3]);
            }
            (void)valid;
            const bool stop = publish_and_vote(&ctl->bar_out[n & 1], tid, ctl->abort != 0);
            PROF_MARK();
            PROF_DUMP("value_side lean compute");
            if (stop) break;
        }
        if (!ctl->abort && a.Send && d0 + row < a.D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) a.Send[((size_t)bh * kM + sb + s) * a.D + d0 + row] = S[s];
        }
    }
    lean_finish(ctl, tid, warp, tmem, dev_status);
}

// ======================================================================================
// key_side: out_i = (uq_i * qscale_i) S + sum_j A_ij xv_j,  A_ij = sum_s uq_i[s] uk_j[s] decay_ij[s]
//   uq_d / uk_d hold the decayed bf16 rows (first 64 of every 128): forward uq exp(G), uk exp(-G);
//   reverse uq exp(-G), uk exp(G).
// ======================================================================================
template <bool REV, bool PAIRS>
__global__ void __launch_bounds__(kLeanThreads, 1)
key_side_lean_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapUq,
                     const __grid_constant__ CUtensorMap mapUk, const __grid_constant__ CUtensorMap mapO,
                     KeySideArgs a, const int* __restrict__ strong_flag, int32_t* dev_status) {
    if (strong_flag[blockIdx.x] != 0) return;       // the general kernel takes this (batch, head)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sXv = smem;                       // xv tile, 2 stages of 2 panels              (64 KB)
                                                     //   ... a stage also holds the chunk's output rows once
                                                     //   its tile is consumed
    unsigned char* sQK = sXv + 4 * kPanelB;          // decayed uq (K-major A [128][64]) and uk (K-major /
                                                     //   MN-major B [128][64]), each with its rounding residual:
                                                     //   2 stages of 4 panels [uq_hi, uk_hi, uq_lo, uk_lo] (128 KB)
    unsigned char* sSb = sQK + 8 * kPanelB;          // state copy, K-major B [128 (channel)][64], and its
                                                     //   rounding residual                        (32 KB)
    LeanCtl* ctl = reinterpret_cast<LeanCtl*>(sSb + 2 * kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / a.H, h = bh % a.H;
    const int d0 = slice * kDST;

    lean_ctl_init(ctl, tid, warp);
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (a.T + kCT - 1) / kCT;
    auto chunk_t0 = [&](int n) { return (REV ? nchunks - 1 - n : n) * kCT; };

    if (warp == kCopyWarp) {
        if (elect_one()) {
            // =============================== copy lane: every tile load and store
            auto load_v = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                mbar_expect_tx(&ctl->bar_x2[st], 2 * kPanelB);
                tma_load_4d(sXv + (2 * st) * kPanelB, &mapV, &ctl->bar_x2[st], d0, h, t, b);
                tma_load_4d(sXv + (2 * st + 1) * kPanelB, &mapV, &ctl->bar_x2[st], d0 + 64, h, t, b);
            };
            auto load_qk = [&](int n) {
                const int t = chunk_t0(n), st = n & 1;
                mbar_expect_tx(&ctl->bar_w[st], 4 * kPanelB);
                tma_load_4d(sQK + (4 * st) * kPanelB, &mapUq, &ctl->bar_w[st], 0, h, t, b);
                tma_load_4d(sQK + (4 * st + 1) * kPanelB, &mapUk, &ctl->bar_w[st], 0, h, t, b);
                tma_load_4d(sQK + (4 * st + 2) * kPanelB, &mapUq, &ctl->bar_w[st], 64, h, t, b);
                tma_load_4d(sQK + (4 * st + 3) * kPanelB, &mapUk, &ctl->bar_w[st], 64, h, t, b);
            };
            auto store_out = [&](int n) {
                const int t = chunk_t0(n);
                const unsigned char* sOut = sXv + 2 * (n & 1) * kPanelB;
                tma_store_4d(&mapO, sOut, d0, h, t, b);
                if (d0 + 64 < a.D) tma_store_4d(&mapO, sOut + kPanelB, d0 + 64, h, t, b);
                bulk_commit();
            };
            prefetch_tmap(&mapV); prefetch_tmap(&mapUq); prefetch_tmap(&mapUk); prefetch_tmap(&mapO);
            load_qk(0);
            load_v(0);
            if (nchunks > 1) {
                load_qk(1);
                load_v(1);
            }
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                // the decayed uq / uk rows of chunk n are consumed once its state products are done: their
                // buffer takes the rows of chunk n+2
                LEAN_WAIT(&ctl->bar_free1[n & 1], (n >> 1) & 1);
                if (n + 2 < nchunks) load_qk(n + 2);
                // the xv tile is consumed once the intra-chunk product is done; the compute threads then
                // stage the output rows in its place, and when those have left the buffer takes the tile
                // of chunk n+2
                LEAN_WAIT(&ctl->bar_out[n & 1], (n >> 1) & 1);
                if (ctl->abort) break;
                store_out(n);
                bulk_wait_read();
                if (n + 2 < nchunks) load_v(n + 2);
            }
        }
    } else if (warp == kMmaWarp) {
        if (elect_one()) {
            // =============================== MMA lane
            constexpr uint32_t idescA = make_idesc(128, 128, false, false);   // Q~ K~^T
            constexpr uint32_t idescO = make_idesc(128, kDST, false, false);  // Q~ x state copy (K-major B)
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);  // xv^T (MN-major A) x [K~_hi | K~_lo] (MN-major B)
            constexpr uint32_t idescV = make_idesc(128, kDST, false, true);   // A x xv (MN-major B)
            const uint64_t dS = desc_kmajor(smem_u32(sSb), 0), dSl = desc_kmajor(smem_u32(sSb + kPanelB), 0);
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            auto issue_a = [&](int n) {
                // A = Q~ K~^T with both factors as bf16 high/low pairs (the low x low term is dropped)
                const uint32_t qk = smem_u32(sQK + 4 * (n & 1) * kPanelB);
                const uint64_t dQt = desc_kmajor(qk, 0), dKt = desc_kmajor(qk + kPanelB, 0);
                const uint64_t dQl = desc_kmajor(qk + 2 * kPanelB, 0), dKl = desc_kmajor(qk + 3 * kPanelB, 0);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + kLkA, desc_advance(dQt, kmaj(kk)), desc_advance(dKt, kmaj(kk)), idescA, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kLkA, desc_advance(dQl, kmaj(kk)), desc_advance(dKt, kmaj(kk)), idescA, true);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(tmem + kLkA, desc_advance(dQt, kmaj(kk)), desc_advance(dKl, kmaj(kk)), idescA, true);
                }
                mma_commit(&ctl->bar_p);
            };
            LEAN_WAIT(&ctl->bar_w[0], 0);
            tc_fence_after_sync();
            issue_a(0);
            PROF_DECL
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int it = n;
                (void)it;
                const uint64_t dV = desc_mnmajor(smem_u32(sXv + 2 * (n & 1) * kPanelB), 0, kPanelB);
                const uint32_t accO = tmem + kLkO + 128 * (n & 1);
                const uint32_t qk = smem_u32(sQK + 4 * (n & 1) * kPanelB);
                const uint64_t dQt = desc_kmajor(qk, 0), dQl = desc_kmajor(qk + 2 * kPanelB, 0);
                // the decayed uk read MN-major, its high and low parts as one N = 128 operand (the panels
                // of a stage are [uq_hi, uk_hi, uq_lo, uk_lo]: the low part is two panels on)
                const uint64_t dKtm = desc_mnmajor(qk + kPanelB, 0, 2 * kPanelB);
                PROF_MARK();
                // state products of chunk n: the state copy was written at the end of chunk n-1 (which also
                // says that the accumulators they overwrite have been read)
                LEAN_WAIT(&ctl->bar_x2[n & 1], (n >> 1) & 1);
                PROF_MARK();
                LEAN_WAIT(&ctl->bar_sb, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + kLkU, desc_advance(dV, mnmaj(kk)), desc_advance(dKtm, mnmaj(kk)), idescU, kk > 0);
                // inter-chunk product with both factors as bf16 high/low pairs (low x low dropped)
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(accO, desc_advance(dQt, kmaj(kk)), desc_advance(dS, kmaj(kk)), idescO, kk > 0);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(accO, desc_advance(dQl, kmaj(kk)), desc_advance(dS, kmaj(kk)), idescO, true);
#pragma unroll
                    for (int kk = 0; kk < kM / 16; ++kk)
                        mma_bf16(accO, desc_advance(dQt, kmaj(kk)), desc_advance(dSl, kmaj(kk)), idescO, true);
                }
                mma_commit(&ctl->bar_mma1);
                mma_commit(&ctl->bar_free1[n & 1]);
                PROF_MARK();
                // intra-chunk product (masked A and its rounding residual) on top of the inter-chunk one
                LEAN_WAIT(&ctl->bar_pm, n & 1);
                tc_fence_after_sync();
                PROF_MARK();
                // (the masked A and its rounding residual are bf16 rows in tensor memory, in place of A)
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(accO, tmem + kLkA + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)), idescV, true);
                if (PAIRS) {
#pragma unroll
                    for (int kk = 0; kk < kCT / 16; ++kk)
                        mma_bf16_ta(accO, tmem + kLkA + 64 * (kk >> 2) + 32 + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)),
                                    idescV, true);
                }
                mma_commit(&ctl->bar_mma2);
                PROF_MARK();
                // the A accumulator is free: the next chunk's A queues right behind
                if (n + 1 < nchunks) {
                    LEAN_WAIT(&ctl->bar_w[(n + 1) & 1], ((n + 1) >> 1) & 1);
                    tc_fence_after_sync();
                    PROF_MARK();
                    issue_a(n + 1);
                }
                PROF_MARK();
                PROF_DUMP("key_side lean mma");
            }
        }
    } else if (tid < kComputeThreads) {
        // =============================== compute threads
        // state slice, transposed: S[c = row][s], slots sb .. sb+31
        float S[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) S[s] = (a.S0 && d0 + row < a.D) ? a.S0[((size_t)bh * kM + sb + s) * a.D + d0 + row] : 0.f;

        // G of the last valid row of chunk n (threads 0..63, one slot each)
        auto chunk_gc = [&](int n) {
            const int t0 = chunk_t0(n);
            const int last = min(t0 + kCT, a.T) - 1;
            return a.G[(((size_t)b * a.T + last) * a.H + h) * kM + tid];
        };
        float g_next = 0.f;      // gc of chunk n+1, loaded one chunk ahead
        if (tid < kM) {
            ctl->egc[0][tid] = __expf(chunk_gc(0));
            if (nchunks > 1) g_next = chunk_gc(1);
        }
        compute_sync();
        // bf16 copy of the state for the first chunk's inter-chunk product (reverse: scaled by the
        // chunk's total decay, which the decayed uq rows leave out)
        if (REV) store_state_row_split<true>(sSb, sSb + kPanelB, row, sb, S, ctl->egc[0]);
        else store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);
        publish(&ctl->bar_sb, tid);

        for (int n = 0; n < nchunks; ++n) {
            const float* egc = ctl->egc[n & 1];
            if (tid < kM && n + 1 < nchunks) {
                ctl->egc[(n + 1) & 1][tid] = __expf(g_next);
                if (n + 2 < nchunks) g_next = chunk_gc(n + 2);
            }
            // ---- masked A rows as a bf16 high/low pair (the barrier inside also publishes egc)
            LEAN_WAIT(&ctl->bar_p, n & 1);
            tc_fence_after_sync();
            mask_row_in_tmem<REV, PAIRS>(tmem, wq, row, half, kLkA);
            publish(&ctl->bar_pm, tid);

            // ---- state update from U^T: forward S <- exp(G_C) (S + U^T), reverse S <- exp(G_C) S + U^T
            LEAN_WAIT(&ctl->bar_mma1, n & 1);
            tc_fence_after_sync();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, kLkU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, kLkU + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; ++e) v[e] += vl[e];          // high + low part of the decayed uk
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        S[e + t] = REV ? fmaf(S[e + t], ecv[t], v[e + t]) : (S[e + t] + v[e + t]) * ecv[t];
                }
            }
            if (REV) store_state_row_split<true>(sSb, sSb + kPanelB, row, sb, S, ctl->egc[(n + 1) & 1]);
            else store_state_row_split<false>(sSb, sSb + kPanelB, row, sb, S, nullptr);
            publish(&ctl->bar_sb, tid);

            // ---- output rows -> bf16, staged for the tiled store (clipped at the sequence end)
            LEAN_WAIT(&ctl->bar_mma2, n & 1);
            tc_fence_after_sync();
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                float v[32];
                tmem_ld32(tmem_row_addr(tmem, wq, kLkO + 128 * (n & 1) + 64 * half + c0), v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float x[8] = {v[8 * c], v[8 * c + 1], v[8 * c + 2], v[8 * c + 3],
                                        v[8 * c + 4], v[8 * c + 5], v[8 * c + 6], v[8 * c + 7]};
                    store_chunk(sXv + (2 * (n & 1) + half) * kPanelB, row, (c0 >> 3) + c, x);
                }
            }
            if (publish_and_vote(&ctl->bar_out[n & 1], tid, ctl->abort != 0)) break;
        }
        if (!ctl->abort && a.Send && d0 + row < a.D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) a.Send[((size_t)bh * kM + sb + s) * a.D + d0 + row] = S[s];
        }
    }
    lean_finish(ctl, tid, warp, tmem, dev_status);
}

// ======================================================================================
// End state only (segment-parallel scheduling runs every segment once from empty memories just
// for its end memories).  Both primitives update their state the same way,
//     U_n = X_n^T [W_hi | W_lo]_n,   forward S <- exp(G_C) (S + U_n),   reverse S <- exp(G_C) S + U_n,
// with X the d-sized tile that enters the state (xk of value_side, xv of key_side) and W the
// decayed slot-sized rows beside it (wd, uk_d), and no product depends on the state: the chunk
// chain is copy -> product -> read-out, with three tile stages and two accumulators, and reads
// each of the two streams once.
// ======================================================================================
constexpr int kScanStages = 3;

struct ScanCtl {
    uint64_t bar_x[kScanStages];      // (TMA) the tiles of a chunk have landed
    uint64_t bar_free[kScanStages];   // (tcgen05.commit) ... and have been consumed by the chunk's product
    uint64_t bar_u[2];                // (tcgen05.commit) the product of a chunk is complete, by chunk parity
    uint64_t bar_acc[2];              // (compute threads) ... and has been read out
    uint32_t tmem_slot;
    volatile int abort;
    alignas(16) float egc[2][kM];     // exp(G of the chunk's last valid row), by chunk parity
};

template <bool REV>
__global__ void __launch_bounds__(kLeanThreads, 1)
state_scan_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                  const float* __restrict__ G, const float* __restrict__ S0, float* __restrict__ Send, int T, int H,
                  int D, const int* __restrict__ strong_flag, int32_t* dev_status) {
    if (strong_flag[blockIdx.x] != 0) return;       // the general kernel takes this (batch, head)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // a stage: X tile (2 panels of 64 channels) and the decayed rows [hi 64 | lo 64] (2 panels)
    ScanCtl* ctl = reinterpret_cast<ScanCtl*>(smem + kScanStages * 4 * kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;          // this thread's first slot
    const int bh = blockIdx.x, slice = blockIdx.y, b = bh / H, h = bh % H;
    const int d0 = slice * kDST;

    if (tid == 0) {
        for (int i = 0; i < kScanStages; ++i) {
            mbar_init(&ctl->bar_x[i], 1);
            mbar_init(&ctl->bar_free[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&ctl->bar_u[i], 1);
            mbar_init(&ctl->bar_acc[i], 1);
        }
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
    auto chunk_t0 = [&](int n) { return (REV ? nchunks - 1 - n : n) * kCT; };

    if (warp == kCopyWarp) {
        if (elect_one()) {
            // =============================== copy lane
            auto load = [&](int n) {
                const int t = chunk_t0(n), st = n % kScanStages;
                unsigned char* sX = smem + 4 * st * kPanelB;
                mbar_expect_tx(&ctl->bar_x[st], 4 * kPanelB);
                tma_load_4d(sX, &mapX, &ctl->bar_x[st], d0, h, t, b);
                tma_load_4d(sX + kPanelB, &mapX, &ctl->bar_x[st], d0 + 64, h, t, b);
                tma_load_4d(sX + 2 * kPanelB, &mapW, &ctl->bar_x[st], 0, h, t, b);
                tma_load_4d(sX + 3 * kPanelB, &mapW, &ctl->bar_x[st], 64, h, t, b);
            };
            prefetch_tmap(&mapX); prefetch_tmap(&mapW);
            for (int n = 0; n < kScanStages && n < nchunks; ++n) load(n);
            for (int n = 0; n + kScanStages < nchunks && !ctl->abort; ++n) {
                LEAN_WAIT(&ctl->bar_free[n % kScanStages], (n / kScanStages) & 1);
                if (ctl->abort) break;
                load(n + kScanStages);
            }
        }
    } else if (warp == kMmaWarp) {
        if (elect_one()) {
            // =============================== MMA lane
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);   // X^T (MN-major A) x [W_hi | W_lo] (MN-major B)
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int st = n % kScanStages;
                const uint32_t sX = smem_u32(smem + 4 * st * kPanelB);
                const uint64_t dX = desc_mnmajor(sX, 0, kPanelB), dW = desc_mnmajor(sX + 2 * kPanelB, 0, kPanelB);
                LEAN_WAIT(&ctl->bar_x[st], (n / kScanStages) & 1);
                // the accumulator of chunk n-2 must have been read out
                if (n >= 2) LEAN_WAIT(&ctl->bar_acc[n & 1], ((n - 2) >> 1) & 1);
                if (ctl->abort) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + 128 * (n & 1), desc_advance(dX, mnmaj(kk)), desc_advance(dW, mnmaj(kk)), idescU, kk > 0);
                mma_commit(&ctl->bar_u[n & 1]);
                mma_commit(&ctl->bar_free[st]);
            }
        }
    } else if (tid < kComputeThreads) {
        // =============================== compute threads: S[c = row][s], slots sb .. sb+31
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
        for (int n = 0; n < nchunks; ++n) {
            const float* egc = ctl->egc[n & 1];
            if (tid < kM && n + 1 < nchunks) {
                ctl->egc[(n + 1) & 1][tid] = __expf(g_next);
                if (n + 2 < nchunks) g_next = chunk_gc(n + 2);
            }
            LEAN_WAIT(&ctl->bar_u[n & 1], (n >> 1) & 1);
            tc_fence_after_sync();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, 128 * (n & 1) + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, 128 * (n & 1) + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float u = v[e + t] + vl[e + t];
                        S[e + t] = REV ? fmaf(S[e + t], ecv[t], u) : (S[e + t] + u) * ecv[t];
                    }
                }
            }
            // (the barrier inside also publishes the next chunk's egc)
            if (publish_and_vote(&ctl->bar_acc[n & 1], tid, ctl->abort != 0)) break;
        }
        if (!ctl->abort && Send && d0 + row < D) {
#pragma unroll
            for (int s = 0; s < kHS; ++s) Send[((size_t)bh * kM + sb + s) * D + d0 + row] = S[s];
        }
    }
    lean_finish(ctl, tid, warp, tmem, dev_status);
}

constexpr size_t kSmemStateScan = 1024 + kScanStages * 4 * kPanelB + sizeof(ScanCtl);
constexpr size_t kSmemLeanValue = 1024 + 14 * kPanelB + sizeof(LeanCtl);   // value_side: 8 + 4 + 2 panels
constexpr size_t kSmemLeanKey = 1024 + 14 * kPanelB + sizeof(LeanCtl);     // key_side: 4 + 8 + 2 panels

}  // namespace

namespace {
// X: [B,T,H,D] bf16, the tile that enters the state; W: [B,T,H,2M] bf16 decayed rows [hi | lo]
cudaError_t launch_state_scan(const void* X, const void* W, const float* G, const float* S0, float* Send, int B, int T,
                              int H, int D, int reverse, const int* strong_flag, cudaStream_t st, int32_t* dev_status) {
    CUtensorMap mx, mw;
    cudaError_t e = make_tensor_map_bthd(&mx, X, B, T, H, D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, W, B, T, H, 2 * kM, kCT, 2);
    if (e != cudaSuccess) return e;
    dim3 grid(B * H, tc_value_side_slices(D));
    if (reverse) {
        e = prepare(state_scan_kernel<true>, kSmemStateScan, kLeanThreads);
        if (e != cudaSuccess) return e;
        state_scan_kernel<true><<<grid, kLeanThreads, kSmemStateScan, st>>>(mx, mw, G, S0, Send, T, H, D, strong_flag, dev_status);
    } else {
        e = prepare(state_scan_kernel<false>, kSmemStateScan, kLeanThreads);
        if (e != cudaSuccess) return e;
        state_scan_kernel<false><<<grid, kLeanThreads, kSmemStateScan, st>>>(mx, mw, G, S0, Send, T, H, D, strong_flag, dev_status);
    }
    return cudaGetLastError();
}
}  // namespace

cudaError_t launch_value_side_lean(const ValueSideArgs& a, int reverse, const int* strong_flag, cudaStream_t st,
                                   int32_t* dev_status) {
    if (a.state_only)
        return launch_state_scan(a.xk, a.wd, a.G, a.S0, a.Send, a.B, a.T, a.H, a.D, reverse, strong_flag, st, dev_status);
    CUtensorMap mq, mk, mw, mo;
    cudaError_t e = make_tensor_map_bthd(&mq, a.xq, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_sliced(&mo, a.out, tc_value_side_slices(a.D), a.B, a.T, a.H, kM, kCT, 4);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mk, a.xk, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, a.wd, a.B, a.T, a.H, 2 * kM, kCT, 2);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
    auto launch = [&](auto kernel) {
        cudaError_t e2 = prepare(kernel, kSmemLeanValue, kLeanThreads);
        if (e2 != cudaSuccess) return e2;
        kernel<<<grid, kLeanThreads, kSmemLeanValue, st>>>(mq, mk, mw, mo, a, strong_flag, dev_status);
        return cudaGetLastError();
    };
    if (reverse) return a.single ? launch(value_side_lean_kernel<true, false>) : launch(value_side_lean_kernel<true, true>);
    return a.single ? launch(value_side_lean_kernel<false, false>) : launch(value_side_lean_kernel<false, true>);
}

cudaError_t launch_key_side_lean(const KeySideArgs& a, int reverse, const int* strong_flag, cudaStream_t st,
                                 int32_t* dev_status) {
    if (a.state_only)
        return launch_state_scan(a.xv, a.uk_d, a.G, a.S0, a.Send, a.B, a.T, a.H, a.D, reverse, strong_flag, st, dev_status);
    CUtensorMap mv, muq, muk, mo;
    cudaError_t e = make_tensor_map_bthd(&mv, a.xv, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mo, a.out, a.B, a.T, a.H, a.D, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muq, a.uq_d, a.B, a.T, a.H, 2 * kM, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&muk, a.uk_d, a.B, a.T, a.H, 2 * kM, kCT, 2);
    if (e != cudaSuccess) return e;
    dim3 grid(a.B * a.H, tc_value_side_slices(a.D));
    auto launch = [&](auto kernel) {
        cudaError_t e2 = prepare(kernel, kSmemLeanKey, kLeanThreads);
        if (e2 != cudaSuccess) return e2;
        kernel<<<grid, kLeanThreads, kSmemLeanKey, st>>>(mv, muq, muk, mo, a, strong_flag, dev_status);
        return cudaGetLastError();
    };
    if (reverse) return a.single ? launch(key_side_lean_kernel<true, false>) : launch(key_side_lean_kernel<true, true>);
    return a.single ? launch(key_side_lean_kernel<false, false>) : launch(key_side_lean_kernel<false, true>);
}

}  // namespace gsa
