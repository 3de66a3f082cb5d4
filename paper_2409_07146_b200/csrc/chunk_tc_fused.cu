// Fused chunk kernel of the GSA layer: a value_side scan, the slot non-linearity and a key_side
// scan in ONE kernel, so that the slot-sized rows between the two passes never leave the chip.
//
//   forward  (Algorithm 1, forward pass: pass 1 -> softmax over the slots -> pass 2)
//       o' = value_side(q, k, 1-a)      p = softmax(scale o')      o  = key_side(p, 1-a, v)
//   backward (Algorithm 1, backward pass: gradient of pass 2's queries -> dsoftmax -> gradient of
//   pass 1's queries; both scans run forward in time)
//       dp = value_side(dO, v, 1-a)     dz = scale dsoftmax(o', dp) dq = key_side(dz, 1-a, k)
//
// One thread-block cluster per (batch, head): CTA r of the cluster owns the r-th 128-wide slice of
// the first pass's head dimension AND the r-th slice of the second pass's (d_k / 128 == d_v / 128
// == cluster size: 1, 2 or 4).  Per chunk of 128 tokens every CTA
//   1. runs the first pass on its slice (its partial sums of the 128 x 64 slot rows),
//   2. stages its partial sums and sends every row to the CTA that owns the row (rows are dealt out
//      evenly: 128 / cluster size each): one asynchronous bulk copy per peer, shared memory to the
//      peer's shared memory, completing on the peer's mbarrier,
//   3. sums the slices of its rows, applies the pending row factor exp(G), the non-linearity, writes
//      the decayed bf16 high/low rows of the result into its own operand buffer and copies them
//      into the operand buffer of every peer (bulk copies again),
//   4. runs the second pass on its slice with that operand.
// The first pass of chunk n+1 is queued behind the second pass of chunk n; all tiles are
// single-staged (the two passes keep 14 of the 14 panels of shared memory busy), refilled as soon
// as their last reader is done.  Thread roles, tile geometry, operand pairs and bounded waits are
// those of the pipelined kernels (chunk_tc_lean.cu).  Traffic between the CTAs of a cluster is
// point-to-point bulk copies between shared memories and relaxed mbarrier arrivals: no thread runs
// a cluster-scope fence.  Every tensor map covers this GPU's memory; no copy is multicast.
#include <string.h>

#include "chunk_tc_shared.cuh"

namespace gsa {
namespace {
using namespace tc;
using namespace tcchunk;

constexpr int kFThreads = kComputeThreads + 64;
constexpr int kFMma = kComputeThreads, kFCopy = kComputeThreads + 32;
// accumulator columns: first product of either pass (P, then A), state update of either pass (U),
// first-pass rows (inter + intra, [high | low] weight parts), second-pass rows (inter + intra)
constexpr int cP = 0, cU = 128, cO1 = 256, cO2 = 384;

struct FusedCtl {
    // filled by TMA
    uint64_t bar_x1, bar_w, bar_xv;
    // signalled by tcgen05.commit, for the compute threads ...
    uint64_t bar_p1, bar_s1, bar_o1, bar_p2, bar_s2, bar_o2;
    // ... and for the copy lane (same commits as bar_s1 / bar_s2)
    uint64_t bar_fx1, bar_fw;
    // signalled by this CTA's compute threads (one arrival after their barrier)
    uint64_t bar_init, bar_pm1, bar_sb1, bar_pm2, bar_sb2, bar_out, bar_rxdone;
    // signalled by every CTA of the cluster (count = cluster size; relaxed arrivals, they carry no data)
    uint64_t bar_rxfree;    // every CTA's landing buffer for partial sums is free
    uint64_t bar_pfree;     // every CTA's second-pass operand buffer is free
    uint64_t bar_txdone;    // (count = peers) my staged partial sums have been copied out
    // one local arrival that announces the bytes expected + the peers' bulk copies
    uint64_t bar_rxfull;    // every peer's partial sums of my rows have landed
    uint64_t bar_pready;    // every row of the second-pass operand is in place
    uint32_t tmem_slot;
    volatile int abort;
    alignas(16) float egc[2][kM];
};

#define FUSED_WAIT(bar, parity)                                             \
    do {                                                                    \
        if (!ctl->abort && !mbar_wait(bar, parity)) ctl->abort = 1;         \
    } while (0)
#define FUSED_WAIT_CLUSTER(bar, parity)                                     \
    do {                                                                    \
        if (!ctl->abort && !mbar_wait_cluster(bar, parity)) ctl->abort = 1; \
    } while (0)

// ---- cluster helpers (all of them are valid in a launch without cluster dimensions: rank 0 of 1)
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t peer_addr(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
// an arrival that orders nothing: it only tells the peer that a buffer of this CTA may be rewritten
__device__ __forceinline__ void mbar_arrive_peer(uint32_t addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// `bytes` (a multiple of 16) from this CTA's shared memory to a peer's, completing on the peer's mbarrier
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_peer, uint32_t src_local, uint32_t bytes, uint32_t bar_peer) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_peer), "r"(src_local), "r"(bytes), "r"(bar_peer)
                 : "memory");
}
// bounded wait that also acquires what other CTAs of the cluster wrote before their arrival
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    uint64_t start = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
        if ((it & 63u) == 63u) {
            const uint64_t now = global_timer_ns();
            if (start == 0) start = now;
            else if (now - start > kWaitLimitNs) return false;
        }
    }
}
// all threads of all CTAs of the cluster
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

struct FusedArgs {
    const float* G;                    // chunk-local cumulative log gate [B,T,H,M]
    const float *S1_0, *S2_0;          // states entering the two scans (nullable), memory layout [B,H,M,D]
    float *S1_end, *S2_end;            // states after the last chunk (nullable)
    int B, T, H, D1, D2;
    float scale;
    int act;
    // forward: the scaled logits are written here (nullable); backward: they are read from here
    float* ok;
    // backward only: u = p dp + o' do' (fp32 rows), and the decayed bf16 [high | low] rows of p and dz
    float* u;
    __nv_bfloat16* Pd;
    __nv_bfloat16* Zd;
};

// (x0, x1) as a packed bf16 pair and the packed rounding residuals
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// MODE 0: forward (softmax between the passes); MODE 1: backward (dsoftmax between the passes).
// NSL: CTAs per cluster = 128-wide slices of either head dimension.
template <int MODE, int NSL>
__global__ void __launch_bounds__(kFThreads, 1)
fused_pair_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                  const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapV,
                  const __grid_constant__ CUtensorMap mapO, FusedArgs a, const int* __restrict__ strong_flag,
                  int32_t* dev_status) {
    constexpr int RPC = kCT / NSL;          // chunk rows whose slot rows this CTA finishes
    constexpr int TPR = 2 * NSL;            // threads per such row
    constexpr int SPT = kM / TPR;           // slots per thread there (32, 16 or 8)
    const int bh = blockIdx.x / NSL;
    if (strong_flag[bh] != 0) return;       // the general kernels take this (batch, head): the whole cluster leaves
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sXq = smem;                       // first pass: xq tile (2 panels); once consumed, the landing
                                                     //   buffer of the peers' partial sums [source CTA][row][64] fp32
    unsigned char* sXk = sXq + 2 * kPanelB;          // first pass: xk tile (2 panels); once consumed, the staging
                                                     //   buffer of my partial sums [owner CTA][row][64] fp32
    unsigned char* sW = sXk + 2 * kPanelB;           // decayed input gate [hi 64 | lo 64], MN-major B of the first
                                                     //   pass, K-major / MN-major B of the second (2 panels)
    unsigned char* sS1 = sW + 2 * kPanelB;           // first-pass state copy, MN-major B [128][hi | lo]
    unsigned char* sXv = sS1 + 2 * kPanelB;          // second pass: xv tile (2 panels); then its output rows
    unsigned char* sP = sXv + 2 * kPanelB;           // second-pass queries, K-major A [128][64], high and low panel
    unsigned char* sS2 = sP + 2 * kPanelB;           // second-pass state copy, K-major B [128 (channel)][64], high and low
    FusedCtl* ctl = reinterpret_cast<FusedCtl*>(sS2 + 2 * kPanelB);

    const int tid = threadIdx.x, warp = tid >> 5, wq = warp & 3, half = (tid >> 7) & 1, row = tid & 127;
    const int sb = kHS * half;
    const int rank = (int)cluster_rank();            // == blockIdx.x % NSL
    const int b = bh / a.H, h = bh % a.H;
    const int d0 = rank * kDST;

    if (tid == 0) {
        uint64_t* one[] = {&ctl->bar_x1, &ctl->bar_w, &ctl->bar_xv, &ctl->bar_p1, &ctl->bar_s1, &ctl->bar_o1,
                           &ctl->bar_p2, &ctl->bar_s2, &ctl->bar_o2, &ctl->bar_fx1, &ctl->bar_fw, &ctl->bar_init,
                           &ctl->bar_pm1, &ctl->bar_sb1, &ctl->bar_pm2, &ctl->bar_sb2, &ctl->bar_out, &ctl->bar_rxdone};
        for (uint64_t* bar : one) mbar_init(bar, 1);
        mbar_init(&ctl->bar_rxfree, NSL);
        mbar_init(&ctl->bar_pfree, NSL);
        mbar_init(&ctl->bar_txdone, NSL > 1 ? NSL - 1 : 1);
        mbar_init(&ctl->bar_rxfull, 1);
        mbar_init(&ctl->bar_pready, 1);
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
    cluster_sync_all();                     // every CTA's barriers exist before anyone signals them
    const uint32_t tmem = ctl->tmem_slot;
    const int nchunks = (a.T + kCT - 1) / kCT;

    if (warp == kFCopy / 32) {
        if (elect_one()) {
            // =============================== copy lane: every tile load and store
            auto load_xk = [&](int n) {      // (expects the whole first-pass tile pair)
                mbar_expect_tx(&ctl->bar_x1, 4 * kPanelB);
                tma_load_4d(sXk, &mapK, &ctl->bar_x1, d0, h, n * kCT, b);
                tma_load_4d(sXk + kPanelB, &mapK, &ctl->bar_x1, d0 + 64, h, n * kCT, b);
            };
            auto load_xq = [&](int n) {
                tma_load_4d(sXq, &mapQ, &ctl->bar_x1, d0, h, n * kCT, b);
                tma_load_4d(sXq + kPanelB, &mapQ, &ctl->bar_x1, d0 + 64, h, n * kCT, b);
            };
            auto load_w = [&](int n) {
                mbar_expect_tx(&ctl->bar_w, 2 * kPanelB);
                tma_load_4d(sW, &mapW, &ctl->bar_w, 0, h, n * kCT, b);
                tma_load_4d(sW + kPanelB, &mapW, &ctl->bar_w, 64, h, n * kCT, b);
            };
            auto load_xv = [&](int n) {
                mbar_expect_tx(&ctl->bar_xv, 2 * kPanelB);
                tma_load_4d(sXv, &mapV, &ctl->bar_xv, d0, h, n * kCT, b);
                tma_load_4d(sXv + kPanelB, &mapV, &ctl->bar_xv, d0 + 64, h, n * kCT, b);
            };
            prefetch_tmap(&mapQ); prefetch_tmap(&mapK); prefetch_tmap(&mapW); prefetch_tmap(&mapV); prefetch_tmap(&mapO);
            load_xk(0);
            load_xq(0);
            load_w(0);
            load_xv(0);
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const uint32_t ph = n & 1;
                const bool more = n + 1 < nchunks;
                // the first pass's tiles are consumed once its state products are done; their places then hold
                // this CTA's staged partial sums (xk) and the peers' (xq): free again once the peers have copied
                // theirs out and this CTA has summed its rows
                FUSED_WAIT(&ctl->bar_fx1, ph);
                if (NSL > 1) FUSED_WAIT(&ctl->bar_txdone, ph);
                FUSED_WAIT(&ctl->bar_rxdone, ph);
                if (more && !ctl->abort) {
                    load_xk(n + 1);
                    load_xq(n + 1);
                }
                // the decayed input gate is consumed once the second pass's state products are done
                FUSED_WAIT(&ctl->bar_fw, ph);
                if (more && !ctl->abort) load_w(n + 1);
                // the xv tile is consumed once the second intra-chunk product is done; the output rows are
                // staged in its place, and when those have left the buffer takes the next tile
                FUSED_WAIT(&ctl->bar_out, ph);
                if (ctl->abort) break;
                tma_store_4d(&mapO, sXv, d0, h, n * kCT, b);
                tma_store_4d(&mapO, sXv + kPanelB, d0 + 64, h, n * kCT, b);
                bulk_commit();
                bulk_wait_read();
                if (more) load_xv(n + 1);
            }
        }
    } else if (warp == kFMma / 32) {
        if (elect_one()) {
            // =============================== MMA lane
            constexpr uint32_t idescP = make_idesc(128, 128, false, false);     // xq xk^T
            constexpr uint32_t idescO1 = make_idesc(128, 2 * kM, false, true);  // xq x [S_hi | S_lo] (MN-major B)
            constexpr uint32_t idescU = make_idesc(128, 2 * kM, true, true);    // x^T (MN-major A) x [W_hi | W_lo]
            constexpr uint32_t idescI = make_idesc(128, 2 * kM, false, true);   // masked P (tensor memory) x [W_hi | W_lo]
            constexpr uint32_t idescA = make_idesc(128, 128, false, false);     // Q~ K~^T
            constexpr uint32_t idescO2 = make_idesc(128, kDST, false, false);   // Q~ x state copy (K-major B)
            constexpr uint32_t idescV = make_idesc(128, kDST, false, true);     // masked A x xv (MN-major B)
            auto kmaj = [](int kk) { return (uint32_t)((kk >> 2) * kPanelB + (kk & 3) * 32); };
            auto mnmaj = [](int kk) { return (uint32_t)(kk * 2048); };
            const uint64_t dQk = desc_kmajor(smem_u32(sXq), 0), dKk = desc_kmajor(smem_u32(sXk), 0);
            const uint64_t dKm = desc_mnmajor(smem_u32(sXk), 0, kPanelB);
            const uint64_t dWm = desc_mnmajor(smem_u32(sW), 0, kPanelB);          // [W_hi | W_lo], N = 128
            const uint64_t dWk = desc_kmajor(smem_u32(sW), 0), dWkl = desc_kmajor(smem_u32(sW + kPanelB), 0);
            const uint64_t dS1 = desc_mnmajor(smem_u32(sS1), 0, kPanelB);
            const uint64_t dV = desc_mnmajor(smem_u32(sXv), 0, kPanelB);
            const uint64_t dPh = desc_kmajor(smem_u32(sP), 0), dPl = desc_kmajor(smem_u32(sP + kPanelB), 0);
            const uint64_t dS2 = desc_kmajor(smem_u32(sS2), 0), dS2l = desc_kmajor(smem_u32(sS2 + kPanelB), 0);
            FUSED_WAIT(&ctl->bar_init, 0);
            PROF_DECL
            for (int n = 0; n < nchunks && !ctl->abort; ++n) {
                const int it = n;
                (void)it;
                const uint32_t ph = n & 1;
                PROF_MARK();
                // ---- first pass: P = xq xk^T
                FUSED_WAIT(&ctl->bar_x1, ph);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + cP, desc_advance(dQk, kmaj(kk)), desc_advance(dKk, kmaj(kk)), idescP, kk > 0);
                mma_commit(&ctl->bar_p1);
                // state products: U = xk^T [W], rows = xq [S] (the U accumulator is shared with the second
                // pass: its previous contents were read when that pass's state copy was written)
                PROF_MARK();
                FUSED_WAIT(&ctl->bar_w, ph);
                PROF_MARK();
                if (n >= 1) FUSED_WAIT(&ctl->bar_sb2, (n - 1) & 1);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + cU, desc_advance(dKm, mnmaj(kk)), desc_advance(dWm, mnmaj(kk)), idescU, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kDST / 16; ++kk)
                    mma_bf16(tmem + cO1, desc_advance(dQk, kmaj(kk)), desc_advance(dS1, mnmaj(kk)), idescO1, kk > 0);
                mma_commit(&ctl->bar_s1);
                mma_commit(&ctl->bar_fx1);
                // intra-chunk product on top: masked P (bf16 high, then low part, in tensor memory) x [W]
                PROF_MARK();
                FUSED_WAIT(&ctl->bar_pm1, ph);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + cO1, tmem + cP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dWm, mnmaj(kk)), idescI, true);
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + cO1, tmem + cP + 64 * (kk >> 2) + 32 + 8 * (kk & 3), desc_advance(dWm, mnmaj(kk)), idescI,
                                true);
                mma_commit(&ctl->bar_o1);
                // ---- second pass: its state update needs no queries, U = xv^T [W] (the first pass's U has been
                // read once that pass's state copy is written)
                PROF_MARK();
                FUSED_WAIT(&ctl->bar_xv, ph);
                PROF_MARK();
                FUSED_WAIT(&ctl->bar_sb1, ph);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16(tmem + cU, desc_advance(dV, mnmaj(kk)), desc_advance(dWm, mnmaj(kk)), idescU, kk > 0);
                // A = Q~ K~^T and rows = Q~ [S] once the queries of the chunk have landed from every CTA
                // (high/low pairs on both factors, low x low dropped)
                PROF_MARK();
                FUSED_WAIT_CLUSTER(&ctl->bar_pready, ph);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cP, desc_advance(dPh, kmaj(kk)), desc_advance(dWk, kmaj(kk)), idescA, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cP, desc_advance(dPl, kmaj(kk)), desc_advance(dWk, kmaj(kk)), idescA, true);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cP, desc_advance(dPh, kmaj(kk)), desc_advance(dWkl, kmaj(kk)), idescA, true);
                mma_commit(&ctl->bar_p2);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cO2, desc_advance(dPh, kmaj(kk)), desc_advance(dS2, kmaj(kk)), idescO2, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cO2, desc_advance(dPl, kmaj(kk)), desc_advance(dS2, kmaj(kk)), idescO2, true);
#pragma unroll
                for (int kk = 0; kk < kM / 16; ++kk)
                    mma_bf16(tmem + cO2, desc_advance(dPh, kmaj(kk)), desc_advance(dS2l, kmaj(kk)), idescO2, true);
                mma_commit(&ctl->bar_s2);
                mma_commit(&ctl->bar_fw);
                // intra-chunk product on top: masked A (high, low) x xv
                PROF_MARK();
                FUSED_WAIT(&ctl->bar_pm2, ph);
                tc_fence_after_sync();
                PROF_MARK();
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + cO2, tmem + cP + 64 * (kk >> 2) + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)), idescV, true);
#pragma unroll
                for (int kk = 0; kk < kCT / 16; ++kk)
                    mma_bf16_ta(tmem + cO2, tmem + cP + 64 * (kk >> 2) + 32 + 8 * (kk & 3), desc_advance(dV, mnmaj(kk)), idescV,
                                true);
                mma_commit(&ctl->bar_o2);
                PROF_MARK();
                PROF_DUMP("fused mma");
            }
        }
    } else if (tid < kComputeThreads) {
        // =============================== compute threads
        // state slices, row = channel: S1[c][s] (first pass), S2[c][s] (second pass, transposed), slots sb .. sb+31
        float S1[kHS], S2[kHS];
#pragma unroll
        for (int s = 0; s < kHS; ++s) {
            S1[s] = a.S1_0 ? a.S1_0[((size_t)bh * kM + sb + s) * a.D1 + d0 + row] : 0.f;
            S2[s] = a.S2_0 ? a.S2_0[((size_t)bh * kM + sb + s) * a.D2 + d0 + row] : 0.f;
        }
        store_state_row_split<false>(sS1, sS1 + kPanelB, row, sb, S1, nullptr);
        store_state_row_split<false>(sS2, sS2 + kPanelB, row, sb, S2, nullptr);
        auto chunk_gc = [&](int n) {
            const int last = min(n * kCT + kCT, a.T) - 1;
            return a.G[(((size_t)b * a.T + last) * a.H + h) * kM + tid];
        };
        float g_next = 0.f;
        if (tid < kM) {
            ctl->egc[0][tid] = __expf(chunk_gc(0));
            if (nchunks > 1) g_next = chunk_gc(1);
        }
        publish(&ctl->bar_init, tid);

        // the rows this CTA finishes: local row lr of the chunk's rows [rank * RPC, rank * RPC + RPC), part
        // `part` of its 64 slots
        const int lr = tid / TPR, part = tid % TPR;
        const int gr = rank * RPC + lr;              // row of the chunk
        const int s0 = part * SPT;                   // first slot
        // where this thread stages its first-pass partial sums: block of the CTA that owns the row (row / RPC),
        // row (row % RPC) of it; 16-byte cells of a 256-byte row are XOR-swizzled by the row (bank conflicts)
        unsigned char* tx_row = sXk + (size_t)(row * kM) * 4;
        const uint32_t swz_tx = (uint32_t)((row % RPC) & 7), swz_rx = (uint32_t)(lr & 7);
        constexpr uint32_t kBlockB = RPC * kM * 4;            // bytes of one CTA's rows: 32 KB / cluster size

        PROF_DECL
        for (int n = 0; n < nchunks; ++n) {
            const int it = n;
            (void)it;
            PROF_MARK();
            const uint32_t ph = n & 1;
            const int valid = min(kCT, a.T - n * kCT);
            const float* egc = ctl->egc[n & 1];
            if (tid < kM && n + 1 < nchunks) {
                ctl->egc[(n + 1) & 1][tid] = __expf(g_next);
                if (n + 2 < nchunks) g_next = chunk_gc(n + 2);
            }
            // ---- first pass: masked P rows (the barrier inside also publishes egc)
            FUSED_WAIT(&ctl->bar_p1, ph);
            tc_fence_after_sync();
            PROF_MARK();
            mask_row_in_tmem<false, true>(tmem, wq, row, half, cP);
            publish(&ctl->bar_pm1, tid);
            PROF_MARK();

            // ---- first-pass state: S1 <- exp(G_C) (S1 + U)
            FUSED_WAIT(&ctl->bar_s1, ph);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, cU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, cU + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; e += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) S1[e + t] = (S1[e + t] + (v[e + t] + vl[e + t])) * ecv[t];
                }
            }
            store_state_row_split<false>(sS1, sS1 + kPanelB, row, sb, S1, nullptr);
            publish(&ctl->bar_sb1, tid);
            // this CTA's xq tile has been consumed (bar_s1 covers P and the state products): its place may
            // take the peers' partial sums
            if (tid < NSL) mbar_arrive_peer(peer_addr(smem_u32(&ctl->bar_rxfree), (uint32_t)tid));

            PROF_MARK();
            // ---- row factor and (backward) logits of the rows this thread will finish, ahead of their use
            const int grow = n * kCT + min(gr, valid - 1);
            const size_t mrow = (((size_t)b * a.T + grow) * a.H + h) * kM + s0;
            float eg[SPT], zin[MODE == 1 ? SPT : 1];
#pragma unroll
            for (int i = 0; i < SPT; i += 4) {
                const float4 g4 = *reinterpret_cast<const float4*>(a.G + mrow + i);
                eg[i] = g4.x; eg[i + 1] = g4.y; eg[i + 2] = g4.z; eg[i + 3] = g4.w;
                if constexpr (MODE == 1) {
                    const float4 z4 = *reinterpret_cast<const float4*>(a.ok + mrow + i);
                    zin[i] = z4.x; zin[i + 1] = z4.y; zin[i + 2] = z4.z; zin[i + 3] = z4.w;
                }
            }

            // ---- first-pass rows (inter + intra, high + low weight parts) -> the CTA that owns the row
            FUSED_WAIT(&ctl->bar_o1, ph);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float vo[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, cO1 + sb), vo);
                tmem_ld32(tmem_row_addr(tmem, wq, cO1 + kM + sb), vl);
#pragma unroll
                for (int e = 0; e < kHS; ++e) vo[e] += vl[e];
#pragma unroll
                for (int c = 0; c < kHS / 4; ++c)
                    *reinterpret_cast<float4*>(tx_row + (((uint32_t)(sb / 4 + c) ^ swz_tx) * 16u)) =
                        make_float4(vo[4 * c], vo[4 * c + 1], vo[4 * c + 2], vo[4 * c + 3]);
            }
            PROF_MARK();
            fence_async_smem();
            tc_fence_before_sync();
            compute_sync();
            if (tid == 0) {
                // the rows that peers own go out, one bulk copy per peer, once every landing buffer is free
                if (NSL > 1) {
                    FUSED_WAIT(&ctl->bar_rxfree, ph);
                    mbar_expect_tx(&ctl->bar_rxfull, (NSL - 1) * kBlockB);
                    if (!ctl->abort) {
#pragma unroll
                        for (int d = 0; d < NSL; ++d) {
                            if (d == rank) continue;
                            bulk_copy_to_peer(peer_addr(smem_u32(sXq) + (uint32_t)rank * kBlockB, (uint32_t)d),
                                              smem_u32(sXk) + (uint32_t)d * kBlockB, kBlockB,
                                              peer_addr(smem_u32(&ctl->bar_rxfull), (uint32_t)d));
                        }
                    }
                } else {
                    mbar_arrive(&ctl->bar_rxfull);
                }
            }
            PROF_MARK();

            // ---- sum the slices of my rows, row factor, non-linearity
            FUSED_WAIT_CLUSTER(&ctl->bar_rxfull, ph);
            PROF_MARK();
            // (the peers' copies into my landing buffer are done: their staging buffers may be refilled)
            if (NSL > 1 && tid < NSL && tid != rank) mbar_arrive_peer(peer_addr(smem_u32(&ctl->bar_txdone), (uint32_t)tid));
            float z[SPT];
#pragma unroll
            for (int i = 0; i < SPT; ++i) z[i] = 0.f;
#pragma unroll
            for (int src = 0; src < NSL; ++src) {
                const unsigned char* rrow = (src == rank ? sXk : sXq) + (size_t)((src * RPC + lr) * kM) * 4;
#pragma unroll
                for (int c = 0; c < SPT / 4; ++c) {
                    const float4 t = *reinterpret_cast<const float4*>(rrow + (((uint32_t)(s0 / 4 + c) ^ swz_rx) * 16u));
                    z[4 * c] += t.x; z[4 * c + 1] += t.y; z[4 * c + 2] += t.z; z[4 * c + 3] += t.w;
                }
            }
#pragma unroll
            for (int i = 0; i < SPT; ++i) eg[i] = __expf(eg[i]);
            float e[SPT], dzv[MODE == 1 ? SPT : 1], uv[MODE == 1 ? SPT : 1];
            if constexpr (MODE == 0) {
                float zmax = -INFINITY;
#pragma unroll
                for (int i = 0; i < SPT; ++i) {
                    z[i] = z[i] * eg[i] * a.scale;
                    zmax = fmaxf(zmax, z[i]);
                }
                if (a.act == GSA_ACT_SOFTMAX) {
#pragma unroll
                    for (int o = TPR / 2; o; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
                    float den = 0.f;
#pragma unroll
                    for (int i = 0; i < SPT; ++i) { e[i] = __expf(z[i] - zmax); den += e[i]; }
#pragma unroll
                    for (int o = TPR / 2; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
                    const float inv = 1.f / den;
#pragma unroll
                    for (int i = 0; i < SPT; ++i) e[i] *= inv;
                } else {
#pragma unroll
                    for (int i = 0; i < SPT; ++i) e[i] = slot_act_value(z[i], a.act);
                }
                if (a.ok != nullptr && gr < valid) {
#pragma unroll
                    for (int i = 0; i < SPT; i += 4)
                        *reinterpret_cast<float4*>(a.ok + mrow + i) = make_float4(z[i], z[i + 1], z[i + 2], z[i + 3]);
                }
            } else {
                // z = gradient w.r.t. the second pass's queries; zin = the scaled logits
                float zmax = -INFINITY;
#pragma unroll
                for (int i = 0; i < SPT; ++i) {
                    z[i] *= eg[i];
                    zmax = fmaxf(zmax, zin[i]);
                }
                if (a.act == GSA_ACT_SOFTMAX) {
#pragma unroll
                    for (int o = TPR / 2; o; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
                    float den = 0.f;
#pragma unroll
                    for (int i = 0; i < SPT; ++i) { e[i] = __expf(zin[i] - zmax); den += e[i]; }
#pragma unroll
                    for (int o = TPR / 2; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
                    const float inv = 1.f / den;
                    float pdp = 0.f;
#pragma unroll
                    for (int i = 0; i < SPT; ++i) { e[i] *= inv; pdp += e[i] * z[i]; }
#pragma unroll
                    for (int o = TPR / 2; o; o >>= 1) pdp += __shfl_xor_sync(0xffffffffu, pdp, o);
#pragma unroll
                    for (int i = 0; i < SPT; ++i) {
                        const float dok = e[i] * (z[i] - pdp);
                        dzv[i] = a.scale * dok;
                        uv[i] = e[i] * z[i] + zin[i] * dok;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < SPT; ++i) {
                        e[i] = slot_act_value(zin[i], a.act);
                        const float dok = slot_act_slope(zin[i], a.act) * z[i];
                        dzv[i] = a.scale * dok;
                        uv[i] = e[i] * z[i] + zin[i] * dok;
                    }
                }
                if (gr < valid) {
                    __nv_bfloat16* prow = a.Pd + 2 * (mrow - s0);
                    __nv_bfloat16* zrow = a.Zd + 2 * (mrow - s0);
#pragma unroll
                    for (int i = 0; i < SPT; i += 4)
                        *reinterpret_cast<float4*>(a.u + mrow + i) = make_float4(uv[i], uv[i + 1], uv[i + 2], uv[i + 3]);
#pragma unroll
                    for (int i = 0; i < SPT; i += 8) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) split2(e[i + 2 * t] * eg[i + 2 * t], e[i + 2 * t + 1] * eg[i + 2 * t + 1], hi[t], lo[t]);
                        *reinterpret_cast<uint4*>(prow + s0 + i) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<uint4*>(prow + kM + s0 + i) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
#pragma unroll
                        for (int t = 0; t < 4; ++t) split2(dzv[i + 2 * t] * eg[i + 2 * t], dzv[i + 2 * t + 1] * eg[i + 2 * t + 1], hi[t], lo[t]);
                        *reinterpret_cast<uint4*>(zrow + s0 + i) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                        *reinterpret_cast<uint4*>(zrow + kM + s0 + i) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    }
                }
            }
            // ---- the second pass's queries (forward: p exp(G); backward: dz exp(G)) as bf16 high / low rows of
            // EVERY CTA's operand buffer: those buffers were consumed by the previous chunk's second pass
            PROF_MARK();
#pragma unroll
            for (int i = 0; i < SPT; i += 8) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float x0, x1;
                    if constexpr (MODE == 0) { x0 = e[i + 2 * t]; x1 = e[i + 2 * t + 1]; }
                    else { x0 = dzv[i + 2 * t]; x1 = dzv[i + 2 * t + 1]; }
                    split2(x0 * eg[i + 2 * t], x1 * eg[i + 2 * t + 1], hi[t], lo[t]);
                }
                unsigned char* cell = sP + swz128((uint32_t)gr, (uint32_t)((s0 + i) >> 3));
                *reinterpret_cast<uint4*>(cell) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(cell + kPanelB) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
            PROF_MARK();
            fence_async_smem();
            compute_sync();
            if (tid == 0) {
                // my rows of the operand (RPC rows of 128 bytes, high and low panel) to every peer, once all
                // operand buffers have been consumed by the previous chunk's second pass
                if (NSL > 1) {
                    if (n >= 1) FUSED_WAIT(&ctl->bar_pfree, (n - 1) & 1);
                    mbar_expect_tx(&ctl->bar_pready, (NSL - 1) * 2 * RPC * 128);
                    if (!ctl->abort) {
                        const uint32_t rows = smem_u32(sP) + (uint32_t)(rank * RPC) * 128u;
#pragma unroll
                        for (int d = 0; d < NSL; ++d) {
                            if (d == rank) continue;
                            const uint32_t bar = peer_addr(smem_u32(&ctl->bar_pready), (uint32_t)d);
                            bulk_copy_to_peer(peer_addr(rows, (uint32_t)d), rows, RPC * 128, bar);
                            bulk_copy_to_peer(peer_addr(rows + kPanelB, (uint32_t)d), rows + kPanelB, RPC * 128, bar);
                        }
                    }
                } else {
                    mbar_arrive(&ctl->bar_pready);
                }
                mbar_arrive(&ctl->bar_rxdone);
            }
            PROF_MARK();

            // ---- second pass: masked A rows
            FUSED_WAIT(&ctl->bar_p2, ph);
            tc_fence_after_sync();
            PROF_MARK();
            mask_row_in_tmem<false, true>(tmem, wq, row, half, cP);
            publish(&ctl->bar_pm2, tid);
            PROF_MARK();

            // ---- second-pass state: S2 <- exp(G_C) (S2 + U^T)
            FUSED_WAIT(&ctl->bar_s2, ph);
            tc_fence_after_sync();
            PROF_MARK();
            {
                float v[kHS], vl[kHS];
                tmem_ld32(tmem_row_addr(tmem, wq, cU + sb), v);
                tmem_ld32(tmem_row_addr(tmem, wq, cU + kM + sb), vl);
#pragma unroll
                for (int e2 = 0; e2 < kHS; e2 += 4) {
                    const float4 ec = *reinterpret_cast<const float4*>(&egc[sb + e2]);
                    const float ecv[4] = {ec.x, ec.y, ec.z, ec.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) S2[e2 + t] = (S2[e2 + t] + (v[e2 + t] + vl[e2 + t])) * ecv[t];
                }
            }
            store_state_row_split<false>(sS2, sS2 + kPanelB, row, sb, S2, nullptr);
            publish(&ctl->bar_sb2, tid);
            // this CTA's query buffer has been consumed (bar_s2 covers A and the state products)
            if (tid < NSL) mbar_arrive_peer(peer_addr(smem_u32(&ctl->bar_pfree), (uint32_t)tid));

            // ---- second-pass rows -> bf16, staged in the xv tile for the tiled store (clipped at the sequence end)
            PROF_MARK();
            FUSED_WAIT(&ctl->bar_o2, ph);
            tc_fence_after_sync();
            PROF_MARK();
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                float v[32];
                tmem_ld32(tmem_row_addr(tmem, wq, cO2 + 64 * half + c0), v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float x[8] = {v[8 * c], v[8 * c + 1], v[8 * c + 2], v[8 * c + 3],
                                        v[8 * c + 4], v[8 * c + 5], v[8 * c + 6], v[8 * c + 7]};
                    store_chunk(sXv + half * kPanelB, row, (c0 >> 3) + c, x);
                }
            }
            const bool stop = publish_and_vote(&ctl->bar_out, tid, ctl->abort != 0);
            PROF_MARK();
            PROF_DUMP("fused compute");
            if (stop) break;
        }
        if (!ctl->abort) {
            if (a.S1_end) {
#pragma unroll
                for (int s = 0; s < kHS; ++s) a.S1_end[((size_t)bh * kM + sb + s) * a.D1 + d0 + row] = S1[s];
            }
            if (a.S2_end) {
#pragma unroll
                for (int s = 0; s < kHS; ++s) a.S2_end[((size_t)bh * kM + sb + s) * a.D2 + d0 + row] = S2[s];
            }
        }
    }
    // ---- all roles meet; no CTA of the cluster leaves (and gives up its shared memory) while a peer may
    // still write to it
    tc_fence_before_sync();
    __syncthreads();
    if (ctl->abort) {
        if (tid == 0 && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

constexpr size_t kSmemFused = 1024 + 14 * kPanelB + sizeof(FusedCtl);

template <int MODE, int NSL>
cudaError_t launch_one(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mw, const CUtensorMap& mv,
                       const CUtensorMap& mo, const FusedArgs& a, const int* strong, cudaStream_t st, int32_t* dev_status) {
    auto kernel = fused_pair_kernel<MODE, NSL>;
    cudaError_t e = prepare(kernel, kSmemFused, kFThreads);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(a.B * a.H * NSL));
    cfg.blockDim = dim3(kFThreads);
    cfg.dynamicSmemBytes = kSmemFused;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = NSL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (NSL > 1) {
        int nclusters = 0;
        e = cudaOccupancyMaxActiveClusters(&nclusters, kernel, &cfg);
        if (e != cudaSuccess) return e;
        if (nclusters < 1) return cudaErrorLaunchOutOfResources;
    }
    return cudaLaunchKernelEx(&cfg, kernel, mq, mk, mw, mv, mo, a, strong, dev_status);
}

}  // namespace

bool fused_pair_supported(int d_k, int d_v, int M) {
    if (M != kM || d_k != d_v) return false;
    return d_k == 128 || d_k == 256 || d_k == 512;
}

// mode 0: xq1 = q, xk1 = k, xv = v, out = o; mode 1: xq1 = dO, xk1 = v, xv = k, out = dq.
cudaError_t launch_fused_pair(int mode, const void* xq1, const void* xk1, const void* wd, const void* xv, void* out,
                              const float* G, const float* S1_0, const float* S2_0, float* S1_end, float* S2_end, int B,
                              int T, int H, int D1, int D2, float scale, int act, float* ok, float* u, void* Pd,
                              void* Zd, const int* strong_flag, cudaStream_t st, int32_t* dev_status) {
    if (D1 != D2 || D1 % kDST != 0 || strong_flag == nullptr || wd == nullptr) return cudaErrorInvalidValue;
    if (mode == 1 && (ok == nullptr || u == nullptr || Pd == nullptr || Zd == nullptr)) return cudaErrorInvalidValue;
    CUtensorMap mq, mk, mw, mv, mo;
    cudaError_t e = make_tensor_map_bthd(&mq, xq1, B, T, H, D1, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mk, xk1, B, T, H, D1, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mw, wd, B, T, H, 2 * kM, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mv, xv, B, T, H, D2, kCT, 2);
    if (e == cudaSuccess) e = make_tensor_map_bthd(&mo, out, B, T, H, D2, kCT, 2);
    if (e != cudaSuccess) return e;
    FusedArgs a{G, S1_0, S2_0, S1_end, S2_end, B, T, H, D1, D2, scale, act, ok, u,
                static_cast<__nv_bfloat16*>(Pd), static_cast<__nv_bfloat16*>(Zd)};
    const int nsl = D1 / kDST;
#define GSA_FUSED_CASE(MODE_, NSL_) \
    if (mode == MODE_ && nsl == NSL_) return launch_one<MODE_, NSL_>(mq, mk, mw, mv, mo, a, strong_flag, st, dev_status)
    GSA_FUSED_CASE(0, 1);
    GSA_FUSED_CASE(0, 2);
    GSA_FUSED_CASE(0, 4);
    GSA_FUSED_CASE(1, 1);
    GSA_FUSED_CASE(1, 2);
    GSA_FUSED_CASE(1, 4);
#undef GSA_FUSED_CASE
    return cudaErrorNotSupported;
}

}  // namespace gsa
