// Pieces shared by the tensor-core chunk kernels (the general ones, which also carry the
// strong-decay path, and the pipelined lean ones): tile geometry, accumulator columns, row
// access to swizzled fp32 tiles, operand-row stores and the compute-thread barrier.
#pragma once
#include <stdio.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace gsa {
namespace tcchunk {
using namespace tc;

constexpr int kCT = 128;               // chunk length of the tensor-core kernels
constexpr int kDST = 128;              // head-dimension slice per CTA
constexpr int kM = 64;                 // slots
constexpr int kPanelB = 128 * 128;     // bytes of a 128-row operand panel
constexpr uint32_t kTmemCols = 512;
constexpr int kComputeThreads = 256;   // 8 warps: two threads per chunk row
constexpr int kThreads = kComputeThreads + 32;   // + the issuing warp (TMA and MMA), one lane active
constexpr int kHS = kM / 2;            // slots per thread

// accumulator columns
constexpr int kColP = 0;       // P / A           [128 x 128]
constexpr int kColO = 128;     // inter (+ intra for key_side) output
constexpr int kColU = 256;     // state update    [128 x 64] (value_side: [128 x 128], high | low weight parts)
constexpr int kColO2 = 384;    // value_side: intra-chunk output [128 x 128], high | low weight parts

// Optional phase timing for development builds (-DGSA_TC_PROF): CTA 0 prints, for its fifth
// chunk, the SM clock at each phase boundary.
#ifdef GSA_TC_PROF
#define PROF_DECL long long prof_t[32]; int prof_n = 0;
#define PROF_MARK() do { if (prof_n < 32) prof_t[prof_n++] = clock64(); } while (0)
#ifdef GSA_TC_PROF_ABS
#define PROF_DUMP(name) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (tid == 0 || tid == 256) && (it == 5 || it == 6)) { \
    long long b_ = prof_t[0] % 1000000; for (int i_ = prof_n; i_ < 16; ++i_) prof_t[i_] = prof_t[0]; \
    printf("%s tid %d it %d base %lld: %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld %lld\n", name, (int)tid, it, b_, \
           prof_t[1] - prof_t[0], prof_t[2] - prof_t[0], prof_t[3] - prof_t[0], prof_t[4] - prof_t[0], prof_t[5] - prof_t[0], \
           prof_t[6] - prof_t[0], prof_t[7] - prof_t[0], prof_t[8] - prof_t[0], prof_t[9] - prof_t[0], prof_t[10] - prof_t[0], \
           prof_t[11] - prof_t[0], prof_t[12] - prof_t[0], prof_t[13] - prof_t[0], prof_t[14] - prof_t[0], prof_t[15] - prof_t[0]); } \
    prof_n = 0; } while (0)
#else
#define PROF_DUMP(name) do { if (blockIdx.x == 0 && blockIdx.y == 0 && ((tid == 0 && it == 6) || (tid == 256 && it == 4))) { \
    printf("%s:", name); for (int i_ = 1; i_ < prof_n; ++i_) printf(" %lld", prof_t[i_] - prof_t[i_ - 1]); printf("\n"); } prof_n = 0; } while (0)
#endif
#else
#define PROF_DECL
#define PROF_MARK() do {} while (0)
#define PROF_DUMP(name) do {} while (0)
#endif

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
// 8 consecutive floats from a 16-byte aligned plain (unswizzled) row
__device__ __forceinline__ void tile_free_row8(const float* p, float (&x)[8]) {
    const float4 t0 = *reinterpret_cast<const float4*>(p);
    const float4 t1 = *reinterpret_cast<const float4*>(p + 4);
    x[0] = t0.x; x[1] = t0.y; x[2] = t0.z; x[3] = t0.w;
    x[4] = t1.x; x[5] = t1.y; x[6] = t1.z; x[7] = t1.w;
}
__device__ __forceinline__ float tile_elem(const unsigned char* tile, int row, int s) {
    return *reinterpret_cast<const float*>(tile + (s >> 5) * kPanelB + swz128(row, (s & 31) >> 2) + (s & 3) * 4);
}

// bf16 copy of this thread's half state row (32 values from slot sb on, optionally scaled
// per slot) into row `row` of a one-panel operand
template <bool SCALE>
__device__ __forceinline__ void store_state_row(unsigned char* panel, int row, int sb, const float (&S)[kHS],
                                                const float* scale) {
#pragma unroll
    for (int c = 0; c < kHS / 8; ++c) {
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = SCALE ? S[8 * c + e] * scale[sb + 8 * c + e] : S[8 * c + e];
        store_chunk(panel, row, (sb >> 3) + c, x);
    }
}

// The same as a bf16 pair: the rounded copy and its rounding residual, in two panels
template <bool SCALE>
__device__ __forceinline__ void store_state_row_split(unsigned char* panel_hi, unsigned char* panel_lo, int row, int sb,
                                                      const float (&S)[kHS], const float* scale) {
#pragma unroll
    for (int c = 0; c < kHS / 8; ++c) {
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = SCALE ? S[8 * c + e] * scale[sb + 8 * c + e] : S[8 * c + e];
        store_chunk_split(panel_hi, panel_lo, row, (sb >> 3) + c, x);
    }
}

// Barrier over the 256 compute threads only (the issuing warp runs ahead on its own).
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool compute_sync_and(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool compute_sync_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}

// rows published and consumed: shared-memory writes to the async proxy, accumulator reads
// ordered before the barrier, then one arrival for the issuing lane
__device__ __forceinline__ void publish(uint64_t* bar, int tid) {
    fence_async_smem();
    tc_fence_before_sync();
    compute_sync();
    if (tid == 0) mbar_arrive(bar);
}
// the same at the end of a chunk, with the vote on leaving the loop
__device__ __forceinline__ bool publish_and_vote(uint64_t* bar, int tid, bool stop) {
    fence_async_smem();
    tc_fence_before_sync();
    const bool any = compute_sync_or(stop);
    if (tid == 0) mbar_arrive(bar);
    return any;
}

// masked accumulator row -> bf16 K-major operand row (two 64-column panels); with SPLIT the
// rounding residual goes to a second operand of the same shape (dst_lo)
template <bool REV, bool SPLIT>
__device__ __forceinline__ void store_masked_row(uint32_t tmem, int wq, int row, int half, unsigned char* dst,
                                                 unsigned char* dst_lo) {
    unsigned char* panel = dst + half * kPanelB;      // columns 64 half .. 64 half + 63
    unsigned char* panel_lo = dst_lo + half * kPanelB;
#pragma unroll 1
    for (int c0 = 0; c0 < 64; c0 += 32) {
        float v[32];
        tmem_ld32(tmem_row_addr(tmem, wq, kColP + 64 * half + c0), v);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int j = 64 * half + c0 + 8 * c + e;
                const bool keep = REV ? (j >= row) : (j <= row);
                x[e] = keep ? v[8 * c + e] : 0.f;
            }
            if (SPLIT) store_chunk_split(panel, panel_lo, row, (c0 >> 3) + c, x);
            else store_chunk(panel, row, (c0 >> 3) + c, x);
        }
    }
}

// The same into tensor memory, in place: the thread's 64 fp32 columns (64 half .. 64 half + 63 from
// `col0` on) become bf16 pairs in the first 32 of them -- the A operand of the next product, K step
// kk at column col0 + 64 (kk >> 2) + 8 (kk & 3).  With SPLIT the rounding residual follows in the
// other 32 columns (K step kk at + 32).  Every thread overwrites only columns it has read itself.
template <bool REV, bool SPLIT>
__device__ __forceinline__ void mask_row_in_tmem(uint32_t tmem, int wq, int row, int half, int col0) {
    const int base = col0 + 64 * half;
    uint32_t hi[32], lo[SPLIT ? 32 : 1];
#pragma unroll
    for (int c0 = 0; c0 < 64; c0 += 32) {
        float v[32];
        tmem_ld32(tmem_row_addr(tmem, wq, base + c0), v);
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
            const int j = 64 * half + c0 + e;
            const float x0 = (REV ? (j >= row) : (j <= row)) ? v[e] : 0.f;
            const float x1 = (REV ? (j + 1 >= row) : (j + 1 <= row)) ? v[e + 1] : 0.f;
            hi[(c0 + e) >> 1] = pack_bf16(x0, x1);
            if (SPLIT) {
                const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&hi[(c0 + e) >> 1]);
                lo[(c0 + e) >> 1] = pack_bf16(x0 - __bfloat162float(h.x), x1 - __bfloat162float(h.y));
            }
        }
        if (!SPLIT) {
            // the 16 packed columns of this batch land on columns already read
            const uint32_t (&r)[16] = *reinterpret_cast<const uint32_t (*)[16]>(&hi[c0 >> 1]);
            tmem_st16(tmem_row_addr(tmem, wq, base + (c0 >> 1)), r);
        }
    }
    if (SPLIT) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const uint32_t (&rh)[16] = *reinterpret_cast<const uint32_t (*)[16]>(&hi[16 * q]);
            const uint32_t (&rl)[16] = *reinterpret_cast<const uint32_t (*)[16]>(&lo[SPLIT ? 16 * q : 0]);
            tmem_st16(tmem_row_addr(tmem, wq, base + 16 * q), rh);
            tmem_st16(tmem_row_addr(tmem, wq, base + 32 + 16 * q), rl);
        }
    }
    tmem_st_wait();
}

// wait helper of the loops below: a wait that expires flags the CTA
#define WAIT_OR_ABORT(bar, parity)                          \
    do {                                                    \
        if (!mbar_wait(bar, parity)) ctl->abort = 1;        \
    } while (0)

template <typename K>
cudaError_t prepare(K kernel, size_t smem, int threads = kThreads) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // each CTA takes the whole tensor memory of its SM: make sure no second CTA can be co-resident
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
    if (e != cudaSuccess) return e;
    return per_sm == 1 ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

}  // namespace tcchunk
}  // namespace gsa
