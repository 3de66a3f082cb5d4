// Self-test of the tcgen05 building blocks: one 128-row product per operand-layout
// combination that the chunk kernels use, on caller-provided 128 x 128 bf16 matrices.
// It exists so that a wrong matrix descriptor or swizzle shows up in isolation.
#include "common.cuh"
#include "gsa_dev.h"
#include "tc_common.cuh"

namespace gsa {

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t get_encoder(EncodeFn* out) {
    static EncodeFn encode = nullptr;
    if (encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    *out = encode;
    return cudaSuccess;
}
}  // namespace

cudaError_t make_tensor_map_sliced(CUtensorMap* map, const void* base, int nslice, int B, int T, int H, int D,
                                   int box_rows, int elem_bytes) {
    EncodeFn encode;
    cudaError_t e = get_encoder(&encode);
    if (e != cudaSuccess) return e;
    const cuuint64_t eb = (cuuint64_t)elem_bytes;
    const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B, (cuuint64_t)nslice};
    const cuuint64_t strides[4] = {(cuuint64_t)D * eb, (cuuint64_t)H * D * eb, (cuuint64_t)T * H * D * eb,
                                   (cuuint64_t)B * T * H * D * eb};
    const cuuint32_t box[5] = {(cuuint32_t)(128 / elem_bytes), 1, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    const cuuint32_t rank = nslice > 0 ? 5 : 4;
    CUresult r = encode(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                        rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t make_tensor_map_bthd(CUtensorMap* map, const void* base, int B, int T, int H, int D, int box_rows,
                                 int elem_bytes) {
    return make_tensor_map_sliced(map, base, 0, B, T, H, D, box_rows, elem_bytes);
}

namespace {
using namespace tc;

constexpr int kPanel = 128 * 128;   // bytes of a 128-row panel

__global__ void __launch_bounds__(128) tc_selftest_kernel(const __grid_constant__ CUtensorMap mapX,
                                                          const __grid_constant__ CUtensorMap mapY,
                                                          const __nv_bfloat16* __restrict__ X,
                                                          const __nv_bfloat16* __restrict__ Y, int mode,
                                                          float* __restrict__ D, int32_t* dev_status) {
    extern __shared__ unsigned char smem_raw[];
    // align by pointer arithmetic (not an integer round trip) so accesses stay in the shared window
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sX = smem;                  // 2 panels (TMA)
    unsigned char* sY = smem + 2 * kPanel;     // 2 panels (TMA)
    unsigned char* sW = smem + 4 * kPanel;     // 2 panels written by threads
    __shared__ uint64_t bar_load, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;

    if (tid == 0) {
        mbar_init(&bar_load, 1);
        mbar_init(&bar_mma, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&tmem_slot, 256);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;

    if (tid == 0) {
        mbar_expect_tx(&bar_load, 4 * kPanel);
        tma_load_4d(sX, &mapX, &bar_load, 0, 0, 0, 0);
        tma_load_4d(sX + kPanel, &mapX, &bar_load, 64, 0, 0, 0);
        tma_load_4d(sY, &mapY, &bar_load, 0, 0, 0, 0);
        tma_load_4d(sY + kPanel, &mapY, &bar_load, 64, 0, 0, 0);
    }
    // operands written by threads
    if (mode == 1) {          // A = X as K-major panels: thread = row
        for (int c = 0; c < 16; ++c) {
            float x[8];
            for (int e = 0; e < 8; ++e) x[e] = __bfloat162float(X[tid * 128 + c * 8 + e]);
            store_chunk(sW + (c >> 3) * kPanel, tid, c & 7, x);
        }
    } else if (mode == 2) {   // B K-major [N = 64 rows s][K = 128 (j)]: Z[s][j] = Y[s][j]; thread j writes column j
        for (int s = 0; s < 64; ++s)
            store_elem(sW + (tid >> 6) * (64 * 128), s, tid & 63, __bfloat162float(Y[s * 128 + tid]));
    } else if (mode == 3) {   // B MN-major [K = 128 rows c][N = 64]: Sb[c][s] = Y[c][s]; thread c writes its row
        for (int c = 0; c < 8; ++c) {
            float x[8];
            for (int e = 0; e < 8; ++e) x[e] = __bfloat162float(Y[tid * 128 + c * 8 + e]);
            store_chunk(sW, tid, c, x);
        }
    }
    else if (mode >= 4) {   // A = X in tensor memory: thread = row = lane, 64 packed columns from 128 on
        for (int c0 = 0; c0 < 64; c0 += 16) {
            uint32_t r[16];
            for (int e = 0; e < 16; ++e)
                r[e] = pack_bf16(__bfloat162float(X[tid * 128 + 2 * (c0 + e)]), __bfloat162float(X[tid * 128 + 2 * (c0 + e) + 1]));
            tmem_st16(tmem_row_addr(tmem, warp, 128 + c0), r);
        }
        tmem_st_wait();
        tc_fence_before_sync();
    }
    fence_async_smem();
    __syncthreads();
    bool ok = mbar_wait(&bar_load, 0);
    const int N = (mode <= 1 || mode >= 4) ? 128 : 64;
    if (ok && tid == 0) {
        tc_fence_after_sync();
        const uint32_t aX = smem_u32(sX), aY = smem_u32(sY), aW = smem_u32(sW);
        for (int kk = 0; kk < 8; ++kk) {
            uint64_t da, db;
            uint32_t idesc;
            if (mode == 0) {
                da = desc_kmajor(aX + (kk >> 2) * kPanel, kk);
                db = desc_kmajor(aY + (kk >> 2) * kPanel, kk);
                idesc = make_idesc(128, 128, false, false);
            } else if (mode == 1) {
                da = desc_kmajor(aW + (kk >> 2) * kPanel, kk);
                db = desc_mnmajor(aY, kk, kPanel);
                idesc = make_idesc(128, 128, false, true);
            } else if (mode == 2) {
                da = desc_mnmajor(aX, kk, kPanel);
                db = desc_kmajor(aW + (kk >> 2) * (64 * 128), kk);
                idesc = make_idesc(128, 64, true, false);
            } else if (mode == 3) {
                da = desc_kmajor(aX + (kk >> 2) * kPanel, kk);
                db = desc_mnmajor(aW, kk, kPanel);
                idesc = make_idesc(128, 64, false, true);
            } else {
                // A from tensor memory; B = Y K-major (mode 4: X Y^T) or MN-major (mode 5: X Y)
                db = mode == 4 ? desc_kmajor(aY + (kk >> 2) * kPanel, kk) : desc_mnmajor(aY, kk, kPanel);
                idesc = make_idesc(128, 128, false, mode == 5);
                mma_bf16_ta(tmem, tmem + 128 + 8 * kk, db, idesc, kk > 0);
                continue;
            }
            mma_bf16(tmem, da, db, idesc, kk > 0);
        }
        mma_commit(&bar_mma);
    }
    ok = ok && mbar_wait(&bar_mma, 0);
    tc_fence_after_sync();
    if (ok) {
        for (int c0 = 0; c0 < N; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_row_addr(tmem, warp, c0), v);
            for (int e = 0; e < 16; ++e) D[tid * N + c0 + e] = v[e];
        }
    } else if (dev_status != nullptr) {
        *dev_status = GSA_ERR_TIMEOUT;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem, 256);
    }
}
// The bounded wait itself: one CTA waits on an mbarrier that nothing will ever signal, with the
// given limit; the wait must give up, the CTA must report GSA_ERR_TIMEOUT through dev_status the way
// the chunk kernels do (flag, release tensor memory, return), and the context must stay usable.
__global__ void __launch_bounds__(128) wait_expiry_kernel(uint64_t limit_ns, int32_t* dev_status, uint32_t* waited_us) {
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&tmem_slot, 32);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint64_t t0 = global_timer_ns();
    const bool done = mbar_wait(&bar, 0, limit_ns);          // nobody arrives: must expire
    const uint64_t t1 = global_timer_ns();
    if (tid == 0) {
        if (!done && dev_status != nullptr) *dev_status = GSA_ERR_TIMEOUT;
        if (waited_us != nullptr) *waited_us = (uint32_t)((t1 - t0) / 1000u);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_slot, 32);
    }
}
}  // namespace
}  // namespace gsa

extern "C" GSA_API gsa_status_t gsa_wait_selftest(uint32_t limit_us, void* stream, int32_t* dev_status, uint32_t* waited_us) {
    if (limit_us < 1 || limit_us > 100000 || dev_status == nullptr) return GSA_ERR_INVALID_ARG;    // at most 0.1 s
    gsa::wait_expiry_kernel<<<1, 128, 0, static_cast<cudaStream_t>(stream)>>>((uint64_t)limit_us * 1000ull, dev_status, waited_us);
    return cudaGetLastError() == cudaSuccess ? GSA_OK : GSA_ERR_CUDA;
}

extern "C" GSA_API gsa_status_t gsa_tc_selftest(int32_t mode, const void* X, const void* Y, float* D, void* stream,
                                                int32_t* dev_status) {
    using namespace gsa;
    if (mode < 0 || mode > 5 || X == nullptr || Y == nullptr || D == nullptr) return GSA_ERR_INVALID_ARG;
    CUtensorMap mx, my;
    if (make_tensor_map_bthd(&mx, X, 1, 128, 1, 128, 128, 2) != cudaSuccess) return GSA_ERR_CUDA;
    if (make_tensor_map_bthd(&my, Y, 1, 128, 1, 128, 128, 2) != cudaSuccess) return GSA_ERR_CUDA;
    const size_t smem = 6 * kPanel + 1024;
    if (cudaFuncSetAttribute(tc_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return GSA_ERR_CUDA;
    tc_selftest_kernel<<<1, 128, smem, static_cast<cudaStream_t>(stream)>>>(
        mx, my, (const __nv_bfloat16*)X, (const __nv_bfloat16*)Y, mode, D, dev_status);
    return cudaGetLastError() == cudaSuccess ? GSA_OK : GSA_ERR_CUDA;
}
