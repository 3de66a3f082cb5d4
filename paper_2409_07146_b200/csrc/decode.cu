// Recurrent decode step of Gated Slot Attention: one iteration of Eq. 6 per (sequence, head).
//
// Per pair the kernel reads and rewrites both slot memories once (m*(d_k+d_v) fp32 each
// way) and does about one FMA per two bytes moved, so it is a pure HBM stream.  One CTA of
// 8 warps owns one pair; a warp owns a memory row at a time, with 16-byte accesses that
// cover the row contiguously (coalesced); rows are loaded in batches before any is used so
// that several 512-byte requests per warp are in flight.  The key memory is updated and
// read first (slot logits), then the softmax, then the value memory is updated and summed.
#include "common.cuh"

namespace gsa {

template <typename IO>
__device__ __forceinline__ float io_to_float(IO x);
template <>
__device__ __forceinline__ float io_to_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ float io_to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename IO>
__device__ __forceinline__ IO float_to_io(float x);
template <>
__device__ __forceinline__ float float_to_io<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 float_to_io<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

constexpr int kDecodeWarps = 8;

// One memory row of D floats per warp: lane l owns the float4s l, l+32, ... (D >= 128) or
// one float2 (D == 64).
template <int D>
struct RowVec {
    static constexpr int kW = (D >= 128) ? 4 : 2;      // floats per access
    static constexpr int kN = D / (32 * kW);           // accesses per lane
    float v[kN][kW];
    __device__ __forceinline__ void load(const float* row, int lane) {
#pragma unroll
        for (int r = 0; r < kN; ++r) {
            if constexpr (kW == 4) {
                float4 t = *reinterpret_cast<const float4*>(row + (lane + 32 * r) * 4);
                v[r][0] = t.x; v[r][1] = t.y; v[r][2] = t.z; v[r][3] = t.w;
            } else {
                float2 t = *reinterpret_cast<const float2*>(row + (lane + 32 * r) * 2);
                v[r][0] = t.x; v[r][1] = t.y;
            }
        }
    }
    __device__ __forceinline__ void store(float* row, int lane) const {
#pragma unroll
        for (int r = 0; r < kN; ++r) {
            if constexpr (kW == 4)
                *reinterpret_cast<float4*>(row + (lane + 32 * r) * 4) = make_float4(v[r][0], v[r][1], v[r][2], v[r][3]);
            else
                *reinterpret_cast<float2*>(row + (lane + 32 * r) * 2) = make_float2(v[r][0], v[r][1]);
        }
    }
    template <typename IO>
    __device__ __forceinline__ void load_io(const IO* row, int lane) {
#pragma unroll
        for (int r = 0; r < kN; ++r)
#pragma unroll
            for (int w = 0; w < kW; ++w) v[r][w] = io_to_float<IO>(row[(lane + 32 * r) * kW + w]);
    }
    // the layer's feature map (Sec. 3.3), applied as the token's q, k, v are loaded
    __device__ __forceinline__ void swish() {
#pragma unroll
        for (int r = 0; r < kN; ++r)
#pragma unroll
            for (int w = 0; w < kW; ++w) v[r][w] = v[r][w] / (1.f + __expf(-v[r][w]));
    }
};

template <typename IO, int DK, int DV, int M>
__global__ void __launch_bounds__(kDecodeWarps * 32)
decode_step_kernel(const IO* __restrict__ q, const IO* __restrict__ k, const IO* __restrict__ v,
                   const void* __restrict__ gate_raw, int gate_bf16, int gate_row_of_head, int feature_map, int gate_kind, float inv_tau, float scale, int act,
                   float* __restrict__ Ks, float* __restrict__ Vs, IO* __restrict__ o) {
    constexpr int RPW = M / kDecodeWarps;  // memory rows per warp
    const size_t pair = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __shared__ float s_z[M];
    __shared__ float s_p[M];
    __shared__ float s_o[kDecodeWarps][DV];

    float* Kp = Ks + pair * (size_t)M * DK;
    float* Vp = Vs + pair * (size_t)M * DV;

    RowVec<DK> qv, kv;
    RowVec<DV> vv;
    qv.load_io(q + pair * DK, lane);
    kv.load_io(k + pair * DK, lane);
    vv.load_io(v + pair * DV, lane);
    if (feature_map == GSA_FEAT_SWISH) { qv.swish(); kv.swish(); vv.swish(); }
    float a[RPW], ia[RPW];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        // (data-independent decay: one gate row per head, shared by all sequences; gate_row_of_head = H then)
        const size_t gi = (gate_row_of_head ? pair % gate_row_of_head : pair) * M + warp * RPW + r;
        float gt = gate_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(gate_raw)[gi])
                             : static_cast<const float*>(gate_raw)[gi];
        if (gate_kind == GSA_GATE_LOGITS) gt = log_gate_from_logit(gt, inv_tau);
        if (gate_kind != GSA_GATE_A) { a[r] = __expf(gt); ia[r] = -expm1f(gt); }
        else { a[r] = gt; ia[r] = 1.f - gt; }
    }

    // K~ <- a K~ + (1-a) k ; z = scale * K~ q.  Rows go through registers in batches whose
    // loads are all issued before the first use.
    constexpr int KB = (RPW * (DK / 32) <= 32) ? RPW : (32 / (DK / 32));
#pragma unroll
    for (int r0 = 0; r0 < RPW; r0 += KB) {
        RowVec<DK> kr[KB];
#pragma unroll
        for (int r = 0; r < KB; ++r) kr[r].load(Kp + (size_t)(warp * RPW + r0 + r) * DK, lane);
#pragma unroll
        for (int r = 0; r < KB; ++r) {
            float dot = 0.f;
#pragma unroll
            for (int i = 0; i < RowVec<DK>::kN; ++i)
#pragma unroll
                for (int w = 0; w < RowVec<DK>::kW; ++w) {
                    const float x = fmaf(a[r0 + r], kr[r].v[i][w], ia[r0 + r] * kv.v[i][w]);
                    kr[r].v[i][w] = x;
                    dot = fmaf(x, qv.v[i][w], dot);
                }
            kr[r].store(Kp + (size_t)(warp * RPW + r0 + r) * DK, lane);
#pragma unroll
            for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
            if (lane == 0) s_z[warp * RPW + r0 + r] = dot * scale;
        }
    }
    __syncthreads();
    // softmax over the m slots, or its element-wise replacement
    if (warp == 0 && act != GSA_ACT_SOFTMAX) {
#pragma unroll
        for (int r = 0; r < M / 32; ++r) s_p[lane + 32 * r] = slot_act_value(s_z[lane + 32 * r], act);
    } else if (warp == 0) {
        float z[M / 32], zmax = -INFINITY;
#pragma unroll
        for (int r = 0; r < M / 32; ++r) { z[r] = s_z[lane + 32 * r]; zmax = fmaxf(zmax, z[r]); }
#pragma unroll
        for (int off = 16; off; off >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, off));
        float den = 0.f;
#pragma unroll
        for (int r = 0; r < M / 32; ++r) { z[r] = __expf(z[r] - zmax); den += z[r]; }
#pragma unroll
        for (int off = 16; off; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
        const float inv = 1.f / den;
#pragma unroll
        for (int r = 0; r < M / 32; ++r) s_p[lane + 32 * r] = z[r] * inv;
    }
    __syncthreads();
    // V~ <- a V~ + (1-a) v ; o = V~^T p: each warp sums its rows, then the 8 partial rows
    // are added in a fixed order
    RowVec<DV> acc;
#pragma unroll
    for (int i = 0; i < RowVec<DV>::kN; ++i)
#pragma unroll
        for (int w = 0; w < RowVec<DV>::kW; ++w) acc.v[i][w] = 0.f;
    constexpr int VB = (RPW * (DV / 32) <= 32) ? RPW : (32 / (DV / 32));
#pragma unroll
    for (int r0 = 0; r0 < RPW; r0 += VB) {
        RowVec<DV> vr[VB];
#pragma unroll
        for (int r = 0; r < VB; ++r) vr[r].load(Vp + (size_t)(warp * RPW + r0 + r) * DV, lane);
#pragma unroll
        for (int r = 0; r < VB; ++r) {
            const float pr = s_p[warp * RPW + r0 + r];
#pragma unroll
            for (int i = 0; i < RowVec<DV>::kN; ++i)
#pragma unroll
                for (int w = 0; w < RowVec<DV>::kW; ++w) {
                    const float x = fmaf(a[r0 + r], vr[r].v[i][w], ia[r0 + r] * vv.v[i][w]);
                    vr[r].v[i][w] = x;
                    acc.v[i][w] = fmaf(pr, x, acc.v[i][w]);
                }
            vr[r].store(Vp + (size_t)(warp * RPW + r0 + r) * DV, lane);
        }
    }
    acc.store(&s_o[warp][0], lane);
    __syncthreads();
    for (int c = threadIdx.x; c < DV; c += kDecodeWarps * 32) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) sum += s_o[w][c];
        o[pair * DV + c] = float_to_io<IO>(sum);
    }
}

template <typename IO, int DK, int DV>
static cudaError_t launch_decode_m(const gsa_params_t& p, const IO* q, const IO* k, const IO* v,
                                   const float* gate, float* Ks, float* Vs, IO* o, cudaStream_t st) {
    const unsigned pairs = (unsigned)p.B * (unsigned)p.H;
    const int is_log = p.gate_kind;
    const float inv_tau = p.tau > 0.f ? 1.f / p.tau : 0.f;
    if (p.m == 128)
        decode_step_kernel<IO, DK, DV, 128><<<pairs, kDecodeWarps * 32, 0, st>>>(q, k, v, gate, p.gate_dtype == GSA_BF16, p.gate_broadcast ? p.H : 0, p.feature_map, is_log, inv_tau, p.scale, p.slot_act, Ks, Vs, o);
    else if (p.m == 64)
        decode_step_kernel<IO, DK, DV, 64><<<pairs, kDecodeWarps * 32, 0, st>>>(q, k, v, gate, p.gate_dtype == GSA_BF16, p.gate_broadcast ? p.H : 0, p.feature_map, is_log, inv_tau, p.scale, p.slot_act, Ks, Vs, o);
    else
        decode_step_kernel<IO, DK, DV, 32><<<pairs, kDecodeWarps * 32, 0, st>>>(q, k, v, gate, p.gate_dtype == GSA_BF16, p.gate_broadcast ? p.H : 0, p.feature_map, is_log, inv_tau, p.scale, p.slot_act, Ks, Vs, o);
    return cudaGetLastError();
}

template <typename IO, int DK>
static cudaError_t launch_decode_dv(const gsa_params_t& p, const IO* q, const IO* k, const IO* v,
                                    const float* gate, float* Ks, float* Vs, IO* o, cudaStream_t st) {
    switch (p.d_v) {
        case 64: return launch_decode_m<IO, DK, 64>(p, q, k, v, gate, Ks, Vs, o, st);
        case 128: return launch_decode_m<IO, DK, 128>(p, q, k, v, gate, Ks, Vs, o, st);
        case 256: return launch_decode_m<IO, DK, 256>(p, q, k, v, gate, Ks, Vs, o, st);
        default: return launch_decode_m<IO, DK, 512>(p, q, k, v, gate, Ks, Vs, o, st);
    }
}

template <typename IO>
static cudaError_t launch_decode_io(const gsa_params_t& p, const void* q, const void* k, const void* v,
                                    const float* gate, float* Ks, float* Vs, void* o, cudaStream_t st) {
    const IO* q_ = (const IO*)q; const IO* k_ = (const IO*)k; const IO* v_ = (const IO*)v; IO* o_ = (IO*)o;
    switch (p.d_k) {
        case 64: return launch_decode_dv<IO, 64>(p, q_, k_, v_, gate, Ks, Vs, o_, st);
        case 128: return launch_decode_dv<IO, 128>(p, q_, k_, v_, gate, Ks, Vs, o_, st);
        case 256: return launch_decode_dv<IO, 256>(p, q_, k_, v_, gate, Ks, Vs, o_, st);
        default: return launch_decode_dv<IO, 512>(p, q_, k_, v_, gate, Ks, Vs, o_, st);
    }
}

cudaError_t launch_decode(const gsa_params_t& p, const void* q, const void* k, const void* v,
                          const float* gate, float* Ks, float* Vs, void* o, cudaStream_t st) {
    if (p.io == GSA_BF16) return launch_decode_io<__nv_bfloat16>(p, q, k, v, gate, Ks, Vs, o, st);
    return launch_decode_io<float>(p, q, k, v, gate, Ks, Vs, o, st);
}

}  // namespace gsa
