// Shared declarations of the GSA CUDA library (internal; the public surface is include/gsa.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gsa.h"

namespace gsa {

constexpr int kChunk = 64;            // C of the chunkwise form, fp32 CUDA-core kernels (tensor-core kernels: 128)
constexpr float kLogGateMin = -100.f; // clamp of log a (exp(-100) == 0 in fp32)
// A chunk whose total log-decay stays above this bound uses the factorised
// decay exp(G_i) * exp(-G_j) (one reference point per chunk); below it the
// exponent differences are taken explicitly so nothing can overflow.
constexpr float kFactorisedDecayMin = -60.f;

template <typename T> struct IoTraits;
template <> struct IoTraits<float> {
    static constexpr int kVec = 4;  // elements per 16-byte access
};
template <> struct IoTraits<__nv_bfloat16> {
    static constexpr int kVec = 8;
};

// 16-byte global load of kVec consecutive elements, widened to fp32.
__device__ __forceinline__ void load_vec(const float* p, float (&out)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float (&out)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f = __bfloat1622float2(h[i]);
        out[2 * i] = f.x; out[2 * i + 1] = f.y;
    }
}
__device__ __forceinline__ void store_vec(float* p, const float (&in)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(in[0], in[1], in[2], in[3]);
}
__device__ __forceinline__ void store_vec(__nv_bfloat16* p, const float (&in)[8]) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = v;
}
__device__ __forceinline__ void store_vec4(float* p, const float (&in)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(in[0], in[1], in[2], in[3]);
}
__device__ __forceinline__ void store_vec4(__nv_bfloat16* p, const float (&in)[4]) {
    uint2 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
    h[0] = __floats2bfloat162_rn(in[0], in[1]);
    h[1] = __floats2bfloat162_rn(in[2], in[3]);
    *reinterpret_cast<uint2*>(p) = v;
}

// ---- arguments of the two chunk primitives (both passes, forward and time-reversed) ----
//
// value_side ("gsa_fwd" of Algorithm 1 with GATE_K = False, the pass-1 form):
//     out_i[s] = sum_{j<=i} <xq_i, xk_j> w_j[s] prod_{r=j+1..i} a_r[s]   (+ state term)
//   xq, xk: [B,T,H,D] io; w, G: [B,T,H,M] fp32; state S (D x M), given/returned in the
//   memory layout [B,H,M,D].  The contraction over D is split into `nslice` slices of
//   width D/nslice; slice z writes its partial sums to out + z * B*T*H*M.
//
// key_side ("gsa_fwd" with GATE_K = True, the pass-2 form):
//     out_i = sum_{j<=i} (sum_s uq_i[s] uk_j[s] prod_{r=j+1..i} a_r[s]) xv_j   (+ state term)
//   uq, uk, G: [B,T,H,M] fp32; xv, out: [B,T,H,D] io; state S (M x D) in [B,H,M,D].
//
// reverse = 1 sums over i >= j instead (same decay product): the gradients w.r.t. keys,
// values and the input gate are such time-reversed runs.
struct ValueSideArgs {
    const void* xq; const void* xk;   // io
    const float* w; const float* G;
    const float* S0;                  // nullable
    float* Send;                      // nullable
    float* out;                       // [nslice][B,T,H,M]
    int B, T, H, D;
    // tensor-core path: the weights already multiplied by their decay factor, bf16 rows of 2M
    // [high part | rounding residual] of w exp(-G) (forward) or w exp(G) (reverse); nullable
    const void* wd;
    // only the end state matters to the caller (first run of the segment-parallel forward): kernels
    // may leave `out` unwritten where computing it is expensive
    int state_only;
    int single;                       // tensor-core kernels: derived operands as one bf16 value (GSA_TC_SINGLE)
};
struct KeySideArgs {
    const float* uq; const float* uk; const float* G;
    const void* xv;                   // io
    const float* S0;                  // nullable
    float* Send;                      // nullable
    void* out;                        // io [B,T,H,D]
    int B, T, H, D;
    // tensor-core path: decayed bf16 rows of 2M (the first M are used): forward uq exp(G) and
    // uk exp(-G), reverse uq exp(-G) and uk exp(G); nullable (both or neither)
    const void* uq_d; const void* uk_d;
    int state_only;                   // as in ValueSideArgs
    int single;                       // as in ValueSideArgs
};

// Element-wise replacements of the slot softmax (gsa_act_t other than GSA_ACT_SOFTMAX): f(z) and f'(z).
__device__ __forceinline__ float slot_act_value(float z, int act) {
    const float r = fmaxf(z, 0.f);
    if (act == GSA_ACT_NONE) return z;
    if (act == GSA_ACT_RELU) return r;
    if (act == GSA_ACT_SWISH) return z / (1.f + __expf(-z));
    return r * r;
}
__device__ __forceinline__ float slot_act_slope(float z, int act) {
    if (act == GSA_ACT_NONE) return 1.f;
    if (act == GSA_ACT_RELU) return z > 0.f ? 1.f : 0.f;
    if (act == GSA_ACT_SWISH) {
        const float sg = 1.f / (1.f + __expf(-z));
        return sg * (1.f + z * (1.f - sg));
    }
    return 2.f * fmaxf(z, 0.f);
}

// GSA_GATE_LOGITS: log a = -softplus(-x) / tau (a = sigmoid(x)^(1/tau), Sec. 3.3) and the factor
// d(log a)/dx = sigmoid(-x) / tau of the gate gradient.
__device__ __forceinline__ float log_gate_from_logit(float x, float inv_tau) {
    return -(fmaxf(-x, 0.f) + log1pf(__expf(-fabsf(x)))) * inv_tau;
}
__device__ __forceinline__ float dlog_gate_dlogit(float x, float inv_tau) {
    return inv_tau / (1.f + __expf(x));
}

// The pipelined tensor-core value_side kernel leaves the row factor of its partial sums --
// exp(G_i) of a forward run, exp(-G_i) of a time-reversed one -- to the element-wise kernel that
// consumes them (slot softmax forward / backward, gate gradient), which sums the D/128 slices
// anyway.  strong[(b * nseg + segment) * H + h] != 0 marks the (batch, head) pairs that the general
// kernel wrote, with the factor already applied.  G == nullptr: nothing is pending.
struct PendingDecay {
    const float* G;
    const int* strong;
    int T, H, nseg;
    // != 0: the slot kernel serves ONLY the pairs flagged in `strong` (the fused chunk kernel has done
    // the others on chip): rows with a pending factor are skipped
    int strong_only;
    // row r = t * H + h of batch element b of a [B,T,H,M] tensor (32-bit arithmetic: T * H < 2^31)
    __host__ __device__ bool pending(int b, int r) const {
        if (G == nullptr) return false;
        const int t = r / H, h = r - t * H;
        const int seg = nseg == 1 ? 0 : t / (T / nseg);
        return strong[(b * nseg + seg) * H + h] == 0;
    }
};

// launchers (definitions in the .cu files); all return cudaGetLastError() of the launch
// strong_flag (nullable, [B*H] ints, zeroed by the caller): set to 1 for every (b,h) that has a
// chunk whose total log-decay is below kFactorisedDecayMin (nseg > 1: [B*nseg*H], per segment).
// decayed (nullable, bf16 [B,T,H,2M]): rows [high part | rounding residual] of I exp(-G), the
// input-gate operand of the pipelined tensor-core kernels.  fast_log: take log a with the
// hardware base-2 logarithm (absolute error 2^-21.4 for a in [0.5, 1], 3 ulp below), for bf16 io.
// gate_kind: gsa_gate_t (a, log a, or logits with inv_tau = 1/tau)
cudaError_t launch_gate_cumsum(const float* gate, int gate_kind, float inv_tau, float* G, float* I,
                               int B, int T, int H, int M, int chunk, int* strong_flag, int nseg,
                               void* decayed, int fast_log, cudaStream_t st, const int* cu_seqlens = nullptr,
                               int nseq = 0);
// ABC (Eq. 3-4): write weights phi (cumulative softmax over time of the scores) into I, zeros into G, phi as the
// decayed bf16 rows; and the gradient w.r.t. the scores from phi and the input-gate gradient partial sums
cudaError_t launch_abc_write(const float* s_in, float* G, float* I, void* decayed, int B, int T, int H, int M, cudaStream_t st);
cudaError_t launch_abc_grad(const float* phi, const float* dIk, int nsk, const float* dIv, int nsv, float* ds, int B, int T,
                            int H, int M, cudaStream_t st);
// a gate row [n] spread over `rows` rows; column sums of [rows, n] (scratch: column_sum_parts(rows) * n floats)
cudaError_t launch_broadcast_rows(const float* row, float* out, size_t rows, int n, cudaStream_t st);
size_t column_sum_parts(size_t rows);
cudaError_t launch_column_sum(const float* in, float* part, float* out, size_t rows, int n, cudaStream_t st);
// n bfloat16 values -> fp32 (a gate tensor given in bfloat16)
cudaError_t launch_widen_bf16(const void* in, float* out, size_t n, cudaStream_t st);
// Segment-parallel scheduling (T cut into nseg segments run as independent sequences): per-segment
// log-decay [B,nseg,H,M] from G, and the start memories [B,nseg,H,M,D] of every segment from the
// end memories of the segments run from empty memories.
cudaError_t launch_segment_logdecay(const float* G, float* seg_logdecay, int B, int T, int H, int M, int nseg,
                                    int chunk, cudaStream_t st);
cudaError_t launch_segment_combine(const float* seg_logdecay, const float* local_end, const float* S0,
                                   float* start, float* final_state, int B, int H, int M, int D, int nseg,
                                   int reverse, cudaStream_t st);
cudaError_t launch_shard_combine(const float* logdecay_all, const float* local_all, const float* S0, float* start,
                                 float* final_state, int B, int H, int M, int D, int nshard, int rank, int reverse,
                                 cudaStream_t st);
// G, p_decayed / dz_decayed (nullable together; bf16 [rows, 2M]): rows [high | residual] of
// p exp(G) and dz exp(G), operands of the pipelined tensor-core kernels.
// (tensors [B, rows_per_batch = T*H, M])
// act: gsa_act_t (the softmax over the slots or an element-wise replacement)
cudaError_t launch_slot_softmax_fwd(const float* part, int nslice, float scale, int act, float* ok,
                                    float* p, int B, int rows_per_batch, int M, const float* G, void* p_decayed,
                                    PendingDecay pend, cudaStream_t st, int m_active = 0);
cudaError_t launch_slot_softmax_bwd(const float* ok, const float* dp_part, int nslice,
                                    float scale, int act, float* p, float* dz, float* u, int B, int rows_per_batch,
                                    int M, const float* G, void* p_decayed, void* dz_decayed,
                                    PendingDecay pend, cudaStream_t st, int m_active = 0);
// m_active (0 = all M): slots from m_active on are padding and take no part in the non-linearity.
// rows of n_in floats -> rows of n_out floats (tail filled with `fill`, or cut)
cudaError_t launch_resize_rows(const float* in, float* out, size_t rows, int n_in, int n_out, float fill, cudaStream_t st);
cudaError_t launch_gate_grad(const float* u, const float* I, const float* dIk_part, int nsk,
                             const float* dIv_part, int nsv, const float* gate,
                             int gate_kind, float inv_tau, const float* dKT, const float* KT,
                             const float* dVT, const float* VT, int d_k, int d_v,
                             float* chunk_tot, float* dgate, int B, int T, int H, int M,
                             PendingDecay pend, cudaStream_t st, int32_t* dev_status);
int gate_grad_blocks(int T);       // entries per (b,h,slot) of launch_gate_grad's scratch
cudaError_t launch_value_side_simt(const ValueSideArgs& a, int io, int M, int reverse,
                                   cudaStream_t st);
cudaError_t launch_key_side_simt(const KeySideArgs& a, int io, int M, int reverse,
                                 cudaStream_t st);
// tcgen05 (bf16 tensor-core) versions of the two primitives; bf16 io only.
bool tc_supported(int d_k, int d_v, int M);
bool tc_dim_ok(int D);
int tc_value_side_slices(int D);
int tc_chunk();                    // chunk length of the tensor-core kernels   // how many partial-sum slices value_side writes for width D
cudaError_t launch_value_side_tc(const ValueSideArgs& a, int M, int reverse, const int* strong_flag,
                                 cudaStream_t st, int32_t* dev_status);
cudaError_t launch_key_side_tc(const KeySideArgs& a, int M, int reverse, const int* strong_flag,
                               cudaStream_t st, int32_t* dev_status);
// the pipelined kernels for the (batch, head) pairs without a strong-decay chunk (strong_flag 0);
// they need the pre-decayed operands of the argument structs
cudaError_t launch_value_side_lean(const ValueSideArgs& a, int reverse, const int* strong_flag, cudaStream_t st,
                                   int32_t* dev_status);
cudaError_t launch_key_side_lean(const KeySideArgs& a, int reverse, const int* strong_flag, cudaStream_t st,
                                 int32_t* dev_status);
// only the general kernel of a scan (the flagged pairs), on the given stream
cudaError_t launch_value_side_general(const ValueSideArgs& a, int M, int reverse, const int* strong_flag,
                                      cudaStream_t st, int32_t* dev_status);
cudaError_t launch_key_side_general(const KeySideArgs& a, int M, int reverse, const int* strong_flag,
                                    cudaStream_t st, int32_t* dev_status);
// The two reversed scans that share a state (dv with dI^v, dk with dI^k) as one kernel
// (chunk_tc_pair.cu): av / ak are the arguments the single reversed scans would get.
bool rev_pair_supported(const ValueSideArgs& av, const KeySideArgs& ak, int M);
cudaError_t launch_rev_pair_tc(const ValueSideArgs& av, const KeySideArgs& ak, int M, const int* strong_flag,
                               cudaStream_t st, int32_t* dev_status);
// the side stream of the calling host thread on the current device, with its fork / join events
struct SideLane {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};
cudaError_t side_lane(SideLane** out);
cudaError_t side_lane_release();
// Fused chunk kernel: value_side scan -> slot non-linearity -> key_side scan in one kernel, for the
// (batch, head) pairs without a strong-decay chunk (chunk_tc_fused.cu).
//   mode 0 (forward):  xq1 = q,  xk1 = k, xv = v, out = o;   ok (nullable) receives the scaled logits
//   mode 1 (backward): xq1 = dO, xk1 = v, xv = k, out = dq;  ok holds the scaled logits; u, Pd, Zd are written
bool fused_pair_supported(int d_k, int d_v, int M);
cudaError_t launch_fused_pair(int mode, const void* xq1, const void* xk1, const void* wd, const void* xv, void* out,
                              const float* G, const float* S1_0, const float* S2_0, float* S1_end, float* S2_end, int B,
                              int T, int H, int D1, int D2, float scale, int act, float* ok, float* u, void* Pd,
                              void* Zd, const int* strong_flag, cudaStream_t st, int32_t* dev_status);
// layer pre- and post-operations (layer_ops.cu)
cudaError_t launch_swish_fwd(const void* in, void* out, size_t n, int io, cudaStream_t st);
cudaError_t launch_swish_bwd(const void* x, void* d, size_t n, int io, cudaStream_t st);
int out_norm_max_width(int io);
size_t out_norm_bwd_parts(size_t rows);
cudaError_t launch_out_norm_fwd(const void* o, const float* weight, float eps, void* y, size_t rows, int N, int io,
                                cudaStream_t st);
cudaError_t launch_out_norm_bwd(const void* o, const void* dy, const float* weight, float eps, void* d_o, float* dw_part,
                                float* dweight, size_t rows, int N, int io, cudaStream_t st);
cudaError_t launch_decode(const gsa_params_t& p, const void* q, const void* k, const void* v,
                          const float* gate, float* Ks, float* Vs, void* o, cudaStream_t st);

}  // namespace gsa
