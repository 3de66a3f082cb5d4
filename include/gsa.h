/*
 * libgsa -- Gated Slot Attention layer for NVIDIA B200 (sm_100a), C ABI.
 *
 * The layer (arXiv 2409.07146, Sec. 3.2, Eq. 6), per (batch b, head h):
 *     K~_t = Diag(a_t) K~_{t-1} + (1 - a_t) (x) k_t          (m x d_k)
 *     V~_t = Diag(a_t) V~_{t-1} + (1 - a_t) (x) v_t          (m x d_v)
 *     o_t  = V~_t^T softmax(scale * K~_t q_t)
 * with both memories updated by token t before they are read.  Training and
 * prefill evaluate it in the chunkwise two-pass form of Eq. 7 / Algorithm 1
 * (two gated-linear-attention passes joined by a softmax over the m slots);
 * decoding applies one step of Eq. 6.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, contiguous,
 *     16-byte aligned.  Layouts: q,k,dq,dk [B,T,H,d_k]; v,o,dO,dv [B,T,H,d_v];
 *     gate,dgate,ok [B,T,H,m]; memories and their gradients [B,H,m,d].
 *   - q,k,v,o,dO,dq,dk,dv have the element type `io` (fp32 or bf16); gate, the
 *     slot logits and all memories are always fp32; accumulation is fp32.
 *   - The gate tensor holds a in [0,1] (GSA_GATE_A), log a <= 0 (GSA_GATE_LOG_A) or the
 *     layer's gate pre-activation x with a = sigmoid(x)^(1/tau) (GSA_GATE_LOGITS: Sec. 3.3,
 *     tau = 8 in the paper; the damped sigmoid is then fused into the gate kernel and
 *     `dgate` is the gradient with respect to x).  Internally log a is clamped to >= -100.
 *   - `params` is a HOST pointer.  `stream` is a cudaStream_t passed as void*
 *     (NULL = the legacy default stream).  Work is only enqueued; nothing
 *     synchronises with the host, allocates or frees device memory.
 *   - Kernels that are independent of one another (the five scans of the backward
 *     after the softmax gradient; the general and the pipelined kernel of a scan)
 *     run on internal streams: up to five per calling host thread and device,
 *     with their events, created on first use and kept until gsa_release_streams()
 *     (this is the library's only state: per host thread and device, no device
 *     memory).  They are forked from `stream` and joined back into it by events
 *     inside the call, so ordering with respect to `stream` is that of a plain
 *     in-stream call, and a call can be captured into a CUDA graph.
 *   - `ws` is caller-provided device scratch of at least
 *     gsa_workspace_bytes() bytes, 256-byte aligned; its contents are
 *     undefined afterwards.  Calls that run concurrently need distinct
 *     workspaces.
 *   - Supported: d_k, d_v in {64,128,256,512}; m in {32,64,128}; B,T,H >= 1
 *     (T need not be a multiple of the chunk; the tail chunk is masked).  bf16 io
 *     with m in {32,64} runs on the tensor-core kernels (m = 32 on their 64-slot
 *     tiles with the upper half padded; d = 64 on half a 128-wide slice); fp32 io
 *     and m = 128 run on the fp32 CUDA-core kernels.
 *   - Errors are return codes; arguments are validated before anything is
 *     launched and outputs are untouched when a call fails validation.
 *     No entry point throws, aborts or prints.
 */
#ifndef GSA_H_
#define GSA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GSA_API __attribute__((visibility("default")))
#else
#define GSA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GSA_OK = 0,
    GSA_ERR_INVALID_ARG = 1,  /* null/misaligned pointer, non-positive size, bad enum */
    GSA_ERR_UNSUPPORTED = 2,  /* valid request outside the supported (d, m, dtype) set */
    GSA_ERR_WORKSPACE = 3,    /* ws is NULL or smaller than gsa_workspace_bytes() */
    GSA_ERR_CUDA = 4,         /* a CUDA runtime call or launch failed */
    GSA_ERR_TIMEOUT = 5       /* a bounded device-side wait expired (see dev_status) */
} gsa_status_t;

typedef enum { GSA_F32 = 0, GSA_BF16 = 1 } gsa_dtype_t;
typedef enum {
    GSA_GATE_A = 0, GSA_GATE_LOG_A = 1, GSA_GATE_LOGITS = 2,
    /* ABC, the ungated ancestor of the layer (Eq. 3-4; the "no decay" row of the table of ablations): the
     * gate tensor holds the score logits s_t, the memories only accumulate (a = 1) and the write weights
     * are the cumulative softmax over time phi_t = exp(s_t) / sum_{j<=t} exp(s_j) per slot, formed by the
     * library; dgate is the gradient w.r.t. s.  gsa_fwd and gsa_bwd only; not with packed sequences. */
    GSA_GATE_ABC = 3
} gsa_gate_t;

/* The non-linearity between the two passes: the softmax over the m slots of Eq. 6, or one of the
 * element-wise replacements of the paper's ablation on it (Sec. 4, table of ablations,
 * "Ablations on non-linearity": no softmax, Swish, ReLU, squared ReLU), applied to the scaled
 * slot logits scale * K~_t q_t. */
typedef enum {
    GSA_ACT_SOFTMAX = 0, GSA_ACT_NONE = 1, GSA_ACT_RELU = 2, GSA_ACT_SWISH = 3, GSA_ACT_RELU2 = 4
} gsa_act_t;

/* Tensor-core kernels only: how the operands that the kernels derive on the way (masked
 * intra-chunk products, decayed slot-space rows, state copies) enter the bf16 products.
 * PAIRED carries each as a bfloat16 value plus its rounding residual wherever that costs extra
 * products (fp32-like results: logits, gradients and memories at ~1e-4 of their rms);
 * SINGLE rounds them to one bfloat16 value, as a plain bf16 matrix product of the chunkwise
 * form does: a quarter fewer products per chunk (the step is 8% faster at d = 512), errors of
 * the order of the bfloat16 rounding of those operands -- logits and gate gradient ~1e-2 of
 * their rms, dq and dk 3e-2 to 1e-1 where the gradients are heavy-tailed, i.e. outside the
 * 2e-2 that PAIRED meets for every tensor. */
typedef enum { GSA_TC_PAIRED = 0, GSA_TC_SINGLE = 1 } gsa_tc_operands_t;

/* Which kernels serve the d-sized contractions of the chunk passes. */
typedef enum {
    GSA_IMPL_AUTO = 0,   /* bf16 io: tensor-core kernels; fp32 io: fp32 CUDA-core kernels */
    GSA_IMPL_SIMT = 1,   /* fp32 CUDA-core kernels for either io type */
    GSA_IMPL_TC = 2      /* tcgen05 bf16 tensor-core kernels (bf16 io only) */
} gsa_impl_t;

/* Tensor-core kernels only: whether the slot non-linearity runs inside the chunk kernel. */
typedef enum {
    GSA_FUSE_OFF = 0,    /* separate kernels: pass 1, slot softmax, pass 2 (and dp, dsoftmax, dq in the backward),
                          * the slot-sized rows between them passed through the workspace; the faster form
                          * on B200 as measured, hence the default */
    GSA_FUSE_ON = 1      /* pass 1 -> softmax -> pass 2 (and dp -> dsoftmax -> dq) as ONE kernel wherever the
                          * shape allows it (d_k == d_v in {128, 256, 512}, m = 64, paired operands): the slot
                          * rows between the passes never leave the chip (a cluster of d / 128 CTAs per
                          * (batch, head) exchanges them through distributed shared memory); with
                          * ok_save == NULL the forward then writes nothing but o.  Other shapes fall back
                          * to the separate kernels. */
} gsa_fuse_t;

/* The layer's feature map on q, k, v (Sec. 3.3: q, k, v = Swish(W x)): with GSA_FEAT_SWISH the q, k, v
 * tensors hold the projections' outputs and Swish is applied by the library (one pass over q, k, v
 * in gsa_fwd and gsa_bwd, whose dq, dk, dv are then gradients w.r.t. those pre-activations; at load
 * in gsa_decode_step). */
typedef enum { GSA_FEAT_NONE = 0, GSA_FEAT_SWISH = 1 } gsa_feature_map_t;

typedef struct {
    int32_t B, T, H, d_k, d_v, m;
    int32_t io;         /* gsa_dtype_t */
    int32_t gate_kind;  /* gsa_gate_t */
    float scale;        /* multiplies the slot logits; 1.0f is the paper's layer */
    int32_t impl;       /* gsa_impl_t */
    float tau;          /* GSA_GATE_LOGITS only: damping of the gate, a = sigmoid(x)^(1/tau); > 0 */
    int32_t slot_act;   /* gsa_act_t; 0 = the paper's softmax */
    int32_t tc_operands; /* gsa_tc_operands_t; ignored by the fp32 kernels */
    int32_t fuse;       /* gsa_fuse_t; ignored by the fp32 kernels */
    int32_t gate_dtype; /* gsa_dtype_t of the gate tensor: GSA_F32 (0, the default) or GSA_BF16 (meant for
                         * GSA_GATE_LOG_A and GSA_GATE_LOGITS: bfloat16 cannot tell a = 0.99 from 1, its
                         * logarithm it can); dgate is fp32 either way */
    int32_t feature_map; /* gsa_feature_map_t */
    int32_t gate_broadcast; /* != 0: data-independent decay (table of ablations): the gate tensor is ONE row
                         * [H, m] used for every token of every sequence (any gate_kind but GSA_GATE_ABC), and
                         * dgate is [H, m], the sum of the per-token gate gradients */
    int32_t nseq;       /* packed sequences: number of sequences along T, 0 = none (see cu_seqlens) */
    const int32_t* cu_seqlens; /* DEVICE pointer to nseq + 1 ascending token offsets, cu_seqlens[0] = 0 and
                         * cu_seqlens[nseq] = T, or NULL.  Every batch row then holds nseq sequences back
                         * to back (variable-length batches packed as B = 1): the memories are emptied at
                         * every offset, so each sequence is an independent recurrence; K0 / V0 enter the
                         * first sequence, KT / VT leave the last.  gsa_fwd and gsa_bwd only.  The chunks
                         * that hold an offset run on the strong-decay kernels. */
} gsa_params_t;

enum { GSA_WS_FWD = 0, GSA_WS_BWD = 1, GSA_WS_DECODE = 2, GSA_WS_GATE = 3, GSA_WS_SHARD = 4 };

/* Chunk length C of the chunkwise form that these params select (Algorithm 1 leaves C
 * open): 128 for the tensor-core kernels, 64 for the fp32 CUDA-core kernels; 0 for
 * invalid params. */
GSA_API int32_t gsa_chunk_size(const gsa_params_t* params);

/* Bytes of scratch `which` (GSA_WS_*) needs for these params; 0 for decode and
 * for invalid params.  GSA_WS_GATE: the block that gsa_fwd_save_gate fills for
 * gsa_bwd_saved_gate. */
GSA_API size_t gsa_workspace_bytes(const gsa_params_t* params, int32_t which);

GSA_API const char* gsa_status_string(gsa_status_t status);

/*
 * chunk_cumsum of Algorithm 1 (its "preprocessing" step), in log space: for
 * each chunk of C = gsa_chunk_size(params) tokens, G[i] = sum_{j <= i in chunk} log a_j (log a clamped
 * to >= -100), and the input gate I = 1 - a.  gate, G, I: [B,T,H,m] fp32; G and
 * I are written in full.  Uses no workspace.
 */
GSA_API gsa_status_t gsa_gate_cumsum(const gsa_params_t* params, const float* gate,
                             float* G, float* I, void* stream);

/*
 * ForwardPass of Algorithm 1 == Eq. 6 over whole sequences.
 *   in : q, k, v, gate; K0, V0 initial memories (NULL = zeros)
 *   out: o; ok_save (nullable) the scaled pre-softmax slot logits
 *        scale * K~_t q_t (the "output of the first GLA pass" that the paper
 *        keeps for the backward); KT, VT (nullable) the final memories.
 * dev_status (nullable, device int32): set non-zero by a kernel whose bounded
 * wait expired; read it after synchronising the stream.
 */
GSA_API gsa_status_t gsa_fwd(const gsa_params_t* params, const void* q, const void* k,
                     const void* v, const float* gate, const float* K0,
                     const float* V0, void* o, float* ok_save, float* KT,
                     float* VT, void* ws, size_t ws_bytes, void* stream,
                     int32_t* dev_status);

/*
 * BackwardPass of Algorithm 1: gradients of gsa_fwd's o (and, optionally, of
 * its final memories) w.r.t. every input.  The memories and the softmax are
 * recomputed from the inputs (the paper's recomputation scheme); ok_saved
 * (nullable) is gsa_fwd's ok_save and spares the recomputation of pass 1.
 *   in : q, k, v, gate, K0, V0 (nullable) as given to gsa_fwd; dO;
 *        dKT, dVT gradients w.r.t. the final memories (NULL = zeros)
 *   out: dq, dk, dv; dgate = total derivative w.r.t. the gate tensor as
 *        passed (through the decay and through the coupled input gate 1 - a);
 *        dK0, dV0 (nullable).
 * With GSA_GATE_A the decay part of dgate is d(log a)/a and loses accuracy as
 * a -> 0; GSA_GATE_LOG_A has no such division.
 */
GSA_API gsa_status_t gsa_bwd(const gsa_params_t* params, const void* q, const void* k,
                     const void* v, const float* gate, const float* K0,
                     const float* V0, const float* ok_saved, const void* dO,
                     const float* dKT, const float* dVT, void* dq, void* dk,
                     void* dv, float* dgate, float* dK0, float* dV0, void* ws,
                     size_t ws_bytes, void* stream, int32_t* dev_status);

/*
 * The same two calls for a training step that trades memory for the backward's gate kernel
 * (the save-instead-of-recompute side of the trade-off the paper discusses in Sec. 4,
 * "Efficiency"): gsa_fwd_save_gate leaves the products of chunk_cumsum (the cumulative log
 * gate, the input gate, its decayed bf16 rows and the per-(batch, head) decay flags), on the
 * tensor-core path also the forward's slot weights p (as the backward's reversed scans read them:
 * they depend on the saved logits only, and with them in hand the backward starts its dv scan at
 * once) and, where a long sequence is cut into segments, the segments' decay, the memories entering
 * every segment and the final memories in gate_save, a device block of gsa_workspace_bytes(params, GSA_WS_GATE) bytes, 256-byte
 * aligned, owned by the caller; gsa_bwd_saved_gate reads them from there instead of running
 * the gate kernel (and the segments' forward-direction state runs) again.  Both calls must use the same params and the same gate tensor;
 * nothing checks that.  A missing, misaligned or short block is GSA_ERR_WORKSPACE.
 */
GSA_API gsa_status_t gsa_fwd_save_gate(const gsa_params_t* params, const void* q, const void* k,
                                       const void* v, const float* gate, const float* K0,
                                       const float* V0, void* o, float* ok_save, float* KT,
                                       float* VT, void* gate_save, size_t gate_save_bytes, void* ws,
                                       size_t ws_bytes, void* stream, int32_t* dev_status);
GSA_API gsa_status_t gsa_bwd_saved_gate(const gsa_params_t* params, const void* q, const void* k,
                                        const void* v, const float* gate, const float* K0,
                                        const float* V0, const float* ok_saved, const void* dO,
                                        const float* dKT, const float* dVT, void* dq, void* dk,
                                        void* dv, float* dgate, float* dK0, float* dV0,
                                        const void* gate_saved, size_t gate_saved_bytes, void* ws,
                                        size_t ws_bytes, void* stream, int32_t* dev_status);

/*
 * One recurrent step of Eq. 6 for B independent sequences (params->T is
 * ignored): q,k [B,H,d_k], v,o [B,H,d_v] of type io, gate [B,H,m] fp32;
 * Kstate [B,H,m,d_k] and Vstate [B,H,m,d_v] fp32 are updated IN PLACE (same
 * layout as gsa_fwd's KT/VT, so a prefill hands its memories straight to the
 * decoder).  Works in linear space: a = 0 and a = 1 are exact.  No workspace.
 */
GSA_API gsa_status_t gsa_decode_step(const gsa_params_t* params, const void* q,
                             const void* k, const void* v, const float* gate,
                             float* Kstate, float* Vstate, void* o, void* stream);

/*
 * gsa_fwd without caller-provided scratch (the paper has no counterpart: this is a
 * packaging variant of gsa_fwd, same arguments minus ws / ws_bytes, same results).
 *
 * For callers that cannot allocate device memory around the layer -- code running inside
 * a server's fixed memory plan, a latency-critical loop that must avoid the allocator's
 * lock and implicit synchronisation, a plug-in that is only handed input and output
 * buffers.  The scratch is a fixed array inside the library image: every GPU that loads
 * the library holds GSA_NOALLOC_MAX_WORKSPACE_BYTES (32 MiB) until the process exits.  The call allocates and frees nothing (no cudaMalloc / cudaFree, no allocating
 * library routine).
 *   - Shapes whose gsa_workspace_bytes(params, GSA_WS_FWD) exceeds that maximum are
 *     rejected with GSA_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Like gsa_fwd, the first tensor-core call of a host thread on a device also
 *     creates that thread's side stream and its two events (no device memory).  Make that
 *     first call before any stream capture and outside latency-critical sections; later
 *     calls only read the cached address.
 *   - All calls on a device share the one array: calls that overlap on the GPU (different
 *     streams) race and give wrong results; serialise them or use gsa_fwd with separate
 *     workspaces.  The array keeps the previous call's contents; the forward needs none of
 *     it cleared (it writes every scratch tensor before reading it).
 */
#define GSA_NOALLOC_MAX_WORKSPACE_BYTES ((size_t)32 << 20)
GSA_API gsa_status_t gsa_fwd_noalloc(const gsa_params_t* params, const void* q, const void* k,
                                     const void* v, const float* gate, const float* K0,
                                     const float* V0, void* o, float* ok_save, float* KT,
                                     float* VT, void* stream, int32_t* dev_status);

/*
 * The layer's output path (Sec. 3.3: y = W_o RMSNorm(Swish(concat_h o^h))), element-wise part:
 *   y = w * x / sqrt(mean(x^2) + eps),  x = Swish(o),  mean over the H d_v values of a token.
 * o, y, dy, d_o: [B,T,H,d_v] of the io type; weight (nullable = ones), dweight (nullable): [H d_v] fp32.
 * H d_v must not exceed 4096 (bf16) / 2048 (fp32).  gsa_out_norm_bwd recomputes the norm from o; with
 * dweight != NULL it needs ws of gsa_out_norm_workspace_bytes(params) bytes (256-byte aligned) for the
 * per-block partial sums of the weight gradient, added in a fixed order (deterministic).
 */
GSA_API gsa_status_t gsa_out_norm_fwd(const gsa_params_t* params, const void* o, const float* weight, float eps,
                                      void* y, void* stream);
GSA_API size_t gsa_out_norm_workspace_bytes(const gsa_params_t* params);
GSA_API gsa_status_t gsa_out_norm_bwd(const gsa_params_t* params, const void* o, const void* dy, const float* weight,
                                      float eps, void* d_o, float* dweight, void* ws, size_t ws_bytes, void* stream);

/*
 * Sequence sharding across GPUs (the memories of Eq. 6 are linear in (k, v): the memory after a
 * stretch of tokens is D * (memory before) + (memory of the stretch run from empty memories), D =
 * the product of the stretch's gates).  A sequence cut into R shards, one per GPU, therefore needs
 * ONE exchange: every rank computes the end memories of its shard from empty memories and the
 * shard's log-decay (gsa_shard_states), the R results are gathered on every rank by the caller
 * (an all-gather of m (d_k + d_v + 1) floats per (batch, head) and rank, into local memory), every
 * rank combines them into the memories that enter its shard (gsa_shard_combine) and runs the
 * ordinary gsa_fwd with those as K0 / V0.  The backward uses the same two calls on the memory
 * gradients that gsa_bwd returns for a shard (dK0 / dV0 with zero final-memory gradients are the
 * shard's local contribution; combined from the last shard down with reverse = 1 they give the
 * dKT / dVT of every shard).  Both calls work on this GPU's memory only.
 *
 * gsa_shard_states: k, v, gate of the shard ([B,T,H,.] with T the shard's length) -> KT, VT
 *   [B,H,m,d] (end memories from EMPTY memories) and logdecay [B,H,m] (sum of log a over the shard).
 *   ws: gsa_workspace_bytes(params, GSA_WS_SHARD).  32-slot bf16 layers: GSA_ERR_UNSUPPORTED.
 * gsa_shard_combine: logdecay_all [R,B,H,m] and local_all [R,B,H,m,d] gathered in rank order, S0
 *   (nullable [B,H,m,d]: the memories before the first shard; reverse: the gradient after the last)
 *   -> start (nullable): what enters shard `rank` (reverse = 0: from the left; 1: from the right);
 *   final_state (nullable): what leaves the last shard (reverse: the first).  d = d_k or d_v.
 */
GSA_API gsa_status_t gsa_shard_states(const gsa_params_t* params, const void* k, const void* v,
                                      const float* gate, float* KT, float* VT, float* logdecay,
                                      void* ws, size_t ws_bytes, void* stream, int32_t* dev_status);
GSA_API gsa_status_t gsa_shard_combine(const gsa_params_t* params, int32_t d, int32_t nshard, int32_t rank,
                                       int32_t reverse, const float* logdecay_all, const float* local_all,
                                       const float* S0, float* start, float* final_state, void* stream);

/*
 * Releases the internal streams and events that this HOST thread's calls created on the current
 * device (the side streams described in the conventions above); they are created again by the
 * next call that needs them.  Call it only when none of this thread's gsa_* work is in flight on
 * the device and no capture is open.  No counterpart in the paper.
 */
GSA_API gsa_status_t gsa_release_streams(void);

#ifdef __cplusplus
}
#endif
#endif /* GSA_H_ */
