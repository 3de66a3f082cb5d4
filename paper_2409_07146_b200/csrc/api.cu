// C ABI of the GSA library: argument validation, workspace carving and the order in which
// the kernels of one forward / backward call are enqueued.  No kernel lives here.
#include <string.h>

#include <atomic>
#include <vector>

#include "common.cuh"
#include "gsa_dev.h"

using namespace gsa;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool ok_ptr(const void* p) { return p != nullptr && aligned16(p); }
bool ok_opt(const void* p) { return p == nullptr || aligned16(p); }
bool dim_ok(int d) { return d == 64 || d == 128 || d == 256 || d == 512; }

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr int kPaddedSlots = 64;      // slot width of the tensor-core tiles (see pads_slots)

gsa_status_t check_params(const gsa_params_t* p, bool need_T) {
    if (p == nullptr) return GSA_ERR_INVALID_ARG;
    if (p->B < 1 || p->H < 1 || p->d_k < 1 || p->d_v < 1 || p->m < 1) return GSA_ERR_INVALID_ARG;
    if (need_T && p->T < 1) return GSA_ERR_INVALID_ARG;
    if (p->io != GSA_F32 && p->io != GSA_BF16) return GSA_ERR_INVALID_ARG;
    if (p->gate_kind != GSA_GATE_A && p->gate_kind != GSA_GATE_LOG_A && p->gate_kind != GSA_GATE_LOGITS &&
        p->gate_kind != GSA_GATE_ABC)
        return GSA_ERR_INVALID_ARG;
    if (p->gate_kind == GSA_GATE_ABC && (p->cu_seqlens != nullptr || p->gate_broadcast != 0)) return GSA_ERR_UNSUPPORTED;
    if (p->gate_kind == GSA_GATE_LOGITS && !(p->tau > 0.f)) return GSA_ERR_INVALID_ARG;
    if (p->slot_act < GSA_ACT_SOFTMAX || p->slot_act > GSA_ACT_RELU2) return GSA_ERR_INVALID_ARG;
    if (p->tc_operands != GSA_TC_PAIRED && p->tc_operands != GSA_TC_SINGLE) return GSA_ERR_INVALID_ARG;
    if (p->impl != GSA_IMPL_AUTO && p->impl != GSA_IMPL_SIMT && p->impl != GSA_IMPL_TC)
        return GSA_ERR_INVALID_ARG;
    if (p->fuse != GSA_FUSE_OFF && p->fuse != GSA_FUSE_ON) return GSA_ERR_INVALID_ARG;
    if (p->gate_dtype != GSA_F32 && p->gate_dtype != GSA_BF16) return GSA_ERR_INVALID_ARG;
    if (p->feature_map != GSA_FEAT_NONE && p->feature_map != GSA_FEAT_SWISH) return GSA_ERR_INVALID_ARG;
    if (p->nseq < 0 || (p->nseq == 0) != (p->cu_seqlens == nullptr)) return GSA_ERR_INVALID_ARG;
    if (!(p->scale == p->scale)) return GSA_ERR_INVALID_ARG;
    if (!dim_ok(p->d_k) || !dim_ok(p->d_v)) return GSA_ERR_UNSUPPORTED;
    if (p->m != 32 && p->m != 64 && p->m != 128) return GSA_ERR_UNSUPPORTED;
    if ((long long)p->B * p->H > 0x7fffffffLL / 4) return GSA_ERR_UNSUPPORTED;
    if (p->impl == GSA_IMPL_TC && p->io != GSA_BF16) return GSA_ERR_UNSUPPORTED;
    // the tensor-core kernels asked for by name: no silent fall-back to the CUDA-core kernels
    if (p->impl == GSA_IMPL_TC && !tc_supported(p->d_k, p->d_v, p->m == 32 ? kPaddedSlots : p->m)) return GSA_ERR_UNSUPPORTED;
    return GSA_OK;
}

// Does this call run the tensor-core chunk kernels?
bool use_tc(const gsa_params_t& p) {
    if (p.impl == GSA_IMPL_SIMT) return false;
    return p.io == GSA_BF16 && tc_supported(p.d_k, p.d_v, p.m);
}

// A bf16 layer with 32 slots runs on the tensor-core kernels too: their tiles are 64 slots wide, so the
// call is carried out with 64 slots of which the last 32 are padding -- a gate that keeps everything
// and writes nothing (a = 1), empty memory rows, and a non-linearity that leaves the padding out.
// The gate, the logits, the memories and their gradients are widened / narrowed at the boundary.
bool pads_slots(const gsa_params_t& p) {
    return p.impl != GSA_IMPL_SIMT && p.io == GSA_BF16 && p.m == 32 && tc_supported(p.d_k, p.d_v, kPaddedSlots);
}
gsa_params_t internal_params(const gsa_params_t& p) {
    gsa_params_t q = p;
    if (pads_slots(p)) q.m = kPaddedSlots;
    return q;
}

// Does this call run the slot non-linearity inside the fused chunk kernel?  (The operand pairs are
// built into that kernel: GSA_TC_SINGLE keeps the separate kernels.)
bool use_fused(const gsa_params_t& p) {
    return use_tc(p) && p.fuse == GSA_FUSE_ON && p.tc_operands == GSA_TC_PAIRED &&
           fused_pair_supported(p.d_k, p.d_v, p.m);
}

float inv_tau(const gsa_params_t& p) { return p.tau > 0.f ? 1.f / p.tau : 0.f; }

int chunk_of(const gsa_params_t& p) { return use_tc(p) ? tc_chunk() : kChunk; }

struct Slices { int k, v; };
Slices slices(const gsa_params_t& p) {
    if (use_tc(p)) return {tc_value_side_slices(p.d_k), tc_value_side_slices(p.d_v)};
    return {p.d_k / 64, p.d_v / 64};
}

// Segment-parallel scheduling of the forward: when (batch, head, slice) triples cannot fill the
// GPU, long sequences are cut into nseg segments that run as independent sequences (the
// memories are linear in (k, v), so every segment's start memories follow from a first pass
// that runs the segments from empty memories).  1 = off.
int segments_of(const gsa_params_t& p) {
    if (!use_tc(p)) return 1;
    const int chunk = tc_chunk();
    const long long ctas = (long long)p.B * p.H * tc_value_side_slices(p.d_k < p.d_v ? p.d_k : p.d_v);
    int nseg = 1;
    while (ctas * nseg * 2 <= 160 && p.T % (nseg * 2 * chunk) == 0 && p.T / (nseg * 2) >= 8 * chunk) nseg *= 2;
    return nseg;
}

struct Carver {
    char* base; size_t off;
    float* take(size_t nfloat) {
        float* r = reinterpret_cast<float*>(base + off);
        off += align_up(nfloat * sizeof(float), 256);
        return r;
    }
};

struct Workspace {
    float *G, *I, *okpart, *ok, *p, *dz, *u, *dppart, *dIk, *dIv, *chunk_tot, *KT, *VT;
    int* strong;     // [B*nseg*H] flags: this (b,h) has a chunk that decays too hard for the factorised form
    float *seg_decay, *Kloc, *Vloc, *Kstart, *Vstart;   // segment-parallel scheduling only
    float *dKend, *dVend;                               // ... backward: states entering each segment from the right
    // tensor-core path: bf16 rows [high | residual] of I exp(-G), p exp(G), dz exp(G), each [B,T,H,2m]
    void *Id, *Pd, *Zd;
    size_t bytes;
};

Workspace carve(const gsa_params_t& p, int which, void* ws) {
    Workspace w;
    memset(&w, 0, sizeof(w));
    const size_t mt = (size_t)p.B * p.T * p.H * p.m;
    const Slices s = slices(p);
    Carver c{static_cast<char*>(ws), 0};
    const int nseg = segments_of(p);
    w.strong = reinterpret_cast<int*>(c.take((size_t)p.B * p.H * nseg));
    if (nseg > 1) {
        const size_t pairs = (size_t)p.B * nseg * p.H;
        w.seg_decay = c.take(pairs * p.m);
        w.Kloc = c.take(pairs * p.m * p.d_k);
        w.Vloc = c.take(pairs * p.m * p.d_v);
        w.Kstart = c.take(pairs * p.m * p.d_k);
        w.Vstart = c.take(pairs * p.m * p.d_v);
        if (which == GSA_WS_BWD) {
            w.dKend = c.take(pairs * p.m * p.d_k);
            w.dVend = c.take(pairs * p.m * p.d_v);
        }
    }
    w.G = c.take(mt);
    w.I = c.take(mt);
    w.okpart = c.take(mt * s.k);
    w.ok = c.take(mt);
    w.p = c.take(mt);
    if (use_tc(p)) {           // 2m bf16 per row = m floats
        w.Id = c.take(mt);
        w.Pd = c.take(mt);
        if (which == GSA_WS_BWD) w.Zd = c.take(mt);
    }
    if (which == GSA_WS_BWD) {
        w.dz = c.take(mt);
        w.u = c.take(mt);
        w.dppart = c.take(mt * s.v);
        w.dIk = c.take(mt * s.k);
        w.dIv = c.take(mt * s.v);
        w.chunk_tot = c.take((size_t)p.B * p.H * gate_grad_blocks(p.T) * p.m);
        w.KT = c.take((size_t)p.B * p.H * p.m * p.d_k);
        w.VT = c.take((size_t)p.B * p.H * p.m * p.d_v);
    }
    w.bytes = c.off;
    return w;
}

// The gate kernel's products as a block of their own (GSA_WS_GATE): what the forward can leave for
// the backward of the same call so that the backward does not run the gate kernel again.
// With segment-parallel scheduling the block also carries what the forward's first run found: the
// segments' decay, the memories entering every segment and the final memories.
struct GateSums {
    int* strong; float *G, *I; void* Id;
    float* p; void* Pd;                               // slot weights of the forward (tensor-core path)
    float *seg_decay, *Kstart, *Vstart, *KT, *VT;     // nseg > 1 only
    size_t bytes;
};
GateSums carve_gate(const gsa_params_t& p, void* base) {
    GateSums g;
    memset(&g, 0, sizeof(g));
    const size_t mt = (size_t)p.B * p.T * p.H * p.m;
    const int nseg = segments_of(p);
    Carver c{static_cast<char*>(base), 0};
    g.strong = reinterpret_cast<int*>(c.take((size_t)p.B * p.H * nseg));
    g.G = c.take(mt);
    g.I = c.take(mt);
    g.Id = use_tc(p) ? c.take(mt) : nullptr;
    // the slot weights p (fp32 for the pairs flagged for strong decay, the decayed operand pair for
    // the others) depend on the forward's logits only: kept, they let the backward's dv and dI^v
    // scans start before the softmax gradient is known
    g.p = use_tc(p) ? c.take(mt) : nullptr;
    g.Pd = use_tc(p) ? c.take(mt) : nullptr;
    if (nseg > 1) {
        const size_t pairs = (size_t)p.B * nseg * p.H;
        g.seg_decay = c.take(pairs * p.m);
        g.Kstart = c.take(pairs * p.m * p.d_k);
        g.Vstart = c.take(pairs * p.m * p.d_v);
        g.KT = c.take((size_t)p.B * p.H * p.m * p.d_k);
        g.VT = c.take((size_t)p.B * p.H * p.m * p.d_v);
    }
    g.bytes = c.off;
    return g;
}
// points the workspace's gate products at the block; false if the block is missing or too small
bool use_gate_block(const gsa_params_t& p, Workspace* w, void* block, size_t block_bytes) {
    if (block == nullptr || (reinterpret_cast<uintptr_t>(block) & 255u) != 0) return false;
    const GateSums g = carve_gate(p, block);
    if (block_bytes < g.bytes) return false;
    w->strong = g.strong; w->G = g.G; w->I = g.I; w->Id = g.Id;
    if (g.p != nullptr) { w->p = g.p; w->Pd = g.Pd; }
    if (g.seg_decay != nullptr) {
        w->seg_decay = g.seg_decay; w->Kstart = g.Kstart; w->Vstart = g.Vstart;
        w->KT = g.KT; w->VT = g.VT;      // (the forward's workspace has no KT / VT of its own)
    }
    return true;
}

cudaError_t value_side(const gsa_params_t& p, const ValueSideArgs& a, int reverse, const int* strong,
                       cudaStream_t st, int32_t* dev_status) {
    if (use_tc(p)) {
        ValueSideArgs b = a;
        b.single = p.tc_operands == GSA_TC_SINGLE;
        return launch_value_side_tc(b, p.m, reverse, strong, st, dev_status);
    }
    return launch_value_side_simt(a, p.io, p.m, reverse, st);
}
cudaError_t key_side(const gsa_params_t& p, const KeySideArgs& a, int reverse, const int* strong,
                     cudaStream_t st, int32_t* dev_status) {
    if (use_tc(p)) {
        KeySideArgs b = a;
        b.single = p.tc_operands == GSA_TC_SINGLE;
        return launch_key_side_tc(b, p.m, reverse, strong, st, dev_status);
    }
    return launch_key_side_simt(a, p.io, p.m, reverse, st);
}

// ---- optional per-kernel timing (benchmarks only): while a sink is active on the calling
// host thread, every kernel launch is bracketed by a pair of events on its stream.
struct TimingSink {
    bool active = false;
    int capacity = 0, count = 0;
    std::vector<cudaEvent_t> ev;       // 2 per launch
    std::vector<const char*> labels;
};
thread_local TimingSink g_sink;

// development switch (gsa_dev_pair_scans): the backward's reversed scans as two pair kernels (default)
// or as four single ones
std::atomic<int> g_pair_scans{1};

void timing_before(cudaStream_t st) {
    if (g_sink.active && g_sink.count < g_sink.capacity) cudaEventRecord(g_sink.ev[2 * g_sink.count], st);
}
void timing_after(const char* label, cudaStream_t st) {
    if (g_sink.active && g_sink.count < g_sink.capacity) {
        cudaEventRecord(g_sink.ev[2 * g_sink.count + 1], st);
        g_sink.labels[g_sink.count] = label;
        ++g_sink.count;
    }
}

// ---- the five scans of the backward that follow the softmax gradient are independent: on the
// tensor-core path they run on five streams of the calling host thread (the caller's and four
// of the library's), so that the CTAs of one start as those of another finish and the SMs that
// one scan's 128 CTAs leave idle take CTAs of the next.  Forked and joined by events; with a
// timing sink active they run one after the other instead, so that each is timed alone.
struct ScanLanes {
    cudaStream_t stream[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaStream_t fast = nullptr;       // highest priority: the chain the other scans wait for
    cudaEvent_t fast_done = nullptr;
    cudaEvent_t fork = nullptr, fork_early = nullptr, join[4] = {nullptr, nullptr, nullptr, nullptr};
};
constexpr int kMaxLaneDevices = 64;
thread_local ScanLanes g_scan_lanes[kMaxLaneDevices];

cudaError_t scan_lanes(ScanLanes** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxLaneDevices) return cudaErrorInvalidDevice;
    ScanLanes& l = g_scan_lanes[dev];
    if (l.fork == nullptr) {
        for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
            e = cudaStreamCreateWithFlags(&l.stream[i], cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.join[i], cudaEventDisableTiming);
        }
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.fork_early, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&l.fast_done, cudaEventDisableTiming);
        int least = 0, greatest = 0;
        if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&least, &greatest);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&l.fast, cudaStreamNonBlocking, greatest);
        if (e != cudaSuccess) return e;
    }
    *out = &l;
    return cudaSuccess;
}

cudaError_t scan_lanes_release() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxLaneDevices) return cudaErrorInvalidDevice;
    ScanLanes& l = g_scan_lanes[dev];
    for (int i = 0; i < 4; ++i) {
        if (l.stream[i] != nullptr) cudaStreamDestroy(l.stream[i]);
        if (l.join[i] != nullptr) cudaEventDestroy(l.join[i]);
    }
    if (l.fork != nullptr) cudaEventDestroy(l.fork);
    if (l.fork_early != nullptr) cudaEventDestroy(l.fork_early);
    if (l.fast_done != nullptr) cudaEventDestroy(l.fast_done);
    if (l.fast != nullptr) cudaStreamDestroy(l.fast);
    l = ScanLanes{};
    return cudaSuccess;
}

// Buffers of the padded-slot mode, carved from the tail of the workspace (after the internal one).
struct PadBuffers {
    float *gate, *ok, *dgate;                    // [B,T,H,64]
    float *K0, *V0, *KT, *VT;                    // [B,H,64,d]   (backward: K0, V0, dKT, dVT in; KT = dK0, VT = dV0 out)
    float *dKT, *dVT;
    size_t bytes;
};
PadBuffers carve_pad(const gsa_params_t& p, int which, void* base) {
    PadBuffers b;
    memset(&b, 0, sizeof(b));
    if (!pads_slots(p)) return b;
    const size_t mt = (size_t)p.B * p.T * p.H * kPaddedSlots;
    const size_t sk = (size_t)p.B * p.H * kPaddedSlots * p.d_k, sv = (size_t)p.B * p.H * kPaddedSlots * p.d_v;
    Carver c{static_cast<char*>(base), 0};
    b.gate = c.take(mt);
    b.ok = c.take(mt);
    b.K0 = c.take(sk); b.V0 = c.take(sv); b.KT = c.take(sk); b.VT = c.take(sv);
    if (which == GSA_WS_BWD) {
        b.dgate = c.take(mt);
        b.dKT = c.take(sk); b.dVT = c.take(sv);
    }
    b.bytes = c.off;
    return b;
}
size_t pad_bytes(const gsa_params_t& p, int which) { return carve_pad(p, which, nullptr).bytes; }
// a gate tensor given in bfloat16 is widened to fp32 once, into the last part of the workspace
size_t gate_elems(const gsa_params_t& p) {       // elements of the gate tensor as the caller passes it
    return p.gate_broadcast ? (size_t)p.H * p.m : (size_t)p.B * p.T * p.H * p.m;
}
// Workspace behind the padded-slot buffers: [ widened bf16 gate | gate row spread over all tokens |
// per-token gate gradient | its column-sum scratch ]
struct GateBoundary { size_t conv, spread, dfull, colsum, bytes; };
GateBoundary gate_boundary(const gsa_params_t& p, int which) {
    GateBoundary g{0, 0, 0, 0, 0};
    const size_t mt = align_up((size_t)p.B * p.T * p.H * p.m * sizeof(float), 256);
    if (p.gate_dtype == GSA_BF16) g.conv = align_up(gate_elems(p) * sizeof(float), 256);
    if (p.gate_broadcast) {
        g.spread = mt;
        if (which == GSA_WS_BWD) {
            g.dfull = mt;
            g.colsum = align_up(column_sum_parts((size_t)p.B * p.T) * p.H * p.m * sizeof(float), 256);
        }
    }
    g.bytes = g.conv + g.spread + g.dfull + g.colsum;
    return g;
}
size_t gate_conv_bytes(const gsa_params_t& p, int which = GSA_WS_BWD) { return gate_boundary(p, which).bytes; }
// The layer's feature map: Swish(q), Swish(k), Swish(v) are formed once, in the part of the workspace
// that follows everything else; the scans then read those copies.
struct FeatureBuffers { void *q, *k, *v; size_t bytes; };
FeatureBuffers carve_features(const gsa_params_t& p, void* base) {
    FeatureBuffers f{nullptr, nullptr, nullptr, 0};
    if (p.feature_map != GSA_FEAT_SWISH) return f;
    const size_t e = p.io == GSA_BF16 ? 2 : 4, R = (size_t)p.B * p.T * p.H;
    const size_t nk = align_up(R * p.d_k * e, 256), nv = align_up(R * p.d_v * e, 256);
    char* b = static_cast<char*>(base);
    f.q = b; f.k = b + nk; f.v = b + 2 * nk;
    f.bytes = 2 * nk + nv;
    return f;
}
gsa_status_t apply_feature_map(const gsa_params_t& p, int which, const void** q, const void** k, const void** v, void* ws,
                               size_t ws_bytes, cudaStream_t st) {
    if (p.feature_map != GSA_FEAT_SWISH) return GSA_OK;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    const gsa_params_t pi = internal_params(p);
    const size_t before = carve(pi, which, nullptr).bytes + pad_bytes(p, which) + gate_conv_bytes(p, which);
    const FeatureBuffers f = carve_features(p, static_cast<char*>(ws) + before);
    if (ws_bytes < before + f.bytes) return GSA_ERR_WORKSPACE;
    const size_t R = (size_t)p.B * p.T * p.H;
    if (launch_swish_fwd(*q, f.q, R * p.d_k, p.io, st) != cudaSuccess) return GSA_ERR_CUDA;
    if (launch_swish_fwd(*k, f.k, R * p.d_k, p.io, st) != cudaSuccess) return GSA_ERR_CUDA;
    if (launch_swish_fwd(*v, f.v, R * p.d_v, p.io, st) != cudaSuccess) return GSA_ERR_CUDA;
    *q = f.q; *k = f.k; *v = f.v;
    return GSA_OK;
}

// the fp32 gate tensor of this call (the caller's, or its widened copy behind `before` bytes of workspace)
gsa_status_t gate_as_f32(const gsa_params_t& p, int which, const float* gate, void* ws, size_t ws_bytes, size_t before,
                         cudaStream_t st, const float** out) {
    *out = gate;
    const GateBoundary g = gate_boundary(p, which);
    if (g.bytes == 0) return GSA_OK;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || ws_bytes < before + g.bytes) return GSA_ERR_WORKSPACE;
    char* base = static_cast<char*>(ws) + before;
    if (p.gate_dtype == GSA_BF16) {
        float* buf = reinterpret_cast<float*>(base);
        if (launch_widen_bf16(gate, buf, gate_elems(p), st) != cudaSuccess) return GSA_ERR_CUDA;
        *out = buf;
    }
    if (p.gate_broadcast) {
        float* buf = reinterpret_cast<float*>(base + g.conv);
        if (launch_broadcast_rows(*out, buf, (size_t)p.B * p.T, p.H * p.m, st) != cudaSuccess) return GSA_ERR_CUDA;
        *out = buf;
    }
    return GSA_OK;
}

#define GSA_CUDA(expr)                                  \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) return GSA_ERR_CUDA;    \
    } while (0)
// a kernel launch on stream `st`, timed when a sink is active
#define GSA_LAUNCH(label, expr)                         \
    do {                                                \
        timing_before(st);                              \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) return GSA_ERR_CUDA;    \
        timing_after(label, st);                        \
    } while (0)

}  // namespace

extern "C" {

int32_t gsa_chunk_size(const gsa_params_t* params) {
    if (check_params(params, false) != GSA_OK) return 0;
    return chunk_of(internal_params(*params));
}

const char* gsa_status_string(gsa_status_t status) {
    switch (status) {
        case GSA_OK: return "ok";
        case GSA_ERR_INVALID_ARG: return "invalid argument";
        case GSA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case GSA_ERR_WORKSPACE: return "workspace missing or too small";
        case GSA_ERR_CUDA: return "CUDA error";
        case GSA_ERR_TIMEOUT: return "bounded device-side wait expired";
    }
    return "unknown status";
}

size_t gsa_workspace_bytes(const gsa_params_t* params, int32_t which) {
    if (which == GSA_WS_DECODE) return 0;
    if (which != GSA_WS_FWD && which != GSA_WS_BWD && which != GSA_WS_GATE && which != GSA_WS_SHARD) return 0;
    if (check_params(params, true) != GSA_OK) return 0;
    if (which == GSA_WS_SHARD) {
        if (pads_slots(*params)) return 0;
        const size_t esz = params->io == GSA_BF16 ? 2 : 4;
        return carve(*params, GSA_WS_FWD, nullptr).bytes +
               align_up((size_t)params->B * params->T * params->H * params->d_v * esz, 256);
    }
    const gsa_params_t pi = internal_params(*params);
    if (which == GSA_WS_GATE) return carve_gate(pi, nullptr).bytes;
    return carve(pi, which, nullptr).bytes + pad_bytes(*params, which) + gate_conv_bytes(*params, which) +
           carve_features(*params, nullptr).bytes;
}

gsa_status_t gsa_gate_cumsum(const gsa_params_t* params, const float* gate, float* G, float* I,
                             void* stream) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(gate) || !ok_ptr(G) || !ok_ptr(I)) return GSA_ERR_INVALID_ARG;
    if (params->gate_dtype != GSA_F32 || params->gate_kind == GSA_GATE_ABC || params->gate_broadcast)
        return GSA_ERR_UNSUPPORTED;      // (this query entry point has no workspace)
    const gsa_params_t& p = *params;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GSA_LAUNCH("gate_cumsum", launch_gate_cumsum(gate, p.gate_kind, inv_tau(p), G, I, p.B, p.T,
                                                 p.H, p.m, chunk_of(internal_params(p)), nullptr, 1, nullptr, 0, st,
                                                 p.cu_seqlens, p.nseq));
    return GSA_OK;
}

namespace {
gsa_status_t fwd_core(const gsa_params_t* params, int m_active, const void* q, const void* k, const void* v,
                      const float* gate, const float* K0, const float* V0, void* o,
                      float* ok_save, float* KT, float* VT, bool save_gate, void* gate_save, size_t gate_save_bytes,
                      void* ws, size_t ws_bytes, void* stream, int32_t* dev_status) {
    const gsa_params_t& p = *params;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    Workspace w = carve(p, GSA_WS_FWD, ws);
    if (ws_bytes < w.bytes) return GSA_ERR_WORKSPACE;
    // the gate kernel's products go to the caller's block when the backward is to reuse them
    if (save_gate && !use_gate_block(p, &w, gate_save, gate_save_bytes)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Slices s = slices(p);

    const int nseg = segments_of(p);
    GSA_CUDA(cudaMemsetAsync(w.strong, 0, sizeof(int) * (size_t)p.B * p.H * nseg, st));
    if (p.gate_kind == GSA_GATE_ABC)      // no decay, write weights from the cumulative softmax of the scores
        GSA_LAUNCH("abc_write", launch_abc_write(gate, w.G, w.I, w.Id, p.B, p.T, p.H, p.m, st));
    else
        GSA_LAUNCH("gate_cumsum", launch_gate_cumsum(gate, p.gate_kind, inv_tau(p), w.G, w.I, p.B, p.T,
                                                     p.H, p.m, chunk_of(p), w.strong, nseg, w.Id, p.io == GSA_BF16, st,
                                                     p.cu_seqlens, p.nseq));
    float* ok = ok_save;      // the scaled logits leave the softmax kernel only if the caller keeps them
    // the pipelined kernels leave the row factor of the pass-1 sums to the softmax kernel
    const PendingDecay pend = use_tc(p) ? PendingDecay{w.G, w.strong, p.T, p.H, nseg} : PendingDecay{nullptr, nullptr, 1, 1, 1};
    // [B,T,H,.] cut into nseg segments is the same memory as [B*nseg, T/nseg, H, .]
    const int Bs = p.B * nseg, Ts = p.T / nseg;
    const float *Kin = K0, *Vin = V0;
    float *Kout = KT, *Vout = VT;
    if (nseg > 1) {
        // first pass: every segment from empty memories, only for its end memories (the outputs
        // land in buffers that the second pass overwrites); then the start memories of all
        // segments, and the final memories, by a scan over the segments
        GSA_LAUNCH("segment_logdecay", launch_segment_logdecay(w.G, w.seg_decay, p.B, p.T, p.H, p.m, nseg,
                                                               chunk_of(p), st));
        ValueSideArgs s1{q, k, w.I, w.G, nullptr, w.Kloc, w.okpart, Bs, Ts, p.H, p.d_k, w.Id, 1};
        GSA_LAUNCH("segment_pass1_states", value_side(p, s1, 0, w.strong, st, dev_status));
        KeySideArgs s2{w.I, w.I, w.G, v, nullptr, w.Vloc, o, Bs, Ts, p.H, p.d_v, w.Id, w.Id, 1};
        GSA_LAUNCH("segment_pass2_states", key_side(p, s2, 0, w.strong, st, dev_status));
        // (when the backward is to reuse them, the final memories land in the saved block first)
        float* KTc = save_gate ? w.KT : KT;
        float* VTc = save_gate ? w.VT : VT;
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Kloc, K0, w.Kstart, KTc, p.B, p.H, p.m,
                                                             p.d_k, nseg, 0, st));
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Vloc, V0, w.Vstart, VTc, p.B, p.H, p.m,
                                                             p.d_v, nseg, 0, st));
        if (save_gate && KT != nullptr)
            GSA_CUDA(cudaMemcpyAsync(KT, w.KT, sizeof(float) * (size_t)p.B * p.H * p.m * p.d_k, cudaMemcpyDeviceToDevice, st));
        if (save_gate && VT != nullptr)
            GSA_CUDA(cudaMemcpyAsync(VT, w.VT, sizeof(float) * (size_t)p.B * p.H * p.m * p.d_v, cudaMemcpyDeviceToDevice, st));
        Kin = w.Kstart; Vin = w.Vstart;
        Kout = nullptr; Vout = nullptr;
    }
    // pass 1: o' = GLA(q, k, 1-a) with the decay on the slot (value) side
    ValueSideArgs a1{q, k, w.I, w.G, Kin, Kout, w.okpart, Bs, Ts, p.H, p.d_k, w.Id};
    // pass 2: o = GLA(softmax(o'), 1-a, v) with the decay on the slot (key) side
    KeySideArgs a2{w.p, w.I, w.G, v, Vin, Vout, o, Bs, Ts, p.H, p.d_v, w.Pd, w.Id};
    if (use_fused(p)) {
        // One kernel for pass 1 -> softmax -> pass 2; the logits are written only if the caller wants
        // them.  The (batch, head) pairs flagged for strong decay take the general kernels and the
        // slot kernel (restricted to those pairs) on the side stream, beside the fused kernel.
        PendingDecay only = pend;
        only.strong_only = 1;
        SideLane* side = nullptr;
        GSA_CUDA(side_lane(&side));
        cudaStream_t ss = g_sink.active ? st : side->stream;
        if (!g_sink.active) {
            GSA_CUDA(cudaEventRecord(side->fork, st));
            GSA_CUDA(cudaStreamWaitEvent(ss, side->fork, 0));
        }
        GSA_LAUNCH("fused_fwd", launch_fused_pair(0, q, k, w.Id, v, o, w.G, Kin, Vin, Kout, Vout, Bs, Ts, p.H, p.d_k,
                                                  p.d_v, p.scale, p.slot_act, ok_save, nullptr, nullptr, nullptr, w.strong,
                                                  st, dev_status));
        GSA_CUDA(launch_value_side_general(a1, p.m, 0, w.strong, ss, dev_status));
        GSA_CUDA(launch_slot_softmax_fwd(w.okpart, s.k, p.scale, p.slot_act, ok, w.p, p.B, p.T * p.H, p.m, pend.G, w.Pd, only, ss, m_active));
        GSA_CUDA(launch_key_side_general(a2, p.m, 0, w.strong, ss, dev_status));
        if (!g_sink.active) {
            GSA_CUDA(cudaEventRecord(side->join, ss));
            GSA_CUDA(cudaStreamWaitEvent(st, side->join, 0));
        }
        return GSA_OK;
    }
    GSA_LAUNCH("pass1_value_side", value_side(p, a1, 0, w.strong, st, dev_status));
    GSA_LAUNCH("slot_softmax", launch_slot_softmax_fwd(w.okpart, s.k, p.scale, p.slot_act, ok, w.p, p.B, p.T * p.H, p.m, pend.G, w.Pd,
                                                       pend, st, m_active));
    GSA_LAUNCH("pass2_key_side", key_side(p, a2, 0, w.strong, st, dev_status));
    return GSA_OK;
}

// Validation, and the padded-slot mode around the core (see pads_slots).
gsa_status_t fwd_impl(const gsa_params_t* params, const void* q, const void* k, const void* v,
                      const float* gate, const float* K0, const float* V0, void* o,
                      float* ok_save, float* KT, float* VT, bool save_gate, void* gate_save, size_t gate_save_bytes,
                      void* ws, size_t ws_bytes, void* stream, int32_t* dev_status) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(q) || !ok_ptr(k) || !ok_ptr(v) || !ok_ptr(gate) || !ok_ptr(o)) return GSA_ERR_INVALID_ARG;
    if (!ok_opt(K0) || !ok_opt(V0) || !ok_opt(ok_save) || !ok_opt(KT) || !ok_opt(VT))
        return GSA_ERR_INVALID_ARG;
    {
        // a bfloat16 gate tensor is widened once; everything downstream reads fp32
        const gsa_params_t pi0 = internal_params(*params);
        const size_t before = carve(pi0, GSA_WS_FWD, nullptr).bytes + pad_bytes(*params, GSA_WS_FWD);
        rc = gate_as_f32(*params, GSA_WS_FWD, gate, ws, ws_bytes, before, static_cast<cudaStream_t>(stream), &gate);
        if (rc != GSA_OK) return rc;
        rc = apply_feature_map(*params, GSA_WS_FWD, &q, &k, &v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
        if (rc != GSA_OK) return rc;
    }
    if (!pads_slots(*params))
        return fwd_core(params, 0, q, k, v, gate, K0, V0, o, ok_save, KT, VT, save_gate, gate_save, gate_save_bytes, ws,
                        ws_bytes, stream, dev_status);
    const gsa_params_t& p = *params;
    const gsa_params_t pi = internal_params(p);
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    const size_t core = carve(pi, GSA_WS_FWD, nullptr).bytes;
    const PadBuffers pb = carve_pad(p, GSA_WS_FWD, static_cast<char*>(ws) + core);
    if (ws_bytes < core + pb.bytes) return GSA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)p.B * p.T * p.H, pairs = (size_t)p.B * p.H;
    const int M = kPaddedSlots;
    // a neutral gate for the padding: a = 1 (log a = 0; a logit whose sigmoid is 1 to rounding)
    const float neutral = p.gate_kind == GSA_GATE_A ? 1.f : (p.gate_kind == GSA_GATE_LOG_A ? 0.f : 80.f);
    GSA_CUDA(launch_resize_rows(gate, pb.gate, rows, p.m, M, neutral, st));
    if (K0) GSA_CUDA(launch_resize_rows(K0, pb.K0, pairs, p.m * p.d_k, M * p.d_k, 0.f, st));
    if (V0) GSA_CUDA(launch_resize_rows(V0, pb.V0, pairs, p.m * p.d_v, M * p.d_v, 0.f, st));
    rc = fwd_core(&pi, p.m, q, k, v, pb.gate, K0 ? pb.K0 : nullptr, V0 ? pb.V0 : nullptr, o, ok_save ? pb.ok : nullptr,
                  KT ? pb.KT : nullptr, VT ? pb.VT : nullptr, save_gate, gate_save, gate_save_bytes, ws, core, stream,
                  dev_status);
    if (rc != GSA_OK) return rc;
    if (ok_save) GSA_CUDA(launch_resize_rows(pb.ok, ok_save, rows, M, p.m, 0.f, st));
    if (KT) GSA_CUDA(launch_resize_rows(pb.KT, KT, pairs, M * p.d_k, p.m * p.d_k, 0.f, st));
    if (VT) GSA_CUDA(launch_resize_rows(pb.VT, VT, pairs, M * p.d_v, p.m * p.d_v, 0.f, st));
    return GSA_OK;
}
}  // namespace

gsa_status_t gsa_fwd(const gsa_params_t* params, const void* q, const void* k, const void* v,
                     const float* gate, const float* K0, const float* V0, void* o,
                     float* ok_save, float* KT, float* VT, void* ws, size_t ws_bytes,
                     void* stream, int32_t* dev_status) {
    return fwd_impl(params, q, k, v, gate, K0, V0, o, ok_save, KT, VT, false, nullptr, 0, ws, ws_bytes, stream,
                    dev_status);
}

gsa_status_t gsa_fwd_save_gate(const gsa_params_t* params, const void* q, const void* k, const void* v,
                               const float* gate, const float* K0, const float* V0, void* o,
                               float* ok_save, float* KT, float* VT, void* gate_save, size_t gate_save_bytes,
                               void* ws, size_t ws_bytes, void* stream, int32_t* dev_status) {
    return fwd_impl(params, q, k, v, gate, K0, V0, o, ok_save, KT, VT, true, gate_save, gate_save_bytes, ws,
                    ws_bytes, stream, dev_status);
}

namespace {
gsa_status_t bwd_core(const gsa_params_t* params, int m_active, const void* q, const void* k, const void* v,
                      const float* gate, const float* K0, const float* V0, const float* ok_saved,
                      const void* dO, const float* dKT, const float* dVT, void* dq, void* dk,
                      void* dv, float* dgate, float* dK0, float* dV0, bool gate_is_saved, const void* gate_saved,
                      size_t gate_saved_bytes, void* ws, size_t ws_bytes, void* stream, int32_t* dev_status) {
    const gsa_params_t& p = *params;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    Workspace w = carve(p, GSA_WS_BWD, ws);
    if (ws_bytes < w.bytes) return GSA_ERR_WORKSPACE;
    if (gate_is_saved && !use_gate_block(p, &w, const_cast<void*>(gate_saved), gate_saved_bytes)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Slices s = slices(p);

    // Long sequences with few (batch, head) pairs run as nseg independent segments (see gsa_fwd):
    // [B,T,H,.] viewed as [B*nseg, T/nseg, H, .], every scan starting from the state that enters its
    // segment -- from the left for the forward-direction scans, from the right for the reversed ones.
    const int nseg = segments_of(p);
    const int Bs = p.B * nseg, Ts = p.T / nseg;
    if (!gate_is_saved) {      // (a forward of the same call left the gate kernel's products otherwise)
        GSA_CUDA(cudaMemsetAsync(w.strong, 0, sizeof(int) * (size_t)p.B * p.H * nseg, st));
        if (p.gate_kind == GSA_GATE_ABC)
            GSA_LAUNCH("abc_write", launch_abc_write(gate, w.G, w.I, w.Id, p.B, p.T, p.H, p.m, st));
        else
            GSA_LAUNCH("gate_cumsum", launch_gate_cumsum(gate, p.gate_kind, inv_tau(p), w.G, w.I, p.B, p.T,
                                                         p.H, p.m, chunk_of(p), w.strong, nseg, w.Id, p.io == GSA_BF16, st,
                                                         p.cu_seqlens, p.nseq));
    }
    const float* ok = ok_saved;
    const PendingDecay pend = use_tc(p) ? PendingDecay{w.G, w.strong, p.T, p.H, nseg} : PendingDecay{nullptr, nullptr, 1, 1, 1};
    const float *Kin = K0, *Vin = V0;        // states entering the forward-direction scans
    float* KTout = dKT ? w.KT : nullptr;     // final memories, for the gate gradient's final-memory term
    float* VTout = dVT ? w.VT : nullptr;
    if (nseg > 1 && gate_is_saved) {
        // the forward of the same call left the segments' decay, the memories entering every
        // segment and the final memories in the block
        Kin = w.Kstart; Vin = w.Vstart;
        KTout = nullptr; VTout = nullptr;
    } else if (nseg > 1) {
        GSA_LAUNCH("segment_logdecay", launch_segment_logdecay(w.G, w.seg_decay, p.B, p.T, p.H, p.m, nseg,
                                                               chunk_of(p), st));
        ValueSideArgs s1{q, k, w.I, w.G, nullptr, w.Kloc, w.okpart, Bs, Ts, p.H, p.d_k, w.Id, 1};
        GSA_LAUNCH("segment_pass1_states", value_side(p, s1, 0, w.strong, st, dev_status));
        KeySideArgs s2{w.I, w.I, w.G, v, nullptr, w.Vloc, dv, Bs, Ts, p.H, p.d_v, w.Id, w.Id, 1};
        GSA_LAUNCH("segment_pass2_states", key_side(p, s2, 0, w.strong, st, dev_status));
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Kloc, K0, w.Kstart, KTout, p.B, p.H, p.m,
                                                             p.d_k, nseg, 0, st));
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Vloc, V0, w.Vstart, VTout, p.B, p.H, p.m,
                                                             p.d_v, nseg, 0, st));
        Kin = w.Kstart; Vin = w.Vstart;
        KTout = nullptr; VTout = nullptr;
    }
    if (ok == nullptr) {  // recompute pass 1 and its logits
        ValueSideArgs a1{q, k, w.I, w.G, Kin, nullptr, w.okpart, Bs, Ts, p.H, p.d_k, w.Id};
        GSA_LAUNCH("pass1_value_side", value_side(p, a1, 0, w.strong, st, dev_status));
        GSA_LAUNCH("slot_softmax", launch_slot_softmax_fwd(w.okpart, s.k, p.scale, p.slot_act, w.ok, w.p, p.B, p.T * p.H, p.m, pend.G,
                                                           nullptr, pend, st, m_active));
        ok = w.ok;
    }
    // gradient w.r.t. the pass-2 queries p: the pass-1 form on (dO, v, 1-a); carries V~
    ValueSideArgs adp{dO, v, w.I, w.G, Vin, VTout, w.dppart, Bs, Ts, p.H, p.d_v, w.Id};
    // dq: the pass-2 form on (dz, 1-a, k); carries K~
    KeySideArgs adq{w.dz, w.I, w.G, k, Kin, KTout, dq, Bs, Ts, p.H, p.d_k, w.Zd, w.Id};
    const bool fused = use_fused(p);
    // With the forward's slot weights in the saved block (and the logits saved, so that nothing here
    // rewrites them), the dv and dI^v scans depend on nothing this call computes: they start at once,
    // on two of the library's streams, beside the dp scan and the softmax gradient.
    const bool early = gate_is_saved && ok_saved != nullptr && use_tc(p) && !fused && nseg == 1 && !g_sink.active;
    ScanLanes* lanes = nullptr;
    if (use_tc(p) && !g_sink.active) GSA_CUDA(scan_lanes(&lanes));
    if (early) {
        GSA_CUDA(cudaEventRecord(lanes->fork_early, st));
        for (int i = 0; i < 2; ++i) GSA_CUDA(cudaStreamWaitEvent(lanes->stream[i], lanes->fork_early, 0));
        GSA_CUDA(cudaStreamWaitEvent(lanes->fast, lanes->fork_early, 0));
    }
    // (the chain dp -> softmax gradient, which three more scans wait for, goes first wherever an SM is free:
    // it runs on the library's high-priority stream, the early scans fill what it leaves)
    cudaStream_t sc = early ? lanes->fast : st;
    if (fused) {
        // One kernel for dp -> dsoftmax -> dq (it also leaves u and the decayed rows of p and dz for the
        // reversed scans); the flagged pairs take the general kernels on the side stream.
        PendingDecay only = pend;
        only.strong_only = 1;
        SideLane* side = nullptr;
        GSA_CUDA(side_lane(&side));
        cudaStream_t ss = g_sink.active ? st : side->stream;
        if (!g_sink.active) {
            GSA_CUDA(cudaEventRecord(side->fork, st));
            GSA_CUDA(cudaStreamWaitEvent(ss, side->fork, 0));
        }
        GSA_LAUNCH("fused_bwd", launch_fused_pair(1, dO, v, w.Id, k, dq, w.G, Vin, Kin, VTout, KTout, Bs, Ts, p.H, p.d_v,
                                                  p.d_k, p.scale, p.slot_act, const_cast<float*>(ok), w.u, w.Pd, w.Zd,
                                                  w.strong, st, dev_status));
        GSA_CUDA(launch_value_side_general(adp, p.m, 0, w.strong, ss, dev_status));
        GSA_CUDA(launch_slot_softmax_bwd(ok, w.dppart, s.v, p.scale, p.slot_act, w.p, w.dz, w.u, p.B, p.T * p.H, p.m, pend.G,
                                         w.Pd, w.Zd, only, ss, m_active));
        GSA_CUDA(launch_key_side_general(adq, p.m, 0, w.strong, ss, dev_status));
        if (!g_sink.active) {
            GSA_CUDA(cudaEventRecord(side->join, ss));
            GSA_CUDA(cudaStreamWaitEvent(st, side->join, 0));
        }
    } else {
        GSA_LAUNCH("bwd_dp_value_side", value_side(p, adp, 0, w.strong, sc, dev_status));
        if (early) {
            KeySideArgs adv{w.I, w.p, w.G, dO, dVT, dV0, dv, Bs, Ts, p.H, p.d_v, w.Id, w.Pd};
            ValueSideArgs adIv{v, dO, w.p, w.G, dVT, nullptr, w.dIv, Bs, Ts, p.H, p.d_v, w.Pd};
            adv.single = adIv.single = p.tc_operands == GSA_TC_SINGLE;
            if (g_pair_scans.load(std::memory_order_relaxed) != 0 && rev_pair_supported(adIv, adv, p.m)) {
                GSA_CUDA(launch_rev_pair_tc(adIv, adv, p.m, w.strong, lanes->stream[0], dev_status));
            } else {
                GSA_CUDA(key_side(p, adv, 1, w.strong, lanes->stream[0], dev_status));
                GSA_CUDA(value_side(p, adIv, 1, w.strong, lanes->stream[1], dev_status));
            }
        }
        // (started early, the dv / dI^v scans are reading the forward's p: it is not written again)
        GSA_LAUNCH("slot_softmax_bwd", launch_slot_softmax_bwd(ok, w.dppart, s.v, p.scale, p.slot_act, early ? nullptr : w.p, w.dz, w.u,
                                                               p.B, p.T * p.H, p.m, pend.G, early ? nullptr : w.Pd, w.Zd, pend, sc,
                                                               m_active));
        if (early) {
            GSA_CUDA(cudaEventRecord(lanes->fast_done, sc));
            GSA_CUDA(cudaStreamWaitEvent(st, lanes->fast_done, 0));
        }
    }
    const float *dKin = dKT, *dVin = dVT;    // states entering the reversed scans (from the right)
    float *dK0out = dK0, *dV0out = dV0;
    if (nseg > 1) {
        // reversed scans of every segment from empty states, for their end states only (the outputs
        // land in dk / dv, which the real scans overwrite); then the states entering every segment,
        // and dK0 / dV0, by a scan over the segments from the last one down
        KeySideArgs r1{w.I, w.dz, w.G, q, nullptr, w.Kloc, dk, Bs, Ts, p.H, p.d_k, w.Id, w.Zd, 1};
        GSA_LAUNCH("segment_dk_states", key_side(p, r1, 1, w.strong, st, dev_status));
        KeySideArgs r2{w.I, w.p, w.G, dO, nullptr, w.Vloc, dv, Bs, Ts, p.H, p.d_v, w.Id, w.Pd, 1};
        GSA_LAUNCH("segment_dv_states", key_side(p, r2, 1, w.strong, st, dev_status));
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Kloc, dKT, w.dKend, dK0, p.B, p.H, p.m,
                                                             p.d_k, nseg, 1, st));
        GSA_LAUNCH("segment_combine", launch_segment_combine(w.seg_decay, w.Vloc, dVT, w.dVend, dV0, p.B, p.H, p.m,
                                                             p.d_v, nseg, 1, st));
        dKin = w.dKend; dVin = w.dVend;
        dK0out = nullptr; dV0out = nullptr;
    }
    // time-reversed runs: dv and dI^v share the state dV~; dk and dI^k share dK~
    KeySideArgs adv{w.I, w.p, w.G, dO, dVin, dV0out, dv, Bs, Ts, p.H, p.d_v, w.Id, w.Pd};
    ValueSideArgs adIv{v, dO, w.p, w.G, dVin, nullptr, w.dIv, Bs, Ts, p.H, p.d_v, w.Pd};
    KeySideArgs adk{w.I, w.dz, w.G, q, dKin, dK0out, dk, Bs, Ts, p.H, p.d_k, w.Id, w.Zd};
    ValueSideArgs adIk{k, q, w.dz, w.G, dKin, nullptr, w.dIk, Bs, Ts, p.H, p.d_k, w.Zd};
    // the reversed scans that share a state run as one kernel each (dv with dI^v, dk with dI^k)
    ValueSideArgs pIv = adIv, pIk = adIk;
    KeySideArgs pv = adv, pk = adk;
    pIv.single = pIk.single = pv.single = pk.single = p.tc_operands == GSA_TC_SINGLE;
    const bool paired = use_tc(p) && g_pair_scans.load(std::memory_order_relaxed) != 0 &&
                        rev_pair_supported(pIv, pv, p.m) && rev_pair_supported(pIk, pk, p.m);
    if (paired && !g_sink.active) {
        GSA_CUDA(cudaEventRecord(lanes->fork, st));
        for (int i = early ? 1 : 0; i < 2; ++i) GSA_CUDA(cudaStreamWaitEvent(lanes->stream[i], lanes->fork, 0));
        if (!fused) GSA_CUDA(key_side(p, adq, 0, w.strong, st, dev_status));
        if (!early) GSA_CUDA(launch_rev_pair_tc(pIv, pv, p.m, w.strong, lanes->stream[0], dev_status));
        GSA_CUDA(launch_rev_pair_tc(pIk, pk, p.m, w.strong, lanes->stream[1], dev_status));
        for (int i = 0; i < 2; ++i) {
            GSA_CUDA(cudaEventRecord(lanes->join[i], lanes->stream[i]));
            GSA_CUDA(cudaStreamWaitEvent(st, lanes->join[i], 0));
        }
    } else if (paired) {
        if (!fused) GSA_LAUNCH("bwd_dq_key_side", key_side(p, adq, 0, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dv_dIv_pair_rev", launch_rev_pair_tc(pIv, pv, p.m, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dk_dIk_pair_rev", launch_rev_pair_tc(pIk, pk, p.m, w.strong, st, dev_status));
    } else if (use_tc(p) && !g_sink.active) {
        // the five scans side by side (see ScanLanes)
        GSA_CUDA(cudaEventRecord(lanes->fork, st));
        for (int i = early ? 2 : 0; i < 4; ++i) GSA_CUDA(cudaStreamWaitEvent(lanes->stream[i], lanes->fork, 0));
        if (!fused) GSA_CUDA(key_side(p, adq, 0, w.strong, st, dev_status));
        if (!early) {
            GSA_CUDA(key_side(p, adv, 1, w.strong, lanes->stream[0], dev_status));
            GSA_CUDA(value_side(p, adIv, 1, w.strong, lanes->stream[1], dev_status));
        }
        GSA_CUDA(key_side(p, adk, 1, w.strong, lanes->stream[2], dev_status));
        GSA_CUDA(value_side(p, adIk, 1, w.strong, lanes->stream[3], dev_status));
        for (int i = 0; i < 4; ++i) {
            GSA_CUDA(cudaEventRecord(lanes->join[i], lanes->stream[i]));
            GSA_CUDA(cudaStreamWaitEvent(st, lanes->join[i], 0));
        }
    } else {
        if (!fused) GSA_LAUNCH("bwd_dq_key_side", key_side(p, adq, 0, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dv_key_side_rev", key_side(p, adv, 1, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dIv_value_side_rev", value_side(p, adIv, 1, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dk_key_side_rev", key_side(p, adk, 1, w.strong, st, dev_status));
        GSA_LAUNCH("bwd_dIk_value_side_rev", value_side(p, adIk, 1, w.strong, st, dev_status));
    }
    if (p.gate_kind == GSA_GATE_ABC) {
        // no decay path: the scores' gradient follows from that of the write weights (G == 0: no row factor pending)
        GSA_LAUNCH("abc_grad", launch_abc_grad(w.I, w.dIk, s.k, w.dIv, s.v, dgate, p.B, p.T, p.H, p.m, st));
        return GSA_OK;
    }
    // forget-gate gradient: reversed cumulative sum over the whole sequence
    GSA_LAUNCH("gate_grad", launch_gate_grad(w.u, w.I, w.dIk, s.k, w.dIv, s.v, gate, p.gate_kind, inv_tau(p),
                              dKT, w.KT, dVT, w.VT, p.d_k, p.d_v, w.chunk_tot, dgate, p.B, p.T,
                              p.H, p.m, pend, st, dev_status));
    return GSA_OK;
}

gsa_status_t bwd_impl(const gsa_params_t* params, const void* q, const void* k, const void* v,
                      const float* gate, const float* K0, const float* V0, const float* ok_saved,
                      const void* dO, const float* dKT, const float* dVT, void* dq, void* dk,
                      void* dv, float* dgate, float* dK0, float* dV0, bool gate_is_saved, const void* gate_saved,
                      size_t gate_saved_bytes, void* ws, size_t ws_bytes, void* stream, int32_t* dev_status) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(q) || !ok_ptr(k) || !ok_ptr(v) || !ok_ptr(gate) || !ok_ptr(dO) || !ok_ptr(dq) ||
        !ok_ptr(dk) || !ok_ptr(dv) || !ok_ptr(dgate))
        return GSA_ERR_INVALID_ARG;
    if (!ok_opt(K0) || !ok_opt(V0) || !ok_opt(ok_saved) || !ok_opt(dKT) || !ok_opt(dVT) ||
        !ok_opt(dK0) || !ok_opt(dV0))
        return GSA_ERR_INVALID_ARG;
    const void *q_raw = q, *k_raw = k, *v_raw = v;
    float *dgate_row = nullptr, *colsum = nullptr;
    {
        const gsa_params_t pi0 = internal_params(*params);
        const size_t before = carve(pi0, GSA_WS_BWD, nullptr).bytes + pad_bytes(*params, GSA_WS_BWD);
        rc = gate_as_f32(*params, GSA_WS_BWD, gate, ws, ws_bytes, before, static_cast<cudaStream_t>(stream), &gate);
        if (rc != GSA_OK) return rc;
        rc = apply_feature_map(*params, GSA_WS_BWD, &q, &k, &v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
        if (rc != GSA_OK) return rc;
        if (params->gate_broadcast) {        // the per-token gate gradient lands in the workspace; its sum is returned
            const GateBoundary g = gate_boundary(*params, GSA_WS_BWD);
            char* base = static_cast<char*>(ws) + before;
            dgate_row = dgate;
            dgate = reinterpret_cast<float*>(base + g.conv + g.spread);
            colsum = reinterpret_cast<float*>(base + g.conv + g.spread + g.dfull);
        }
    }
    // with the feature map, dq / dk / dv are turned into gradients w.r.t. the pre-activations at the end
    auto finish = [&](gsa_status_t r) -> gsa_status_t {
        if (r != GSA_OK) return r;
        cudaStream_t s2 = static_cast<cudaStream_t>(stream);
        if (dgate_row != nullptr &&
            launch_column_sum(dgate, colsum, dgate_row, (size_t)params->B * params->T, params->H * params->m, s2) != cudaSuccess)
            return GSA_ERR_CUDA;
        if (params->feature_map != GSA_FEAT_SWISH) return GSA_OK;
        const size_t R = (size_t)params->B * params->T * params->H;
        if (launch_swish_bwd(q_raw, dq, R * params->d_k, params->io, s2) != cudaSuccess) return GSA_ERR_CUDA;
        if (launch_swish_bwd(k_raw, dk, R * params->d_k, params->io, s2) != cudaSuccess) return GSA_ERR_CUDA;
        if (launch_swish_bwd(v_raw, dv, R * params->d_v, params->io, s2) != cudaSuccess) return GSA_ERR_CUDA;
        return GSA_OK;
    };
    if (!pads_slots(*params))
        return finish(bwd_core(params, 0, q, k, v, gate, K0, V0, ok_saved, dO, dKT, dVT, dq, dk, dv, dgate, dK0, dV0,
                               gate_is_saved, gate_saved, gate_saved_bytes, ws, ws_bytes, stream, dev_status));
    const gsa_params_t& p = *params;
    const gsa_params_t pi = internal_params(p);
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    const size_t core = carve(pi, GSA_WS_BWD, nullptr).bytes;
    const PadBuffers pb = carve_pad(p, GSA_WS_BWD, static_cast<char*>(ws) + core);
    if (ws_bytes < core + pb.bytes) return GSA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)p.B * p.T * p.H, pairs = (size_t)p.B * p.H;
    const int M = kPaddedSlots;
    const float neutral = p.gate_kind == GSA_GATE_A ? 1.f : (p.gate_kind == GSA_GATE_LOG_A ? 0.f : 80.f);
    GSA_CUDA(launch_resize_rows(gate, pb.gate, rows, p.m, M, neutral, st));
    if (ok_saved) GSA_CUDA(launch_resize_rows(ok_saved, pb.ok, rows, p.m, M, 0.f, st));
    if (K0) GSA_CUDA(launch_resize_rows(K0, pb.K0, pairs, p.m * p.d_k, M * p.d_k, 0.f, st));
    if (V0) GSA_CUDA(launch_resize_rows(V0, pb.V0, pairs, p.m * p.d_v, M * p.d_v, 0.f, st));
    if (dKT) GSA_CUDA(launch_resize_rows(dKT, pb.dKT, pairs, p.m * p.d_k, M * p.d_k, 0.f, st));
    if (dVT) GSA_CUDA(launch_resize_rows(dVT, pb.dVT, pairs, p.m * p.d_v, M * p.d_v, 0.f, st));
    rc = bwd_core(&pi, p.m, q, k, v, pb.gate, K0 ? pb.K0 : nullptr, V0 ? pb.V0 : nullptr, ok_saved ? pb.ok : nullptr, dO,
                  dKT ? pb.dKT : nullptr, dVT ? pb.dVT : nullptr, dq, dk, dv, pb.dgate, dK0 ? pb.KT : nullptr,
                  dV0 ? pb.VT : nullptr, gate_is_saved, gate_saved, gate_saved_bytes, ws, core, stream, dev_status);
    if (rc != GSA_OK) return rc;
    GSA_CUDA(launch_resize_rows(pb.dgate, dgate, rows, M, p.m, 0.f, st));
    if (dK0) GSA_CUDA(launch_resize_rows(pb.KT, dK0, pairs, M * p.d_k, p.m * p.d_k, 0.f, st));
    if (dV0) GSA_CUDA(launch_resize_rows(pb.VT, dV0, pairs, M * p.d_v, p.m * p.d_v, 0.f, st));
    return finish(GSA_OK);
}
}  // namespace

gsa_status_t gsa_bwd(const gsa_params_t* params, const void* q, const void* k, const void* v,
                     const float* gate, const float* K0, const float* V0, const float* ok_saved,
                     const void* dO, const float* dKT, const float* dVT, void* dq, void* dk,
                     void* dv, float* dgate, float* dK0, float* dV0, void* ws, size_t ws_bytes,
                     void* stream, int32_t* dev_status) {
    return bwd_impl(params, q, k, v, gate, K0, V0, ok_saved, dO, dKT, dVT, dq, dk, dv, dgate, dK0, dV0, false,
                    nullptr, 0, ws, ws_bytes, stream, dev_status);
}

gsa_status_t gsa_bwd_saved_gate(const gsa_params_t* params, const void* q, const void* k, const void* v,
                                const float* gate, const float* K0, const float* V0, const float* ok_saved,
                                const void* dO, const float* dKT, const float* dVT, void* dq, void* dk,
                                void* dv, float* dgate, float* dK0, float* dV0, const void* gate_saved,
                                size_t gate_saved_bytes, void* ws, size_t ws_bytes, void* stream,
                                int32_t* dev_status) {
    return bwd_impl(params, q, k, v, gate, K0, V0, ok_saved, dO, dKT, dVT, dq, dk, dv, dgate, dK0, dV0, true,
                    gate_saved, gate_saved_bytes, ws, ws_bytes, stream, dev_status);
}

gsa_status_t gsa_decode_step(const gsa_params_t* params, const void* q, const void* k,
                             const void* v, const float* gate, float* Kstate, float* Vstate,
                             void* o, void* stream) {
    gsa_status_t rc = check_params(params, false);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(q) || !ok_ptr(k) || !ok_ptr(v) || !ok_ptr(gate) || !ok_ptr(Kstate) ||
        !ok_ptr(Vstate) || !ok_ptr(o))
        return GSA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->gate_kind == GSA_GATE_ABC) return GSA_ERR_UNSUPPORTED;      // (the running normaliser is not a state here)
    GSA_LAUNCH("decode_step", launch_decode(*params, q, k, v, gate, Kstate, Vstate, o, st));
    return GSA_OK;
}

// ---- sequence sharding across GPUs: the two local steps around the exchange of shard memories
gsa_status_t gsa_shard_states(const gsa_params_t* params, const void* k, const void* v, const float* gate,
                              float* KT, float* VT, float* logdecay, void* ws, size_t ws_bytes, void* stream,
                              int32_t* dev_status) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (pads_slots(*params) || params->gate_dtype != GSA_F32 || params->cu_seqlens != nullptr ||
        params->feature_map != GSA_FEAT_NONE || params->gate_kind == GSA_GATE_ABC || params->gate_broadcast)
        return GSA_ERR_UNSUPPORTED;
    if (!ok_ptr(k) || !ok_ptr(v) || !ok_ptr(gate) || !ok_ptr(KT) || !ok_ptr(VT) || !ok_ptr(logdecay)) return GSA_ERR_INVALID_ARG;
    const gsa_params_t& p = *params;
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return GSA_ERR_WORKSPACE;
    Workspace w = carve(p, GSA_WS_FWD, ws);
    const size_t esz = p.io == GSA_BF16 ? 2 : 4;
    const size_t obytes = align_up((size_t)p.B * p.T * p.H * p.d_v * esz, 256);
    if (ws_bytes < w.bytes + obytes) return GSA_ERR_WORKSPACE;
    void* oscratch = static_cast<char*>(ws) + w.bytes;      // the scans' token outputs are not wanted: they land here
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // one "segment" per batch element: the whole shard from empty memories, end memories only
    GSA_CUDA(cudaMemsetAsync(w.strong, 0, sizeof(int) * (size_t)p.B * p.H * segments_of(p), st));
    GSA_LAUNCH("gate_cumsum", launch_gate_cumsum(gate, p.gate_kind, inv_tau(p), w.G, w.I, p.B, p.T, p.H, p.m, chunk_of(p),
                                                 w.strong, 1, w.Id, p.io == GSA_BF16, st));
    GSA_LAUNCH("segment_logdecay", launch_segment_logdecay(w.G, logdecay, p.B, p.T, p.H, p.m, 1, chunk_of(p), st));
    ValueSideArgs s1{k, k, w.I, w.G, nullptr, KT, w.okpart, p.B, p.T, p.H, p.d_k, w.Id, 1};
    GSA_LAUNCH("segment_pass1_states", value_side(p, s1, 0, w.strong, st, dev_status));
    KeySideArgs s2{w.I, w.I, w.G, v, nullptr, VT, oscratch, p.B, p.T, p.H, p.d_v, w.Id, w.Id, 1};
    GSA_LAUNCH("segment_pass2_states", key_side(p, s2, 0, w.strong, st, dev_status));
    return GSA_OK;
}

gsa_status_t gsa_shard_combine(const gsa_params_t* params, int32_t d, int32_t nshard, int32_t rank, int32_t reverse,
                               const float* logdecay_all, const float* local_all, const float* S0, float* start,
                               float* final_state, void* stream) {
    gsa_status_t rc = check_params(params, false);
    if (rc != GSA_OK) return rc;
    if (nshard < 1 || rank < 0 || rank >= nshard || d < 1) return GSA_ERR_INVALID_ARG;
    if (!ok_ptr(logdecay_all) || !ok_ptr(local_all) || !ok_opt(S0) || !ok_opt(start) || !ok_opt(final_state))
        return GSA_ERR_INVALID_ARG;
    const gsa_params_t& p = *params;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GSA_LAUNCH("shard_combine", launch_shard_combine(logdecay_all, local_all, S0, start, final_state, p.B, p.H, p.m, d, nshard,
                                                     rank, reverse != 0, st));
    return GSA_OK;
}

gsa_status_t gsa_out_norm_fwd(const gsa_params_t* params, const void* o, const float* weight, float eps, void* y,
                              void* stream) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(o) || !ok_ptr(y) || !ok_opt(weight) || !(eps >= 0.f)) return GSA_ERR_INVALID_ARG;
    const gsa_params_t& p = *params;
    if (p.H * p.d_v > out_norm_max_width(p.io)) return GSA_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GSA_LAUNCH("out_norm", launch_out_norm_fwd(o, weight, eps, y, (size_t)p.B * p.T, p.H * p.d_v, p.io, st));
    return GSA_OK;
}

size_t gsa_out_norm_workspace_bytes(const gsa_params_t* params) {
    if (check_params(params, true) != GSA_OK) return 0;
    return align_up(out_norm_bwd_parts((size_t)params->B * params->T) * params->H * params->d_v * sizeof(float), 256);
}

gsa_status_t gsa_out_norm_bwd(const gsa_params_t* params, const void* o, const void* dy, const float* weight, float eps,
                              void* d_o, float* dweight, void* ws, size_t ws_bytes, void* stream) {
    gsa_status_t rc = check_params(params, true);
    if (rc != GSA_OK) return rc;
    if (!ok_ptr(o) || !ok_ptr(dy) || !ok_ptr(d_o) || !ok_opt(weight) || !ok_opt(dweight) || !(eps >= 0.f))
        return GSA_ERR_INVALID_ARG;
    const gsa_params_t& p = *params;
    if (p.H * p.d_v > out_norm_max_width(p.io)) return GSA_ERR_UNSUPPORTED;
    if (dweight != nullptr && (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 ||
                               ws_bytes < gsa_out_norm_workspace_bytes(params)))
        return GSA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    GSA_LAUNCH("out_norm_bwd", launch_out_norm_bwd(o, dy, weight, eps, d_o, static_cast<float*>(ws), dweight,
                                                   (size_t)p.B * p.T, p.H * p.d_v, p.io, st));
    return GSA_OK;
}

gsa_status_t gsa_release_streams(void) {
    if (scan_lanes_release() != cudaSuccess || side_lane_release() != cudaSuccess) return GSA_ERR_CUDA;
    return GSA_OK;
}

int32_t gsa_dev_pair_scans(int32_t enable) { return g_pair_scans.exchange(enable != 0 ? 1 : 0); }

gsa_status_t gsa_timing_begin(int32_t capacity) {
    if (capacity < 1 || capacity > (1 << 20) || g_sink.active) return GSA_ERR_INVALID_ARG;
    g_sink.ev.assign(2 * (size_t)capacity, nullptr);
    g_sink.labels.assign(capacity, nullptr);
    for (auto& e : g_sink.ev)
        if (cudaEventCreate(&e) != cudaSuccess) return GSA_ERR_CUDA;
    g_sink.capacity = capacity;
    g_sink.count = 0;
    g_sink.active = true;
    return GSA_OK;
}

int32_t gsa_timing_end(float* ms, const char** labels, int32_t capacity) {
    if (!g_sink.active) return -1;
    g_sink.active = false;
    const int n = g_sink.count < capacity ? g_sink.count : capacity;
    int rc = n;
    if (g_sink.count > 0 && cudaEventSynchronize(g_sink.ev[2 * g_sink.count - 1]) != cudaSuccess) rc = -1;
    for (int i = 0; i < n && rc >= 0; ++i) {
        if (cudaEventElapsedTime(&ms[i], g_sink.ev[2 * i], g_sink.ev[2 * i + 1]) != cudaSuccess) rc = -1;
        labels[i] = g_sink.labels[i];
    }
    for (auto& e : g_sink.ev)
        if (e) cudaEventDestroy(e);
    g_sink.ev.clear();
    g_sink.labels.clear();
    return rc;
}

}  // extern "C"
