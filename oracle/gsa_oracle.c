/*
 * Gated Slot Attention -- sequential fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GSA layer computes.  It shares no code with the CUDA library and nothing in
 * the product path may call it; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg do.
 *
 * What it follows (arXiv 2409.07146):
 *   - forward / decode: the slot recurrence of Eq. 6 (Sec. 3.2, "GSA: ABC with
 *     gating mechanism"), read out with Eq. 2 (o_t = V~_t^T f(K~_t q_t)):
 *         K~_t = Diag(a_t) K~_{t-1} + (1 - a_t) (x) k_t
 *         V~_t = Diag(a_t) V~_{t-1} + (1 - a_t) (x) v_t
 *         o_t  = V~_t^T softmax(scale * K~_t q_t)
 *     Both memories include token t before they are read (the causal mask of
 *     Eq. 1 is inclusive of i = j).
 *   - backward: the reverse-mode derivative of exactly that recurrence, taken
 *     one time step at a time (no chunking).  The paper only sketches a
 *     chunkwise backward (Algorithm 1); the gradient of Eq. 6 is unique, so the
 *     oracle differentiates Eq. 6 itself.
 *
 * Pins (tests, CPU only): brute-force unrolled O(T^2) form of Eq. 7, a == 0
 * => o_t = v_t, m == 1 => first-order IIR filter, a == 1 => softmax attention
 * over the fixed initial slots, constant-gate closed form, state carry,
 * decode == forward, finite differences and autograd of the unrolled form for
 * every gradient.  The element-wise replacements of the softmax (the paper's
 * ablation on the non-linearity; `act`) are pinned by the same unrolled form
 * with the library's activation functions and its autograd.
 *
 * Layout: q,k [B,T,H,d_k], v,o [B,T,H,d_v], gate [B,T,H,m], states
 * [B,H,m,d], everything contiguous double.  The gate tensor holds a (linear,
 * in [0,1]) when gate_is_log == 0 and g = log a (<= 0) when gate_is_log == 1;
 * in log space a = exp(g) and 1 - a = -expm1(g).
 * (b,h) pairs in [bh_begin, bh_end) are processed; pairs are independent, so a
 * caller may split the range over threads.
 * Return value: 0 on success, -1 on bad arguments, -2 on allocation failure.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

static void gate_pair(double gate, int gate_is_log, double *a, double *ia)
{
    if (gate_is_log) {
        *a = exp(gate);
        *ia = -expm1(gate);
    } else {
        *a = gate;
        *ia = 1.0 - gate;
    }
}

/* The non-linearity between the two passes.  Eq. 6 has the softmax over the m
 * slots; the paper's ablation on it (Table "ablations", "Ablations on
 * non-linearity") drops it or replaces it by an element-wise function. */
enum { ACT_SOFTMAX = 0, ACT_NONE = 1, ACT_RELU = 2, ACT_SWISH = 3, ACT_RELU2 = 4 };

static void slot_act(int act, int m, const double *z, double *p)
{
    if (act == ACT_SOFTMAX) {
        double zmax = -INFINITY, den = 0.0;
        for (int s = 0; s < m; ++s) if (z[s] > zmax) zmax = z[s];
        for (int s = 0; s < m; ++s) { p[s] = exp(z[s] - zmax); den += p[s]; }
        for (int s = 0; s < m; ++s) p[s] /= den;
        return;
    }
    for (int s = 0; s < m; ++s) {
        double x = z[s], r = x > 0.0 ? x : 0.0;
        if (act == ACT_NONE) p[s] = x;
        else if (act == ACT_RELU) p[s] = r;
        else if (act == ACT_SWISH) p[s] = x / (1.0 + exp(-x));
        else p[s] = r * r;
    }
}

/* dz = (dp/dz)^T dp for the same function. */
static void slot_act_bwd(int act, int m, const double *z, const double *p,
                         const double *dp, double *dz)
{
    if (act == ACT_SOFTMAX) {
        double pdp = 0.0;
        for (int s = 0; s < m; ++s) pdp += p[s] * dp[s];
        for (int s = 0; s < m; ++s) dz[s] = p[s] * (dp[s] - pdp);
        return;
    }
    for (int s = 0; s < m; ++s) {
        double x = z[s], g;
        if (act == ACT_NONE) g = 1.0;
        else if (act == ACT_RELU) g = x > 0.0 ? 1.0 : 0.0;
        else if (act == ACT_SWISH) {
            double sg = 1.0 / (1.0 + exp(-x));
            g = sg + x * sg * (1.0 - sg);
        } else g = x > 0.0 ? 2.0 * x : 0.0;
        dz[s] = g * dp[s];
    }
}

/* One step of Eq. 6 for one head: update K (m x dk), V (m x dv) in place, then
 * read out.  z (m) receives the scaled logits, p (m) the softmax, o (dv) the
 * output. */
static void gsa_step(int dk, int dv, int m, int gate_is_log, int act, double scale,
                     const double *q, const double *k, const double *v,
                     const double *gate, double *K, double *V,
                     double *z, double *p, double *o)
{
    for (int s = 0; s < m; ++s) {
        double a, ia;
        gate_pair(gate[s], gate_is_log, &a, &ia);
        double *Ks = K + (size_t)s * dk;
        double *Vs = V + (size_t)s * dv;
        for (int c = 0; c < dk; ++c) Ks[c] = a * Ks[c] + ia * k[c];
        for (int c = 0; c < dv; ++c) Vs[c] = a * Vs[c] + ia * v[c];
    }
    for (int s = 0; s < m; ++s) {
        const double *Ks = K + (size_t)s * dk;
        double acc = 0.0;
        for (int c = 0; c < dk; ++c) acc += Ks[c] * q[c];
        z[s] = scale * acc;
    }
    slot_act(act, m, z, p);
    for (int c = 0; c < dv; ++c) o[c] = 0.0;
    for (int s = 0; s < m; ++s) {
        const double *Vs = V + (size_t)s * dv;
        for (int c = 0; c < dv; ++c) o[c] += p[s] * Vs[c];
    }
}

/* Forward over whole sequences (Eq. 6).  ok (nullable) receives the scaled
 * pre-softmax logits [B,T,H,m]; KT, VT (nullable) the final memories. */
int gsa_oracle_fwd(int B, int T, int H, int dk, int dv, int m, int gate_is_log,
                   int act, double scale, const double *q, const double *k,
                   const double *v, const double *gate, const double *K0,
                   const double *V0, double *o, double *ok, double *KT,
                   double *VT, int bh_begin, int bh_end)
{
    if (B < 1 || T < 0 || H < 1 || dk < 1 || dv < 1 || m < 1) return -1;
    if (act < ACT_SOFTMAX || act > ACT_RELU2) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    double *K = malloc(sizeof(double) * (size_t)m * dk);
    double *V = malloc(sizeof(double) * (size_t)m * dv);
    double *z = malloc(sizeof(double) * m);
    double *p = malloc(sizeof(double) * m);
    if (!K || !V || !z || !p) { free(K); free(V); free(z); free(p); return -2; }
    for (int bh = bh_begin; bh < bh_end; ++bh) {
        int b = bh / H, h = bh % H;
        if (K0) memcpy(K, K0 + (size_t)bh * m * dk, sizeof(double) * (size_t)m * dk);
        else memset(K, 0, sizeof(double) * (size_t)m * dk);
        if (V0) memcpy(V, V0 + (size_t)bh * m * dv, sizeof(double) * (size_t)m * dv);
        else memset(V, 0, sizeof(double) * (size_t)m * dv);
        for (int t = 0; t < T; ++t) {
            size_t row = ((size_t)b * T + t) * H + h;
            gsa_step(dk, dv, m, gate_is_log, act, scale, q + row * dk, k + row * dk,
                     v + row * dv, gate + row * m, K, V, z, p, o + row * dv);
            if (ok) memcpy(ok + row * m, z, sizeof(double) * m);
        }
        if (KT) memcpy(KT + (size_t)bh * m * dk, K, sizeof(double) * (size_t)m * dk);
        if (VT) memcpy(VT + (size_t)bh * m * dv, V, sizeof(double) * (size_t)m * dv);
    }
    free(K); free(V); free(z); free(p);
    return 0;
}

/* Single-token recurrent step (one iteration of Eq. 6) for S sequences:
 * q,k [S,H,d_k], v,o [S,H,d_v], gate [S,H,m], states [S,H,m,d] updated in
 * place.  Pairs (sequence, head) in [sh_begin, sh_end) are processed. */
int gsa_oracle_decode_step(int S, int H, int dk, int dv, int m, int gate_is_log,
                           int act, double scale, const double *q, const double *k,
                           const double *v, const double *gate, double *Kstate,
                           double *Vstate, double *o, int sh_begin, int sh_end)
{
    if (S < 1 || H < 1 || dk < 1 || dv < 1 || m < 1) return -1;
    if (act < ACT_SOFTMAX || act > ACT_RELU2) return -1;
    if (sh_begin < 0 || sh_end > S * H || sh_begin > sh_end) return -1;
    double *z = malloc(sizeof(double) * m);
    double *p = malloc(sizeof(double) * m);
    if (!z || !p) { free(z); free(p); return -2; }
    for (int sh = sh_begin; sh < sh_end; ++sh) {
        gsa_step(dk, dv, m, gate_is_log, act, scale, q + (size_t)sh * dk,
                 k + (size_t)sh * dk, v + (size_t)sh * dv, gate + (size_t)sh * m,
                 Kstate + (size_t)sh * m * dk, Vstate + (size_t)sh * m * dv, z, p,
                 o + (size_t)sh * dv);
    }
    free(z); free(p);
    return 0;
}

/* Backward of Eq. 6 by a plain reverse sweep.
 *
 * The forward is replayed first and every memory K~_t, V~_t (t = 0..T) is kept,
 * so the sweep reads exactly the values the forward produced.  With
 * dK (m x dk), dV (m x dv) the gradients w.r.t. the memories *after* step t
 * (started from dKT, dVT or zero), step t contributes, in this order:
 *     dV     += p_t (x) do_t                       (o_t = V~_t^T p_t)
 *     dp      = V~_t do_t
 *     dz      = p_t * (dp - <p_t, dp>)              (softmax; f'(z) * dp for an
 *                                                   element-wise replacement f)
 *     dq_t    = scale * K~_t^T dz                   (z = scale K~_t q_t)
 *     dK     += scale * dz (x) q_t
 *     dk_t    = dK^T (1 - a_t),  dv_t = dV^T (1 - a_t)
 *     da_t[s] = <dK[s], K~_{t-1}[s] - k_t> + <dV[s], V~_{t-1}[s] - v_t>
 *     dK[s]  *= a_t[s],  dV[s] *= a_t[s]            (pass to step t-1)
 * dK0, dV0 are what is left after t = 1.  dgate is the total derivative w.r.t.
 * the gate tensor as passed: da when it holds a, a * da when it holds log a.
 * Nullable: K0, V0, dKT, dVT (read as zero); dK0, dV0 (not written). */
int gsa_oracle_bwd(int B, int T, int H, int dk, int dv, int m, int gate_is_log,
                   int act, double scale, const double *q, const double *k,
                   const double *v, const double *gate, const double *K0,
                   const double *V0, const double *dO, const double *dKT,
                   const double *dVT, double *dq, double *dkk, double *dvv,
                   double *dgate, double *dK0, double *dV0, int bh_begin,
                   int bh_end)
{
    if (B < 1 || T < 0 || H < 1 || dk < 1 || dv < 1 || m < 1) return -1;
    if (act < ACT_SOFTMAX || act > ACT_RELU2) return -1;
    if (bh_begin < 0 || bh_end > B * H || bh_begin > bh_end) return -1;
    size_t nK = (size_t)m * dk, nV = (size_t)m * dv;
    double *Ks = malloc(sizeof(double) * nK * (size_t)(T + 1));
    double *Vs = malloc(sizeof(double) * nV * (size_t)(T + 1));
    double *gK = malloc(sizeof(double) * nK);
    double *gV = malloc(sizeof(double) * nV);
    double *z = malloc(sizeof(double) * m);
    double *p = malloc(sizeof(double) * m);
    double *dp = malloc(sizeof(double) * m);
    double *dz = malloc(sizeof(double) * m);
    double *otmp = malloc(sizeof(double) * dv);
    if (!Ks || !Vs || !gK || !gV || !z || !p || !dp || !dz || !otmp) {
        free(Ks); free(Vs); free(gK); free(gV); free(z); free(p); free(dp);
        free(dz); free(otmp);
        return -2;
    }
    for (int bh = bh_begin; bh < bh_end; ++bh) {
        int b = bh / H, h = bh % H;
        if (K0) memcpy(Ks, K0 + (size_t)bh * nK, sizeof(double) * nK);
        else memset(Ks, 0, sizeof(double) * nK);
        if (V0) memcpy(Vs, V0 + (size_t)bh * nV, sizeof(double) * nV);
        else memset(Vs, 0, sizeof(double) * nV);
        /* replay the forward, keeping every memory */
        for (int t = 0; t < T; ++t) {
            size_t row = ((size_t)b * T + t) * H + h;
            double *Kt = Ks + nK * (size_t)(t + 1), *Vt = Vs + nV * (size_t)(t + 1);
            memcpy(Kt, Ks + nK * (size_t)t, sizeof(double) * nK);
            memcpy(Vt, Vs + nV * (size_t)t, sizeof(double) * nV);
            gsa_step(dk, dv, m, gate_is_log, act, scale, q + row * dk, k + row * dk,
                     v + row * dv, gate + row * m, Kt, Vt, z, p, otmp);
        }
        if (dKT) memcpy(gK, dKT + (size_t)bh * nK, sizeof(double) * nK);
        else memset(gK, 0, sizeof(double) * nK);
        if (dVT) memcpy(gV, dVT + (size_t)bh * nV, sizeof(double) * nV);
        else memset(gV, 0, sizeof(double) * nV);
        for (int t = T - 1; t >= 0; --t) {
            size_t row = ((size_t)b * T + t) * H + h;
            const double *Kt = Ks + nK * (size_t)(t + 1), *Vt = Vs + nV * (size_t)(t + 1);
            const double *Kp = Ks + nK * (size_t)t, *Vp = Vs + nV * (size_t)t;
            const double *qt = q + row * dk, *kt = k + row * dk, *vt = v + row * dv;
            const double *dot = dO + row * dv;
            /* logits and slot weights of this step, recomputed from the stored K~_t */
            for (int s = 0; s < m; ++s) {
                double acc = 0.0;
                for (int c = 0; c < dk; ++c) acc += Kt[(size_t)s * dk + c] * qt[c];
                z[s] = scale * acc;
            }
            slot_act(act, m, z, p);
            for (int s = 0; s < m; ++s) {
                double acc = 0.0;
                for (int c = 0; c < dv; ++c) {
                    gV[(size_t)s * dv + c] += p[s] * dot[c];
                    acc += Vt[(size_t)s * dv + c] * dot[c];
                }
                dp[s] = acc;
            }
            slot_act_bwd(act, m, z, p, dp, dz);
            for (int c = 0; c < dk; ++c) {
                double acc = 0.0;
                for (int s = 0; s < m; ++s) acc += Kt[(size_t)s * dk + c] * dz[s];
                dq[row * dk + c] = scale * acc;
            }
            for (int s = 0; s < m; ++s)
                for (int c = 0; c < dk; ++c) gK[(size_t)s * dk + c] += scale * dz[s] * qt[c];
            for (int c = 0; c < dk; ++c) dkk[row * dk + c] = 0.0;
            for (int c = 0; c < dv; ++c) dvv[row * dv + c] = 0.0;
            for (int s = 0; s < m; ++s) {
                double a, ia;
                gate_pair(gate[row * m + s], gate_is_log, &a, &ia);
                double da = 0.0;
                for (int c = 0; c < dk; ++c) {
                    double g = gK[(size_t)s * dk + c];
                    dkk[row * dk + c] += ia * g;
                    da += g * (Kp[(size_t)s * dk + c] - kt[c]);
                    gK[(size_t)s * dk + c] = a * g;
                }
                for (int c = 0; c < dv; ++c) {
                    double g = gV[(size_t)s * dv + c];
                    dvv[row * dv + c] += ia * g;
                    da += g * (Vp[(size_t)s * dv + c] - vt[c]);
                    gV[(size_t)s * dv + c] = a * g;
                }
                dgate[row * m + s] = gate_is_log ? a * da : da;
            }
        }
        if (dK0) memcpy(dK0 + (size_t)bh * nK, gK, sizeof(double) * nK);
        if (dV0) memcpy(dV0 + (size_t)bh * nV, gV, sizeof(double) * nV);
    }
    free(Ks); free(Vs); free(gK); free(gV); free(z); free(p); free(dp); free(dz);
    free(otmp);
    return 0;
}
