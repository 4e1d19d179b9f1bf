// L step: the penalty gradient mu (w - theta) - lambda added to the loss gradient
// and one optimizer step (SGD with momentum, or Adam) in a single pass over the
// multi-tensor list. Every value is produced by single IEEE fp32 operations in a
// fixed order (see include/condensa_cstep.h).
#pragma once
#include "common.cuh"

namespace cs {

enum { OPT_SGD = 0, OPT_ADAM = 1 };

struct OptDesc {
    float *w;
    const float *theta;
    const float *lam;
    const float *grad;
    float *buf1;
    float *buf2;
    long long numel;
    int pad;        // groups of four start at element -pad
    int vec_ok;     // all arrays reach 16-byte alignment at the same elements
};

struct OptParams {
    const OptDesc *td;
    const long long *item_prefix;
    int T;
    long long n_items;
    float mu, lr, momentum, wd, beta1, beta2, eps;
    float c1, c2, step_size, sqrt_bc2;      // 1-beta1, 1-beta2, lr/(1-beta1^t), sqrt(1-beta2^t)
};

template <int KIND>
__device__ __forceinline__ void lstep_elem(const OptParams &P, float &w, float th, float lam, float gr,
                                           float &b1, float &b2, bool has_b1)
{
    const float p = __fmul_rn(P.mu, __fsub_rn(w, th));
    float g = __fadd_rn(gr, __fsub_rn(p, lam));        // lam is +0 when absent: p - 0 == p
    if (P.wd != 0.0f) g = __fadd_rn(g, __fmul_rn(P.wd, w));
    if (KIND == OPT_SGD) {
        float b = g;
        if (has_b1) {
            b = __fadd_rn(__fmul_rn(P.momentum, b1), g);
            b1 = b;
        }
        w = __fsub_rn(w, __fmul_rn(P.lr, b));
    } else {
        const float m = __fadd_rn(__fmul_rn(P.beta1, b1), __fmul_rn(P.c1, g));
        const float v = __fadd_rn(__fmul_rn(P.beta2, b2), __fmul_rn(P.c2, __fmul_rn(g, g)));
        b1 = m;
        b2 = v;
        const float dn = __fadd_rn(__fdiv_rn(__fsqrt_rn(v), P.sqrt_bc2), P.eps);
        w = __fsub_rn(w, __fmul_rn(P.step_size, __fdiv_rn(m, dn)));
    }
}

// Work items: GROUPS_PER_ITEM groups of four elements of one tensor.
template <int KIND>
__global__ void __launch_bounds__(THREADS, 3) k_lstep(OptParams P)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const OptDesc d = P.td[t];
        const long long local = item - P.item_prefix[t];
        const long long e_first = 4 * (local * GROUPS_PER_ITEM) - d.pad;
        const bool has_lam = d.lam != nullptr, has_b1 = d.buf1 != nullptr;
        const bool fast = d.vec_ok && e_first >= 0 && e_first + 4 * GROUPS_PER_ITEM <= d.numel;
        if (fast) {
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                float4 wv[2], tv[2], lv[2], gv[2], b1v[2], b2v[2];
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const long long go = (2 * half + i) * THREADS + threadIdx.x;
                    wv[i] = reinterpret_cast<const float4 *>(d.w + e_first)[go];
                    tv[i] = __ldg(reinterpret_cast<const float4 *>(d.theta + e_first) + go);
                    gv[i] = __ldg(reinterpret_cast<const float4 *>(d.grad + e_first) + go);
                    lv[i] = has_lam ? __ldg(reinterpret_cast<const float4 *>(d.lam + e_first) + go) : make_float4(0.f, 0.f, 0.f, 0.f);
                    b1v[i] = has_b1 ? reinterpret_cast<const float4 *>(d.buf1 + e_first)[go] : make_float4(0.f, 0.f, 0.f, 0.f);
                    b2v[i] = (KIND == OPT_ADAM) ? reinterpret_cast<const float4 *>(d.buf2 + e_first)[go] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const long long go = (2 * half + i) * THREADS + threadIdx.x;
                    float w[4] = {wv[i].x, wv[i].y, wv[i].z, wv[i].w};
                    const float th[4] = {tv[i].x, tv[i].y, tv[i].z, tv[i].w};
                    const float l[4] = {lv[i].x, lv[i].y, lv[i].z, lv[i].w};
                    const float g[4] = {gv[i].x, gv[i].y, gv[i].z, gv[i].w};
                    float b1[4] = {b1v[i].x, b1v[i].y, b1v[i].z, b1v[i].w};
                    float b2[4] = {b2v[i].x, b2v[i].y, b2v[i].z, b2v[i].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) lstep_elem<KIND>(P, w[j], th[j], l[j], g[j], b1[j], b2[j], has_b1);
                    reinterpret_cast<float4 *>(d.w + e_first)[go] = make_float4(w[0], w[1], w[2], w[3]);
                    if (has_b1) reinterpret_cast<float4 *>(d.buf1 + e_first)[go] = make_float4(b1[0], b1[1], b1[2], b1[3]);
                    if (KIND == OPT_ADAM) reinterpret_cast<float4 *>(d.buf2 + e_first)[go] = make_float4(b2[0], b2[1], b2[2], b2[3]);
                }
            }
        } else {
            const long long lo = e_first < 0 ? 0 : e_first;
            const long long hi = (e_first + 4 * GROUPS_PER_ITEM < d.numel) ? e_first + 4 * GROUPS_PER_ITEM : d.numel;
            for (long long e = lo + threadIdx.x; e < hi; e += THREADS) {
                float w = d.w[e];
                float b1 = has_b1 ? d.buf1[e] : 0.0f;
                float b2 = (KIND == OPT_ADAM) ? d.buf2[e] : 0.0f;
                lstep_elem<KIND>(P, w, d.theta[e], has_lam ? d.lam[e] : 0.0f, d.grad[e], b1, b2, has_b1);
                d.w[e] = w;
                if (has_b1) d.buf1[e] = b1;
                if (KIND == OPT_ADAM) d.buf2[e] = b2;
            }
        }
    }
}

}  // namespace cs
