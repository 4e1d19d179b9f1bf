// Elementwise passes over a multi-tensor descriptor table: projection with a
// known cut-off, fp16 quantisation, multiplier update, penalty gradient.
// A linear work item is GROUPS_PER_ITEM groups of 4 consecutive elements; groups
// start at element -pad so that full groups are 16-byte aligned in every array.
#pragma once
#include "common.cuh"

namespace cs {

enum { M_KEEPALL = 0, M_PRUNE = 1, M_FILTER = 2, M_LAGRANGE = 3, M_BLOCKGEN = 4 };

// Structure id of element e of a tensor cut into n-D blocks (row-major block numbering).
__device__ __forceinline__ u64 blockgen_sid(const TensorDesc &d, long long e)
{
    if (d.nd == 2) {
        long long r, c;
        if (d.numel < 0x7FFFFFFFll) {
            const u32 rr = (u32)e / (u32)d.d1;
            r = rr;
            c = (u32)e - rr * (u32)d.d1;
            return (u64)d.unit_prefix + (u64)((u32)r / (u32)d.bh) * (u64)d.nbc + (u32)c / (u32)d.bw;
        }
        r = e / d.d1;
        c = e - r * d.d1;
        return (u64)d.unit_prefix + (u64)(r / d.bh) * (u64)d.nbc + (u64)(c / d.bw);
    }
    long long rest = e;
    int bc[4];
#pragma unroll
    for (int q = 3; q >= 0; --q) { bc[q] = (int)(rest % d.sh[q]) / d.bs[q]; rest /= d.sh[q]; }
    return (u64)d.unit_prefix + (u64)((((long long)bc[0] * d.nb[1] + bc[1]) * d.nb[2] + bc[2]) * d.nb[3] + bc[3]);
}

constexpr int LIN_UNROLL = GROUPS_PER_ITEM / THREADS;   // 4 groups per thread per item

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 ld4_ro(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ void st4(float *p, const float *v)
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}

// One work item of tensor d. tau_* is the cut-off for M_PRUNE / M_FILTER.
template <int MODE>
__device__ __forceinline__ void process_linear_item(const Params &P, const TensorDesc &d,
                                                    long long item_local, u64 tau_key, u64 tau_id)
{
    const long long ng = (d.numel + d.pad + 3) >> 2;
    const long long g0 = item_local * GROUPS_PER_ITEM;
    const long long g1 = (g0 + GROUPS_PER_ITEM < ng) ? g0 + GROUPS_PER_ITEM : ng;
    const bool has_lam = d.lam != nullptr;
    const unsigned fuse = P.fuse;
    const float mu = P.mu;
    const float *__restrict__ wp = d.w;
    const float *lp = d.lam;

    float w[LIN_UNROLL][4], l[LIN_UNROLL][4], t[LIN_UNROLL][4];
    bool live[LIN_UNROLL], full[LIN_UNROLL];

#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        const long long g = g0 + it * THREADS + threadIdx.x;
        const long long e0 = 4 * g - d.pad;
        live[it] = g < g1;
        full[it] = live[it] && d.vec_ok && e0 >= 0 && e0 + 4 <= d.numel;
        if (full[it]) {
            float4 a = ld4_ro(wp + e0);
            w[it][0] = a.x; w[it][1] = a.y; w[it][2] = a.z; w[it][3] = a.w;
            if (has_lam) {
                float4 b = ld4(lp + e0);
                l[it][0] = b.x; l[it][1] = b.y; l[it][2] = b.z; l[it][3] = b.w;
            } else {
                l[it][0] = l[it][1] = l[it][2] = l[it][3] = 0.0f;
            }
            if (MODE == M_LAGRANGE) {
                float4 c = ld4(d.theta + e0);
                t[it][0] = c.x; t[it][1] = c.y; t[it][2] = c.z; t[it][3] = c.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + j;
                const bool ok = live[it] && e >= 0 && e < d.numel;
                w[it][j] = ok ? wp[e] : 0.0f;
                l[it][j] = (ok && has_lam) ? lp[e] : 0.0f;
                if (MODE == M_LAGRANGE) t[it][j] = ok ? d.theta[e] : 0.0f;
            }
        }
    }

#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        if (!live[it]) continue;
        const long long g = g0 + it * THREADS + threadIdx.x;
        const long long e0 = 4 * g - d.pad;
        Out o[4];
        // structure id of lane 0 for the filter decision
        long long f0 = 0, r0 = 0;
        if (MODE == M_FILTER && d.ranked) {
            const long long eb = e0 < 0 ? 0 : e0;
            if (d.numel < 0x7FFFFFFFll) {
                f0 = (long long)((u32)eb / (u32)d.d1);
            } else {
                f0 = eb / d.d1;
            }
            r0 = eb - f0 * d.d1;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long e = e0 + j;
            if (MODE == M_LAGRANGE) {
                o[j] = finish_given(w[it][j], l[it][j], t[it][j], mu, fuse, has_lam);
            } else {
                const float u = form_u(w[it][j], l[it][j], mu, has_lam);
                bool keep = true;
                if (MODE == M_PRUNE) {
                    keep = keep_by_cutoff(key_of_u(u), (u64)(d.elem_prefix + e), tau_key, tau_id);
                } else if (MODE == M_FILTER) {
                    if (d.ranked && e >= 0 && e < d.numel) {
                        long long f = f0, r = r0 + (e - (e0 < 0 ? 0 : e0));
                        while (r >= d.d1) { r -= d.d1; ++f; }
                        const u64 sid = (u64)(d.unit_prefix + f);
                        keep = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                    }
                } else if (MODE == M_BLOCKGEN) {
                    if (d.ranked && e >= 0 && e < d.numel) {
                        const u64 sid = blockgen_sid(d, e);
                        keep = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                    }
                }
                o[j] = finish(w[it][j], l[it][j], u, keep, mu, fuse, has_lam);
            }
        }
        const bool wr_lam = (fuse & FUSE_LAMBDA) && has_lam;
        const bool wr_grad = (fuse & FUSE_PENALTY) && d.grad != nullptr;
        if (full[it]) {
            if (MODE != M_LAGRANGE) {
                float v[4] = {o[0].theta, o[1].theta, o[2].theta, o[3].theta};
                st4(d.theta + e0, v);
                if (d.mask) {
                    const u32 mm = (u32)o[0].m | ((u32)o[1].m << 8) | ((u32)o[2].m << 16) | ((u32)o[3].m << 24);
                    *reinterpret_cast<u32 *>(d.mask + e0) = mm;
                }
                if (d.theta_h) {
                    uint2 hh;
                    hh.x = (u32)o[0].th | ((u32)o[1].th << 16);
                    hh.y = (u32)o[2].th | ((u32)o[3].th << 16);
                    *reinterpret_cast<uint2 *>(d.theta_h + e0) = hh;
                }
            }
            if (wr_lam) {
                float v[4] = {o[0].lam, o[1].lam, o[2].lam, o[3].lam};
                st4(d.lam + e0, v);
            }
            if (wr_grad) {
                float v[4] = {o[0].grad, o[1].grad, o[2].grad, o[3].grad};
                st4(d.grad + e0, v);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + j;
                if (e < 0 || e >= d.numel) continue;
                if (MODE != M_LAGRANGE) {
                    d.theta[e] = o[j].theta;
                    if (d.mask) d.mask[e] = o[j].m;
                    if (d.theta_h) d.theta_h[e] = o[j].th;
                }
                if (wr_lam) d.lam[e] = o[j].lam;
                if (wr_grad) d.grad[e] = o[j].grad;
            }
        }
    }
}

// Lean form of the same work for items whose 1024 groups all exist and are 16-byte
// aligned in every array (elem_item_is_fast): 32-bit indexing inside the item,
// no per-lane validity, outputs stored group by group.
template <int MODE, bool H>
__device__ __forceinline__ void process_linear_item_fast(const Params &P, const TensorDesc &d, long long local,
                                                         u64 tau_key, u64 tau_id)
{
    const long long e_base = 4 * (local * GROUPS_PER_ITEM) - d.pad;
    const bool has_lam = d.lam != nullptr;
    const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
    const int fp16 = quant_code(P.fuse);     // quantisation of theta
    const float mu = P.mu;
    const u32 tau32 = tau_key > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)tau_key;     // KEY_NONE keeps nothing
    const float4 *wp = reinterpret_cast<const float4 *>(d.w + e_base) + threadIdx.x;
    float4 wv[LIN_UNROLL], lv[LIN_UNROLL], tv[LIN_UNROLL];
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) wv[it] = __ldg(wp + it * THREADS);
    if (has_lam) {
        const float4 *lp = reinterpret_cast<const float4 *>(d.lam + e_base) + threadIdx.x;
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) lv[it] = lp[it * THREADS];
    } else {
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) lv[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (MODE == M_LAGRANGE) {
        const float4 *tp = reinterpret_cast<const float4 *>(d.theta + e_base) + threadIdx.x;
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) tv[it] = tp[it * THREADS];
    }
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        const float w[4] = {wv[it].x, wv[it].y, wv[it].z, wv[it].w};
        const float l[4] = {lv[it].x, lv[it].y, lv[it].z, lv[it].w};
        float th[4], ln[4], g[4];
        u32 m = 0x01010101u;
        unsigned short h[4] = {0, 0, 0, 0};
        const u32 eo = 4u * (u32)(it * THREADS + threadIdx.x);        // element offset inside the item
        if (MODE == M_LAGRANGE) {
            th[0] = tv[it].x; th[1] = tv[it].y; th[2] = tv[it].z; th[3] = tv[it].w;
        } else {
            float u[4];
            form_u4(w, l, mu, has_lam, u);
            bool keep[4] = {true, true, true, true};
            if (MODE == M_PRUNE) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const u32 key = __float_as_uint(u[j]) & 0x7FFFFFFFu;
                    keep[j] = key > tau32;
                    if (key == tau32 && tau_key <= 0x7FFFFFFFull)       // tie with the threshold: the index decides
                        keep[j] = (u64)(d.elem_prefix + e_base) + eo + j <= tau_id;
                }
            } else if (MODE == M_FILTER) {
                if (d.ranked) {
                    const long long e0 = e_base + eo;
                    long long f = (d.numel < 0x7FFFFFFFll) ? (long long)((u32)e0 / (u32)d.d1) : e0 / d.d1;
                    long long r = e0 - f * d.d1;
                    if (r + 3 < d.d1) {             // the four elements lie in one filter (nearly always): one decision
                        const u64 sid = (u64)(d.unit_prefix + f);
                        const bool kp = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                        keep[0] = keep[1] = keep[2] = keep[3] = kp;
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (r >= d.d1) { r -= d.d1; ++f; while (r >= d.d1) { r -= d.d1; ++f; } }
                            const u64 sid = (u64)(d.unit_prefix + f);
                            keep[j] = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                            ++r;
                        }
                    }
                }
            }
            else if (MODE == M_BLOCKGEN) {
                if (d.ranked && d.nd == 2 && d.numel < 0x7FFFFFFFll) {
                    // row, column and block coordinates once per group, then walked element by element
                    const u32 C = (u32)d.d1, bh = (u32)d.bh, bw = (u32)d.bw;
                    const u32 e0 = (u32)(e_base + eo);
                    u32 r = e0 / C, c = e0 - r * C;
                    u32 br = r / bh, cb = c / bw, cm = c - cb * bw;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (c >= C) { c = 0; ++r; br = r / bh; cb = 0; cm = 0; }
                        const u64 sid = (u64)d.unit_prefix + (u64)br * (u64)d.nbc + cb;
                        keep[j] = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                        ++c;
                        if (++cm == bw) { cm = 0; ++cb; }
                    }
                } else if (d.ranked) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const u64 sid = blockgen_sid(d, e_base + eo + j);
                        keep[j] = keep_by_cutoff(P.arr_key[sid], sid, tau_key, tau_id);
                    }
                }
            }
            m = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                th[j] = keep[j] ? u[j] : 0.0f;
                m |= keep[j] ? (1u << (8 * j)) : 0u;
            }
            if (H) {
                half4(th, h, fp16 ? fp16 : 1);
                if (fp16) widen4(h, th, th, fp16);
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float p = __fmul_rn(mu, __fsub_rn(w[j], th[j]));
            ln[j] = upd ? __fsub_rn(l[j], p) : l[j];
            g[j] = __fsub_rn(p, ln[j]);
        }
        const long long go = it * THREADS + threadIdx.x;
        if (MODE != M_LAGRANGE) {
            reinterpret_cast<float4 *>(d.theta + e_base)[go] = make_float4(th[0], th[1], th[2], th[3]);
            if (d.mask) reinterpret_cast<u32 *>(d.mask + e_base)[go] = m;
            if (H && d.theta_h) reinterpret_cast<uint2 *>(d.theta_h + e_base)[go] =
                make_uint2((u32)h[0] | ((u32)h[1] << 16), (u32)h[2] | ((u32)h[3] << 16));
        }
        if (upd) reinterpret_cast<float4 *>(d.lam + e_base)[go] = make_float4(ln[0], ln[1], ln[2], ln[3]);
        if (wr_grad) reinterpret_cast<float4 *>(d.grad + e_base)[go] = make_float4(g[0], g[1], g[2], g[3]);
    }
}

// The linear work items of the whole list, strided over the CTAs of the grid.
template <int MODE, bool H>
__device__ __forceinline__ void apply_linear_items(const Params &P, u64 tau_key, u64 tau_id)
{
    long long t_first = 0, t_end = -1;
    TensorDesc d;
    d.numel = 0; d.pad = 0; d.vec_ok = 0;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        if (item >= t_end) {
            const int t = find_tensor(P.item_prefix, P.T, item);
            d = P.td[t];
            t_first = P.item_prefix[t];
            t_end = P.item_prefix[t + 1];
        }
        const long long local = item - t_first;
        if (elem_item_is_fast(d, local)) process_linear_item_fast<MODE, H>(P, d, local, tau_key, tau_id);
        else process_linear_item<MODE>(P, d, local, tau_key, tau_id);
    }
}

// Persistent CTAs stride over the linear work items of the whole list. H: the
// binary16 bits are needed (fp16 fuse or a theta_h output).
template <int MODE, bool H>
__global__ void __launch_bounds__(THREADS, 3) k_apply_linear(Params P)
{
    u64 tau_key = 0, tau_id = 0;
    pdl_wait();                     // a no-op unless the launch was made dependent on the kernel ahead
    if (MODE == M_PRUNE || MODE == M_FILTER || MODE == M_BLOCKGEN) {
        if (P.ctl->sel.onepass) return;      // the single-pass kernel has written everything
        tau_key = P.ctl->tau_key;
        tau_id = P.ctl->tau_id;
    }
    apply_linear_items<MODE, H>(P, tau_key, tau_id);
}

}  // namespace cs
