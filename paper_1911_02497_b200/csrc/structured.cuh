// Structured pruning kernels: 4x4 block projection with a known cut-off, and
// the fp64 filter norms (segment partial sums + in-order combine).
#pragma once
#include "common.cuh"
#include "elementwise.cuh"
#include "select.cuh"

namespace cs {

// Final write of one 4x4 block given the keep decision.
__device__ __forceinline__ void store_block(const TensorDesc &d, const BlockData &bd, const float *u,
                                            bool keep, float mu, unsigned fuse)
{
    const bool has_lam = d.lam != nullptr;
    const bool wr_lam = (fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (fuse & FUSE_PENALTY) && d.grad != nullptr;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        Out o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            o[j] = finish(bd.w[4 * i + j], bd.l[4 * i + j], u[4 * i + j], keep, mu, fuse, has_lam);
        const long long off = (bd.r0 + i) * d.d1 + bd.c0;
        if (bd.full) {
            float v[4] = {o[0].theta, o[1].theta, o[2].theta, o[3].theta};
            st4(d.theta + off, v);
            if (d.mask) {
                const u32 mm = (u32)o[0].m | ((u32)o[1].m << 8) | ((u32)o[2].m << 16) | ((u32)o[3].m << 24);
                *reinterpret_cast<u32 *>(d.mask + off) = mm;
            }
            if (d.theta_h) {
                uint2 hh;
                hh.x = (u32)o[0].th | ((u32)o[1].th << 16);
                hh.y = (u32)o[2].th | ((u32)o[3].th << 16);
                *reinterpret_cast<uint2 *>(d.theta_h + off) = hh;
            }
            if (wr_lam) {
                float v2[4] = {o[0].lam, o[1].lam, o[2].lam, o[3].lam};
                st4(d.lam + off, v2);
            }
            if (wr_grad) {
                float v3[4] = {o[0].grad, o[1].grad, o[2].grad, o[3].grad};
                st4(d.grad + off, v3);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (bd.r0 + i >= d.d0 || bd.c0 + j >= d.d1) continue;
                d.theta[off + j] = o[j].theta;
                if (d.mask) d.mask[off + j] = o[j].m;
                if (d.theta_h) d.theta_h[off + j] = o[j].th;
                if (wr_lam) d.lam[off + j] = o[j].lam;
                if (wr_grad) d.grad[off + j] = o[j].grad;
            }
        }
    }
}

// Projection pass of block pruning. Work items: BLOCKS_PER_ITEM blocks for
// ranked (2-D) tensors, linear items for tensors that pass through.
__device__ __forceinline__ void apply_block_items(const Params &P, u64 tau_key, u64 tau_id)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long local = item - P.item_prefix[t];
        if (!d.ranked) {
            process_linear_item<M_KEEPALL>(P, d, local, 0, 0);
            continue;
        }
        const bool has_lam = d.lam != nullptr;
#pragma unroll 1
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const long long b = local * BLOCKS_PER_ITEM + it * THREADS + threadIdx.x;
            if (b >= d.n_units) continue;
            BlockData bd;
            float u[16];
            load_block(d, b, bd);
            const u64 key = block_key(bd, P.mu, has_lam, u);
            const bool keep = keep_by_cutoff(key, (u64)(d.unit_prefix + b), tau_key, tau_id);
            store_block(d, bd, u, keep, P.mu, P.fuse);
        }
    }
}

// The same for bh x bw blocks (the fall-back of the single-pass route).
__device__ __forceinline__ void apply_blockg_items(const Params &P, u64 tau_key, u64 tau_id)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long local = item - P.item_prefix[t];
        if (!d.ranked) {
            process_linear_item<M_KEEPALL>(P, d, local, 0, 0);
            continue;
        }
#pragma unroll 1
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const long long b = local * BLOCKS_PER_ITEM + it * THREADS + threadIdx.x;
            if (b >= d.n_units) continue;
            const u64 key = blockg_key_global(d, b, P.mu);
            blockg_write_global(P, d, b, keep_by_cutoff(key, (u64)(d.unit_prefix + b), tau_key, tau_id), nullptr, 0, 1);
        }
    }
}

__global__ void __launch_bounds__(THREADS) k_apply_block(Params P)
{
    if (P.ctl->sel.onepass) return;          // the single-pass kernel has written everything
    apply_block_items(P, P.ctl->tau_key, P.ctl->tau_id);
}

// Projection with the exact cut-off at the end of the selection kernel (declared
// there): used when a call that went for the single pass had to fall back.
template <int SRC>
__device__ __noinline__ void apply_after_select(const Params &P, int need_h)
{
    // the cut-off was written by another CTA of this launch: read it past the L1
    const u64 tau_key = __ldcg(&P.ctl->tau_key), tau_id = __ldcg(&P.ctl->tau_id);
    if (SRC == SRC_ELEM) {
        if (need_h) apply_linear_items<M_PRUNE, true>(P, tau_key, tau_id);
        else apply_linear_items<M_PRUNE, false>(P, tau_key, tau_id);
    } else if (SRC == SRC_BLOCK) {
        apply_block_items(P, tau_key, tau_id);
    } else if (SRC == SRC_BLOCKG) {
        apply_blockg_items(P, tau_key, tau_id);
    }
}

// Filter norms, step 1: one warp per segment of SEG elements of one filter.
// Lane l adds the elements of the 4-element groups l, l+32, l+64, ... of the
// segment, each group in index order, then the 32 lane sums are combined by a
// fixed butterfly; the value depends only on the segment's contents and length,
// never on where the filter sits or how it is aligned (the 128-bit and the
// scalar path add in the same order).
// Work items: (filter, segment) pairs of ranked tensors, WARPS per CTA step.
__global__ void __launch_bounds__(THREADS) k_filter_partial(Params P)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int crit = P.crit;
    pdl_launch_dependents();        // the kernels behind may set themselves up (they wait before reading the sums)
    const long long n_work = P.n_items;
    for (long long base = (long long)blockIdx.x * WARPS; base < n_work; base += (long long)gridDim.x * WARPS) {
        const long long item = base + warp;
        if (item >= n_work) continue;
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long local = item - P.item_prefix[t];
        const long long nseg = (d.d1 + SEG - 1) / SEG;
        const long long f = local / nseg, sgm = local - f * nseg;
        const long long j0 = sgm * SEG;
        const long long j1 = (j0 + SEG < d.d1) ? j0 + SEG : d.d1;
        const float *__restrict__ wp = d.w + f * d.d1 + j0;
        const float *lp = d.lam ? d.lam + f * d.d1 + j0 : nullptr;
        const bool has_lam = lp != nullptr;
        const int n = (int)(j1 - j0);                    // elements in this segment
        const bool vec = ((uintptr_t)wp % 16 == 0) && (!has_lam || (uintptr_t)lp % 16 == 0);
        double acc = 0.0;
        const int ngroups = n >> 2;                      // full groups of four
        if (vec) {
            int gidx = lane;
            for (; gidx + 3 * 32 < ngroups; gidx += 4 * 32) {
                float4 wv[4], lv[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    wv[q] = __ldg(reinterpret_cast<const float4 *>(wp) + gidx + q * 32);
                    lv[q] = has_lam ? reinterpret_cast<const float4 *>(lp)[gidx + q * 32] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float w4[4] = {wv[q].x, wv[q].y, wv[q].z, wv[q].w};
                    const float l4[4] = {lv[q].x, lv[q].y, lv[q].z, lv[q].w};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        acc = crit_add(acc, form_u(w4[c], l4[c], P.mu, has_lam), crit);
                    }
                }
            }
            for (; gidx < ngroups; gidx += 32) {
                const float4 a = __ldg(reinterpret_cast<const float4 *>(wp) + gidx);
                const float4 b = has_lam ? reinterpret_cast<const float4 *>(lp)[gidx] : make_float4(0.f, 0.f, 0.f, 0.f);
                const float w4[4] = {a.x, a.y, a.z, a.w};
                const float l4[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    acc = crit_add(acc, form_u(w4[c], l4[c], P.mu, has_lam), crit);
                }
            }
        } else {
            for (int gidx = lane; gidx < ngroups; gidx += 32) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int j = 4 * gidx + c;
                    acc = crit_add(acc, form_u(__ldg(wp + j), has_lam ? lp[j] : 0.0f, P.mu, has_lam), crit);
                }
            }
        }
        // the last, incomplete group belongs to the lane whose turn it is
        if ((n & 3) && lane == (ngroups & 31)) {
            for (int j = 4 * ngroups; j < n; ++j) {
                acc = crit_add(acc, form_u(__ldg(wp + j), has_lam ? lp[j] : 0.0f, P.mu, has_lam), crit);
            }
        }
        for (int o = 16; o > 0; o >>= 1) acc = crit_join(acc, __shfl_xor_sync(0xffffffffu, acc, o), crit);
        if (lane == 0) P.partial[item] = acc;
    }
}

// General n-D blocks: one thread per block goes over the elements of the block that exist, in
// row-major order (the order of the plain definition, so the fp64 value is bit-identical),
// with the criterion of the call. Work items: BLOCKS_PER_ITEM blocks of a ranked tensor.
__global__ void __launch_bounds__(THREADS) k_blockgen_norms(Params P)
{
    const int crit = P.crit;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long local = item - P.item_prefix[t];
        const bool has_lam = d.lam != nullptr;
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const long long b = local * BLOCKS_PER_ITEM + it * THREADS + threadIdx.x;
            if (b >= d.n_units) continue;
            if (d.nd == 2 && crit == CRIT_L2) {     // blocks of a matrix by the L2 norm: rows fetched ahead, a row's loads together
                P.arr_key[d.unit_prefix + b] = blockg_key_global(d, b, P.mu);
                continue;
            }
            long long rest = b;
            int bc[4];
#pragma unroll
            for (int q = 3; q >= 0; --q) { bc[q] = (int)(rest % d.nb[q]); rest /= d.nb[q]; }
            int lo[4], hi[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                lo[q] = bc[q] * d.bs[q];
                hi[q] = lo[q] + d.bs[q] < d.sh[q] ? lo[q] + d.bs[q] : d.sh[q];
            }
            double acc = 0.0;
            for (int i0 = lo[0]; i0 < hi[0]; ++i0)
                for (int i1 = lo[1]; i1 < hi[1]; ++i1)
                    for (int i2 = lo[2]; i2 < hi[2]; ++i2) {
                        const long long row = (((long long)i0 * d.sh[1] + i1) * d.sh[2] + i2) * d.sh[3];
                        for (int i3 = lo[3]; i3 < hi[3]; ++i3) {
                            const long long e = row + i3;
                            acc = crit_add(acc, form_u(d.w[e], has_lam ? d.lam[e] : 0.0f, P.mu, has_lam), crit);
                        }
                    }
            P.arr_key[d.unit_prefix + b] = (u64)__double_as_longlong(acc);
        }
    }
}

// Filter norms, step 2: nu_f = partial sums added in segment order (fp64 bits).
__device__ __forceinline__ u64 filter_norm_key(const Params &P, long long sid)
{
    // tensor that owns structure sid
    int lo = 0, hi = P.T - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (P.td[mid].unit_prefix <= sid) lo = mid; else hi = mid - 1;
    }
    // skip tensors without ranked structures that share the same prefix
    int t = lo;
    while (t > 0 && P.td[t].n_units == 0) --t;
    const TensorDesc &d = P.td[t];
    const long long f = sid - d.unit_prefix;
    const long long nseg = (d.d1 + SEG - 1) / SEG;
    const double *p = P.partial + P.item_prefix[t] + f * nseg;
    double acc = 0.0;
    for (long long sgm = 0; sgm < nseg; ++sgm) acc = crit_join(acc, p[sgm], P.crit);
    return (u64)__double_as_longlong(acc);
}

__global__ void __launch_bounds__(THREADS) k_filter_combine(Params P)
{
    const long long stride = (long long)gridDim.x * THREADS;
    for (long long sid = (long long)blockIdx.x * THREADS + threadIdx.x; sid < P.S; sid += stride)
        P.arr_key[sid] = filter_norm_key(P, sid);
}

}  // namespace cs
