// Aligned interior work items of the single-pass projection: the kernels that
// move almost all of the bytes. No CTA-wide barrier inside the item loop:
// candidates are staged per warp in shared memory and flushed to the list with
// one global atomic per flush.
#pragma once
#include "common.cuh"
#include "fused.cuh"

namespace cs {

// ---------------------------------------------------------------- unstructured
constexpr int ESTG = 64;        // staged candidates per warp

struct ElemFastShared {
    u32 hist[NBINS];            // the first four members mirror FusedShared (edge items reuse them)
    u32 cnt[2];
    u64 base[2];
    u64 red[WARPS];
    u32 wcount[WARPS];
    u64 id[WARPS][ESTG];
    u32 key[WARPS][ESTG];
    float lam[WARPS][ESTG];
};

// The journal entry is written for every staged candidate: entries staged by an
// earlier item of this CTA may belong to another tensor (one with multipliers)
// than the item that triggers the flush; tensors without multipliers stage 0.
__device__ __forceinline__ void elem_flush(const Params &P, ElemFastShared &sh, u32 limit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncwarp();
    u32 c = sh.wcount[warp];
    if (c > limit) {
        if (c > ESTG) c = ESTG;        // entries past the staging area went straight to the list
        u64 base = 0;
        if (lane == 0) base = atomicAdd(&P.ctl->list_count[0], (u64)c);
        base = __shfl_sync(0xffffffffu, base, 0);
        for (u32 i = lane; i < c; i += 32) {
            const u64 pos = base + i;
            if (pos < P.cap) {
                P.list_key[pos] = (u64)sh.key[warp][i];
                P.list_id[pos] = sh.id[warp][i];
                P.jr_lam[pos] = sh.lam[warp][i];
            }
        }
        __syncwarp();
        if (lane == 0) sh.wcount[warp] = 0;
    }
    __syncwarp();
}

template <bool H, bool G>
__global__ void __launch_bounds__(THREADS, 3) k_fused_elem(Params P)
{
    __shared__ ElemFastShared sh;
    if (!P.ctl->sel.onepass) return;
    const Bracket br = load_bracket(P.ctl->sel);
    for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
    if (threadIdx.x < WARPS) sh.wcount[threadIdx.x] = 0;
    __syncthreads();
    const int fp16 = (P.fuse & FUSE_BF16) ? 2 : (P.fuse & FUSE_FP16) ? 1 : 0;     // quantisation of theta
    const u32 lo = (u32)br.lo, range = (u32)br.hi - (u32)br.lo, guess = (u32)br.guess;
    const float mu = P.mu;
    const int warp = threadIdx.x >> 5;
    u32 n_above = 0;
    long long t_first = 0, t_end = -1, fast_lo = 0, fast_hi = 0;
    struct { const float *w; float *lam, *theta, *grad; uint8_t *mask; uint16_t *theta_h; long long elem_prefix; int pad; } d;
    d.w = nullptr; d.lam = d.theta = d.grad = nullptr; d.mask = nullptr; d.theta_h = nullptr;
    d.elem_prefix = 0; d.pad = 0;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        if (item >= t_end) {        // look the tensor up only when the items leave it
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc &g = P.td[t];
            t_first = P.item_prefix[t];
            t_end = P.item_prefix[t + 1];
            // fast items form a range of local indices (same rule as elem_item_is_fast)
            fast_lo = g.pad ? 1 : 0;
            fast_hi = g.vec_ok ? (g.numel + g.pad) / (4 * GROUPS_PER_ITEM) : 0;
            d.w = g.w; d.lam = g.lam; d.theta = g.theta; d.grad = g.grad; d.mask = g.mask; d.theta_h = g.theta_h;
            d.elem_prefix = g.elem_prefix; d.pad = g.pad;
        }
        const long long local = item - t_first;
        if (local < fast_lo || local >= fast_hi) continue;
        const long long e_base = 4 * (local * GROUPS_PER_ITEM) - d.pad;
        const bool has_lam = d.lam != nullptr;
        const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
        const float4 *wp = reinterpret_cast<const float4 *>(d.w + e_base) + threadIdx.x;
        float4 wv[LIN_UNROLL], lv[LIN_UNROLL];
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
        u32 nkeep = 0, candm = 0;       // candm bit 4*it+j: element lies in the bracket
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) {
            const float w[4] = {wv[it].x, wv[it].y, wv[it].z, wv[it].w};
            const float l[4] = {lv[it].x, lv[it].y, lv[it].z, lv[it].w};
            float u[4], th[4], ln[4], g[4];
            form_u4(w, l, mu, has_lam, u);
            u32 m = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const u32 key = __float_as_uint(u[j]) & 0x7FFFFFFFu;
                const bool keep = key >= guess;
                th[j] = keep ? u[j] : 0.0f;
                m |= keep ? (1u << (8 * j)) : 0u;
                candm |= (key - lo <= range) ? (1u << (4 * it + j)) : 0u;
            }
            nkeep += __popc(m);
            unsigned short h[4];
            if (H) {
                half4(th, h, fp16 ? fp16 : 1);     // 16-bit code of theta (zeroed entries give +0)
                if (fp16) widen4(h, th, th, fp16);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float p = __fmul_rn(mu, __fsub_rn(w[j], th[j]));
                ln[j] = upd ? __fsub_rn(l[j], p) : l[j];
                g[j] = __fsub_rn(p, ln[j]);
            }
            const long long go = it * THREADS + threadIdx.x;      // group offset inside the item
            reinterpret_cast<float4 *>(d.theta + e_base)[go] = make_float4(th[0], th[1], th[2], th[3]);
            if (d.mask) reinterpret_cast<u32 *>(d.mask + e_base)[go] = m;
            if (H && d.theta_h) reinterpret_cast<uint2 *>(d.theta_h + e_base)[go] =
                make_uint2((u32)h[0] | ((u32)h[1] << 16), (u32)h[2] | ((u32)h[3] << 16));
            if (upd) reinterpret_cast<float4 *>(d.lam + e_base)[go] = make_float4(ln[0], ln[1], ln[2], ln[3]);
            if (G && d.grad) reinterpret_cast<float4 *>(d.grad + e_base)[go] = make_float4(g[0], g[1], g[2], g[3]);
        }
        // the few elements inside the bracket: once per item, from the lambda still in registers
        u32 ncandkeep = 0;
        while (candm) {
            const int qb = __ffs(candm) - 1;
            candm &= candm - 1;
            float ll = 0.0f;
#pragma unroll
            for (int a = 0; a < LIN_UNROLL; ++a) {      // select without indexing the registers
                if (qb == 4 * a + 0) ll = lv[a].x;
                if (qb == 4 * a + 1) ll = lv[a].y;
                if (qb == 4 * a + 2) ll = lv[a].z;
                if (qb == 4 * a + 3) ll = lv[a].w;
            }
            const u32 eo = 4u * (u32)((qb >> 2) * THREADS + threadIdx.x) + (u32)(qb & 3);
            const float ww = __ldg(d.w + e_base + eo);
            // same operations as above: the key comes out bit-identical
            const float uu = (has_lam && __float_as_uint(ll) != 0u) ? __fsub_rn(ww, __fdiv_rn(ll, mu)) : ww;
            const u32 key = __float_as_uint(uu) & 0x7FFFFFFFu;
            const u64 id = (u64)(d.elem_prefix + e_base) + eo;
            ncandkeep += key >= guess ? 1u : 0u;
            atomicAdd(&sh.hist[bracket_bin(br, (u64)key, id)], 1u);
            const u32 slot = atomicAdd(&sh.wcount[warp], 1u);
            if (slot < ESTG) {
                sh.key[warp][slot] = key;
                sh.id[warp][slot] = id;
                sh.lam[warp][slot] = ll;
            } else {
                const u64 pos = atomicAdd(&P.ctl->list_count[0], 1ull);
                if (pos < P.cap) {
                    P.list_key[pos] = (u64)key;
                    P.list_id[pos] = id;
                    if (has_lam) P.jr_lam[pos] = ll;
                }
            }
        }
        n_above += nkeep - ncandkeep;      // keeps that are not candidates lie above the bracket
        elem_flush(P, sh, ESTG / 2);
    }
    elem_flush(P, sh, 0);
    __syncthreads();
    u64 na = n_above;
    // the items outside the aligned fast path (tensor heads and tails, unaligned
    // tensors), listed by the host
    if (P.n_edge_items > 0) {
        FusedShared &fs = reinterpret_cast<FusedShared &>(sh);
        if (threadIdx.x < 2) fs.cnt[threadIdx.x] = 0;
        __syncthreads();
        const long long *prefix_b = P.edge_items + P.n_edge_items;      // [T+1] projection items per tensor
        int par = 0;
        for (long long i = blockIdx.x; i < P.n_edge_items; i += gridDim.x) {
            const long long item = P.edge_items[i];
            const int t = find_tensor(prefix_b, P.T, item);
            const TensorDesc g = P.td[t];
            fused_elem_item_generic<H>(P, g, item - prefix_b[t], fs, br, par, na, fp16);
            par ^= 1;
        }
        __syncthreads();
    }
    // totals of this CTA
    for (int o = 16; o > 0; o >>= 1) na += __shfl_xor_sync(0xffffffffu, na, o);
    if ((threadIdx.x & 31) == 0) sh.red[warp] = na;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < WARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += THREADS) {
        const u32 hc = sh.hist[i];
        if (hc) atomicAdd(&P.hist[i], (u64)hc);
    }
}

// ---------------------------------------------------------------- 4x4 blocks
#ifndef CS_BLOCK_MINB
#define CS_BLOCK_MINB 2          // resident CTAs per SM the block kernel is compiled for
#endif
constexpr int BSTG = 48;        // staged candidate blocks per warp (a warp adds at most 32 per iteration)

struct BlockFastShared {
    u32 hist[NBINS];            // the first four members mirror FusedShared (edge items reuse them)
    u32 cnt[2];
    u64 base[2];
    u64 red[WARPS];
    u32 wcount[WARPS];
    u64 key[WARPS][BSTG];
    u64 id[WARPS][BSTG];
    float4 lam[WARPS][BSTG][4];
};

__device__ __forceinline__ void block_flush(const Params &P, BlockFastShared &sh, u32 limit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncwarp();
    const u32 c = sh.wcount[warp];
    if (c > limit) {
        u64 base = 0;
        if (lane == 0) base = atomicAdd(&P.ctl->list_count[0], (u64)c);
        base = __shfl_sync(0xffffffffu, base, 0);
        for (u32 i = lane; i < c; i += 32) {
            const u64 pos = base + i;
            if (pos < P.cap) {
                P.list_key[pos] = sh.key[warp][i];
                P.list_id[pos] = sh.id[warp][i];
            }
        }
        for (u32 i = lane; i < 4 * c; i += 32) {      // journal rows, 16 bytes each
            const u64 pos = base + (i >> 2);
            if (pos < P.cap) reinterpret_cast<float4 *>(P.jr_lam + pos * 16)[i & 3] = sh.lam[warp][i >> 2][i & 3];
        }
        __syncwarp();
        if (lane == 0) sh.wcount[warp] = 0;
    }
    __syncwarp();
}

// Every block of a fast item lies in complete block rows of a tensor whose
// arrays are 16-byte aligned, with C % 4 == 0 and fewer than 2^32 elements.
// One thread per block: four 128-bit loads per array (a warp reads 512
// contiguous bytes of each of the four rows), the fp64 sum of squares in
// row-major order, one decision, four rows of outputs.
template <bool H, bool G>
__global__ void __launch_bounds__(THREADS, CS_BLOCK_MINB) k_fused_block(Params P)
{
    __shared__ BlockFastShared sh;
    if (!P.ctl->sel.onepass) return;
    const Bracket br = load_bracket(P.ctl->sel);
    for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
    if (threadIdx.x < WARPS) sh.wcount[threadIdx.x] = 0;
    __syncthreads();
    const int fp16 = (P.fuse & FUSE_BF16) ? 2 : (P.fuse & FUSE_FP16) ? 1 : 0;     // quantisation of theta
    const float mu = P.mu;
    const int warp = threadIdx.x >> 5;
    u32 n_above = 0;
    long long t_first = 0, t_end = -1, n_fast = 0;
    struct { const float *w; float *lam, *theta, *grad; uint8_t *mask; uint16_t *theta_h; u64 unit_prefix; u32 C, nbc; } d;
    d.w = nullptr; d.lam = d.theta = d.grad = nullptr; d.mask = nullptr; d.theta_h = nullptr;
    d.unit_prefix = 0; d.C = d.nbc = 1;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        if (item >= t_end) {        // items of one CTA mostly stay in one tensor: look it up only on leaving
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc &g = P.td[t];
            t_first = P.item_prefix[t];
            t_end = P.item_prefix[t + 1];
            // fast items are the leading ones of a tensor (same rule as block_item_is_fast)
            n_fast = (g.ranked && g.blk_vec_ok && g.numel < 0xFFFFFFFFll) ? ((g.d0 >> 2) * g.nbc) / BLOCKS_PER_ITEM : 0;
            d.w = g.w; d.lam = g.lam; d.theta = g.theta; d.grad = g.grad; d.mask = g.mask; d.theta_h = g.theta_h;
            d.unit_prefix = (u64)g.unit_prefix; d.C = (u32)g.d1; d.nbc = (u32)g.nbc;
        }
        const long long local = item - t_first;
        if (local >= n_fast) continue;
        const u32 C = d.C, nbc = d.nbc;
        const bool has_lam = d.lam != nullptr;
        const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
        u32 b = (u32)(local * BLOCKS_PER_ITEM) + threadIdx.x;
        u32 brow = b / nbc;
        u32 bcol = b - brow * nbc;
#pragma unroll 1
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const u32 off0 = 4u * brow * C + 4u * bcol;
            float4 w4[4], l4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) w4[i] = ld4_ro(d.w + off0 + i * C);
            if (has_lam) {
#pragma unroll
                for (int i = 0; i < 4; ++i) l4[i] = ld4(d.lam + off0 + i * C);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) l4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float w[16], l[16], u[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                w[4 * i] = w4[i].x; w[4 * i + 1] = w4[i].y; w[4 * i + 2] = w4[i].z; w[4 * i + 3] = w4[i].w;
                l[4 * i] = l4[i].x; l[4 * i + 1] = l4[i].y; l[4 * i + 2] = l4[i].z; l[4 * i + 3] = l4[i].w;
            }
            u32 nz = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) nz |= __float_as_uint(l[i]);
            if (nz) {
#pragma unroll
                for (int i = 0; i < 16; ++i) u[i] = __fsub_rn(w[i], __fdiv_rn(l[i], mu));
            } else {                    // every lambda is +0: u is w, bit for bit
#pragma unroll
                for (int i = 0; i < 16; ++i) u[i] = w[i];
            }
            double acc = 0.0;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const double x = (double)u[i];
                acc = __fma_rn(x, x, acc);
            }
            const u64 key = (u64)__double_as_longlong(acc);
            const bool keep = key >= br.guess;
            n_above += key > br.hi ? 1u : 0u;
            if (key >= br.lo && key <= br.hi) {
                const u64 id = d.unit_prefix + b;
                const u32 slot = atomicAdd(&sh.wcount[warp], 1u);
                sh.key[warp][slot] = key;
                sh.id[warp][slot] = id;
#pragma unroll
                for (int i = 0; i < 4; ++i) sh.lam[warp][slot][i] = l4[i];
                atomicAdd(&sh.hist[bracket_bin(br, key, id)], 1u);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float th[4], ln[4], g[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) th[j] = keep ? u[4 * i + j] : 0.0f;
                unsigned short h[4];
                if (H) {
                    half4(th, h, fp16 ? fp16 : 1);
                    if (fp16) widen4(h, th, th, fp16);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float p = __fmul_rn(mu, __fsub_rn(w[4 * i + j], th[j]));
                    ln[j] = upd ? __fsub_rn(l[4 * i + j], p) : l[4 * i + j];
                    g[j] = __fsub_rn(p, ln[j]);
                }
                const u32 off = off0 + i * C;
                *reinterpret_cast<float4 *>(d.theta + off) = make_float4(th[0], th[1], th[2], th[3]);
                if (d.mask) *reinterpret_cast<u32 *>(d.mask + off) = keep ? 0x01010101u : 0u;
                if (H && d.theta_h) *reinterpret_cast<uint2 *>(d.theta_h + off) =
                    make_uint2((u32)h[0] | ((u32)h[1] << 16), (u32)h[2] | ((u32)h[3] << 16));
                if (upd) *reinterpret_cast<float4 *>(d.lam + off) = make_float4(ln[0], ln[1], ln[2], ln[3]);
                if (G && d.grad) *reinterpret_cast<float4 *>(d.grad + off) = make_float4(g[0], g[1], g[2], g[3]);
            }
            block_flush(P, sh, BSTG - 32);
            b += THREADS;
            bcol += THREADS;
            while (bcol >= nbc) { bcol -= nbc; ++brow; }
        }
    }
    block_flush(P, sh, 0);
    __syncthreads();
    u64 na = n_above;
    // the items outside the aligned fast path (tensor tails, ragged or unaligned
    // tensors, tensors that pass through), listed by the host
    if (P.n_edge_items > 0) {
        FusedShared &fs = reinterpret_cast<FusedShared &>(sh);
        if (threadIdx.x < 2) fs.cnt[threadIdx.x] = 0;
        __syncthreads();
        int par = 0;
        for (long long i = blockIdx.x; i < P.n_edge_items; i += gridDim.x) {
            const long long item = P.edge_items[i];
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc g = P.td[t];
            const long long local = item - P.item_prefix[t];
            if (!g.ranked) process_linear_item<M_KEEPALL>(P, g, local, 0, 0);
            else fused_block_item_generic<H>(P, g, local, fs, br, par, na, fp16);
        }
        __syncthreads();
    }
    for (int o = 16; o > 0; o >>= 1) na += __shfl_xor_sync(0xffffffffu, na, o);
    if ((threadIdx.x & 31) == 0) sh.red[warp] = na;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < WARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += THREADS) {
        const u32 hc = sh.hist[i];
        if (hc) atomicAdd(&P.hist[i], (u64)hc);
    }
}

}  // namespace cs
