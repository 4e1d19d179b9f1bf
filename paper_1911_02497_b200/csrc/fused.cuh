// Single-pass projection. With a bracket [lo, hi] that (almost surely) holds the
// threshold, one pass over w and lambda settles every unit outside the bracket
// for good, writes a provisional decision (keep iff key >= guess) for the few
// units inside it, and records those in the candidate list together with their
// original lambda (the multipliers are updated in place, so a later correction
// needs the old values). The exact selection then runs on the list only and
// the units whose provisional decision was wrong are rewritten (repair).
#pragma once
#include "common.cuh"
#include "elementwise.cuh"
#include "select.cuh"
#include "structured.cuh"

namespace cs {

struct Bracket {
    u64 lo, hi, guess, lo_id;
    int shift;
    bool sk;
};

__device__ __forceinline__ Bracket load_bracket(const Sel &s)
{
    Bracket b;
    b.lo = s.lo_key; b.hi = s.hi_key; b.guess = s.guess; b.lo_id = s.lo_id;
    b.shift = s.shift;
    b.sk = s.lo_key == s.hi_key;
    return b;
}

__device__ __forceinline__ u32 bracket_bin(const Bracket &br, u64 key, u64 id)
{
    u64 b = br.sk ? ((id - br.lo_id) >> br.shift) : ((br.hi - key) >> br.shift);
    return (u32)(b > (u64)(NBINS - 1) ? (u64)(NBINS - 1) : b);
}

__device__ __forceinline__ void fused_finish(const Params &P, FusedShared &sh, u64 n_above)
{
    for (int o = 16; o > 0; o >>= 1) n_above += __shfl_xor_sync(0xffffffffu, n_above, o);
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = n_above;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < WARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += THREADS) {
        const u32 h = sh.hist[i];
        if (h) atomicAdd(&P.hist[i], (u64)h);
    }
}

// Final write of one 4x4 block, lean form.
template <bool H>
__device__ __forceinline__ void store_block_lean(const TensorDesc &d, const BlockData &bd, const float *u,
                                                 bool keep, float mu, int fp16, bool upd, bool wr_grad)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        Out o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            o[j] = finish_lean<H>(bd.w[4 * i + j], bd.l[4 * i + j], u[4 * i + j], keep, mu, fp16, upd);
        const long long off = (bd.r0 + i) * d.d1 + bd.c0;
        if (bd.full) {
            *reinterpret_cast<float4 *>(d.theta + off) = make_float4(o[0].theta, o[1].theta, o[2].theta, o[3].theta);
            if (d.mask) *reinterpret_cast<u32 *>(d.mask + off) = keep ? 0x01010101u : 0u;
            if (H && d.theta_h) {
                uint2 hh;
                hh.x = (u32)o[0].th | ((u32)o[1].th << 16);
                hh.y = (u32)o[2].th | ((u32)o[3].th << 16);
                *reinterpret_cast<uint2 *>(d.theta_h + off) = hh;
            }
            if (upd) *reinterpret_cast<float4 *>(d.lam + off) = make_float4(o[0].lam, o[1].lam, o[2].lam, o[3].lam);
            if (wr_grad) *reinterpret_cast<float4 *>(d.grad + off) = make_float4(o[0].grad, o[1].grad, o[2].grad, o[3].grad);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (bd.r0 + i >= d.d0 || bd.c0 + j >= d.d1) continue;
                d.theta[off + j] = o[j].theta;
                if (d.mask) d.mask[off + j] = o[j].m;
                if (H && d.theta_h) d.theta_h[off + j] = o[j].th;
                if (upd) d.lam[off + j] = o[j].lam;
                if (wr_grad) d.grad[off + j] = o[j].grad;
            }
        }
    }
}

// ---------------------------------------------------------------- block pruning
// Generic item: one thread per block, any alignment, ragged edges (2 rounds).
template <bool H>
__device__ __forceinline__ void fused_block_item_generic(const Params &P, const TensorDesc &d, long long local,
                                                         FusedShared &sh, const Bracket &br, int &par,
                                                         u64 &n_above, int fp16)
{
    const bool has_lam = d.lam != nullptr;
    const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
#pragma unroll 1
    for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it, par ^= 1) {
        const long long b = local * BLOCKS_PER_ITEM + it * THREADS + threadIdx.x;
        const bool ok = b < d.n_units && b >= block_fast_end(d);     // the tiled kernel has done the others
        BlockData bd;
        float u[16];
        u64 key = 0;
        const u64 id = (u64)(d.unit_prefix + b);
        if (ok) {
            load_block(d, b, bd);
            key = block_key(bd, P.mu, has_lam, u);
        }
        const bool above = ok && key > br.hi;
        const bool cand = ok && !above && key >= br.lo;
        n_above += above ? 1 : 0;
        u32 my = 0;
        if (cand) {
            my = atomicAdd(&sh.cnt[par], 1u);
            atomicAdd(&sh.hist[bracket_bin(br, key, id)], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const u32 c = sh.cnt[par];
            if (c) sh.base[par] = atomicAdd(&P.ctl->list_count[0], (u64)c);
            sh.cnt[par ^ 1] = 0;
        }
        __syncthreads();
        if (cand) {
            const u64 pos = sh.base[par] + my;
            if (pos < P.cap) {
                P.list_key[pos] = key;
                P.list_id[pos] = id;
                if (has_lam) {
                    float4 *j = reinterpret_cast<float4 *>(P.jr_lam + pos * 16);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        j[q] = make_float4(bd.l[4 * q], bd.l[4 * q + 1], bd.l[4 * q + 2], bd.l[4 * q + 3]);
                }
            }
        }
        if (ok) store_block_lean<H>(d, bd, u, ok && key >= br.guess, P.mu, fp16, upd, wr_grad);
    }
}

// ---------------------------------------------------------------- unstructured
// Generic item: per-lane validity, scalar accesses where needed.
template <bool H>
__device__ __forceinline__ void fused_elem_item_generic(const Params &P, const TensorDesc &d, long long local,
                                                        FusedShared &sh, const Bracket &br, int par,
                                                        u64 &n_above, int fp16)
{
    const u32 lo = (u32)br.lo, hi = (u32)br.hi, guess = (u32)br.guess;
    const long long ng = (d.numel + d.pad + 3) >> 2;
    const long long g0 = local * GROUPS_PER_ITEM;
    const long long g1 = (g0 + GROUPS_PER_ITEM < ng) ? g0 + GROUPS_PER_ITEM : ng;
    const bool has_lam = d.lam != nullptr;
    const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
    float w[LIN_UNROLL][4], l[LIN_UNROLL][4];
    bool full[LIN_UNROLL];
    u32 okm = 0;                 // bit 4*it+j: element exists
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        const long long g = g0 + it * THREADS + threadIdx.x;
        const long long e0 = 4 * g - d.pad;
        const bool live = g < g1;
        full[it] = live && d.vec_ok && e0 >= 0 && e0 + 4 <= d.numel;
        if (full[it]) {
            const float4 a = ld4_ro(d.w + e0);
            w[it][0] = a.x; w[it][1] = a.y; w[it][2] = a.z; w[it][3] = a.w;
            if (has_lam) {
                const float4 b = ld4(d.lam + e0);
                l[it][0] = b.x; l[it][1] = b.y; l[it][2] = b.z; l[it][3] = b.w;
            } else {
                l[it][0] = l[it][1] = l[it][2] = l[it][3] = 0.0f;
            }
            okm |= 0xFu << (4 * it);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + j;
                const bool ok = live && e >= 0 && e < d.numel;
                w[it][j] = ok ? d.w[e] : 0.0f;
                l[it][j] = (ok && has_lam) ? d.lam[e] : 0.0f;
                okm |= (ok ? 1u : 0u) << (4 * it + j);
            }
        }
    }
    float u[LIN_UNROLL][4];
    u32 candm = 0, keepm = 0;
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        form_u4(w[it], l[it], P.mu, has_lam, u[it]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const u32 key = __float_as_uint(u[it][j]) & 0x7FFFFFFFu;
            const bool ok = (okm >> (4 * it + j)) & 1u;
            const bool above = ok && key > hi;
            const bool cand = ok && !above && key >= lo;
            n_above += above ? 1 : 0;
            candm |= (cand ? 1u : 0u) << (4 * it + j);
            keepm |= ((ok && key >= guess) ? 1u : 0u) << (4 * it + j);
        }
    }
    u32 my = 0;
    if (candm) {
        my = atomicAdd(&sh.cnt[par], (u32)__popc(candm));
        u32 mm = candm;
        while (mm) {
            const int q = __ffs(mm) - 1;
            mm &= mm - 1;
            const long long e = 4 * (g0 + (q >> 2) * THREADS + threadIdx.x) - d.pad + (q & 3);
            float uu = 0.0f;
#pragma unroll
            for (int a = 0; a < LIN_UNROLL; ++a)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (q == 4 * a + c) uu = u[a][c];
            const u32 key = __float_as_uint(uu) & 0x7FFFFFFFu;
            atomicAdd(&sh.hist[bracket_bin(br, key, (u64)(d.elem_prefix + e))], 1u);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const u32 c = sh.cnt[par];
        if (c) sh.base[par] = atomicAdd(&P.ctl->list_count[0], (u64)c);
        sh.cnt[par ^ 1] = 0;
    }
    __syncthreads();
    if (candm) {
        u64 pos = sh.base[par] + my;
        u32 mm = candm;
        while (mm) {
            const int q = __ffs(mm) - 1;
            mm &= mm - 1;
            if (pos < P.cap) {
                const long long e = 4 * (g0 + (q >> 2) * THREADS + threadIdx.x) - d.pad + (q & 3);
                float uu = 0.0f, ll = 0.0f;
#pragma unroll
                for (int a = 0; a < LIN_UNROLL; ++a)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (q == 4 * a + c) { uu = u[a][c]; ll = l[a][c]; }
                P.list_key[pos] = (u64)(__float_as_uint(uu) & 0x7FFFFFFFu);
                P.list_id[pos] = (u64)(d.elem_prefix + e);
                if (has_lam) P.jr_lam[pos] = ll;
            }
            ++pos;
        }
    }
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        const long long g = g0 + it * THREADS + threadIdx.x;
        if (g >= g1) continue;
        const long long e0 = 4 * g - d.pad;
        Out o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            o[j] = finish_lean<H>(w[it][j], l[it][j], u[it][j], (keepm >> (4 * it + j)) & 1u, P.mu, fp16, upd);
        if (full[it]) {
            *reinterpret_cast<float4 *>(d.theta + e0) = make_float4(o[0].theta, o[1].theta, o[2].theta, o[3].theta);
            if (d.mask) *reinterpret_cast<u32 *>(d.mask + e0) =
                (u32)o[0].m | ((u32)o[1].m << 8) | ((u32)o[2].m << 16) | ((u32)o[3].m << 24);
            if (H && d.theta_h) {
                uint2 hh;
                hh.x = (u32)o[0].th | ((u32)o[1].th << 16);
                hh.y = (u32)o[2].th | ((u32)o[3].th << 16);
                *reinterpret_cast<uint2 *>(d.theta_h + e0) = hh;
            }
            if (upd) *reinterpret_cast<float4 *>(d.lam + e0) = make_float4(o[0].lam, o[1].lam, o[2].lam, o[3].lam);
            if (wr_grad) *reinterpret_cast<float4 *>(d.grad + e0) = make_float4(o[0].grad, o[1].grad, o[2].grad, o[3].grad);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (!((okm >> (4 * it + j)) & 1u)) continue;
                const long long e = e0 + j;
                d.theta[e] = o[j].theta;
                if (d.mask) d.mask[e] = o[j].m;
                if (H && d.theta_h) d.theta_h[e] = o[j].th;
                if (upd) d.lam[e] = o[j].lam;
                if (wr_grad) d.grad[e] = o[j].grad;
            }
        }
    }
}

// Rewrite one listed unit whose provisional decision was wrong. Called from the
// selection kernels after the cut-off is known. `idx` is the list position (the
// journal holds the original lambda there). An element is rewritten by one thread
// (`part` 0); a block by four, `part` being the row: u comes from the journal by the
// same two operations as everywhere (the norm is not needed again).
template <int SRC>
__device__ __noinline__ void repair_unit(const Params &P, u64 idx, u64 id, bool keep, int part, const long long *pre_s,
                                         const TensorDesc *tdc)
{
    // One copy of this code per kernel and as few instructions as possible: it runs once per
    // call on a few threads, right after a pass that has swept the L2, so its time is the time
    // to fetch its instructions.
    int lo = 0, hi = P.T - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        const long long pre = pre_s ? pre_s[mid] : (SRC == SRC_ELEM) ? P.td[mid].elem_prefix : P.td[mid].unit_prefix;
        if ((u64)pre <= id) lo = mid; else hi = mid - 1;
    }
    const TensorDesc &d = tdc ? tdc[lo] : P.td[lo];
    if (SRC == SRC_BLOCKG) {                    // rows part, part + 8, ... of a bh x bw block
        const long long b = (long long)id - d.unit_prefix;
        if (b < 0 || b >= d.n_units) return;
        blockg_write_global(P, d, b, keep, P.jr_lam + idx * (u64)P.jr_floats, part, (int)RepairLanes<SRC_BLOCKG>::value);
        return;
    }
    const bool has_lam = d.lam != nullptr;
    const bool wr_lam = (P.fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
    long long off;          // first element to rewrite
    int nv;                 // how many consecutive elements
    const float *jr;        // their original multipliers
    if (SRC == SRC_ELEM) {
        off = (long long)id - d.elem_prefix;
        if (off < 0 || off >= d.numel) return;
        nv = 1;
        jr = P.jr_lam + idx;
    } else {
        const long long b = (long long)id - d.unit_prefix;
        if (b < 0 || b >= d.n_units) return;
        const long long br = d.n_units < 0x7FFFFFFFll ? (long long)((u32)b / (u32)d.nbc) : b / d.nbc;
        const long long bc = b - br * d.nbc;
        const long long r = 4 * br + part, c0 = 4 * bc;
        if (r >= d.d0) return;
        off = r * d.d1 + c0;
        nv = d.d1 - c0 < 4 ? (int)(d.d1 - c0) : 4;           // columns of this row that exist
        jr = P.jr_lam + idx * 16 + 4 * part;
    }
    float w[4], l[4];
    const bool vec = SRC == SRC_BLOCK && nv == 4 && d.blk_vec_ok;      // a whole aligned row of a block
    if (vec) {
        const float4 a = ld4_ro(d.w + off);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
        const float4 q = has_lam ? __ldcg(reinterpret_cast<const float4 *>(jr)) : make_float4(0.f, 0.f, 0.f, 0.f);
        l[0] = q.x; l[1] = q.y; l[2] = q.z; l[3] = q.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            w[j] = j < nv ? __ldg(d.w + off + j) : 0.0f;
            l[j] = (j < nv && has_lam) ? __ldcg(jr + j) : 0.0f;
        }
    }
    float th[4], ln[4], gr[4];
    unsigned short hb[4];
    unsigned char mk[4];
#pragma unroll 1
    for (int j = 0; j < nv; ++j) {
        const Out o = finish(w[j], l[j], form_u(w[j], l[j], P.mu, has_lam), keep, P.mu, P.fuse, has_lam);
        th[j] = o.theta; ln[j] = o.lam; gr[j] = o.grad; hb[j] = o.th; mk[j] = o.m;
    }
    if (vec) {
        *reinterpret_cast<float4 *>(d.theta + off) = make_float4(th[0], th[1], th[2], th[3]);
        if (d.mask) *reinterpret_cast<u32 *>(d.mask + off) = keep ? 0x01010101u : 0u;
        if (d.theta_h) *reinterpret_cast<uint2 *>(d.theta_h + off) =
            make_uint2((u32)hb[0] | ((u32)hb[1] << 16), (u32)hb[2] | ((u32)hb[3] << 16));
        if (wr_lam) *reinterpret_cast<float4 *>(d.lam + off) = make_float4(ln[0], ln[1], ln[2], ln[3]);
        if (wr_grad) *reinterpret_cast<float4 *>(d.grad + off) = make_float4(gr[0], gr[1], gr[2], gr[3]);
    } else {
        for (int j = 0; j < nv; ++j) {
            d.theta[off + j] = th[j];
            if (d.mask) d.mask[off + j] = mk[j];
            if (d.theta_h) d.theta_h[off + j] = hb[j];
            if (wr_lam) d.lam[off + j] = ln[j];
            if (wr_grad) d.grad[off + j] = gr[j];
        }
    }
}

}  // namespace cs
