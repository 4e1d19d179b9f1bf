// Exact selection of the rank-k unit in (key descending, id ascending) order
// by range-partition histogram passes, without sorting.
//
// A pass ("scan") visits units, drops those outside the current bracket,
// bins the rest into NBINS equal power-of-two-wide bins (by key, or by id once
// the key range is a single value) and optionally appends them to a candidate
// list. The "pick" finds the bin that holds the wanted rank and makes it the
// new bracket. Passes run over the source until the bracket fits the list,
// then over the list, until at most FIN units are left, which are ranked
// directly. One cooperative kernel drives the loop with grid-wide barriers.
#pragma once
#include "common.cuh"

namespace cs {

namespace cg = cooperative_groups;

constexpr int REPAIR_TD_CACHE = 16;

struct ScanShared {
    u32 hist[NBINS];
    u64 stg_key[WARPS][WSTG];      // the two staging arrays are adjacent: the direct ranking uses
    u64 stg_id[WARPS][WSTG];       // them as one array of 2 * WARPS * WSTG values
    u64 red[WARPS];
    Sel sel;
    u64 pick_before;
    u64 pick_count;
    int pick_bin;
    int fin_hit;
    u64 rk_value;                  // direct ranking: value found, entries before it, entries equal to it
    u32 rk_before, rk_count;
    TensorDesc tdc[REPAIR_TD_CACHE];   // descriptors of short tensor lists, for the rewrites
};
static_assert(offsetof(ScanShared, stg_id) == offsetof(ScanShared, stg_key) + sizeof(u64) * WARPS * WSTG,
              "staging arrays must be adjacent");
static_assert(FIN <= 2 * WARPS * WSTG, "the direct ranking keeps FIN values in the staging arrays");

struct ScanCtx {
    u64 n_above;     // per thread
    u32 wc;          // staged entries of this warp (warp uniform)
    bool sk;         // bracket is a single key: bin by id
    bool do_list;
    int list_sel;
};

__device__ __forceinline__ void scan_begin(ScanShared &sh, ScanCtx &c, bool do_list)
{
    for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
    c.n_above = 0;
    c.wc = 0;
    c.sk = sh.sel.lo_key == sh.sel.hi_key;
    c.do_list = do_list;
    c.list_sel = sh.sel.list_sel;
    __syncthreads();
}

__device__ __forceinline__ void flush_warp(const Params &P, ScanShared &sh, ScanCtx &c)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u64 base = 0;
    if (lane == 0 && c.wc) base = atomicAdd(&P.ctl->list_count[c.list_sel], (u64)c.wc);
    base = __shfl_sync(0xffffffffu, base, 0);
    for (u32 i = lane; i < c.wc; i += 32) {
        const u64 pos = base + i;
        if (pos < P.cap) {
            P.list_key[pos] = sh.stg_key[warp][i];
            P.list_id[pos] = sh.stg_id[warp][i];
        }
    }
    c.wc = 0;
    __syncwarp();
}

// Classify one unit per lane. Must be called by all 32 lanes of a warp together.
__device__ __forceinline__ void scan_emit(const Params &P, ScanShared &sh, ScanCtx &c, u64 key,
                                          u64 id, bool active)
{
    const Sel &s = sh.sel;
    bool in = false;
    if (active) {
        const bool above = key > s.hi_key || (c.sk && key == s.hi_key && id < s.lo_id);
        const bool below = key < s.lo_key || (c.sk && key == s.lo_key && id > s.hi_id);
        in = !above && !below;
        c.n_above += above ? 1 : 0;
    }
    if (in) {
        u64 b = c.sk ? ((id - s.lo_id) >> s.shift) : ((s.hi_key - key) >> s.shift);
        if (b > (u64)(NBINS - 1)) b = NBINS - 1;
        atomicAdd(&sh.hist[(u32)b], 1u);
    }
    if (c.do_list) {
        const unsigned bal = __ballot_sync(0xffffffffu, in);
        if (bal) {
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (in) {
                const u32 pos = c.wc + __popc(bal & ((1u << lane) - 1u));
                sh.stg_key[warp][pos] = key;
                sh.stg_id[warp][pos] = id;
            }
            c.wc += __popc(bal);
            __syncwarp();
            if (c.wc > WSTG - 32) flush_warp(P, sh, c);
        }
    }
}

__device__ __forceinline__ void scan_end(const Params &P, ScanShared &sh, ScanCtx &c, int slot)
{
    if (c.do_list) flush_warp(P, sh, c);
    // units above the bracket seen by this CTA
    u64 v = c.n_above;
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < WARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[slot], tot);
    }
    u64 *gh = P.hist + (size_t)slot * NBINS;
    for (int i = threadIdx.x; i < NBINS; i += THREADS) {
        const u32 h = sh.hist[i];
        if (h) atomicAdd(&gh[i], (u64)h);
    }
    __syncthreads();
}

// ---------------------------------------------------------------- sources
// Unstructured: key of every element of every tensor.
__device__ __forceinline__ void scan_source_elem(const Params &P, ScanShared &sh, ScanCtx &c)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long ng = (d.numel + d.pad + 3) >> 2;
        const long long g0 = (item - P.item_prefix[t]) * GROUPS_PER_ITEM;
        const long long g1 = (g0 + GROUPS_PER_ITEM < ng) ? g0 + GROUPS_PER_ITEM : ng;
        const bool has_lam = d.lam != nullptr;
        float w[GROUPS_PER_ITEM / THREADS][4], l[GROUPS_PER_ITEM / THREADS][4];
#pragma unroll
        for (int it = 0; it < GROUPS_PER_ITEM / THREADS; ++it) {
            const long long g = g0 + it * THREADS + threadIdx.x;
            const long long e0 = 4 * g - d.pad;
            const bool live = g < g1;
            const bool full = live && d.vec_ok && e0 >= 0 && e0 + 4 <= d.numel;
            if (full) {
                const float4 a = __ldg(reinterpret_cast<const float4 *>(d.w + e0));
                w[it][0] = a.x; w[it][1] = a.y; w[it][2] = a.z; w[it][3] = a.w;
                if (has_lam) {
                    const float4 b = *reinterpret_cast<const float4 *>(d.lam + e0);
                    l[it][0] = b.x; l[it][1] = b.y; l[it][2] = b.z; l[it][3] = b.w;
                } else {
                    l[it][0] = l[it][1] = l[it][2] = l[it][3] = 0.0f;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const long long e = e0 + j;
                    const bool ok = live && e >= 0 && e < d.numel;
                    w[it][j] = ok ? d.w[e] : 0.0f;
                    l[it][j] = (ok && has_lam) ? d.lam[e] : 0.0f;
                }
            }
        }
#pragma unroll
        for (int it = 0; it < GROUPS_PER_ITEM / THREADS; ++it) {
            const long long g = g0 + it * THREADS + threadIdx.x;
            const long long e0 = 4 * g - d.pad;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + j;
                const bool ok = g < g1 && e >= 0 && e < d.numel;
                const float u = form_u(w[it][j], l[it][j], P.mu, has_lam);
                scan_emit(P, sh, c, key_of_u(u), (u64)(d.elem_prefix + e), ok);
            }
        }
    }
}

// nu of one 4x4 block: fp64 sum of u^2, row by row. Elements outside the tensor
// count as zero. Returns the fp64 bit pattern.
struct BlockData {
    float w[16], l[16];
    bool full;
    long long r0, c0;
};

__device__ __forceinline__ void load_block(const TensorDesc &d, long long b, BlockData &bd)
{
    long long br;
    if (d.n_units < 0x7FFFFFFFll) br = (long long)((u32)b / (u32)d.nbc);
    else br = b / d.nbc;
    const long long bc = b - br * d.nbc;
    bd.r0 = br * 4;
    bd.c0 = bc * 4;
    bd.full = d.blk_vec_ok && bd.r0 + 4 <= d.d0;
    const bool has_lam = d.lam != nullptr;
    if (bd.full) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long off = (bd.r0 + i) * d.d1 + bd.c0;
            const float4 a = __ldg(reinterpret_cast<const float4 *>(d.w + off));
            bd.w[4 * i + 0] = a.x; bd.w[4 * i + 1] = a.y; bd.w[4 * i + 2] = a.z; bd.w[4 * i + 3] = a.w;
            if (has_lam) {
                const float4 q = *reinterpret_cast<const float4 *>(d.lam + off);
                bd.l[4 * i + 0] = q.x; bd.l[4 * i + 1] = q.y; bd.l[4 * i + 2] = q.z; bd.l[4 * i + 3] = q.w;
            } else {
                bd.l[4 * i + 0] = bd.l[4 * i + 1] = bd.l[4 * i + 2] = bd.l[4 * i + 3] = 0.0f;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long r = bd.r0 + i, cc = bd.c0 + j;
                const bool ok = r < d.d0 && cc < d.d1;
                const long long off = r * d.d1 + cc;
                bd.w[4 * i + j] = ok ? d.w[off] : 0.0f;
                bd.l[4 * i + j] = (ok && has_lam) ? d.lam[off] : 0.0f;
            }
    }
}

__device__ __forceinline__ u64 block_key(const BlockData &bd, float mu, bool has_lam, float *u)
{
    u32 nz = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) nz |= __float_as_uint(bd.l[i]);
    if (has_lam && nz) {
#pragma unroll
        for (int i = 0; i < 16; ++i) u[i] = __fsub_rn(bd.w[i], __fdiv_rn(bd.l[i], mu));
    } else {                           // every lambda is +0: w - (+0) is w, bit for bit
#pragma unroll
        for (int i = 0; i < 16; ++i) u[i] = bd.w[i];
    }
    double acc = 0.0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const double x = (double)u[i];
        acc = __fma_rn(x, x, acc);     // x*x is exact in fp64, so this is (acc + x*x) rounded once
    }
    return (u64)__double_as_longlong(acc);
}

// Block b of tensor d: first row and column, rows and columns that exist.
struct BlockExt {
    long long r0, c0;
    int nr, nc;
};

__device__ __forceinline__ BlockExt blockg_ext(const TensorDesc &d, long long b)
{
    BlockExt e;
    const long long br = d.n_units < 0x7FFFFFFFll ? (long long)((u32)b / (u32)d.nbc) : b / d.nbc;
    const long long bc = b - br * d.nbc;
    e.r0 = br * d.bh;
    e.c0 = bc * d.bw;
    e.nr = (int)(d.d0 - e.r0 < d.bh ? d.d0 - e.r0 : d.bh);
    e.nc = (int)(d.d1 - e.c0 < d.bw ? d.d1 - e.c0 : d.bw);
    return e;
}

// nu of block b straight from global memory: fp64 sum of u^2 over the elements that exist,
// row by row. Returns the fp64 bit pattern.
__device__ __forceinline__ u64 blockg_key_global(const TensorDesc &d, long long b, float mu)
{
    const BlockExt e = blockg_ext(d, b);
    const bool has_lam = d.lam != nullptr;
    // the rows are fetched one after the other by the loop below (its bounds are not known at
    // compile time): ask for all of them first, so that the loop finds them on the way
    for (int r = 0; r < e.nr; ++r) {
        const long long off = (e.r0 + r) * d.d1 + e.c0;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(d.w + off));
        if (has_lam) asm volatile("prefetch.global.L2 [%0];" ::"l"(d.lam + off));
        if (((uintptr_t)(d.w + off) & 127u) + 4u * (u32)e.nc > 128u) {       // the row piece crosses a 128-byte line
            asm volatile("prefetch.global.L2 [%0];" ::"l"(d.w + off + e.nc - 1));
            if (has_lam) asm volatile("prefetch.global.L2 [%0];" ::"l"(d.lam + off + e.nc - 1));
        }
    }
    double acc = 0.0;
    if (e.nc <= 8) {
        // a row at a time: its loads leave together (one round trip per row, not one per element)
        for (int r = 0; r < e.nr; ++r) {
            const long long off = (e.r0 + r) * d.d1 + e.c0;
            float wv[8], lv[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                wv[c] = c < e.nc ? __ldg(d.w + off + c) : 0.0f;
                lv[c] = (c < e.nc && has_lam) ? d.lam[off + c] : 0.0f;
            }
#pragma unroll
            for (int c = 0; c < 8; ++c)
                if (c < e.nc) {
                    const double x = (double)form_u(wv[c], lv[c], mu, has_lam);
                    acc = __fma_rn(x, x, acc);
                }
        }
        return (u64)__double_as_longlong(acc);
    }
    for (int r = 0; r < e.nr; ++r) {
        const long long off = (e.r0 + r) * d.d1 + e.c0;
        for (int c = 0; c < e.nc; ++c) {
            const double x = (double)form_u(__ldg(d.w + off + c), has_lam ? d.lam[off + c] : 0.0f, mu, has_lam);
            acc = __fma_rn(x, x, acc);
        }
    }
    return (u64)__double_as_longlong(acc);
}

// Final write of the rows r_first, r_first + r_step, ... of block b from global memory. `jr`,
// when given, holds the block's original multipliers (row-major, d.bw floats per row) and is
// read instead of lambda, which an earlier pass may have updated in place.
__device__ __forceinline__ void blockg_write_global(const Params &P, const TensorDesc &d, long long b, bool keep,
                                                    const float *jr, int r_first, int r_step)
{
    const BlockExt e = blockg_ext(d, b);
    const bool has_lam = d.lam != nullptr;
    const bool wr_lam = (P.fuse & FUSE_LAMBDA) && has_lam;
    const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
    for (int r = r_first; r < e.nr; r += r_step) {
        const long long off = (e.r0 + r) * d.d1 + e.c0;
        for (int c = 0; c < e.nc; ++c) {
            const float w = __ldg(d.w + off + c);
            const float l = has_lam ? (jr ? __ldcg(jr + r * d.bw + c) : d.lam[off + c]) : 0.0f;
            const Out o = finish(w, l, form_u(w, l, P.mu, has_lam), keep, P.mu, P.fuse, has_lam);
            d.theta[off + c] = o.theta;
            if (d.mask) d.mask[off + c] = o.m;
            if (d.theta_h) d.theta_h[off + c] = o.th;
            if (wr_lam) d.lam[off + c] = o.lam;
            if (wr_grad) d.grad[off + c] = o.grad;
        }
    }
}

// The same scan for bh x bw blocks.
__device__ __forceinline__ void scan_source_blockg(const Params &P, ScanShared &sh, ScanCtx &c)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long b0 = (item - P.item_prefix[t]) * BLOCKS_PER_ITEM;
#pragma unroll 1
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const long long b = b0 + it * THREADS + threadIdx.x;
            const bool ok = b < d.n_units;
            scan_emit(P, sh, c, ok ? blockg_key_global(d, b, P.mu) : 0, (u64)(d.unit_prefix + b), ok);
        }
    }
}

// Block items exist for ranked (2-D) tensors only in the scan decomposition.
__device__ __forceinline__ void scan_source_block(const Params &P, ScanShared &sh, ScanCtx &c)
{
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        const TensorDesc d = P.td[t];
        const long long b0 = (item - P.item_prefix[t]) * BLOCKS_PER_ITEM;
        const bool has_lam = d.lam != nullptr;
#pragma unroll 1
        for (int it = 0; it < BLOCKS_PER_ITEM / THREADS; ++it) {
            const long long b = b0 + it * THREADS + threadIdx.x;
            const bool ok = b < d.n_units;
            u64 key = 0;
            if (ok) {
                BlockData bd;
                float u[16];
                load_block(d, b, bd);
                key = block_key(bd, P.mu, has_lam, u);
            }
            scan_emit(P, sh, c, key, (u64)(d.unit_prefix + b), ok);
        }
    }
}

__device__ __forceinline__ void scan_source_array(const Params &P, ScanShared &sh, ScanCtx &c)
{
    const long long stride = (long long)gridDim.x * THREADS;
    for (long long base = (long long)blockIdx.x * THREADS; base < P.S; base += stride) {
        const long long i = base + threadIdx.x;
        const bool ok = i < P.S;
        scan_emit(P, sh, c, ok ? P.arr_key[i] : 0, (u64)i, ok);
    }
}

template <int SRC>
__device__ __noinline__ void scan_source(const Params &P, ScanShared &sh, bool do_list, int slot)
{
    ScanCtx c;
    scan_begin(sh, c, do_list);
    if (SRC == SRC_ELEM) scan_source_elem(P, sh, c);
    else if (SRC == SRC_BLOCK) scan_source_block(P, sh, c);
    else if (SRC == SRC_BLOCKG) scan_source_blockg(P, sh, c);
    else scan_source_array(P, sh, c);
    scan_end(P, sh, c, slot);
}

__device__ __noinline__ void scan_list(const Params &P, ScanShared &sh, int slot, u64 n_list)
{
    ScanCtx c;
    scan_begin(sh, c, false);
    // several entries per thread are fetched before the first is used: the walk is
    // a few rounds per thread and would otherwise pay one memory round trip per entry
    constexpr int R = 8;
    const u64 chunk = (u64)R * THREADS;
    for (u64 base = (u64)blockIdx.x * chunk; base < n_list; base += (u64)gridDim.x * chunk) {
        u64 key[R], id[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const u64 i = base + (u64)r * THREADS + threadIdx.x;
            key[r] = i < n_list ? __ldcg(&P.list_key[i]) : 0;
            id[r] = i < n_list ? __ldcg(&P.list_id[i]) : 0;
        }
#pragma unroll
        for (int r = 0; r < R; ++r)
            scan_emit(P, sh, c, key[r], id[r], base + (u64)r * THREADS + threadIdx.x < n_list);
    }
    scan_end(P, sh, c, slot);
}

// ---------------------------------------------------------------- pick
__device__ __forceinline__ void set_shift(Sel &s)
{
    const u64 range = (s.lo_key == s.hi_key) ? (s.hi_id - s.lo_id) : (s.hi_key - s.lo_key);
    const int bl = bit_length(range);
    s.shift = bl > LOG_NBINS ? bl - LOG_NBINS : 0;
}

// All threads of the CTA; every CTA computes the same new state from the same
// global histogram. `src_scan`: the scan that filled the histogram visited the
// whole source (its count of units above the bracket is then complete).
// `may_fall_back`: a sampled single-pass bracket that turns out not to hold the rank
// is replaced by the full range (the caller then runs the two-pass route) when the
// call allows it; otherwise, and in the kernel that must not change anything, it is
// error 10.
__device__ __noinline__ void block_pick(const Params &P, ScanShared &sh, bool src_scan, u64 max_key,
                                        bool may_fall_back = false)
{
    Sel &s = sh.sel;
    const u64 *gh = P.hist + (size_t)s.slot * NBINS;
    constexpr int PER = NBINS / THREADS;
    u64 cnt[PER];
    u64 tsum = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        cnt[j] = __ldcg(&gh[threadIdx.x * PER + j]);
        tsum += cnt[j];
    }
    // exclusive scan of tsum over the CTA
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u64 inc = tsum;
    for (int o = 1; o < 32; o <<= 1) {
        const u64 v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) sh.red[warp] = inc;
    if (threadIdx.x == 0) sh.pick_bin = -1;
    __syncthreads();
    u64 wbase = 0, total = 0;
    for (int i = 0; i < WARPS; ++i) {
        if (i < warp) wbase += sh.red[i];
        total += sh.red[i];
    }
    const u64 excl = wbase + inc - tsum;
    const u64 above_scan = __ldcg(&P.ctl->scan_above[s.slot]);
    const u64 n_above = s.above_known ? s.n_above : above_scan;
    const bool valid = s.k > n_above && (s.k - n_above) <= total;
    const u64 r = s.k - n_above;
    if (valid && r > excl && r <= excl + tsum) {
        u64 run = excl;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (r > run && r <= run + cnt[j]) {
                sh.pick_bin = threadIdx.x * PER + j;
                sh.pick_before = run;
                sh.pick_count = cnt[j];
            }
            run += cnt[j];
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        s.passes += 1;
        if (s.above_known && src_scan && above_scan != s.n_above) s.error = 1;
        const bool sk = s.lo_key == s.hi_key;
        if (!valid) {
            if (s.onepass) {
                if (may_fall_back && P.miss_fallback) {
                    // the sampled bracket missed, but nothing the first pass wrote is needed
                    // again: start over on the full key range; the projection follows the
                    // selection and overwrites every output
                    s.onepass = 0;
                    s.lo_key = 0;
                    s.hi_key = max_key;
                    s.n_above = 0;
                    s.pop = s.S;
                } else {
                    s.error = 10;   // the sampled bracket missed: outputs already written are wrong
                    s.done = 1;
                }
            } else if (s.above_known) {
                s.error = 2;        // a histogram-derived bracket must hold the rank
                s.done = 1;
            } else if (s.k <= n_above) {
                // wanted unit ranks before the sampled bracket
                if (sk && s.lo_id > 0) { s.error = 3; s.done = 1; }
                s.lo_key = s.hi_key + 1;
                s.hi_key = max_key;
                s.n_above = 0;
                s.pop = n_above;
            } else {
                if (s.lo_key == 0) { s.error = 4; s.done = 1; }
                s.n_above = n_above + total;
                s.hi_key = s.lo_key - 1;
                s.lo_key = 0;
                s.pop = s.S - s.n_above;
            }
            s.lo_id = 0;
            s.hi_id = s.S - 1;
            s.above_known = 1;
            s.list_valid = 0;
            s.sampled = 0;
            if (s.lo_key > s.hi_key) { s.error = 4; s.done = 1; }
        } else {
            if (sk && !s.key_fixed) {
                s.key_fixed = 1;
                s.n_gt = n_above;
                s.n_tie = total;
            }
            const int b = sh.pick_bin;
            if (b < 0) { s.error = 5; s.done = 1; }
            s.n_above = n_above + sh.pick_before;
            s.above_known = 1;
            s.pop = sh.pick_count;
            if (!sk) {
                const u64 width = 1ull << s.shift;
                const u64 nh = s.hi_key - ((u64)b << s.shift);
                u64 nl = (nh - s.lo_key >= width - 1) ? nh - (width - 1) : s.lo_key;
                s.hi_key = nh;
                s.lo_key = nl;
                if (nl == nh && !s.key_fixed) {
                    s.key_fixed = 1;
                    s.n_gt = s.n_above;
                    s.n_tie = s.pop;
                    s.lo_id = 0;
                    s.hi_id = s.S - 1;
                }
            } else {
                const u64 width = 1ull << s.shift;
                const u64 nl = s.lo_id + ((u64)b << s.shift);
                const u64 nh = (s.hi_id - nl >= width - 1) ? nl + (width - 1) : s.hi_id;
                s.lo_id = nl;
                s.hi_id = nh;
            }
            if (s.lo_key == s.hi_key && s.lo_id == s.hi_id) {
                s.done = 1;            // a single unit is left: it is the cut-off
                if (s.pop != 1) s.error = 6;
            }
        }
        set_shift(s);
        if (s.passes >= MAX_SELECT_ITERS && !s.done) { s.error = 7; s.done = 1; }
    }
    __syncthreads();
}

// Value of rank r (1-based) among the entries of v[0..n) that lie in [lo, hi], in
// descending (asc = false) or ascending order, by range-partition passes in shared
// memory (all threads of the CTA). Leaves in sh.rk_value the value, in sh.rk_before
// how many in-range entries rank strictly before it and in sh.rk_count how many
// equal it; sh.fin_hit is -1 if the rank does not exist. At most 7 passes: the
// range shrinks by LOG_NBINS bits per pass.
__device__ __noinline__ void smem_select(const u64 *v, u32 n, u64 lo, u64 hi, bool asc, u64 r, ScanShared &sh)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int PER = NBINS / THREADS;
    u32 before = 0;
    if (threadIdx.x == 0) sh.fin_hit = 0;
    for (int pass = 0; pass < 8; ++pass) {
        const int bl = bit_length(hi - lo);
        const int shift = bl > LOG_NBINS ? bl - LOG_NBINS : 0;
        for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
        __syncthreads();
        for (u32 i = threadIdx.x; i < n; i += THREADS) {
            const u64 x = v[i];
            if (x >= lo && x <= hi) atomicAdd(&sh.hist[(u32)((asc ? x - lo : hi - x) >> shift)], 1u);
        }
        __syncthreads();
        u32 cnt[PER], tsum = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) { cnt[j] = sh.hist[threadIdx.x * PER + j]; tsum += cnt[j]; }
        u32 inc = tsum;
        for (int o = 1; o < 32; o <<= 1) {
            const u32 y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) sh.red[warp] = inc;
        if (threadIdx.x == 0) sh.pick_bin = -1;
        __syncthreads();
        u32 wbase = 0;
        for (int i = 0; i < warp; ++i) wbase += (u32)sh.red[i];
        u32 run = wbase + inc - tsum;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if (r > run && r <= (u64)run + cnt[j]) {
                sh.pick_bin = threadIdx.x * PER + j;
                sh.pick_before = run;
                sh.pick_count = cnt[j];
            }
            run += cnt[j];
        }
        __syncthreads();
        const int b = sh.pick_bin;
        const u32 pb = (u32)sh.pick_before, pc = (u32)sh.pick_count;
        __syncthreads();
        if (b < 0) {                        // the rank does not exist among the entries
            if (threadIdx.x == 0) sh.fin_hit = -1;
            __syncthreads();
            return;
        }
        before += pb;
        r -= pb;
        const u64 width = 1ull << shift;
        if (asc) {
            const u64 nl = lo + ((u64)b << shift);
            hi = (hi - nl >= width - 1) ? nl + (width - 1) : hi;
            lo = nl;
        } else {
            const u64 nh = hi - ((u64)b << shift);
            lo = (nh - lo >= width - 1) ? nh - (width - 1) : lo;
            hi = nh;
        }
        if (pc == 1 && lo != hi) {          // one entry left in the range: it is the value
            for (u32 i = threadIdx.x; i < n; i += THREADS) {
                const u64 x = v[i];
                if (x >= lo && x <= hi) sh.rk_value = x;
            }
            if (threadIdx.x == 0) { sh.rk_before = before; sh.rk_count = 1; }
            __syncthreads();
            return;
        }
        if (lo == hi) {
            if (threadIdx.x == 0) { sh.rk_value = lo; sh.rk_before = before; sh.rk_count = pc; }
            __syncthreads();
            return;
        }
    }
    if (threadIdx.x == 0) sh.fin_hit = -1;
    __syncthreads();
}

// Rank the (at most FIN) bracket members directly. Entries are in fin_key/fin_id.
// The keys go to shared memory and the key of the wanted rank is found there;
// among the entries that carry this key the index decides (lower first), found the
// same way on their indices.
__device__ __noinline__ void final_rank(const Params &P, ScanShared &sh, u32 n)
{
    Sel &s = sh.sel;
    u64 *v = &sh.stg_key[0][0];
    if (n > FIN) n = FIN;
    for (u32 i = threadIdx.x; i < n; i += THREADS) v[i] = __ldcg(&P.fin_key[i]);
    if (n <= (u32)THREADS && threadIdx.x < n) v[FIN / 2 + threadIdx.x] = __ldcg(&P.fin_id[threadIdx.x]);
    if (threadIdx.x == 0) sh.fin_hit = -1;
    __syncthreads();
    const u64 r = s.k - s.n_above;          // 1-based rank inside the bracket
    bool ok = s.k > s.n_above && r <= (u64)n;
    u64 tk = 0, tid = 0;
    u32 gt = 0, eq = 0;
    if (ok && n <= (u32)THREADS) {
        // few survivors: one entry per thread, which counts how many rank before it
        u64 *ids = v + FIN / 2;
        if (threadIdx.x < n) {
            const u64 ki = v[threadIdx.x];
            u32 g = 0, e = 0, lower = 0;
#pragma unroll 8
            for (u32 j = 0; j < n; ++j) {
                const u64 kj = v[j];
                g += (u32)(kj > ki);
                e += (u32)(kj == ki);
            }
            if (e > 1) {                    // equal keys beside itself: the lower index ranks first
                const u64 di = ids[threadIdx.x];
                for (u32 j = 0; j < n; ++j) lower += (u32)(v[j] == ki && ids[j] < di);
            }
            if ((u64)g + lower + 1 == r) {
                sh.fin_hit = (int)threadIdx.x;
                sh.rk_value = ki;
                sh.rk_before = g;
                sh.rk_count = e;
            }
        }
        __syncthreads();
        ok = sh.fin_hit >= 0;
        if (ok) { tk = sh.rk_value; gt = sh.rk_before; eq = sh.rk_count; tid = ids[sh.fin_hit]; }
        __syncthreads();
    } else {
    if (ok) {
        smem_select(v, n, s.lo_key, s.hi_key, false, r, sh);
        ok = sh.fin_hit >= 0;
        tk = sh.rk_value; gt = sh.rk_before; eq = sh.rk_count;
        __syncthreads();
    }
    if (ok) {
        // the (r - gt)-th lowest index among the entries with this key
        for (u32 i = threadIdx.x; i < n; i += THREADS) v[i] = (v[i] == tk) ? __ldcg(&P.fin_id[i]) : ~0ull;
        __syncthreads();
        smem_select(v, n, s.lo_key == s.hi_key ? s.lo_id : 0ull, s.lo_key == s.hi_key ? s.hi_id : s.S - 1, true,
                    r - gt, sh);
        ok = sh.fin_hit >= 0 && sh.rk_count == 1;
        tid = sh.rk_value;
        __syncthreads();
    }
    }
    if (threadIdx.x == 0) {
        if (ok) {
            if (!s.key_fixed) {
                s.key_fixed = 1;
                s.n_gt = s.n_above + gt;
                s.n_tie = eq;
            }
            s.lo_key = s.hi_key = tk;
            s.lo_id = s.hi_id = tid;
        } else {
            s.error = 8;
        }
        s.done = 1;
    }
    __syncthreads();
}

// Control block at the start of a ranking call (one thread).
__device__ __forceinline__ void init_ctl(Ctl *c, const Sel &init)
{
    c->sel = init;
    c->tau_key = KEY_NONE;
    c->tau_id = 0;
    c->scan_above[0] = c->scan_above[1] = c->scan_above[2] = 0;
    c->list_count[0] = c->list_count[1] = 0;
    c->fin_count = 0;
    c->n_repaired = 0;
    c->sample_done = 0;
    c->async_error = 0;
}

// Cut-off and record of the call, from the final selection state (one thread).
__device__ __forceinline__ void write_result(const Params &P, const Sel &s)
{
    Ctl *c = P.ctl;
    Result r;
    r.status = s.error ? -5 : 0;
    r.passes = s.passes;
    r.n_units = (long long)s.S;
    r.n_keep = (long long)s.k;
    r.n_zero = (long long)(s.S - s.k);
    r.sampled = s.sampled;
    r.n_candidates = (long long)(c->list_count[0] + c->list_count[1]);
    r.tau_norm = 0.0f;
    if (s.k == 0 || s.S == 0 || s.error) {
        c->tau_key = KEY_NONE;
        c->tau_id = 0;
        r.tau_key = (P.bits_key >= 63) ? 0x7FF0000000000000ull : 0x7F800000ull;
        r.tau_id = -1;
        r.n_gt = r.n_tie = r.n_tie_kept = 0;
    } else {
        c->tau_key = s.lo_key;
        c->tau_id = s.lo_id;
        r.tau_key = s.lo_key;
        r.tau_id = (long long)s.lo_id;
        r.n_gt = (long long)s.n_gt;
        r.n_tie = (long long)s.n_tie;
        r.n_tie_kept = (long long)(s.k - s.n_gt);
        if (P.bits_key >= 63) {     // structures: the norm for the L2 criterion, else the ranked value itself
            const double v = __longlong_as_double((long long)s.lo_key);
            r.tau_norm = P.crit == CRIT_L2 ? (float)sqrt(v) : (float)v;
        }
    }
    r.n_repaired = 0;      // filled in by the host from the counter once the stream is idle
    r.seed = P.seed;
    c->sel = s;
    c->res = r;
}

// Defined with the projection kernels: the final write with the exact cut-off.
template <int SRC>
__device__ __noinline__ void apply_after_select(const Params &P, int need_h);

// Defined with the single-pass kernels: rewrites one listed unit - an element, or row
// `part` (0..3) of a 4x4 block. `pre_s` / `tdc`, when given, hold the tensors' first unit
// numbers and descriptors in shared memory (no global loads for the owner search).
template <int SRC>
__device__ __noinline__ void repair_unit(const Params &P, u64 idx, u64 id, bool keep, int part, const long long *pre_s,
                                         const TensorDesc *tdc);

// Threads per rewritten unit: a 4 x 4 block is rewritten by four threads, a row each, which keeps
// the dependent chain of one rewrite short; a bh x bw block by eight (rows part, part + 8, ...).
template <int SRC>
struct RepairLanes { static constexpr u32 value = (SRC == SRC_BLOCK) ? 4u : (SRC == SRC_BLOCKG) ? 8u : 1u; };

// Fills the shared-memory copies used by the rewrites (all threads; a barrier must follow).
template <int SRC>
__device__ __forceinline__ void repair_tables(const Params &P, ScanShared &sh, const long long *&pre_s, const TensorDesc *&tdc)
{
    long long *ps = reinterpret_cast<long long *>(sh.hist);
    pre_s = nullptr;
    tdc = nullptr;
    if (P.T <= NBINS / 2) {
        for (int t = threadIdx.x; t < P.T; t += THREADS)
            ps[t] = (SRC == SRC_ELEM) ? P.td[t].elem_prefix : P.td[t].unit_prefix;
        pre_s = ps;
    }
    if (P.T <= REPAIR_TD_CACHE) {
        const int words = P.T * (int)(sizeof(TensorDesc) / sizeof(u32));
        const u32 *src = reinterpret_cast<const u32 *>(P.td);
        u32 *dst = reinterpret_cast<u32 *>(sh.tdc);
        for (int i = threadIdx.x; i < words; i += THREADS) dst[i] = src[i];
        tdc = sh.tdc;
    }
}

// Shared memory of the generic (edge) items of the single-pass kernels: the
// projection items the aligned fast code leaves out (tensor heads and tails,
// unaligned or ragged tensors).
struct FusedShared {
    u32 hist[NBINS];
    u32 cnt[2];
    u64 base[2];
    u64 red[WARPS];
};

// One walk over the candidate list by the whole grid, in chunks strided over the CTAs.
//   gather  units inside the current bracket are copied to the final buffer (to be ranked);
//           otherwise the bracket is one unit, the cut-off, and every entry is decided by it;
//   repair  (single-pass path) a unit whose decision is known by now and differs from the
//           provisional one is rewritten.
// A rewrite is a chain of dependent memory accesses and only a few per cent of the entries
// need one, so a CTA queues them in shared memory while it classifies a chunk and then
// rewrites them, one unit (or block row) per thread. The caller may have fetched this CTA's
// first chunk already (`pre`). Returns this thread's rewrite count.
constexpr int LIST_ROUNDS = 8;                 // list entries per thread and chunk
static_assert(LIST_ROUNDS * THREADS <= WARPS * WSTG, "the queue reuses the staging arrays");

struct ListChunk {
    u64 key[LIST_ROUNDS], id[LIST_ROUNDS];
};

// Entries per thread and chunk for a list of n_list entries: as many as give every CTA of the
// grid one chunk, at most LIST_ROUNDS (a short list is then spread over all CTAs, and so are the
// rewrites it causes).
__device__ __forceinline__ int list_rounds(u64 n_list)
{
    const u64 per = (n_list + (u64)gridDim.x * THREADS - 1) / ((u64)gridDim.x * THREADS);
    return per < 1 ? 1 : per > (u64)LIST_ROUNDS ? LIST_ROUNDS : (int)per;
}

__device__ __forceinline__ void load_list_chunk(const Params &P, u64 base, u64 n_list, int rounds, ListChunk &ch)
{
#pragma unroll
    for (int r = 0; r < LIST_ROUNDS; ++r) {
        const u64 i = base + (u64)r * THREADS + threadIdx.x;
        const bool ok = r < rounds && i < n_list;
        ch.key[r] = ok ? __ldcg(&P.list_key[i]) : 0;
        ch.id[r] = ok ? __ldcg(&P.list_id[i]) : 0;
    }
}

template <int SRC>
__device__ __noinline__ u64 list_walk(const Params &P, ScanShared &sh, bool gather, bool repair, u64 n_list,
                                      const ListChunk *pre)
{
    __shared__ u32 s_qn;
    u64 *q_idx = &sh.stg_key[0][0];
    u64 *q_id = &sh.stg_id[0][0];
    const long long *pre_s = nullptr;
    const TensorDesc *tdc = nullptr;
    __syncthreads();
    if (SRC != SRC_ARRAY && repair) repair_tables<SRC>(P, sh, pre_s, tdc);
    Ctl *c = P.ctl;
    const Sel &s = sh.sel;
    const bool sk = s.lo_key == s.hi_key;
    const int rounds = list_rounds(n_list);
    const u64 chunk = (u64)rounds * THREADS;
    constexpr u32 LPU = RepairLanes<SRC>::value;
    u64 fixed = 0;
    bool have_pre = pre != nullptr;
    for (u64 base = (u64)blockIdx.x * chunk; base < n_list; base += (u64)gridDim.x * chunk) {
        if (threadIdx.x == 0) s_qn = 0;
        __syncthreads();
        ListChunk ch;
        if (have_pre) ch = *pre;
        else load_list_chunk(P, base, n_list, rounds, ch);
        have_pre = false;
#pragma unroll
        for (int r = 0; r < LIST_ROUNDS; ++r) {
            const u64 i = base + (u64)r * THREADS + threadIdx.x;
            if (r >= rounds || i >= n_list) continue;
            const u64 key = ch.key[r], id = ch.id[r];
            bool fin;
            if (gather) {
                const bool above = key > s.hi_key || (sk && key == s.hi_key && id < s.lo_id);
                const bool below = key < s.lo_key || (sk && key == s.lo_key && id > s.hi_id);
                if (!above && !below) {
                    const u32 pos = atomicAdd(&c->fin_count, 1u);
                    if (pos < FIN) { P.fin_key[pos] = key; P.fin_id[pos] = id; P.fin_idx[pos] = i; }
                    continue;
                }
                fin = above;
            } else {
                fin = keep_by_cutoff(key, id, s.lo_key, s.lo_id);
            }
            if (SRC != SRC_ARRAY && repair && fin != (key >= s.guess)) {
                const u32 pos = atomicAdd(&s_qn, 1u);
                q_idx[pos] = i;
                q_id[pos] = id | (fin ? (1ull << 63) : 0ull);
            }
        }
        __syncthreads();
        if (SRC != SRC_ARRAY && repair) {
            const u32 qn = s_qn;
            for (u32 j = threadIdx.x; j < qn * LPU; j += THREADS) {
                const u32 e = j / LPU;
                const u64 packed = q_id[e];
                repair_unit<SRC>(P, q_idx[e], packed & ~(1ull << 63), (packed >> 63) != 0, (int)(j % LPU), pre_s, tdc);
                fixed += (j % LPU) == 0 ? 1 : 0;
            }
        }
        __syncthreads();
    }
    return fixed;
}

// First pass of a ranking call that does not go for the single pass: a plain
// (non-cooperative) scan at full grid.
template <int SRC>
__global__ void __launch_bounds__(THREADS) k_scan(Params P, int do_list)
{
    __shared__ ScanShared sh;
    if (threadIdx.x == 0) sh.sel = P.ctl->sel;
    __syncthreads();
    scan_source<SRC>(P, sh, do_list != 0, sh.sel.slot);
}

// Cooperative driver: picks, further scans, direct ranking of the last few,
// result record. Entered with the histogram of the first scan in slot 0.
// `pre_scan`: no scan kernel ran before this launch (the call went for the single
// pass); if the sample advised against it, the first full histogram pass is
// made here. `post_apply` (1, or 2 when the 16-bit codes are needed): no
// projection kernel follows this launch; after such a fall-back the final write
// is made here too, on the projection work items `prefix_b` / `n_items_b`.
// `do_init`: nothing ran before this launch at all: the histograms and counters are
// cleared and the initial state `init` is installed here first (the one-launch
// route of lists small enough to stay in the L2 between the passes).
template <int SRC>
__global__ void __launch_bounds__(THREADS) k_select(Params P, int first_listed, int pre_scan,
                                                    const long long *prefix_b, long long n_items_b, int post_apply,
                                                    int do_init, Sel init)
{
    __shared__ ScanShared sh;
    __shared__ int s_skip_pick;
    cg::grid_group grid = cg::this_grid();
    const u64 max_key = (P.bits_key >= 63) ? 0x7FFFFFFFFFFFFFFFull : ((1ull << P.bits_key) - 1ull);
    if (do_init) {
        for (int i = blockIdx.x * THREADS + threadIdx.x; i < 3 * NBINS; i += gridDim.x * THREADS) P.hist[i] = 0;
        if (blockIdx.x == 0 && threadIdx.x == 0) init_ctl(P.ctl, init);
        __threadfence();
        grid.sync();
    }
    if (threadIdx.x == 0) {
        if (do_init) sh.sel = init; else sh.sel = P.ctl->sel;
        if (!do_init && P.ctl->async_error) { sh.sel.error = 12; sh.sel.done = 1; }   // a bulk copy never arrived
    }
    __syncthreads();
    if (pre_scan && !sh.sel.onepass && !sh.sel.done) {
        scan_source<SRC>(P, sh, first_listed != 0, sh.sel.slot);
        grid.sync();
    }
    bool src_scan = true, have_pre = false;
    u64 fixed = 0;
    ListChunk pre;
    if (sh.sel.onepass && !sh.sel.done) {
        // single-pass path: this CTA's first chunk of the list is fetched while the pick is made
        const u64 n_all = __ldcg(&P.ctl->list_count[0]);
        if (n_all <= P.cap) {
            const int rounds = list_rounds(n_all);
            load_list_chunk(P, (u64)blockIdx.x * rounds * THREADS, n_all, rounds, pre);
            have_pre = true;
        }
    }
    if (!sh.sel.done) {
        if ((first_listed || sh.sel.onepass) && threadIdx.x == 0) sh.sel.list_valid = 1;
        __syncthreads();
        for (int it = 0; it < MAX_SELECT_ITERS + 2; ++it) {
            // a listing scan that overflowed the list does not count
            if (threadIdx.x == 0) {
                s_skip_pick = 0;
                if (sh.sel.list_valid && __ldcg(&P.ctl->list_count[sh.sel.list_sel]) > P.cap) {
                    sh.sel.list_valid = 0;
                    if (sh.sel.onepass) {
                        if (P.miss_fallback) {
                            // more candidates than the sample predicted: like a missed bracket,
                            // start over on the full key range with a scan of the source
                            Sel &f = sh.sel;
                            f.onepass = 0; f.sampled = 0;
                            f.lo_key = 0; f.hi_key = max_key; f.lo_id = 0; f.hi_id = f.S - 1;
                            f.n_above = 0; f.above_known = 1; f.pop = f.S;
                            set_shift(f);
                            s_skip_pick = 1;
                        } else {
                            sh.sel.error = 11; sh.sel.done = 1;
                        }
                    }
                }
            }
            __syncthreads();
            if (sh.sel.done) break;
            if (!s_skip_pick) {
                block_pick(P, sh, src_scan, max_key, true);
                // clear the histogram slot that the scan after the next one will use
                if (blockIdx.x == 0) {
                    const int z = (sh.sel.slot + 2) % 3;
                    for (int i = threadIdx.x; i < NBINS; i += THREADS) P.hist[(size_t)z * NBINS + i] = 0;
                    if (threadIdx.x == 0) P.ctl->scan_above[z] = 0;
                }
            }
            if (sh.sel.done) break;
            if (sh.sel.list_valid && sh.sel.pop <= FIN) {
                // gather the bracket members from the list, then rank them
                const u64 n_list = __ldcg(&P.ctl->list_count[sh.sel.list_sel]);
                (void)list_walk<SRC>(P, sh, true, false, n_list, (it == 0 && have_pre) ? &pre : nullptr);
                __threadfence();
                grid.sync();
                const u32 n = __ldcg(&P.ctl->fin_count);
                if (threadIdx.x == 0 && (u64)n != sh.sel.pop) sh.sel.error = 9;
                __syncthreads();
                if (!sh.sel.error) final_rank(P, sh, n);
                break;
            }
            // next scan
            if (threadIdx.x == 0) sh.sel.slot = (sh.sel.slot + 1) % 3;
            __syncthreads();
            if (sh.sel.list_valid) {
                scan_list(P, sh, sh.sel.slot, __ldcg(&P.ctl->list_count[sh.sel.list_sel]));
                src_scan = false;
            } else {
                const bool do_list = sh.sel.pop <= P.cap;
                if (do_list && threadIdx.x == 0) sh.sel.list_sel = 1;
                __syncthreads();
                scan_source<SRC>(P, sh, do_list, sh.sel.slot);
                if (do_list && threadIdx.x == 0) sh.sel.list_valid = 1;
                __syncthreads();
                src_scan = true;
            }
            grid.sync();
        }
    }
    if constexpr (SRC != SRC_ARRAY) {
        if (sh.sel.onepass && !sh.sel.error && sh.sel.k > 0) {
            __syncthreads();
            // The cut-off is known: every listed unit whose provisional decision was wrong is
            // rewritten now. This comes last on purpose: the rewrites read w from DRAM, which is
            // still busy taking the single pass's writes out of the L2 when this kernel starts;
            // the pick, the gather and the ranking before it work out of the L2.
            fixed += list_walk<SRC>(P, sh, false, true, __ldcg(&P.ctl->list_count[0]), nullptr);
        }
        if (fixed) atomicAdd(&P.ctl->n_repaired, fixed);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) write_result(P, sh.sel);
    if constexpr (SRC != SRC_ARRAY) {
        if (post_apply && !sh.sel.onepass) {       // the same on every CTA: all derive the state from the same global data
            __threadfence();
            grid.sync();
            Params Pb = P;
            Pb.item_prefix = prefix_b;
            Pb.n_items = n_items_b;
            apply_after_select<SRC>(Pb, post_apply == 2);
        }
    }
}

// Start of every ranking call: clears the histograms and counters and installs
// the initial selection state.
__global__ void __launch_bounds__(THREADS) k_init(Params P, Sel init)
{
    const int n = 3 * NBINS;
    for (int i = blockIdx.x * THREADS + threadIdx.x; i < n; i += gridDim.x * THREADS) P.hist[i] = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) init_ctl(P.ctl, init);
}

}  // namespace cs
