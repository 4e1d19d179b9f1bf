// Unstructured pruning of a short list in one cooperative launch, with the list in registers.
//
// A list of at most PS_MAX_ITEMS linear work items (one per CTA: 4096 elements, 16 per thread -
// about 1.2 M parameters on 148 SMs) is read from memory ONCE: every thread keeps its w, lambda
// and u in registers across the grid barriers while the CTAs agree on the threshold by three
// histogram levels over the 31-bit key (11 + 11 + 9 bits, most significant first; shared-memory
// histograms merged into a global one, one grid barrier per level; plain shared-memory atomics:
// electing one lane per bin with match.any was measured slower, here and in the grid-wide scan,
// although the first level is the exponent and most lanes hit a handful of bins), then, only
// if the threshold key is shared by more units than may be kept, by two more levels over the
// index (the tie rule). The projection is written from the same registers. No sample, no
// candidate list, no second read: the configuration-1/2-sized lists are latency, not bandwidth.
#pragma once
#include "common.cuh"
#include "elementwise.cuh"
#include "select.cuh"

namespace cs {

constexpr int PS_ELEMS = 4 * LIN_UNROLL;        // elements a thread holds

struct SmallPruneShared {
    u32 hist[NBINS];
    u64 red[WARPS];
    int pick_bin;
    u64 pick_before, pick_count;
};

// One histogram level. `val[j]` with `live` bit j set takes part when it matches `want` above the
// level's bits; bins are numbered so that a scan in ascending bin order visits the units in
// ranking order (descending keys: desc = true; ascending indices: desc = false). Returns with
// sh.pick_* set for rank r (1-based) and r reduced to the rank inside the picked bin.
template <class V>
__device__ __forceinline__ void ps_level(const Params &P, SmallPruneShared &sh, cg::grid_group &grid, int slot,
                                         const V *val, u32 live, int shift, int bits, V want_above, bool desc, u64 &r)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 nb = 1u << bits;
    for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < PS_ELEMS; ++j) {
        const bool in = ((live >> j) & 1u) && (V)(val[j] >> (shift + bits)) == want_above;
        u32 b = (u32)(val[j] >> shift) & (nb - 1u);
        if (desc) b = nb - 1u - b;
        if (in) atomicAdd(&sh.hist[b], 1u);
    }
    __syncthreads();
    u64 *gh = P.hist + (size_t)slot * NBINS;
    for (int i = threadIdx.x; i < (int)nb; i += THREADS) {
        const u32 h = sh.hist[i];
        if (h) atomicAdd(&gh[i], (u64)h);
    }
    __threadfence();
    grid.sync();
    // every CTA scans the merged histogram and arrives at the same bin
    constexpr int PER = NBINS / THREADS;
    u64 cnt[PER], tsum = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int i = threadIdx.x * PER + j;
        cnt[j] = i < (int)nb ? __ldcg(&gh[i]) : 0;
        tsum += cnt[j];
    }
    u64 inc = tsum;
    for (int o = 1; o < 32; o <<= 1) {
        const u64 v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) sh.red[warp] = inc;
    if (threadIdx.x == 0) sh.pick_bin = -1;
    __syncthreads();
    u64 run = inc - tsum;
    for (int i = 0; i < warp; ++i) run += sh.red[i];
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        if (r > run && r <= run + cnt[j]) {
            sh.pick_bin = threadIdx.x * PER + j;
            sh.pick_before = run;
            sh.pick_count = cnt[j];
        }
        run += cnt[j];
    }
    __syncthreads();
    r -= sh.pick_bin >= 0 ? sh.pick_before : 0;
}

__global__ void __launch_bounds__(THREADS, 2) k_prune_small(Params P, Sel init)
{
    __shared__ SmallPruneShared sh;
    cg::grid_group grid = cg::this_grid();
    const int gsize = gridDim.x * THREADS, gtid = blockIdx.x * THREADS + threadIdx.x;
    // ---- this CTA's work item into registers (the host has made sure there is at most one per CTA)
    const long long item = blockIdx.x;
    const bool has_item = item < P.n_items;
    TensorDesc d;
    memset(&d, 0, sizeof(d));
    long long g0 = 0, g1 = 0;
    if (has_item) {
        const int t = find_tensor(P.item_prefix, P.T, item);
        d = P.td[t];
        const long long ng = (d.numel + d.pad + 3) >> 2;
        g0 = (item - P.item_prefix[t]) * GROUPS_PER_ITEM;
        g1 = (g0 + GROUPS_PER_ITEM < ng) ? g0 + GROUPS_PER_ITEM : ng;
    }
    const bool has_lam = d.lam != nullptr;
    float w[PS_ELEMS], l[PS_ELEMS];
    u32 live = 0, fullm = 0;
#pragma unroll
    for (int it = 0; it < LIN_UNROLL; ++it) {
        const long long g = g0 + it * THREADS + threadIdx.x;
        const long long e0 = 4 * g - d.pad;
        const bool lv = has_item && g < g1;
        const bool full = lv && d.vec_ok && e0 >= 0 && e0 + 4 <= d.numel;
        if (full) {
            const float4 a = ld4_ro(d.w + e0);
            w[4 * it] = a.x; w[4 * it + 1] = a.y; w[4 * it + 2] = a.z; w[4 * it + 3] = a.w;
            if (has_lam) {
                const float4 b = ld4(d.lam + e0);
                l[4 * it] = b.x; l[4 * it + 1] = b.y; l[4 * it + 2] = b.z; l[4 * it + 3] = b.w;
            } else {
                l[4 * it] = l[4 * it + 1] = l[4 * it + 2] = l[4 * it + 3] = 0.0f;
            }
            live |= 0xFu << (4 * it);
            fullm |= 1u << it;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long e = e0 + j;
                const bool ok = lv && e >= 0 && e < d.numel;
                w[4 * it + j] = ok ? d.w[e] : 0.0f;
                l[4 * it + j] = (ok && has_lam) ? d.lam[e] : 0.0f;
                live |= (ok ? 1u : 0u) << (4 * it + j);
            }
        }
    }
    // ---- start of the call: clear the histograms, install the state
    for (int i = gtid; i < 3 * NBINS; i += gsize) P.hist[i] = 0;
    if (gtid == 0) init_ctl(P.ctl, init);
    float u[PS_ELEMS];
    u32 key[PS_ELEMS];
#pragma unroll
    for (int j = 0; j < PS_ELEMS; ++j) {
        u[j] = form_u(w[j], l[j], P.mu, has_lam);
        key[j] = __float_as_uint(u[j]) & 0x7FFFFFFFu;
    }
    __threadfence();
    grid.sync();
    // ---- the key of rank k: three levels, most significant bits first
    const u64 k = init.k, S = init.S;
    u64 tau_key = KEY_NONE, tau_id = 0, n_gt = 0, n_tie = 0;
    bool by_id = false, bad = false;
    int passes = 0;
    if (k > 0 && S > 0) {
        u64 r = k;
        u32 prefix = 0;
        const int shifts[3] = {20, 9, 0}, nbits[3] = {11, 11, 9};
#pragma unroll 1
        for (int lv = 0; lv < 3; ++lv) {
            ps_level<u32>(P, sh, grid, lv, key, live, shifts[lv], nbits[lv], prefix, true, r);
            ++passes;
            if (sh.pick_bin < 0) { bad = true; break; }
            n_gt += sh.pick_before;
            prefix = (prefix << nbits[lv]) | (((1u << nbits[lv]) - 1u) - (u32)sh.pick_bin);
            n_tie = sh.pick_count;
            __syncthreads();
        }
        tau_key = prefix;
        // ---- among the units that carry this key the lowest r indices are kept
        u64 id[PS_ELEMS];
        u32 tie = 0;
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = 4 * it + j;
                id[q] = (u64)(d.elem_prefix + 4 * (g0 + it * THREADS + threadIdx.x) - d.pad + j);
                tie |= (((live >> q) & 1u) && key[q] == (u32)tau_key ? 1u : 0u) << q;
            }
        if (!bad && r < n_tie) {
            // not every tie is kept: the index of rank r among them, two levels over the index
            // (the histogram slots of the first two levels are free again; clear them first)
            by_id = true;
            for (int i = gtid; i < 2 * NBINS; i += gsize) P.hist[i] = 0;
            __threadfence();
            grid.sync();
            const int idbits = bit_length(S - 1);
            const int lo_bits = idbits > 11 ? (idbits - 11 < 11 ? idbits - 11 : 11) : 0;     // second level
            const int hi_shift = lo_bits;
            const int hi_bits = idbits - lo_bits > 0 ? idbits - lo_bits : 1;
            if (hi_bits > 11) bad = true;                           // more than 2^22 units never come here
            u64 idp = 0;
            if (!bad) {
                ps_level<u64>(P, sh, grid, 0, id, tie, hi_shift, hi_bits, (u64)0, false, r);
                ++passes;
                if (sh.pick_bin < 0) bad = true;
                idp = (u64)(sh.pick_bin < 0 ? 0 : sh.pick_bin);
                __syncthreads();
            }
            if (!bad && lo_bits > 0) {
                ps_level<u64>(P, sh, grid, 1, id, tie, 0, lo_bits, idp, false, r);
                ++passes;
                if (sh.pick_bin < 0) bad = true;
                idp = (idp << lo_bits) | (u64)(sh.pick_bin < 0 ? 0 : sh.pick_bin);
                __syncthreads();
            }
            tau_id = idp;
        } else if (!bad) {
            // every unit with this key is kept: the record wants the largest of their indices
#pragma unroll
            for (int q = 0; q < PS_ELEMS; ++q)
                if ((tie >> q) & 1u) atomicMax(&P.ctl->tau_id, id[q]);
        }
    }
    // ---- projection from the registers
    if (has_item) {
        const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
        const bool wr_grad = (P.fuse & FUSE_PENALTY) && d.grad != nullptr;
        const int qc = quant_code(P.fuse);
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) {
            const long long g = g0 + it * THREADS + threadIdx.x;
            if (g >= g1) continue;
            const long long e0 = 4 * g - d.pad;
            Out o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = 4 * it + j;
                bool keep = (u64)key[q] > tau_key;
                if ((u64)key[q] == tau_key) keep = by_id ? (u64)(d.elem_prefix + e0 + j) <= tau_id : true;
                if (bad) keep = false;
                o[j] = finish_lean<true>(w[q], l[q], u[q], keep, P.mu, qc, upd);
            }
            if ((fullm >> it) & 1u) {
                *reinterpret_cast<float4 *>(d.theta + e0) = make_float4(o[0].theta, o[1].theta, o[2].theta, o[3].theta);
                if (d.mask) *reinterpret_cast<u32 *>(d.mask + e0) =
                    (u32)o[0].m | ((u32)o[1].m << 8) | ((u32)o[2].m << 16) | ((u32)o[3].m << 24);
                if (d.theta_h) *reinterpret_cast<uint2 *>(d.theta_h + e0) =
                    make_uint2((u32)o[0].th | ((u32)o[1].th << 16), (u32)o[2].th | ((u32)o[3].th << 16));
                if (upd) *reinterpret_cast<float4 *>(d.lam + e0) = make_float4(o[0].lam, o[1].lam, o[2].lam, o[3].lam);
                if (wr_grad) *reinterpret_cast<float4 *>(d.grad + e0) = make_float4(o[0].grad, o[1].grad, o[2].grad, o[3].grad);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (!((live >> (4 * it + j)) & 1u)) continue;
                    const long long e = e0 + j;
                    d.theta[e] = o[j].theta;
                    if (d.mask) d.mask[e] = o[j].m;
                    if (d.theta_h) d.theta_h[e] = o[j].th;
                    if (upd) d.lam[e] = o[j].lam;
                    if (wr_grad) d.grad[e] = o[j].grad;
                }
            }
        }
    }
    // ---- record (the index of the weakest kept unit is taken from Ctl.tau_id by the host)
    if (gtid == 0) {
        Ctl *c = P.ctl;
        Result res;
        res.status = bad ? -5 : 0;
        res.passes = passes;
        res.n_units = (long long)S;
        res.n_keep = (long long)k;
        res.n_zero = (long long)(S - k);
        res.sampled = 0;
        res.n_candidates = 0;
        res.n_repaired = 0;
        res.seed = P.seed;
        res.tau_norm = 0.0f;
        if (k == 0 || S == 0 || bad) {
            c->tau_key = KEY_NONE;
            res.tau_key = 0x7F800000ull;
            res.tau_id = -1;
            res.n_gt = res.n_tie = res.n_tie_kept = 0;
        } else {
            c->tau_key = tau_key;
            if (by_id) c->tau_id = tau_id;
            res.tau_key = tau_key;
            res.tau_id = by_id ? (long long)tau_id : 0;      // all ties kept: the largest tie index is in Ctl.tau_id
            res.n_gt = (long long)n_gt;
            res.n_tie = (long long)n_tie;
            res.n_tie_kept = (long long)(k - n_gt);
        }
        c->sel.error = bad ? 13 : 0;
        c->res = res;
    }
}

}  // namespace cs
