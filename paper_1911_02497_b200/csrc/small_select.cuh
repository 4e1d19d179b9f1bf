// Exact selection on a short key array in one CTA.
//
// Filter, neuron and general block pruning rank a few thousand structures: the
// keys (fp64 bit patterns of nu) already sit in an array. For such sizes the
// grid-wide machinery (start kernel, scan, cooperative select) is all launch and
// barrier latency, so one 1024-thread CTA does the whole job in shared memory:
// most-significant-digit-first radix passes over the keys until the rank-k key
// is the only one left in its bin (or all 63 bits are fixed), then the counts
// around it and, among equal keys, the index-order tie rule. The outcome (cut-off,
// record, final selection state) is what k_select would have produced.
#pragma once
#include "common.cuh"
#include "select.cuh"
#include "structured.cuh"

namespace cs {

constexpr int SMALL_THREADS = 1024;
constexpr int SMALL_S_MAX = 16384;       // keys held in shared memory (128 KB)

constexpr int SMALL_T_CACHE = 512;       // tensors whose ranges are cached in shared memory

struct SmallShared {
    long long t_units[SMALL_T_CACHE + 1];  // first structure of every tensor (+ total)
    long long t_items[SMALL_T_CACHE];      // first partial sum of every tensor
    int t_nseg[SMALL_T_CACHE];             // partial sums per filter
    u32 hist[NBINS];
    u32 wsum[SMALL_THREADS / 32];
    u32 pick_bin, pick_before, pick_count;
    u64 tau;
    u32 tau_id;
    u32 n_gt, n_tie;
};

// Inclusive scan of one u32 per thread over the CTA; returns the exclusive value.
__device__ __forceinline__ u32 small_excl_scan(u32 v, u32 *wsum)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u32 inc = v;
    for (int o = 1; o < 32; o <<= 1) {
        const u32 y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    __syncthreads();                       // wsum may still be read from an earlier call
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    u32 base = 0;
    for (int i = 0; i < warp; ++i) base += wsum[i];
    return base + inc - v;
}

// `combine`: the keys are first formed from the filter partial sums (and stored
// to the key array, which the projection reads).
__global__ void __launch_bounds__(SMALL_THREADS) k_select_small(Params P, Sel init, int combine)
{
    extern __shared__ __align__(16) u64 skey[];        // [S]
    __shared__ SmallShared sh;
    Ctl *c = P.ctl;
    pdl_launch_dependents();
    pdl_wait();                     // the partial sums (or the value array) of the kernel ahead
    const u32 S = (u32)init.S;
    if (combine && P.T <= SMALL_T_CACHE) {
        // tensor ranges first (one round trip), then every key needs only its partial sums
        for (int t = threadIdx.x; t < P.T; t += SMALL_THREADS) {
            const TensorDesc &d = P.td[t];
            sh.t_units[t] = d.unit_prefix;
            sh.t_items[t] = P.item_prefix[t];
            sh.t_nseg[t] = (int)((d.d1 + SEG - 1) / SEG);
        }
        if (threadIdx.x == 0) sh.t_units[P.T] = (long long)S;
        __syncthreads();
        for (u32 i = threadIdx.x; i < S; i += SMALL_THREADS) {
            int lo = 0, hi = P.T - 1;          // the tensor with t_units[t] <= i < t_units[t + 1]
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (sh.t_units[mid] <= (long long)i) lo = mid; else hi = mid - 1;
            }
            while (lo > 0 && sh.t_units[lo + 1] == sh.t_units[lo]) --lo;      // tensors without ranked structures
            const int nseg = sh.t_nseg[lo];
            const double *p = P.partial + sh.t_items[lo] + ((long long)i - sh.t_units[lo]) * nseg;
            double acc = 0.0;
            for (int sgm = 0; sgm < nseg; ++sgm) acc = crit_join(acc, p[sgm], P.crit);      // segment order, as k_filter_combine
            const u64 key = (u64)__double_as_longlong(acc);
            P.arr_key[i] = key;
            skey[i] = key;
        }
    } else if (combine) {
        for (u32 i = threadIdx.x; i < S; i += SMALL_THREADS) {
            const u64 key = filter_norm_key(P, (long long)i);
            P.arr_key[i] = key;
            skey[i] = key;
        }
    } else {
        for (u32 i = threadIdx.x; i < S; i += SMALL_THREADS) skey[i] = P.arr_key[i];
    }
    if (threadIdx.x == 0) {
        // what the start kernel of the general path does
        c->tau_key = KEY_NONE;
        c->tau_id = 0;
        c->scan_above[0] = c->scan_above[1] = c->scan_above[2] = 0;
        c->list_count[0] = init.S;         // every unit counts as a candidate here
        c->list_count[1] = 0;
        c->fin_count = 0;
        c->n_repaired = 0;
        c->sample_done = 0;
        c->async_error = 0;
    }
    __syncthreads();
    if (init.done) {                       // nothing to rank (k == 0 or S == 0)
        if (threadIdx.x == 0) write_result(P, init);
        return;
    }
    // ---- the key of rank k (1-based, largest first) ----
    u64 prefix = 0, prefix_mask = 0;       // bits fixed so far
    u32 r = (u32)init.k;                   // rank among the keys that match the prefix
    int passes = 0;
    bool unique = false;
    for (int top = 63; top > 0 && !unique; top -= LOG_NBINS) {
        const int bits = top >= LOG_NBINS ? LOG_NBINS : top;
        const int shift = top - bits;
        const u32 dmask = (1u << bits) - 1u;
        for (int i = threadIdx.x; i < NBINS; i += SMALL_THREADS) sh.hist[i] = 0;
        __syncthreads();
        for (u32 i = threadIdx.x; i < S; i += SMALL_THREADS) {
            const u64 key = skey[i];
            if ((key & prefix_mask) == prefix) atomicAdd(&sh.hist[(u32)(key >> shift) & dmask], 1u);
        }
        __syncthreads();
        // bins in descending digit order, two per thread
        const u32 c0 = sh.hist[NBINS - 1 - 2 * threadIdx.x], c1 = sh.hist[NBINS - 2 - 2 * threadIdx.x];
        const u32 excl = small_excl_scan(c0 + c1, sh.wsum);
        if (r > excl && r <= excl + c0) { sh.pick_bin = NBINS - 1 - 2 * threadIdx.x; sh.pick_before = excl; sh.pick_count = c0; }
        else if (r > excl + c0 && r <= excl + c0 + c1) { sh.pick_bin = NBINS - 2 - 2 * threadIdx.x; sh.pick_before = excl + c0; sh.pick_count = c1; }
        __syncthreads();
        prefix |= (u64)sh.pick_bin << shift;
        prefix_mask |= (u64)dmask << shift;
        r -= sh.pick_before;
        unique = sh.pick_count == 1;
        ++passes;
        __syncthreads();
    }
    if (unique && prefix_mask != 0x7FFFFFFFFFFFFFFFull) {
        // one key carries the prefix: it is the cut-off key
        for (u32 i = threadIdx.x; i < S; i += SMALL_THREADS)
            if ((skey[i] & prefix_mask) == prefix) sh.tau = skey[i];
        __syncthreads();
    } else {
        if (threadIdx.x == 0) sh.tau = prefix;
        __syncthreads();
    }
    const u64 tau = sh.tau;
    // ---- counts around it and the tie rule: among equal keys the lower index ranks first ----
    const u32 per = (S + SMALL_THREADS - 1) / SMALL_THREADS;
    const u32 i0 = threadIdx.x * per, i1 = i0 + per < S ? i0 + per : S;
    u32 gt = 0, eq = 0;
    for (u32 i = i0; i < i1; ++i) {
        const u64 key = skey[i];
        gt += key > tau ? 1u : 0u;
        eq += key == tau ? 1u : 0u;
    }
    const u32 gt_excl = small_excl_scan(gt, sh.wsum);
    if (threadIdx.x == SMALL_THREADS - 1) sh.n_gt = gt_excl + gt;
    const u32 eq_excl = small_excl_scan(eq, sh.wsum);
    if (threadIdx.x == SMALL_THREADS - 1) sh.n_tie = eq_excl + eq;
    __syncthreads();
    const u32 q = (u32)init.k - sh.n_gt;               // ties that are kept (>= 1)
    if (q > eq_excl && q <= eq_excl + eq) {
        u32 seen = eq_excl;
        for (u32 i = i0; i < i1; ++i)
            if (skey[i] == tau && ++seen == q) sh.tau_id = i;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        Sel s = init;
        s.passes = passes;
        s.pop = 1;
        if (q < 1 || q > sh.n_tie) {
            s.error = 8;                   // the counts contradict the selected key
        } else {
            s.lo_key = s.hi_key = tau;
            s.lo_id = s.hi_id = sh.tau_id;
            s.n_above = init.k - 1;
            s.n_gt = sh.n_gt;
            s.n_tie = sh.n_tie;
            s.key_fixed = 1;
        }
        s.done = 1;
        s.list_valid = 1;
        write_result(P, s);
    }
}

}  // namespace cs
