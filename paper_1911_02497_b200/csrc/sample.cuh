// Bracketing the threshold from a random sample of units.
//
// n_sample units at hashed positions (with replacement) are keyed; the last
// CTA to finish reads the keys back and finds a key range [lo0, hi0] that holds
// the sample order statistics at ranks n_sample*p -/+ 9 standard deviations
// (p = k / S). The rank-k unit of the whole population lies in that range
// unless a ~9-sigma event happens, and whether it does is checked exactly
// afterwards from the full pass's counts - the sample only decides how little
// work the exact selection has to do, never the result.
#pragma once
#include <type_traits>
#include "common.cuh"
#include "select.cuh"

namespace cs {

constexpr int SAMPLE_THREADS = 1024;
constexpr int SAMPLE_KEYS_PER_THREAD = 16;          // n_sample = 16384 keys for one CTA ...
constexpr int SAMPLE_KEYS_PER_THREAD_BIG = 32;      // ... 32768 for long unstructured lists (31-bit keys: half the registers)

constexpr int SAMPLE_TD_CACHE = 16;

struct SampleShared {
    u32 hist[NBINS];
    u64 red[32];
    u64 red2[32];
    u64 rank_before[3];
    u32 rank_bin[3];
    u32 last;
    TensorDesc tdc[SAMPLE_TD_CACHE];
};

// Key of unit `unit`. `tdc`, when given, is a copy of the descriptor table in shared memory
// (short tensor lists): the owner search then needs no global loads.
template <int SRC>
__device__ __forceinline__ u64 unit_key(const Params &P, u64 unit, const TensorDesc *tdc)
{
    const TensorDesc *tab = tdc ? tdc : P.td;
    int lo = 0, hi = P.T - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        const long long pre = (SRC == SRC_ELEM) ? tab[mid].elem_prefix : tab[mid].unit_prefix;
        if ((u64)pre <= unit) lo = mid; else hi = mid - 1;
    }
    const TensorDesc &d = tab[lo];
    const bool has_lam = d.lam != nullptr;
    if (SRC == SRC_ELEM) {
        const long long e = (long long)unit - d.elem_prefix;
        if (e < 0 || e >= d.numel) return 0;
        return key_of_u(form_u(d.w[e], has_lam ? d.lam[e] : 0.0f, P.mu, has_lam));
    } else if (SRC == SRC_BLOCKG) {
        const long long b = (long long)unit - d.unit_prefix;
        if (b < 0 || b >= d.n_units) return 0;
        return blockg_key_global(d, b, P.mu);
    } else {
        const long long b = (long long)unit - d.unit_prefix;
        if (b < 0 || b >= d.n_units) return 0;
        BlockData bd;
        float u[16];
        load_block(d, b, bd);
        return block_key(bd, P.mu, has_lam, u);
    }
}

// CTA-wide sum of a u64 (all SAMPLE_THREADS threads).
__device__ __forceinline__ u64 cta_sum(u64 v, u64 *red)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    u64 t = 0;
    for (int i = 0; i < SAMPLE_THREADS / 32; ++i) t += red[i];
    return t;
}

template <int SRC, int KPT>
__global__ void __launch_bounds__(SAMPLE_THREADS) k_sample(Params P, Sel init)
{
    typedef typename std::conditional<SRC == SRC_ELEM, u32, u64>::type KeyT;     // element keys have 31 bits
    __shared__ SampleShared sh;
    Ctl *ctl = P.ctl;
    pdl_launch_dependents();        // the single-pass kernel behind may set itself up meanwhile
    // what the plain start kernel does: clear histograms (all CTAs share the work)
    for (int i = blockIdx.x * SAMPLE_THREADS + threadIdx.x; i < 3 * NBINS; i += gridDim.x * SAMPLE_THREADS)
        P.hist[i] = 0;
    // the sampling itself is spread over many CTAs (few threads each) so that the
    // random reads of one SM do not queue behind each other
    const TensorDesc *tdc = nullptr;
    if (P.T <= SAMPLE_TD_CACHE) {
        const int words = P.T * (int)(sizeof(TensorDesc) / sizeof(u32));
        const u32 *src = reinterpret_cast<const u32 *>(P.td);
        u32 *dst = reinterpret_cast<u32 *>(sh.tdc);
        for (int i = threadIdx.x; i < words; i += SAMPLE_THREADS) dst[i] = src[i];
        tdc = sh.tdc;
        __syncthreads();
    }
    const int per_cta = (P.n_sample + gridDim.x - 1) / gridDim.x;
    const int j = blockIdx.x * per_cta + threadIdx.x;
    if (threadIdx.x < per_cta && j < P.n_sample) {
        // hashed twice, so that the positions of two seeds are unrelated however close the seeds are
        const u64 unit = __umul64hi(mix64(mix64(P.seed) ^ (u64)j), (u64)P.S);   // uniform on [0, S)
        P.sample_key[j] = unit_key<SRC>(P, unit, tdc);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const u32 prev = atomicAdd(&ctl->sample_done, 1u);
        sh.last = (prev == gridDim.x - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (!sh.last) return;
    __threadfence();

    // ---- last CTA: bracket from the sample ----
    const int m = P.n_sample;
    KeyT key[KPT];
    u64 mn = ~0ull, mx = 0;
#pragma unroll
    for (int q = 0; q < KPT; ++q) {
        const int idx = q * SAMPLE_THREADS + threadIdx.x;
        key[q] = idx < m ? (KeyT)__ldcg(&P.sample_key[idx]) : (KeyT)0;
        if (idx < m) { mn = key[q] < mn ? key[q] : mn; mx = key[q] > mx ? key[q] : mx; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const u64 a = __shfl_xor_sync(0xffffffffu, mn, o), b = __shfl_xor_sync(0xffffffffu, mx, o);
        mn = a < mn ? a : mn; mx = b > mx ? b : mx;
    }
    if ((threadIdx.x & 31) == 0) { sh.red[threadIdx.x >> 5] = mn; sh.red2[threadIdx.x >> 5] = mx; }
    __syncthreads();
    u64 lo = ~0ull, hi = 0;
    for (int i = 0; i < SAMPLE_THREADS / 32; ++i) {
        lo = sh.red[i] < lo ? sh.red[i] : lo;
        hi = sh.red2[i] > hi ? sh.red2[i] : hi;
    }
    __syncthreads();
    const u64 max_key = (P.bits_key >= 63) ? 0x7FFFFFFFFFFFFFFFull : ((1ull << P.bits_key) - 1ull);
    const double p = (double)init.k / (double)init.S;
    const double mp = (double)m * p;
    const double delta = 9.0 * sqrt((double)m * p * (1.0 - p)) + 2.0;
    long long r_hi = (long long)floor(mp - delta), r_lo = (long long)ceil(mp + delta);
    long long r_mid = (long long)floor(mp + 0.5);
    const bool open_top = r_hi < 1, open_bot = r_lo > m;
    if (r_hi < 1) r_hi = 1;
    if (r_lo > m) r_lo = m;
    if (r_mid < 1) r_mid = 1;
    if (r_mid > m) r_mid = m;
    const u64 ranks[3] = {(u64)r_hi, (u64)r_mid, (u64)r_lo};

    u64 above = 0;          // samples ranked before the current range
    int shift = 0;
    u64 hi0 = hi, lo0 = lo, guess = lo;
    for (int pass = 0; pass < 8; ++pass) {
        const int bl = bit_length(hi - lo);
        shift = bl > LOG_NBINS ? bl - LOG_NBINS : 0;
        for (int i = threadIdx.x; i < NBINS; i += SAMPLE_THREADS) sh.hist[i] = 0;
        if (threadIdx.x < 3) { sh.rank_bin[threadIdx.x] = 0; sh.rank_before[threadIdx.x] = 0; }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < KPT; ++q) {
            const int idx = q * SAMPLE_THREADS + threadIdx.x;
            if (idx < m && key[q] >= lo && key[q] <= hi) {
                u64 b = (hi - key[q]) >> shift;
                if (b > NBINS - 1) b = NBINS - 1;
                atomicAdd(&sh.hist[(u32)b], 1u);
            }
        }
        __syncthreads();
        // exclusive scan over bins, two per thread
        const u32 c0 = sh.hist[2 * threadIdx.x], c1 = sh.hist[2 * threadIdx.x + 1];
        u64 inc = (u64)c0 + c1;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (int o = 1; o < 32; o <<= 1) {
            const u64 v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        if (lane == 31) sh.red[warp] = inc;
        __syncthreads();
        u64 wbase = 0;
        for (int i = 0; i < warp; ++i) wbase += sh.red[i];
        const u64 excl = wbase + inc - ((u64)c0 + c1);
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const u64 want = ranks[r] - above;      // ranks lie inside the range by construction
            if (want > excl && want <= excl + c0) { sh.rank_bin[r] = 2 * threadIdx.x; sh.rank_before[r] = excl; }
            else if (want > excl + c0 && want <= excl + c0 + c1) { sh.rank_bin[r] = 2 * threadIdx.x + 1; sh.rank_before[r] = excl + c0; }
        }
        __syncthreads();
        const u32 b_hi = sh.rank_bin[0], b_mid = sh.rank_bin[1], b_lo = sh.rank_bin[2];
        const u64 width = 1ull << shift;
        const u64 e_hi = hi - ((u64)b_hi << shift);                               // upper edge of b_hi
        const u64 lo_edge = hi - ((u64)b_lo << shift);                            // upper edge of b_lo
        const u64 e_lo = (lo_edge - lo >= width - 1) ? lo_edge - (width - 1) : lo;   // lower edge of b_lo
        const u64 mid_edge = hi - ((u64)b_mid << shift);
        const u64 e_mid = (mid_edge - lo >= width - 1) ? mid_edge - (width - 1) : lo;
        hi0 = e_hi; lo0 = e_lo;
        {
            // the guess: inside the bin of the sample's rank m*p, by linear interpolation over the
            // bin's population (a whole bin width of bias would cost as many wrong provisional
            // decisions as the bin holds units of the full list)
            const u64 c_mid = sh.hist[b_mid];
            const u64 pos = ranks[1] - above - sh.rank_before[1];           // 1 .. c_mid, counted from the upper edge
            const u64 span = mid_edge - e_mid;
            const u64 down = c_mid ? (u64)((double)span * (((double)pos - 0.5) / (double)c_mid)) : 0;
            guess = mid_edge - (down > span ? span : down);
        }
        const u64 before_hi = sh.rank_before[0];
        __syncthreads();
        if (b_lo - b_hi >= 16 || shift == 0) break;
        above += before_hi;
        hi = e_hi;
        lo = e_lo;
    }
    if (open_top) hi0 = max_key;
    if (open_bot) lo0 = 0;
    if (guess < lo0) guess = lo0;
    if (guess > hi0) guess = hi0;
    u64 inside = 0;
#pragma unroll
    for (int q = 0; q < KPT; ++q) {
        const int idx = q * SAMPLE_THREADS + threadIdx.x;
        inside += (idx < m && key[q] >= lo0 && key[q] <= hi0) ? 1 : 0;
    }
    inside = cta_sum(inside, sh.red);
    if (threadIdx.x == 0) {
        const double predicted = (double)inside * ((double)init.S / (double)m);
        // written field by field into global memory (the state starts as `init`)
        Sel *d = &ctl->sel;
        *d = init;
        if (2.0 * predicted + 1024.0 <= (double)P.onepass_cap) {
            d->lo_key = lo0;
            d->hi_key = hi0;
            d->guess = guess;
            d->above_known = 0;
            d->sampled = 1;
            d->onepass = 1;
            d->pop = 0;
            const int bl = bit_length(lo0 == hi0 ? init.hi_id - init.lo_id : hi0 - lo0);
            d->shift = bl > LOG_NBINS ? bl - LOG_NBINS : 0;
        }
        ctl->tau_key = KEY_NONE;
        ctl->tau_id = 0;
        ctl->scan_above[0] = ctl->scan_above[1] = ctl->scan_above[2] = 0;
        ctl->list_count[0] = ctl->list_count[1] = 0;
        ctl->fin_count = 0;
        ctl->n_repaired = 0;
        ctl->sample_done = 0;
        ctl->async_error = 0;
    }
}

}  // namespace cs
