// Shared device-side definitions of the C-step kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cooperative_groups.h>
#include <stdint.h>

namespace cs {

typedef unsigned long long u64;
typedef unsigned int u32;

constexpr int THREADS = 256;             // every kernel here runs 256-thread CTAs
constexpr int WARPS = THREADS / 32;
constexpr int GROUPS_PER_ITEM = 1024;    // linear work item = 1024 groups of 4 elements
constexpr int BLOCKS_PER_ITEM = 256;     // block work item = 256 4x4 blocks (one per thread: the smaller the item, the smaller the imbalance of the last round)
constexpr int SEG = 2048;                // filter norm segment (elements)
constexpr int LOG_NBINS = 11;
constexpr int NBINS = 1 << LOG_NBINS;    // histogram bins per selection pass
constexpr int FIN = 4096;                // bracket population finished by ranking in shared memory
constexpr int WSTG = 256;                // staged list entries per warp
constexpr int MAX_SELECT_ITERS = 24;
constexpr u64 KEY_NONE = ~0ull;          // cut-off key that keeps nothing

enum { OP_PRUNE = 0, OP_FILTER = 1, OP_BLOCK = 2, OP_QUANTIZE = 3, OP_LAGRANGE = 4, OP_BLOCKGEN = 5 };
enum { FUSE_FP16 = 1, FUSE_LAMBDA = 2, FUSE_PENALTY = 4, FUSE_BF16 = 8, NO_SAMPLING = 64 };
enum { SRC_ELEM = 0, SRC_BLOCK = 1, SRC_ARRAY = 2 };

// One tensor of the list as the kernels see it.
struct TensorDesc {
    const float *w;
    float *lam;
    float *theta;
    uint8_t *mask;
    float *grad;
    uint16_t *theta_h;
    long long numel;
    long long elem_prefix;   // global index of element 0
    long long unit_prefix;   // global id of this tensor's first ranked structure
    long long n_units;       // ranked structures in this tensor (0: passes through)
    long long d0, d1;        // block: rows, cols.  filter: filters, filter length
    long long nbc;           // block: blocks per block row
    int pad;                 // linear groups start at element -pad (0..3)
    int vec_ok;              // linear path may use 128-bit accesses
    int blk_vec_ok;          // block path may use 128-bit accesses
    int ranked;              // takes part in the ranking of the current call
    int bh, bw;              // general block pruning: block height and width
};

// Device-resident record of one ranking call.
struct Result {
    int status, passes;
    long long n_units, n_zero, n_keep;
    u64 tau_key;
    long long tau_id, n_gt, n_tie, n_tie_kept;
    float tau_norm;
    int sampled;
    long long n_candidates;
    long long n_repaired;
    u64 seed;                // seed of the sample positions this call used
};

// Selection state: the bracket is the set of units whose (key, id) lies in
// [lo_key, hi_key] and, when lo_key == hi_key, also in [lo_id, hi_id]. `n_above`
// units are known to rank before the bracket, so the unit looked for (rank k
// overall, 1-based, larger key first, lower id first) has rank k - n_above in it.
struct Sel {
    u64 lo_key, hi_key, lo_id, hi_id;
    u64 n_above, pop;
    u64 k, S;
    u64 n_gt, n_tie;          // fixed when the key range collapses to one value
    int shift;                // bin = (hi_key - key) >> shift, or (id - lo_id) >> shift
    int slot;                 // histogram buffer the last scan filled
    int list_valid;           // the candidate list covers the bracket
    int list_sel;             // which list counter is live (0: first scan, 1: relist)
    int above_known;          // n_above is exact (else taken from the scan's own count)
    int done, error, passes;
    int key_fixed;            // n_gt / n_tie are set
    int sampled;              // the bracket came from a sample (and held so far)
    int onepass;              // the first pass also writes provisional outputs + journal
    int pad1;
    u64 guess;                // provisional rule of the one-pass path: keep iff key >= guess
};

struct Ctl {
    Sel sel;
    u64 tau_key, tau_id;      // final cut-off: keep iff key > tau_key || (== && id <= tau_id)
    u64 scan_above[3];        // per histogram slot: units above the bracket seen by that scan
    u64 list_count[2];
    u32 fin_count;
    u32 sample_done;          // CTAs of the sample kernel that have finished
    u64 n_repaired;           // one-pass: provisional decisions that had to be rewritten
    int async_error;          // a bounded wait for a bulk copy ran out in the single-pass kernel
    Result res;
};

// Kernel argument block.
struct Params {
    const TensorDesc *td;
    const long long *item_prefix;   // [T+1] work items per tensor (kernel specific)
    int T;
    long long n_items;
    float mu;
    unsigned fuse;
    Ctl *ctl;
    u64 *hist;                      // [3][NBINS]
    u64 *list_key, *list_id;        // [cap]
    u64 cap;
    u64 *fin_key, *fin_id;          // [FIN]
    u64 *arr_key;                   // filter: fp64 bits of nu per structure
    double *partial;                // filter: per segment partial sums
    long long S;                    // ranked units
    int bits_key;                   // width of the key in bits (31 or 63)
    u64 *sample_key;                // [n_sample] keys of the sampled units
    int n_sample;
    float *jr_lam;                  // one-pass journal: original lambda of listed units
                                    // (1 float per element, 16 per block)
    u64 onepass_cap;                // candidates the one-pass path accepts (<= cap)
    u64 seed;                       // sample positions
    const long long *edge_items;    // projection work items the aligned fast kernel skips
    long long n_edge_items;
    u64 *fin_idx;                   // [FIN] list position of each entry of the final buffer
    const long long *tile_prefix;   // [T+1] warp tiles per tensor of the tiled block kernel
    long long n_tiles;
    int miss_fallback;              // a missed sample bracket may be repaired by the two-pass route inside the
                                    // same call: nothing the first pass wrote is needed again (no multiplier
                                    // is updated in place)
};

// Which projection work items the fast single-pass kernels take (host and device
// must agree: the host lists the others for the edge kernel).
__host__ __device__ inline bool elem_item_is_fast(const TensorDesc &d, long long local)
{
    const long long e_first = 4 * (local * GROUPS_PER_ITEM) - d.pad;
    return d.vec_ok && e_first >= 0 && e_first + 4 * GROUPS_PER_ITEM <= d.numel;
}

// Block pruning: the blocks [0, block_fast_end) of a tensor - its complete block rows, when
// the arrays are aligned - are done by the tiled single-pass kernel, the others by generic
// code on the work items that reach beyond that bound (listed by the host).
__host__ __device__ inline long long block_fast_end(const TensorDesc &d)
{
    return (d.ranked && d.blk_vec_ok && d.numel < 0xFFFFFFFFll) ? (d.d0 >> 2) * d.nbc : 0;
}

__host__ __device__ inline bool block_item_is_fast(const TensorDesc &d, long long local)
{
    return d.ranked && (local + 1) * BLOCKS_PER_ITEM <= block_fast_end(d);
}

// ---------------------------------------------------------------- arithmetic
// u = w - lambda / mu as two IEEE fp32 operations.
__device__ __forceinline__ float form_u(float w, float lam, float mu, bool has_lam)
{
    // lambda == +0 gives u = w bit for bit (w - (+0) is w for every w, -0 included); taking
    // that branch also keeps the IEEE division off its slow path for a zero numerator
    if (!has_lam || __float_as_uint(lam) == 0u) return w;
    return __fsub_rn(w, __fdiv_rn(lam, mu));
}

// binary32 -> binary16 bits, round to nearest even; NaN -> quiet NaN, sign kept.
__device__ __forceinline__ unsigned short f32_to_f16_bits(float x)
{
    unsigned short h = __half_as_ushort(__float2half_rn(x));
    if (x != x) h = (unsigned short)(((__float_as_uint(x) >> 16) & 0x8000u) | 0x7E00u);
    return h;
}

// binary16 bits -> binary32, exact.
__device__ __forceinline__ float f16_bits_to_f32(unsigned short h)
{
    float f = __half2float(__ushort_as_half(h));
    if ((h & 0x7FFFu) > 0x7C00u)
        f = __uint_as_float((((u32)h & 0x8000u) << 16) | 0x7F800000u | (((u32)h & 0x3FFu) << 13));
    return f;
}

// binary32 -> bfloat16 bits, round to nearest even; NaN -> quiet NaN, sign kept.
__device__ __forceinline__ unsigned short f32_to_bf16_bits(float x)
{
    const u32 b = __float_as_uint(x);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return (unsigned short)(((b >> 16) & 0x8000u) | 0x7FC0u);
    return (unsigned short)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}

__device__ __forceinline__ float bf16_bits_to_f32(unsigned short h) { return __uint_as_float((u32)h << 16); }

struct Out {
    float theta, lam, grad;
    unsigned short th;
    unsigned char m;
};

// Everything that follows the keep decision for one element.
__device__ __forceinline__ Out finish(float w, float lam, float u, bool keep, float mu,
                                      unsigned fuse, bool has_lam)
{
    Out o;
    const bool bf = (fuse & FUSE_BF16) != 0;
    unsigned short hb = keep ? (bf ? f32_to_bf16_bits(u) : f32_to_f16_bits(u)) : (unsigned short)0;
    float th = keep ? (bf ? bf16_bits_to_f32(hb) : (fuse & FUSE_FP16) ? f16_bits_to_f32(hb) : u) : 0.0f;
    float d = __fsub_rn(w, th);
    float p = __fmul_rn(mu, d);
    float lu = has_lam ? lam : 0.0f;
    if ((fuse & FUSE_LAMBDA) && has_lam) lu = __fsub_rn(lam, p);
    o.theta = th;
    o.th = hb;
    o.m = keep ? 1 : 0;
    o.lam = lu;
    o.grad = __fsub_rn(p, lu);
    return o;
}

// Lean form for the hot kernels: H = the binary16 bits are needed (fp16 fuse or
// a theta_h output); `fp16`, `upd` (update lambda) are warp-uniform flags.
// `q` is the quantisation of theta: 0 none, 1 binary16, 2 bfloat16 (theta_h then holds that type).
template <bool H>
__device__ __forceinline__ Out finish_lean(float w, float lam, float u, bool keep, float mu,
                                           int q, bool upd)
{
    Out o;
    float th = keep ? u : 0.0f;
    o.th = 0;
    if (H) {
        const unsigned short hb = keep ? (q == 2 ? f32_to_bf16_bits(u) : f32_to_f16_bits(u)) : (unsigned short)0;
        o.th = hb;
        if (q == 1) th = keep ? f16_bits_to_f32(hb) : 0.0f;
        if (q == 2) th = keep ? bf16_bits_to_f32(hb) : 0.0f;
    }
    const float p = __fmul_rn(mu, __fsub_rn(w, th));
    const float lu = upd ? __fsub_rn(lam, p) : lam;
    o.theta = th;
    o.m = keep ? 1 : 0;
    o.lam = lu;
    o.grad = __fsub_rn(p, lu);
    return o;
}

// u for four elements; skips the divisions when every lambda is +0 (u == w then).
__device__ __forceinline__ void form_u4(const float *w, const float *l, float mu, bool has_lam, float *u)
{
    const bool nz = has_lam && ((__float_as_uint(l[0]) | __float_as_uint(l[1]) |
                                 __float_as_uint(l[2]) | __float_as_uint(l[3])) != 0u);
    if (__any_sync(0xffffffffu, nz)) {
#pragma unroll
        for (int j = 0; j < 4; ++j) u[j] = has_lam ? __fsub_rn(w[j], __fdiv_rn(l[j], mu)) : w[j];
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) u[j] = w[j];
    }
}

// binary16 bits of four values with the plain hardware conversion; the rare
// NaN (whose sign must be kept) is patched on a side path.
__device__ __forceinline__ void half4(const float *x, unsigned short *h, int q = 1)
{
    if (q == 2) {        // bfloat16: integer rounding, NaN included
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = f32_to_bf16_bits(x[j]);
        return;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) h[j] = __half_as_ushort(__float2half_rn(x[j]));
    const float s = (x[0] + x[1]) + (x[2] + x[3]);
    if (s != s) {        // a NaN among them (or inf - inf): take the exact route
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = f32_to_f16_bits(x[j]);
    }
}

__device__ __forceinline__ void widen4(const unsigned short *h, const float *x, float *o, int q = 1)
{
    if (q == 2) {
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = bf16_bits_to_f32(h[j]);
        return;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = __half2float(__ushort_as_half(h[j]));
    const float s = (x[0] + x[1]) + (x[2] + x[3]);
    if (s != s) {
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = f16_bits_to_f32(h[j]);
    }
}

// splitmix64 output function: position hash of the sampler.
__device__ __forceinline__ u64 mix64(u64 z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27; z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

// Same with theta supplied (multiplier update / penalty gradient only).
__device__ __forceinline__ Out finish_given(float w, float lam, float th, float mu, unsigned fuse,
                                            bool has_lam)
{
    Out o;
    float d = __fsub_rn(w, th);
    float p = __fmul_rn(mu, d);
    float lu = has_lam ? lam : 0.0f;
    if ((fuse & FUSE_LAMBDA) && has_lam) lu = __fsub_rn(lam, p);
    o.theta = th;
    o.th = 0;
    o.m = 1;
    o.lam = lu;
    o.grad = __fsub_rn(p, lu);
    return o;
}

__device__ __forceinline__ u64 key_of_u(float u) { return (u64)(__float_as_uint(u) & 0x7FFFFFFFu); }

__device__ __forceinline__ bool keep_by_cutoff(u64 key, u64 id, u64 tau_key, u64 tau_id)
{
    return key > tau_key || (key == tau_key && id <= tau_id);
}

// Tensor that owns work item `item`: largest t with prefix[t] <= item.
__device__ __forceinline__ int find_tensor(const long long *__restrict__ prefix, int T, long long item)
{
    int lo = 0, hi = T - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (prefix[mid] <= item) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ __forceinline__ int bit_length(u64 x) { return x ? 64 - __clzll((long long)x) : 0; }

}  // namespace cs
