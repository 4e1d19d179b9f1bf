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
constexpr int SEG = 512;                 // filter norm segment (elements): one batch of four 128-bit loads per lane,
                                         // and enough segments that the last round of the grid hardly matters
constexpr int LOG_NBINS = 11;
constexpr int NBINS = 1 << LOG_NBINS;    // histogram bins per selection pass
constexpr int FIN = 4096;                // bracket population finished by ranking in shared memory
constexpr int WSTG = 256;                // staged list entries per warp
constexpr int MAX_SELECT_ITERS = 24;
constexpr u64 KEY_NONE = ~0ull;          // cut-off key that keeps nothing

enum { OP_PRUNE = 0, OP_FILTER = 1, OP_BLOCK = 2, OP_QUANTIZE = 3, OP_LAGRANGE = 4, OP_BLOCKGEN = 5,
       OP_BLOCKG1 = 6 };      // OP_BLOCKG1: bh x bw blocks of matrices by the single-pass kernels
enum { FUSE_FP16 = 1, FUSE_LAMBDA = 2, FUSE_PENALTY = 4, FUSE_BF16 = 8, FUSE_E4M3 = 16, FUSE_E5M2 = 32, NO_SAMPLING = 64 };
constexpr unsigned FUSE_QUANT = FUSE_FP16 | FUSE_BF16 | FUSE_E4M3 | FUSE_E5M2;
constexpr unsigned FUSE_KERNEL_BITS = 63u;      // the fuse bits the kernels see
enum { SRC_ELEM = 0, SRC_BLOCK = 1, SRC_ARRAY = 2, SRC_BLOCKG = 3 };    // SRC_BLOCKG: bh x bw blocks of matrices
enum { CRIT_L2 = 0, CRIT_L1 = 1, CRIT_MAX = 2 };

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
    int bh, bw;              // general block pruning of matrices: block height and width
    int nd;                  // general n-D block pruning: dimensions cut (2: the fields above serve)
    int sh[4], bs[4], nb[4]; // ... extents, block extents and blocks per dimension, right-aligned to four
    int tile_rows;           // tiled bh x bw kernel: block rows of one tile of this tensor (set by the host)
};
static_assert(sizeof(TensorDesc) % 8 == 0, "descriptor tables are copied word by word");

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
    int crit;                       // structured pruning: value a structure is ranked by (CRIT_*)
    int miss_fallback;              // a missed sample bracket may be repaired by the two-pass route inside the
                                    // same call: nothing the first pass wrote is needed again (no multiplier
                                    // is updated in place)
    int jr_floats;                  // journal floats per listed unit (1, 16, or bh * bw of the call)
    int bt_arr_bytes;               // tiled bh x bw kernel: bytes of w (or lambda) one tile buffer holds ...
    int bt_stages;                  // ... and the number of tile buffers
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

// The same for bh x bw blocks: complete block rows of an aligned matrix, when one block row
// (bh matrix rows) fits a tile buffer of `arr_bytes` bytes per array. (Tiles that are column
// chunks of a block row were measured too: the time of a tile hardly depends on its size, so
// twice as many tiles took twice as long, more than the route over the norm array.)
__host__ __device__ inline long long blockg_fast_end(const TensorDesc &d, int arr_bytes)
{
    if (!d.ranked || !d.blk_vec_ok || d.numel >= 0xFFFFFFFFll) return 0;
    if ((long long)d.bh * d.d1 * 4 > (long long)arr_bytes) return 0;
    return (d.d0 / d.bh) * d.nbc;
}

__host__ __device__ inline bool blockg_item_is_fast(const TensorDesc &d, long long local, int arr_bytes)
{
    return d.ranked && (local + 1) * BLOCKS_PER_ITEM <= blockg_fast_end(d, arr_bytes);
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

// Quantisation of theta named by the fuse bits: 0 none, 1 binary16, 2 bfloat16, 3 E4M3, 4 E5M2.
__device__ __forceinline__ int quant_code(unsigned fuse)
{
    return (fuse & FUSE_E5M2) ? 4 : (fuse & FUSE_E4M3) ? 3 : (fuse & FUSE_BF16) ? 2 : (fuse & FUSE_FP16) ? 1 : 0;
}

// binary32 -> 8-bit floating point (fmt 0: E4M3, bias 7, no infinity, largest finite 448;
// fmt 1: E5M2, bias 15, largest finite 57344), round to nearest even, saturating: what
// rounds beyond the largest finite value, infinity included, becomes that value; NaN
// becomes S.1111111. In the normal range the fraction is rounded by one integer addition
// (a carry runs into the exponent, as it should) and the exponent rebiased; below the
// smallest normal one IEEE addition of the power of two whose unit in the last place is
// the smallest subnormal does the rounding, and the low bits of the sum are the code.
__device__ __forceinline__ unsigned short f32_to_fp8_bits(float x, int fmt)
{
    const u32 b = __float_as_uint(x), a = b & 0x7FFFFFFFu, sign = (b >> 24) & 0x80u;
    if (a > 0x7F800000u) return (unsigned short)(sign | 0x7Fu);
    const int drop = fmt ? 21 : 20;                               // fraction bits that go
    const u32 maxcode = fmt ? 0x7Bu : 0x7Eu;
    const u32 min_normal = fmt ? 0x38800000u : 0x3C800000u;       // 2^-14, 2^-6
    u32 q;
    if (a >= min_normal) {
        const u32 r = a + ((1u << (drop - 1)) - 1u) + ((a >> drop) & 1u);
        q = (r - ((fmt ? 112u : 120u) << 23)) >> drop;
        if (q > maxcode) q = maxcode;
    } else {
        const float magic = fmt ? 128.0f : 16384.0f;              // 2^7, 2^14: ulp 2^-16, 2^-9
        q = __float_as_uint(__fadd_rn(__uint_as_float(a), magic)) - __float_as_uint(magic);
    }
    return (unsigned short)(sign | q);
}

// 8-bit floating point -> binary32, exact: the code's bits, moved to the place of a binary32
// exponent and fraction, times the power of two between the two exponent biases (this also
// turns the format's subnormals into the right values).
__device__ __forceinline__ float fp8_bits_to_f32(unsigned short h, int fmt)
{
    const u32 mag = (u32)h & 0x7Fu, sign = ((u32)h & 0x80u) << 24;
    if (fmt == 0 && mag == 0x7Fu) return __uint_as_float(sign | 0x7FC00000u);
    if (fmt == 1 && mag >= 0x7Cu) return __uint_as_float(sign | 0x7F800000u | (mag > 0x7Cu ? 0x400000u : 0u));
    const float f = __fmul_rn(__uint_as_float(mag << (fmt ? 21 : 20)), fmt ? 5.192296858534828e33f : 1.329227995784916e36f);   // 2^112, 2^120
    return __uint_as_float(__float_as_uint(f) | sign);
}

// Code and widened value for quantisation q (1..4) of x.
__device__ __forceinline__ unsigned short quant_bits(float x, int q)
{
    return q == 1 ? f32_to_f16_bits(x) : q == 2 ? f32_to_bf16_bits(x) : f32_to_fp8_bits(x, q - 3);
}
__device__ __forceinline__ float quant_widen(unsigned short h, int q)
{
    return q == 1 ? f16_bits_to_f32(h) : q == 2 ? bf16_bits_to_f32(h) : fp8_bits_to_f32(h, q - 3);
}

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
    const int q = quant_code(fuse);
    unsigned short hb = keep ? quant_bits(u, q ? q : 1) : (unsigned short)0;
    float th = keep ? (q ? quant_widen(hb, q) : u) : 0.0f;
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
        const unsigned short hb = keep ? quant_bits(u, q ? q : 1) : (unsigned short)0;
        o.th = hb;
        if (q) th = keep ? quant_widen(hb, q) : 0.0f;
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
    if (q >= 2) {        // bfloat16 and the 8-bit formats: integer rounding, NaN included
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = quant_bits(x[j], q);
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
    if (q >= 2) {
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = quant_widen(h[j], q);
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

// One element's contribution to the value a structure is ranked by, and the combination of
// two partial values (sums for the norms, the larger one for the maximum; a NaN stays).
__device__ __forceinline__ double crit_add(double acc, float u, int crit)
{
    const double x = (double)u;
    if (crit == CRIT_L2) return __fma_rn(x, x, acc);         // x*x is exact in fp64: (acc + x*x) rounded once
    const double a = fabs(x);
    if (crit == CRIT_L1) return __dadd_rn(acc, a);
    return (a > acc || a != a) ? a : acc;
}
__device__ __forceinline__ double crit_join(double a, double b, int crit)
{
    if (crit != CRIT_MAX) return __dadd_rn(a, b);
    return (b > a || b != b) ? b : a;
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

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start before the kernel ahead of it in the stream has finished; pdl_wait() returns when that
// kernel has completed and its writes are visible (a no-op for a normal launch);
// pdl_launch_dependents() lets the kernel behind start as early as resources allow.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ int bit_length(u64 x) { return x ? 64 - __clzll((long long)x) : 0; }

}  // namespace cs
