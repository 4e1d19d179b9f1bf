/*
 * condensa_cstep.h - C ABI of the B200 (sm_100a) C-step library.
 *
 * The C-step of the learning-compression (L-C) scheme (paper Section 3.3): given
 * the current weights w, the multipliers lambda and the penalty weight mu, form
 *
 *      u = w - lambda / mu
 *
 * and replace theta by the compression mapping C(u) = argmin_Theta ||u - D(Theta)||^2
 * (Section 3.3, text under Eq. 1), followed by the augmented-Lagrangian updates
 *
 *      lambda <- lambda - mu (w - theta)          (multiplier update)
 *      g       = mu (w - theta) - lambda          (penalty gradient the L step adds)
 *
 * The compression mappings offered are the paper's pre-built schemes (Table 1):
 * Prune() (unstructured magnitude pruning), FilterPrune (3-D blocks),
 * BlockPrune (2-D blocks), Quantize(float16) and Compose([Prune, Quantize]).
 * One sparsity is applied globally over the whole tensor list (Section 3: the
 * L-C optimizer "distributes this global sparsity across all the layers").
 *
 * Conventions
 *  - Every function returns CONDENSA_OK (0) or a negative CONDENSA_ERR_* code and
 *    never throws. condensa_last_error() gives a text for the last failure of a
 *    context.
 *  - All tensor pointers in condensa_tensor are DEVICE pointers on the context's
 *    device unless a function says "host". They are owned by the caller, must
 *    stay valid until the stream has run the call, are contiguous row-major, and
 *    need only their natural alignment (4 bytes for fp32): 16-byte alignment is
 *    faster but not required.
 *  - Calls are asynchronous and ordered on the `stream` argument (a cudaStream_t
 *    passed as void*; NULL is the legacy default stream). A context's workspace is
 *    shared by its calls: a call on another stream than the previous one first
 *    waits (on the device) for that call's kernels. The library allocates device memory only in
 *    condensa_create() and when a call needs a larger workspace than any call
 *    before it on that context (this synchronises the device once); steady-state
 *    calls allocate nothing and do not synchronise.
 *  - Arguments are checked on the host before anything is launched; on an
 *    argument error no caller buffer has been touched.
 *  - Arithmetic: every fp32 value is produced by single IEEE-754 operations,
 *    round-to-nearest-even, no fused multiply-add, subnormals kept:
 *        q = lambda / mu;  u = w - q;
 *        d = w - theta;    p = mu * d;   lambda' = lambda - p;   g = p - lambda_used
 *    where lambda_used is lambda' when CONDENSA_FUSE_LAMBDA is set and the given
 *    lambda otherwise. Structure norms are accumulated in fp64.
 *  - Ranking: units (elements, filters or blocks) are ordered by key, larger
 *    first, and among equal keys by global index, lower first. With n ranked
 *    units, Z = floor(sparsity * n + 0.5) (computed in double, clamped to [0, n])
 *    units are zeroed: exactly the last Z of that order. "Target sparsity" is the
 *    proportion of zeroed units (Introduction).
 */
#ifndef CONDENSA_CSTEP_H
#define CONDENSA_CSTEP_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define CONDENSA_API __attribute__((visibility("default")))
#else
#define CONDENSA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct condensa_ctx condensa_ctx;   /* opaque: workspace + descriptor cache of one device */

/* One weight tensor of the list. Global element index of element i of tensor t
 * is (sum of numel of tensors before t) + i; structures are numbered the same
 * way, tensor by tensor. */
typedef struct {
    const float *w;       /* in : weights, fp32, never written                              */
    float *lambda;        /* i/o: multipliers, fp32. NULL: treated as 0 and never written    */
    float *theta;         /* out: compressed weights, fp32 (in: for _lagrange_update)        */
    uint8_t *mask;        /* out: 1 byte per element, 1 = in the kept set. NULL: not written */
    float *grad;          /* out: penalty gradient g, fp32, overwritten. NULL: not written   */
    uint16_t *theta_h;    /* out: IEEE binary16 bits of theta. NULL: not written             */
    int64_t numel;        /* number of elements, >= 0                                        */
    int32_t ndim;         /* 1..4; product of shape[0..ndim-1] must equal numel              */
    int64_t shape[4];     /* dim 0 = filters (4-D) or rows (2-D)                             */
} condensa_tensor;

/* `fuse` bits */
enum {
    CONDENSA_FUSE_FP16 = 1,     /* theta = fp16 round-to-nearest-even of kept u, widened back  */
    CONDENSA_FUSE_LAMBDA = 2,   /* update lambda in place                                     */
    CONDENSA_FUSE_PENALTY = 4,  /* write g to grad                                            */
    CONDENSA_FUSE_BF16 = 8,     /* like FUSE_FP16 with bfloat16; theta_h then holds bfloat16 bits  */
    CONDENSA_FUSE_E4M3 = 16,    /* like FUSE_FP16 with the 8-bit format E4M3 (see
                                   condensa_cstep_quantize); theta_h then holds the code in its
                                   low byte                                                     */
    CONDENSA_FUSE_E5M2 = 32,    /* the same with E5M2. At most one of the four types per call   */
    CONDENSA_NO_SAMPLING = 64   /* rank with full histogram passes, then project (two passes over
                                   w and lambda; same results). It also sends rankings of at most
                                   16384 structures (filters, rows, general blocks), which by
                                   default are settled by one CTA in shared memory, through the
                                   grid-wide selection. Default for large inputs is ONE
                                   pass: the threshold is first bracketed from 16384 hashed sample
                                   positions (seed: condensa_set_seed), the pass decides everything
                                   outside the bracket for good and lists the rest, and the exact
                                   selection runs on that list. The bracket is checked exactly
                                   afterwards. Should it miss (probability < 1e-16 for positions
                                   independent of the data), the call falls back to the two-pass
                                   route by itself and returns the exact result whenever the first
                                   pass has not destroyed an input, i.e. unless FUSE_LAMBDA is set
                                   and a tensor has a lambda buffer. In that one case the outputs
                                   of the call are invalid, lambda has been overwritten, and
                                   condensa_get_result() returns CONDENSA_ERR_INTERNAL (CONDENSA_OK
                                   from the call itself is provisional until then) - never silent.
                                   Callers that cannot accept this set CONDENSA_NO_SAMPLING.      */
};

/* return codes */
enum {
    CONDENSA_OK = 0,
    CONDENSA_ERR_INVALID_ARG = -1,   /* bad pointer, size, shape, sparsity, mu, aliasing       */
    CONDENSA_ERR_WORKSPACE = -2,     /* workspace could not be allocated                       */
    CONDENSA_ERR_CUDA = -3,          /* CUDA runtime error, text in condensa_last_error()      */
    CONDENSA_ERR_UNSUPPORTED = -4,   /* dtype or block shape not built                         */
    CONDENSA_ERR_INTERNAL = -5,      /* a device-side consistency check failed (reported by
                                        condensa_get_result)                                   */
    CONDENSA_ERR_TOO_LARGE = -6      /* input larger than a fixed built-in limit               */
};

enum { CONDENSA_DTYPE_FP16 = 1, CONDENSA_DTYPE_BF16 = 2, CONDENSA_DTYPE_FP8_E4M3 = 3, CONDENSA_DTYPE_FP8_E5M2 = 4 };

/* Record of the last ranking call, filled on the device. */
typedef struct {
    int32_t status;        /* CONDENSA_OK or CONDENSA_ERR_INTERNAL                             */
    int32_t passes;        /* histogram passes the selection took (over the source or a list) */
    int64_t n_units;       /* ranked units: elements, filters or blocks                       */
    int64_t n_zero;        /* Z                                                                */
    int64_t n_keep;        /* n_units - Z                                                      */
    uint64_t tau_key;      /* key of the weakest kept unit: bits(|u|) for _prune, the fp64
                              bits of the squared L2 norm for _filter/_block; the bits of
                              +infinity in that format when nothing is kept                   */
    int64_t tau_id;        /* global index of the weakest kept unit, -1 when nothing is kept  */
    int64_t n_gt;          /* units with key  > tau_key                                       */
    int64_t n_tie;         /* units with key == tau_key                                       */
    int64_t n_tie_kept;    /* how many of those are kept (the lowest indices)                 */
    float tau_norm;        /* _filter/_block: (float)sqrt of the weakest kept squared norm    */
    int32_t sampled;       /* 1 when a sample bracket was used and held                       */
    int64_t n_candidates;  /* units that had to be listed for the exact selection             */
    int64_t n_repaired;    /* single-pass path: listed units whose provisional decision was
                              wrong and were rewritten                                        */
    uint64_t seed;         /* seed of the sample positions the call used (condensa_set_seed)  */
} condensa_result;

/* Create a context on CUDA device `device`. workspace_bytes = 0 sizes the
 * workspace on demand; otherwise that much is reserved up front. */
CONDENSA_API int condensa_create(condensa_ctx **out, int device, size_t workspace_bytes);
CONDENSA_API int condensa_destroy(condensa_ctx *ctx);

/* Seed of the hashed sample positions of the single-pass path. Every context draws
 * its own at creation, so that no fixed input can be built against the positions;
 * setting it makes a run reproducible. It never changes a result, only how many
 * units the exact selection has to look at (see CONDENSA_NO_SAMPLING). */
CONDENSA_API int condensa_set_seed(condensa_ctx *ctx, uint64_t seed);

/* Prune() - unstructured magnitude pruning (Table 1; Section 3.3 "pruning").
 * key = bits(u) & 0x7FFFFFFF. theta = u (or fp16(u) with FUSE_FP16: Compose([Prune(),
 * Quantize(float16)]), Evaluation, Objective 1: prune first, then quantise) on the
 * kept set, +0 elsewhere. `tensors` is a HOST array of T entries. */
CONDENSA_API int condensa_cstep_prune(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                         double sparsity, float mu, unsigned fuse, void *stream);

/* FilterPrune - every 4-D tensor is ranked by output filter [f, :, :, :] on the
 * fp64 sum of u^2 (Table 1, "filters (3D blocks)"); `sparsity` is the proportion
 * of filters zeroed. Tensors with ndim != 4 pass through: theta = u, mask = 1. */
CONDENSA_API int condensa_cstep_filter(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                          double sparsity, float mu, unsigned fuse, void *stream);

/* NeuronPrune / StructurePrune (Table 1: neurons are "1D blocks"; StructurePrune
 * "combines neuron and filter pruning"). `kinds` selects the leading-index slices
 * that are ranked together, by the fp64 sum of u^2 like filters:
 *   CONDENSA_STRUCT_FILTER  [f, :, :, :] of every 4-D tensor,
 *   CONDENSA_STRUCT_NEURON  rows [r, :] of every 2-D tensor,
 * or both. Every other tensor passes through. condensa_cstep_filter() is this
 * call with CONDENSA_STRUCT_FILTER. */
enum { CONDENSA_STRUCT_FILTER = 1, CONDENSA_STRUCT_NEURON = 2 };
CONDENSA_API int condensa_cstep_structure(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                                          double sparsity, float mu, int kinds, unsigned fuse,
                                          void *stream);

/* BlockPrune - every 2-D tensor is cut into bh x bw blocks (row-major numbering,
 * blocks that stick out over an edge hold fewer elements) ranked on the fp64 sum
 * of u^2 taken row by row inside the block (Table 1, "n-D blocks of size bs").
 * bh = bw = 4 takes the single-pass kernels, and so do 5 x 5 (the block size of the
 * paper's LSTM run), 3 x 3, 2 x 2, 1 x 8 and 8 x 1 on lists of at least 131072 blocks
 * whose matrices are mostly 16-byte aligned with a width that is a multiple of 4 (the
 * sample-bracket rules of condensa_cstep_prune() then apply: CONDENSA_NO_SAMPLING,
 * result fields `sampled`, `n_candidates`, `n_repaired`). Every other shape with sides
 * up to 4096, and every list the single pass does not take, is ranked in three steps -
 * norms per block, selection on the norm array, elementwise projection - with the same
 * results contract. Tensors with ndim != 2 pass through. */
CONDENSA_API int condensa_cstep_block(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                         double sparsity, float mu, int bh, int bw, unsigned fuse, void *stream);

/* Structured pruning by a specification (Table 1: NeuronPrune(criteria), FilterPrune(criteria),
 * StructurePrune(criteria), BlockPrune(criteria, bs) - "prune based on criteria", blocks of
 * 1, 3 or n dimensions "of size bs"). The calls above are special cases of this one.
 *   kind CONDENSA_SPEC_SLICES  leading-index slices: `kinds` as in condensa_cstep_structure().
 *   kind CONDENSA_SPEC_BLOCKS  every tensor with ndim == spec->ndim is cut into blocks of
 *        block[0] x ... x block[ndim-1] elements, numbered row-major over the grid of blocks;
 *        a block that sticks out over an edge holds fewer elements. Extents up to 4096; tensor
 *        extents below 2^31.
 *   criterion: the value a structure is ranked by, accumulated in fp64 over its elements in
 *        row-major order - CONDENSA_CRIT_L2 the sum of u^2 (the squared L2 norm; this is the
 *        argmin of Section 3.3), CONDENSA_CRIT_L1 the sum of |u|, CONDENSA_CRIT_MAX the largest
 *        |u|. The paper names no criterion; L1 and MAX are the usual alternatives and are not
 *        the projection of Section 3.3. condensa_result.tau_key holds the fp64 bits of the
 *        weakest kept value, tau_norm its square root for L2 and the value itself otherwise.
 * Every other tensor passes through (theta = u, mask = 1). */
enum { CONDENSA_SPEC_SLICES = 0, CONDENSA_SPEC_BLOCKS = 1 };
enum { CONDENSA_CRIT_L2 = 0, CONDENSA_CRIT_L1 = 1, CONDENSA_CRIT_MAX = 2 };
typedef struct {
    int32_t kind;         /* CONDENSA_SPEC_SLICES or CONDENSA_SPEC_BLOCKS              */
    int32_t kinds;        /* SLICES: CONDENSA_STRUCT_FILTER and/or CONDENSA_STRUCT_NEURON */
    int32_t criterion;    /* CONDENSA_CRIT_*                                            */
    int32_t ndim;         /* BLOCKS: number of block extents                            */
    int64_t block[4];     /* BLOCKS: the extents                                        */
} condensa_structure_spec;
CONDENSA_API int condensa_cstep_structured(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                                           double sparsity, float mu, const condensa_structure_spec *spec,
                                           unsigned fuse, void *stream);

/* Quantize(dtype) - theta = round-to-nearest-even of u in `dtype` for every element,
 * mask = 1 (Table 1; Section 2 "low-precision approximation"; Conclusion: further data
 * types for quantization). dtype is
 *   CONDENSA_DTYPE_FP16      IEEE binary16;
 *   CONDENSA_DTYPE_BF16      bfloat16, the upper half of a binary32;
 *   CONDENSA_DTYPE_FP8_E4M3  1 sign, 4 exponent (bias 7), 3 fraction bits, no infinity,
 *                            NaN = S.1111.111, largest finite value 448;
 *   CONDENSA_DTYPE_FP8_E5M2  1 sign, 5 exponent (bias 15), 2 fraction bits, largest
 *                            finite value 57344.
 * theta_h receives the code (16 bits; an 8-bit code in the low byte). Underflow is
 * gradual; NaN becomes a quiet NaN with the same sign. Overflow goes to infinity for the
 * two 16-bit types and SATURATES for the two 8-bit types: whatever rounds beyond the
 * largest finite value, infinity included, becomes that value (an 8-bit codebook with
 * infinities in it would be useless for weights; this is also what the conversion
 * instruction of the GPU does). `fuse` may carry FUSE_LAMBDA / FUSE_PENALTY only. */
CONDENSA_API int condensa_cstep_quantize(condensa_ctx *ctx, const condensa_tensor *tensors, int T, float mu,
                            int dtype, unsigned fuse, void *stream);

/* Multiplier update and/or penalty gradient with theta as given by the caller
 * (augmented-Lagrangian method of the L-C algorithm, Section 3.3). `fuse` is
 * CONDENSA_FUSE_LAMBDA and/or CONDENSA_FUSE_PENALTY. Reads w, theta, lambda. */
CONDENSA_API int condensa_cstep_lagrange_update(condensa_ctx *ctx, const condensa_tensor *tensors, int T,
                                   float mu, unsigned fuse, void *stream);

/* L step helper: the penalty gradient folded into one optimizer step, in a
 * single pass over the list (Section 3.3: the L step trains w "with a quadratic
 * regularization term"; Evaluation, L-C optimizer settings: SGD with momentum
 * 0.9 for the CNNs, Adam for the LSTM; it runs on every minibatch). With `grad`
 * the loss gradient of the minibatch, per element and in this order of single
 * fp32 operations:
 *     d = w - theta;  p = mu*d;  g1 = p - lambda;  g = grad + g1;  [g = g + weight_decay*w]
 *   SGD :  b' = momentum*b + g;                     w' = w - lr*b'
 *   Adam:  m' = beta1*m + (1-beta1)*g;  v' = beta2*v + (1-beta2)*(g*g);
 *          w' = w - (lr/(1-beta1^step)) * ( m' / ( sqrt(v')/sqrt(1-beta2^step) + eps ) )
 * (1-beta in fp32; the two bias corrections in double, rounded once to fp32.)
 * w, buf1 (b or m) and buf2 (v) are updated in place; theta, lambda (NULL: 0) and
 * grad are read. buf1 may be NULL for SGD with momentum == 0. All DEVICE pointers. */
typedef struct {
    float *w;
    const float *theta;
    const float *lambda;
    const float *grad;
    float *buf1;
    float *buf2;
    int64_t numel;
} condensa_opt_tensor;

enum { CONDENSA_OPT_SGD = 0, CONDENSA_OPT_ADAM = 1 };

typedef struct {
    int32_t kind;          /* CONDENSA_OPT_SGD or CONDENSA_OPT_ADAM */
    float lr, momentum, weight_decay, beta1, beta2, eps;
    int64_t step;          /* Adam: 1-based step number */
} condensa_opt;

CONDENSA_API int condensa_lstep_update(condensa_ctx *ctx, const condensa_opt_tensor *tensors, int T,
                                       float mu, const condensa_opt *opt, void *stream);

/* Operation selector for condensa_cstep_host(). */
enum { CONDENSA_OP_PRUNE = 0, CONDENSA_OP_FILTER = 1, CONDENSA_OP_BLOCK = 2,
       CONDENSA_OP_QUANTIZE = 3, CONDENSA_OP_LAGRANGE = 4 };

/* Same operations for weights that live in HOST memory: every pointer in
 * `tensors` is a host pointer (pinned memory makes the copies asynchronous).
 * The call copies w and lambda (and theta for CONDENSA_OP_LAGRANGE) to device
 * buffers the context keeps, runs the operation there, copies every non-NULL
 * output back and returns after the stream has finished. bh/bw are read for
 * CONDENSA_OP_BLOCK only, sparsity for the three pruning operations. */
CONDENSA_API int condensa_cstep_host(condensa_ctx *ctx, int op, const condensa_tensor *tensors, int T,
                        double sparsity, float mu, int bh, int bw, unsigned fuse, void *stream);

/* Workspace a context needs for calls of a given shape, so that condensa_create() can
 * reserve it and no call allocates later: `op` is a CONDENSA_OP_* value (PRUNE, FILTER,
 * BLOCK, QUANTIZE, LAGRANGE), `tensors` / `T` the list (only numel, ndim, shape and the
 * alignment of the pointers are looked at), `spec` the structure specification of a
 * structured call (NULL: filters resp. 4 x 4 blocks by the L2 norm), `fuse` as for the
 * call. Writes the byte count to *bytes. Host only; nothing is launched. */
CONDENSA_API int condensa_workspace_bytes(int op, const condensa_tensor *tensors, int T,
                                          const condensa_structure_spec *spec, unsigned fuse, size_t *bytes);

/* Waits for the stream of the last ranking call and copies its record. */
CONDENSA_API int condensa_get_result(condensa_ctx *ctx, condensa_result *out);

/* Per-kernel device time. While enabled, every kernel launch of this context is
 * bracketed by a pair of CUDA events on its stream (this adds a little latency
 * between kernels, so enable it only to measure). condensa_profile_read() waits
 * for the recorded events and returns, per kernel name, the launches and the
 * summed event time since profiling was enabled. `out` is a HOST array. */
typedef struct {
    char name[48];
    int64_t launches;
    double total_ms;
} condensa_kernel_time;
CONDENSA_API int condensa_profile_enable(condensa_ctx *ctx, int on);
CONDENSA_API int condensa_profile_read(condensa_ctx *ctx, condensa_kernel_time *out, int max_entries,
                                       int *n_out);

/* Number of kernels this context has launched so far. */
CONDENSA_API int64_t condensa_launch_count(const condensa_ctx *ctx);

/* ---- Network thinning (paper, Implementation, "Network Thinning") and the
 * non-zero count of the memory-footprint objective (Evaluation, Objective 1).
 *
 * Structure pruning leaves zero structures (filters, neurons, channels that
 * are zero throughout); thinning finds and removes them so that the tensors
 * become smaller dense ones. The paper's three phases are: build a graph of
 * the network, derive a thinning strategy from the dependencies between
 * nodes, apply it. The first two are host work on the caller's side; these
 * calls are the third phase's device work on one tensor at a time. A tensor
 * is seen as the row-major 3-D view [d0][d1][inner]: a conv weight
 * F x C x kh x kw has d0 = F, d1 = C, inner = kh*kw; a matrix R x C has
 * d0 = R, d1 = C, inner = 1; a bias has d0 = n, d1 = inner = 1.
 * All pointers are DEVICE pointers unless stated; calls are asynchronous on
 * `stream`; a value is zero when it is +0 or -0. */

/* keep[i] = 1 if the slice i along `axis` (0: [i][:][:], 1: [:][i][:]) holds a
 * non-zero value, else 0. `keep` has d0 (axis 0) or d1 (axis 1) bytes and is
 * overwritten. Extents may be 0. */
CONDENSA_API int condensa_thin_flags(condensa_ctx *ctx, const float *theta, int64_t d0, int64_t d1,
                                     int64_t inner, int axis, uint8_t *keep, void *stream);

/* dst = src with the slices removed whose flag is 0: dst is the dense row-major
 * [d0'][d1'][inner] tensor of the entries src[i][j][:] with keep0[i] != 0 and
 * keep1[j] != 0, in their original order. A NULL flag array keeps the whole
 * axis. dims_out (device, two int64) receives d0' and d1'. dst must hold
 * d0' * d1' * inner floats (d0 * d1 * inner always suffices) and must not
 * overlap src. d0, d1 and d1 * inner must be below 2^31. The caller's
 * strategy supplies the flags: e.g. keep0 of a conv layer from its own
 * filters, keep1 from the flags of the layer that feeds it. */
CONDENSA_API int condensa_thin_compact(condensa_ctx *ctx, const float *src, int64_t d0, int64_t d1,
                                       int64_t inner, const uint8_t *keep0, const uint8_t *keep1,
                                       float *dst, int64_t *dims_out, void *stream);

/* The same for a whole list of tensors in three launches (flags of all, index lists of all,
 * gather of all) instead of three per tensor: thinning a network is dozens of small tensors.
 * For every layer l: keep0 (d0 bytes, DEVICE, out) receives the axis-0 flags of src (1 iff
 * the slice holds a non-zero); dst receives src without the axis-0 slices whose flag is 0
 * (if remove_axis0 != 0) and without the axis-1 slices whose flag in layer keep1_from's keep0
 * is 0 (keep1_from = -1: the whole axis stays; that layer's d0 must equal this layer's d1 -
 * e.g. a conv layer loses the input channels that the layer feeding it lost as filters);
 * dims_out (DEVICE, two int64) receives the kept extents. `layers` is a HOST array.
 * Extents and pointer rules as for condensa_thin_compact(). */
typedef struct {
    const float *src;      /* in : [d0][d1][inner], fp32                      */
    int64_t d0, d1, inner;
    uint8_t *keep0;        /* out: axis-0 flags, d0 bytes                     */
    int32_t remove_axis0;  /* remove the axis-0 slices whose flag is 0        */
    int32_t keep1_from;    /* layer whose keep0 removes axis-1 slices, or -1  */
    float *dst;            /* out: the dense smaller tensor                   */
    int64_t *dims_out;     /* out: d0', d1'                                   */
} condensa_thin_layer;
CONDENSA_API int condensa_thin_list(condensa_ctx *ctx, const condensa_thin_layer *layers, int L, void *stream);

/* counts[t] = number of non-zero values of arrays[t] (numel[t] floats each),
 * counts[T] = their sum; the memory footprint is that count times the bytes of
 * a stored value. `arrays` and `numel` are HOST arrays of T entries (the
 * pointers in `arrays` are device pointers); `counts` is a DEVICE array of
 * T + 1 int64, overwritten. */
CONDENSA_API int condensa_count_nonzero(condensa_ctx *ctx, const float *const *arrays, const int64_t *numel,
                                        int T, int64_t *counts, void *stream);

/* condensa_cstep_prune() for callers that must not allocate device memory.
 * (An addition of this library: the paper has no counterpart.)
 *
 * Who needs it: programs in which a pool allocator already owns all device
 * memory, so that a cudaMalloc from a library may fail or eat into the pool's
 * reserve; and latency-critical loops that cannot accept the device-wide
 * synchronisation cudaMalloc/cudaFree imply. The context-based calls allocate
 * a workspace the first time they see a problem size; this call never does:
 * no cudaMalloc, cudaFree, cudaMallocHost or other routine that allocates device
 * or pinned memory, on any call (ordinary host heap is used while the arguments
 * are checked). Its scratch (selection state, histograms, candidate list:
 * 2304 KiB) is a fixed array inside the library image, so every GPU that loads
 * the library holds those bytes until the process exits.
 *
 * Operation: exactly condensa_cstep_prune() on a list of ONE tensor, with the
 * same arithmetic, ranking and tie rule and bit-identical theta, mask, lambda,
 * grad and theta_h. `tensor` is a HOST pointer to one condensa_tensor whose
 * buffers are DEVICE pointers on the CURRENT device (cudaGetDevice); all
 * outputs are the caller's. There is no context and no result record;
 * condensa_noalloc_status() tells whether the device-side checks of the last
 * call passed.
 *
 * Limits and rules:
 *  - tensor->numel <= CONDENSA_NOALLOC_MAX_NUMEL, else CONDENSA_ERR_TOO_LARGE
 *    and nothing is launched or written.
 *  - The first call on each device looks up the scratch's device address (once
 *    per device, with that device current; host threads are serialised for
 *    it). Make that first call outside any stream capture.
 *  - All calls on a device share the one scratch array, which still holds the
 *    previous call's contents; each call clears the parts that must start at
 *    zero on `stream` before using them. Two calls that may overlap on the GPU
 *    (different streams without ordering, or several host threads) race on it
 *    and give wrong results: keep calls on one device ordered.
 *  - The error text of a failed call is condensa_last_error(NULL). */
#define CONDENSA_NOALLOC_MAX_NUMEL 1048576
CONDENSA_API int condensa_cstep_prune_noalloc(const condensa_tensor *tensor, double sparsity,
                                              float mu, unsigned fuse, void *stream);

/* Waits for the stream of the last condensa_cstep_prune_noalloc() call on the
 * current device and returns CONDENSA_OK, or CONDENSA_ERR_INTERNAL if one of its
 * device-side consistency checks failed (the outputs are then invalid). Allocates
 * nothing. (No counterpart in the paper.) */
CONDENSA_API int condensa_noalloc_status(void);

/* Text of the last error on this context (never NULL). ctx may be NULL to get
 * the text of a failed condensa_create() or condensa_cstep_prune_noalloc(). */
CONDENSA_API const char *condensa_last_error(const condensa_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* CONDENSA_CSTEP_H */
