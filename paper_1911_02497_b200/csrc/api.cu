// C ABI of the C-step library: argument checks, descriptor table, workspace,
// kernel sequencing. See include/condensa_cstep.h for the contract.
#include "../../include/condensa_cstep.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <ctime>
#include <functional>
#include <mutex>
#include <random>
#include <string>
#include <vector>

#include "common.cuh"
#include "elementwise.cuh"
#include "select.cuh"
#include "structured.cuh"
#include "fused.cuh"
#include "fused_fast.cuh"
#include "fused_blockg.cuh"
#include "sample.cuh"
#include "lstep.cuh"
#include "thin.cuh"
#include "small_select.cuh"
#include "small_prune.cuh"

using namespace cs;

static_assert(sizeof(condensa_result) == sizeof(cs::Result), "result layouts must agree");

namespace {

std::string g_create_error;

struct KernelInfo {
    int occ = 0;     // CTAs per SM
};

struct DeviceMirror {   // device copies used by condensa_cstep_host
    char *buf = nullptr;
    size_t bytes = 0;
};

}  // namespace

struct condensa_ctx {
    int device = 0;
    int num_sms = 0;
    bool coop = false;
    std::string err;
    char *ws = nullptr;
    size_t ws_bytes = 0;
    char *h_stage = nullptr;        // pinned staging of the descriptor upload
    size_t h_stage_bytes = 0;
    cudaEvent_t stage_ev = nullptr;
    cudaEvent_t tail_ev = nullptr;  // recorded behind the last kernel of every call
    bool tail_recorded = false;
    uint64_t seed = 0;              // sample positions of the single-pass path
    std::vector<char> last_upload;  // what the device descriptor area holds now
    char *last_upload_dst = nullptr;
    int64_t launches = 0;
    cudaStream_t last_stream = nullptr;
    bool has_result = false;
    Ctl *ctl = nullptr;
    int occ_select[4] = {0, 0, 0, 0};
    int occ_stream = 0;
    int occ_filter = 0;
    int occ_prune_small = 0;        // resident CTAs per SM of the register-resident small-list kernel
    bool small_smem_set = false;    // dynamic shared memory limit of k_select_small raised on this device
    bool block_smem_set = false;    // the same for the tiled block kernel
    size_t blockg_smem_set = 0;     // ... and for the tiled bh x bw kernel (bytes it has been allowed so far)
    DeviceMirror mirror;
    // optional per-kernel timing (event pair around every launch)
    bool prof_on = false;
    std::vector<cudaEvent_t> prof_ev;       // start/stop pairs
    std::vector<int> prof_name;             // index into prof_names per pair
    std::vector<std::string> prof_names;
    size_t prof_used = 0;                   // pairs recorded since the last read
    std::vector<double> prof_ms;            // accumulated per name
    std::vector<int64_t> prof_cnt;
};

namespace {

int fail(condensa_ctx *c, int code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    if (c) c->err = buf; else g_create_error = buf;
    return code;
}

#define CU_TRY(ctx, call)                                                                   \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess)                                                              \
            return fail(ctx, CONDENSA_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_));   \
    } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Interval {
    uintptr_t lo, hi;
    bool out;
};

// Layout of one call's workspace.
struct Layout {
    size_t ctl, hist, fin_key, fin_id, fin_idx, desc, list_key, list_id, arr_key, partial, sample, journal, total;
    size_t desc_bytes;
};

struct Plan {
    std::vector<TensorDesc> td;
    std::vector<long long> prefix_a, prefix_b;   // scan / apply work items
    long long n_items_a = 0, n_items_b = 0;
    long long S = 0, N = 0, n_seg = 0;
    u64 cap = 0;
    std::vector<long long> edge_items;           // projection items outside the aligned fast path
    std::vector<long long> tile_prefix;          // block pruning: warp tiles of the aligned interior per tensor
    int bt_arr = 0, bt_stages = 0;               // tiled bh x bw kernel: bytes of one array in a tile buffer, buffers
    int jr_floats = 0;                           // journal floats per listed unit
};

int validate(condensa_ctx *ctx, int op, const condensa_tensor *ts, int T, double s, float mu,
             unsigned fuse)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (!ts || T <= 0 || T > (1 << 20)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor list is empty or NULL");
    if (!(mu > 0.0f) || !std::isfinite(mu)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "mu must be finite and > 0");
    if (op <= CONDENSA_OP_BLOCK && !(s >= 0.0 && s <= 1.0))
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "sparsity must lie in [0, 1]");
    const unsigned known = CONDENSA_FUSE_FP16 | CONDENSA_FUSE_LAMBDA | CONDENSA_FUSE_PENALTY | CONDENSA_FUSE_BF16 |
                           CONDENSA_FUSE_E4M3 | CONDENSA_FUSE_E5M2 | CONDENSA_NO_SAMPLING;
    if (fuse & ~known) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "unknown fuse bits");
    {
        const unsigned qb = fuse & (CONDENSA_FUSE_FP16 | CONDENSA_FUSE_BF16 | CONDENSA_FUSE_E4M3 | CONDENSA_FUSE_E5M2);
        if (qb & (qb - 1)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "at most one quantisation type may be fused");
    }
    std::vector<Interval> iv;
    iv.reserve((size_t)T * 6);
    for (int t = 0; t < T; ++t) {
        const condensa_tensor &x = ts[t];
        if (x.numel < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: numel < 0", t);
        if (x.ndim < 1 || x.ndim > 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: ndim must be 1..4", t);
        long long prod = 1;
        for (int d = 0; d < x.ndim; ++d) {
            if (x.shape[d] < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: negative dimension", t);
            prod *= x.shape[d];
        }
        if (prod != x.numel) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: shape does not match numel", t);
        if (x.numel == 0) continue;
        if (!x.w || !x.theta) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: w and theta must not be NULL", t);
        const uintptr_t p4[4] = {(uintptr_t)x.w, (uintptr_t)x.lambda, (uintptr_t)x.theta, (uintptr_t)x.grad};
        for (int i = 0; i < 4; ++i)
            if (p4[i] % 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: fp32 pointer not 4-byte aligned", t);
        if ((uintptr_t)x.theta_h % 2) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: theta_h not 2-byte aligned", t);
        const size_t n = (size_t)x.numel;
        const bool theta_out = op != CONDENSA_OP_LAGRANGE;
        iv.push_back({(uintptr_t)x.w, (uintptr_t)x.w + 4 * n, false});
        iv.push_back({(uintptr_t)x.theta, (uintptr_t)x.theta + 4 * n, theta_out});
        if (x.lambda) iv.push_back({(uintptr_t)x.lambda, (uintptr_t)x.lambda + 4 * n, (fuse & CONDENSA_FUSE_LAMBDA) != 0});
        if (x.grad && (fuse & CONDENSA_FUSE_PENALTY)) iv.push_back({(uintptr_t)x.grad, (uintptr_t)x.grad + 4 * n, true});
        if (x.mask && theta_out) iv.push_back({(uintptr_t)x.mask, (uintptr_t)x.mask + n, true});
        if (x.theta_h && theta_out) iv.push_back({(uintptr_t)x.theta_h, (uintptr_t)x.theta_h + 2 * n, true});
    }
    std::sort(iv.begin(), iv.end(), [](const Interval &a, const Interval &b) { return a.lo < b.lo; });
    // an output range may overlap nothing else
    uintptr_t reach = 0, reach_out = 0;
    for (size_t i = 0; i < iv.size(); ++i) {
        if (iv[i].lo < reach_out || (iv[i].out && iv[i].lo < reach))
            return fail(ctx, CONDENSA_ERR_INVALID_ARG, "an output buffer overlaps another buffer of the call");
        reach = std::max(reach, iv[i].hi);
        if (iv[i].out) reach_out = std::max(reach_out, iv[i].hi);
    }
    return CONDENSA_OK;
}

// What a structured call ranks: for OP_FILTER which leading-index slices (1 = filters of 4-D tensors,
// 2 = rows of 2-D tensors); for OP_BLOCKGEN the block extents, one per dimension of the tensors
// that are cut; and the criterion.
struct HostSpec {
    int kinds = 1;
    int nd = 2;
    long long bs[4] = {4, 4, 1, 1};
    int crit = CRIT_L2;
};

void build_plan(int op, const condensa_tensor *ts, int T, Plan &pl, const HostSpec &sp = HostSpec())
{
    const int kinds = sp.kinds;
    pl.td.resize(T);
    pl.prefix_a.assign(T + 1, 0);
    pl.prefix_b.assign(T + 1, 0);
    long long eoff = 0, uoff = 0, seg = 0;
    for (int t = 0; t < T; ++t) {
        const condensa_tensor &x = ts[t];
        TensorDesc d;
        memset(&d, 0, sizeof(d));
        d.w = x.w; d.lam = x.lambda; d.theta = x.theta; d.mask = x.mask; d.grad = x.grad; d.theta_h = x.theta_h;
        d.numel = x.numel;
        d.elem_prefix = eoff;
        d.unit_prefix = uoff;
        // linear vector path: all arrays must reach 16-byte alignment at the same element
        const uintptr_t aw = (uintptr_t)x.w;
        const int pad = (int)((aw % 16) / 4);
        bool ok = true;
        const uintptr_t f32p[3] = {(uintptr_t)x.lambda, (uintptr_t)x.theta, (uintptr_t)x.grad};
        for (int i = 0; i < 3; ++i)
            if (f32p[i] && (f32p[i] % 16) != (aw % 16)) ok = false;
        if (x.mask && ((uintptr_t)x.mask % 4) != (uintptr_t)(pad % 4)) ok = false;
        if (x.theta_h && ((uintptr_t)x.theta_h % 8) != (uintptr_t)((2 * pad) % 8)) ok = false;
        d.vec_ok = ok ? 1 : 0;
        d.pad = ok ? pad : 0;
        const long long n_groups = (x.numel + d.pad + 3) / 4;
        const long long lin_items = (n_groups + GROUPS_PER_ITEM - 1) / GROUPS_PER_ITEM;
        long long items_a = 0, items_b = lin_items;
        if (op == OP_PRUNE) {
            d.ranked = x.numel > 0;
            d.n_units = x.numel;
            items_a = lin_items;
        } else if (op == OP_FILTER) {
            d.ranked = (x.numel > 0 && ((x.ndim == 4 && (kinds & 1)) || (x.ndim == 2 && (kinds & 2)))) ? 1 : 0;
            if (d.ranked) {
                d.d0 = x.shape[0];
                d.d1 = x.numel / x.shape[0];
                d.n_units = d.d0;
                items_a = d.d0 * ((d.d1 + SEG - 1) / SEG);
            }
        } else if (op == OP_BLOCKGEN) {
            d.ranked = (x.ndim == sp.nd && x.numel > 0) ? 1 : 0;
            if (d.ranked) {
                d.nd = sp.nd;
                d.n_units = 1;
                for (int q = 0; q < 4; ++q) { d.sh[q] = 1; d.bs[q] = 1; d.nb[q] = 1; }
                for (int q = 0; q < sp.nd; ++q) {          // right-aligned to four dimensions
                    const int r = 4 - sp.nd + q;
                    d.sh[r] = (int)x.shape[q];
                    d.bs[r] = (int)std::min<long long>(sp.bs[q], x.shape[q]);
                    d.nb[r] = (int)((x.shape[q] + sp.bs[q] - 1) / sp.bs[q]);
                    d.n_units *= d.nb[r];
                }
                if (sp.nd == 2) {
                    d.d0 = x.shape[0];
                    d.d1 = x.shape[1];
                    d.bh = d.bs[2];
                    d.bw = d.bs[3];
                    d.nbc = d.nb[3];
                }
                items_a = (d.n_units + BLOCKS_PER_ITEM - 1) / BLOCKS_PER_ITEM;
            }
        } else if (op == OP_BLOCKG1) {
            d.ranked = (x.ndim == 2 && x.numel > 0) ? 1 : 0;
            if (d.ranked) {
                d.nd = 2;
                d.d0 = x.shape[0];
                d.d1 = x.shape[1];
                d.bh = (int)sp.bs[0];            // (not cut down to the shape: the kernels are built for bh x bw)
                d.bw = (int)sp.bs[1];
                d.nbc = (d.d1 + d.bw - 1) / d.bw;
                d.n_units = ((d.d0 + d.bh - 1) / d.bh) * d.nbc;
                // whole block rows go through shared memory by bulk copies: 16-byte rule for every row start
                bool bok = (d.d1 % 4) == 0 && (aw % 16) == 0;
                for (int i = 0; i < 2; ++i)
                    if (f32p[i] % 16) bok = false;
                d.blk_vec_ok = bok ? 1 : 0;
                items_a = (d.n_units + BLOCKS_PER_ITEM - 1) / BLOCKS_PER_ITEM;
                items_b = items_a;
            }
        } else if (op == OP_BLOCK) {
            d.ranked = (x.ndim == 2 && x.numel > 0) ? 1 : 0;
            if (d.ranked) {
                d.d0 = x.shape[0];
                d.d1 = x.shape[1];
                d.nbc = (d.d1 + 3) / 4;
                d.n_units = ((d.d0 + 3) / 4) * d.nbc;
                bool bok = (d.d1 % 4) == 0 && (aw % 16) == 0;
                for (int i = 0; i < 3; ++i)
                    if (f32p[i] % 16) bok = false;
                if ((uintptr_t)x.mask % 4) bok = false;
                if ((uintptr_t)x.theta_h % 8) bok = false;
                d.blk_vec_ok = bok ? 1 : 0;
                items_a = (d.n_units + BLOCKS_PER_ITEM - 1) / BLOCKS_PER_ITEM;
                items_b = items_a;
            }
        }
        pl.td[t] = d;
        pl.prefix_a[t + 1] = pl.prefix_a[t] + items_a;
        pl.prefix_b[t + 1] = pl.prefix_b[t] + items_b;
        eoff += x.numel;
        if (op != OP_PRUNE) uoff += d.n_units;
        if (op == OP_FILTER) seg += items_a;
    }
    pl.N = eoff;
    pl.S = (op == OP_PRUNE) ? eoff : uoff;
    pl.n_seg = seg;
    pl.n_items_a = pl.prefix_a[T];
    pl.n_items_b = pl.prefix_b[T];
    const u64 S = (u64)pl.S;
    u64 cap = S / 8;
    if (cap < 65536) cap = 65536;
    // unstructured lists may list up to 16 Mi candidates (20 bytes each with the journal): the sample
    // bracket of a list of more than 10^8 parameters at a moderate sparsity holds several million
    const u64 cap_max = op == OP_PRUNE ? (1ull << 24) : (1ull << 22);
    if (cap > cap_max) cap = cap_max;
    if (cap > S) cap = S ? S : 1;
    pl.cap = cap;
}

constexpr int N_SAMPLE = SAMPLE_THREADS * SAMPLE_KEYS_PER_THREAD;
constexpr int N_SAMPLE_BIG = SAMPLE_THREADS * SAMPLE_KEYS_PER_THREAD_BIG;
constexpr long long SAMPLE_BIG_FROM = 1ll << 26;     // unstructured lists from this many units take the larger sample
constexpr int SAMPLE_CTAS = 64;
constexpr long long ONE_LAUNCH_MAX_N = 4ll << 20;    // parameters of a list that the one-launch route takes

// journal_floats: floats of original lambda kept per listed unit (0: no single-pass path)
Layout make_layout(int T, const Plan &pl, bool ranking, bool filter, int journal_floats = 0)
{
    Layout L;
    size_t off = 0;
    L.ctl = off; off = align_up(off + sizeof(Ctl), 256);
    L.hist = off; off = align_up(off + sizeof(u64) * 3 * NBINS, 256);
    L.fin_key = off; off = align_up(off + sizeof(u64) * FIN, 256);
    L.fin_id = off; off = align_up(off + sizeof(u64) * FIN, 256);
    L.fin_idx = off; off = align_up(off + sizeof(u64) * FIN, 256);
    L.desc = off;
    L.desc_bytes = sizeof(TensorDesc) * (size_t)T + 2 * sizeof(long long) * (size_t)(T + 1) +
                   sizeof(long long) * (pl.edge_items.size() + pl.tile_prefix.size());
    off = align_up(off + L.desc_bytes, 256);
    L.list_key = off; if (ranking) off = align_up(off + sizeof(u64) * pl.cap, 256);
    L.list_id = off; if (ranking) off = align_up(off + sizeof(u64) * pl.cap, 256);
    L.arr_key = off; if (filter) off = align_up(off + sizeof(u64) * (size_t)std::max<long long>(pl.S, 1), 256);
    L.partial = off; if (filter) off = align_up(off + sizeof(double) * (size_t)std::max<long long>(pl.n_seg, 1), 256);
    L.sample = off; if (journal_floats) off = align_up(off + sizeof(u64) * N_SAMPLE_BIG, 256);
    L.journal = off; if (journal_floats) off = align_up(off + sizeof(float) * (size_t)journal_floats * pl.cap, 256);
    L.total = off;
    return L;
}

int ensure_workspace(condensa_ctx *ctx, size_t bytes, cudaStream_t stream, bool exact = false)
{
    if (bytes <= ctx->ws_bytes) return CONDENSA_OK;
    CU_TRY(ctx, cudaStreamSynchronize(stream));
    if (ctx->last_stream && ctx->last_stream != stream) CU_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    if (ctx->ws) cudaFree(ctx->ws);
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
    ctx->last_upload.clear();
    ctx->last_upload_dst = nullptr;
    ctx->has_result = false;       // the record of an earlier call lived in the old workspace
    ctx->ctl = nullptr;
    const size_t want = exact ? align_up(bytes, 256) : align_up(bytes + bytes / 4, 1 << 20);
    cudaError_t e = cudaMalloc((void **)&ctx->ws, want);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ctx, CONDENSA_ERR_WORKSPACE, "cannot allocate %zu bytes of workspace: %s", want, cudaGetErrorString(e));
    }
    ctx->ws_bytes = want;
    // counters that kernels expect to find at zero on first use
    if ((e = cudaMemset(ctx->ws, 0, std::min<size_t>(want, 1 << 16))) != cudaSuccess)
        return fail(ctx, CONDENSA_ERR_CUDA, "cudaMemset: %s", cudaGetErrorString(e));
    return CONDENSA_OK;
}

// Copies the descriptor table and both prefix arrays to the workspace unless
// the device already holds exactly these bytes.
int upload_image(condensa_ctx *ctx, std::vector<char> &img, char *dst, cudaStream_t stream);

int upload_desc(condensa_ctx *ctx, const Plan &pl, int T, char *dst, size_t bytes, cudaStream_t stream)
{
    std::vector<char> img(bytes);
    char *p = img.data();
    memcpy(p, pl.td.data(), sizeof(TensorDesc) * (size_t)T); p += sizeof(TensorDesc) * (size_t)T;
    memcpy(p, pl.prefix_a.data(), sizeof(long long) * (size_t)(T + 1)); p += sizeof(long long) * (size_t)(T + 1);
    if (!pl.edge_items.empty()) memcpy(p, pl.edge_items.data(), sizeof(long long) * pl.edge_items.size());
    p += sizeof(long long) * pl.edge_items.size();
    memcpy(p, pl.prefix_b.data(), sizeof(long long) * (size_t)(T + 1)); p += sizeof(long long) * (size_t)(T + 1);
    if (!pl.tile_prefix.empty()) memcpy(p, pl.tile_prefix.data(), sizeof(long long) * pl.tile_prefix.size());
    return upload_image(ctx, img, dst, stream);
}

// Copies `img` to `dst` through the pinned staging area unless the device already holds these bytes there.
int upload_image(condensa_ctx *ctx, std::vector<char> &img, char *dst, cudaStream_t stream)
{
    const size_t bytes = img.size();
    if (ctx->last_upload_dst == dst && ctx->last_upload == img) return CONDENSA_OK;
    CU_TRY(ctx, cudaEventSynchronize(ctx->stage_ev));    // the previous upload has left the staging area
    if (bytes > ctx->h_stage_bytes) {
        if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
        ctx->h_stage = nullptr;
        ctx->h_stage_bytes = 0;
        CU_TRY(ctx, cudaMallocHost((void **)&ctx->h_stage, align_up(bytes * 2, 4096)));
        ctx->h_stage_bytes = align_up(bytes * 2, 4096);
    }
    memcpy(ctx->h_stage, img.data(), bytes);
    CU_TRY(ctx, cudaMemcpyAsync(dst, ctx->h_stage, bytes, cudaMemcpyHostToDevice, stream));
    CU_TRY(ctx, cudaEventRecord(ctx->stage_ev, stream));
    ctx->last_upload.swap(img);
    ctx->last_upload_dst = dst;
    return CONDENSA_OK;
}

template <class K>
int occupancy(K kernel)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, THREADS, 0) != cudaSuccess) occ = 1;
    return occ < 1 ? 1 : occ;
}

int stream_grid(condensa_ctx *ctx, long long n_items, int occ)
{
    long long g = (long long)ctx->num_sms * occ;
    if (g > n_items) g = n_items;
    if (g < 1) g = 1;
    return (int)g;
}

int prof_begin(condensa_ctx *ctx, const char *name, cudaStream_t stream)
{
    if (!ctx->prof_on) return 0;
    if (ctx->prof_used * 2 + 2 > ctx->prof_ev.size()) {
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return 0;
            ctx->prof_ev.push_back(e);
        }
    }
    int id = -1;
    for (size_t i = 0; i < ctx->prof_names.size(); ++i)
        if (ctx->prof_names[i] == name) id = (int)i;
    if (id < 0) {
        id = (int)ctx->prof_names.size();
        ctx->prof_names.push_back(name);
        ctx->prof_ms.push_back(0.0);
        ctx->prof_cnt.push_back(0);
    }
    if (ctx->prof_name.size() <= ctx->prof_used) ctx->prof_name.resize(ctx->prof_used + 1);
    ctx->prof_name[ctx->prof_used] = id;
    cudaEventRecord(ctx->prof_ev[ctx->prof_used * 2], stream);
    return 1;
}

void prof_end(condensa_ctx *ctx, int active, cudaStream_t stream)
{
    if (!active) return;
    cudaEventRecord(ctx->prof_ev[ctx->prof_used * 2 + 1], stream);
    ctx->prof_used += 1;
}

// Folds the recorded event pairs into the per-kernel totals (synchronises).
void prof_collect(condensa_ctx *ctx)
{
    for (size_t i = 0; i < ctx->prof_used; ++i) {
        float ms = 0.0f;
        cudaEventSynchronize(ctx->prof_ev[2 * i + 1]);
        if (cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]) == cudaSuccess) {
            ctx->prof_ms[ctx->prof_name[i]] += ms;
            ctx->prof_cnt[ctx->prof_name[i]] += 1;
        }
    }
    ctx->prof_used = 0;
}

// Launch configuration with the programmatic-dependent-launch attribute (dropped while every
// kernel is bracketed by an event pair: nothing can overlap then).
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    PdlLaunch(const condensa_ctx *ctx, int grid, int block, size_t smem, cudaStream_t stream)
    {
        memset(&cfg, 0, sizeof(cfg));
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3((unsigned)block);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cfg.attrs = &attr;
        cfg.numAttrs = ctx->prof_on ? 0 : 1;
    }
};

#define LAUNCH_CHECK(ctx)                                                                    \
    do {                                                                                     \
        cudaError_t e_ = cudaGetLastError();                                                 \
        if (e_ != cudaSuccess)                                                               \
            return fail(ctx, CONDENSA_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e_)); \
        ctx->launches += 1;                                                                  \
    } while (0)

template <int SRC>
int launch_select(condensa_ctx *ctx, Params &P, int first_listed, int pre_scan, cudaStream_t stream,
                  const long long *prefix_b = nullptr, long long n_items_b = 0, int post_apply = 0,
                  const Sel *init = nullptr)
{
    if (!ctx->occ_select[SRC]) ctx->occ_select[SRC] = occupancy(k_select<SRC>);
    const int per_sm = std::min(ctx->occ_select[SRC], 2);
    dim3 grid((unsigned)(ctx->num_sms * per_sm)), block(THREADS);
    int do_init = init ? 1 : 0;
    Sel init_v;
    if (init) init_v = *init; else memset(&init_v, 0, sizeof(init_v));
    void *args[] = {(void *)&P, (void *)&first_listed, (void *)&pre_scan, (void *)&prefix_b, (void *)&n_items_b,
                    (void *)&post_apply, (void *)&do_init, (void *)&init_v};
    const int pa_ = prof_begin(ctx, init ? "k_select_all" : "k_select", stream);
    CU_TRY(ctx, cudaLaunchCooperativeKernel((const void *)k_select<SRC>, grid, block, args, 0, stream));
    ctx->launches += 1;
    prof_end(ctx, pa_, stream);
    return CONDENSA_OK;
}

Sel initial_state(long long S, long long k, int bits_key)
{
    Sel s;
    memset(&s, 0, sizeof(s));
    s.S = (u64)S;
    s.k = (u64)k;
    s.lo_key = 0;
    s.hi_key = bits_key >= 63 ? 0x7FFFFFFFFFFFFFFFull : ((1ull << bits_key) - 1ull);
    s.lo_id = 0;
    s.hi_id = S > 0 ? (u64)S - 1 : 0;
    s.pop = (u64)S;
    s.above_known = 1;
    s.shift = bits_key > LOG_NBINS ? bits_key - LOG_NBINS : 0;
    s.done = (S == 0 || k == 0) ? 1 : 0;
    return s;
}

// Tile buffers of the tiled bh x bw kernel for this plan: three buffers if a block row of every
// large matrix fits then, else two; false when even two do not hold the widest block row or a
// large matrix is not aligned (the caller then takes the route over the norm array).
constexpr size_t SMEM_OPTIN_BYTES = 232448;      // shared memory one CTA may have on this architecture
bool blockg_ring_config(Plan &pl, int T)
{
    const size_t fixed = sizeof(BlockGShared) + 1024 + (size_t)BG_GROUPS * blockg_cand_bytes(pl.jr_floats);
    if (fixed >= SMEM_OPTIN_BYTES) return false;
    long long best_tiled = 0, best_rounds = 0;
    for (int stages = BG_MAX_STAGES; stages >= 2; --stages) {
        // stages * (2.25 * arr + 16) <= what is left
        const size_t per = (SMEM_OPTIN_BYTES - fixed) / (size_t)stages;
        if (per < 1024) continue;
        long long arr = (long long)((per - 16) * 4 / 9);
        arr -= arr % 64;
        long long tiled = 0, rounds = 0;                // units the tiles cover; rounds of one block per thread
        for (int t = 0; t < T; ++t) {
            tiled += blockg_fast_end(pl.td[t], (int)arr);
            rounds += blockg_tile_rounds(pl.td[t], (int)arr);
        }
        // coverage first, then the fewest rounds (the kernel's time follows them, not the bytes of
        // a tile), then the most buffers
        if (tiled > best_tiled || (tiled == best_tiled && tiled > 0 && rounds < best_rounds)) {
            best_tiled = tiled;
            best_rounds = rounds;
            pl.bt_arr = (int)arr;
            pl.bt_stages = stages;
        }
    }
    // (mostly unaligned or very wide matrices: the generic code would do the work, at the speed
    // of the route over the norm array at best)
    return best_tiled > 0 && 2 * best_tiled >= pl.S;
}

// Block shapes the tiled bh x bw kernel is built for (the per-block code is unrolled at compile
// time; 5 x 5 is the block size of the paper's LSTM experiment). Other shapes take the route
// over the norm array.
#define CS_BLOCKG_SHAPES(X) X(5, 5) X(3, 3) X(2, 2) X(1, 8) X(8, 1)
bool blockg_shape_built(long long bh, long long bw)
{
#define CS_X(BH, BW) if (bh == BH && bw == BW) return true;
    CS_BLOCKG_SHAPES(CS_X)
#undef CS_X
    return false;
}

bool blockg_single_pass_candidate(int op, const HostSpec &sp, unsigned fuse)
{
    return op == OP_BLOCKGEN && sp.nd == 2 && sp.crit == CRIT_L2 && blockg_shape_built(sp.bs[0], sp.bs[1]) &&
           !(fuse & CONDENSA_NO_SAMPLING);
}

// Work decomposition and workspace layout of one call (no device work).
Layout plan_call(int op, const condensa_tensor *ts, int T, unsigned fuse, const HostSpec &sp, Plan &pl,
                 bool &ranking, bool &sampling, long long small_items_max = 0, bool *small_prune = nullptr)
{
    build_plan(op, ts, T, pl, sp);
    ranking = op <= OP_BLOCK || op == OP_BLOCKGEN || op == OP_BLOCKG1;
    // single-pass path: unstructured and block pruning of lists too large to list whole
    // an unstructured list of at most one work item per resident CTA stays in registers for the whole call
    const bool reg_resident = op == OP_PRUNE && pl.n_items_b > 0 && pl.n_items_b <= small_items_max;
    if (small_prune) *small_prune = reg_resident;
    sampling = (op == OP_PRUNE || op == OP_BLOCK || op == OP_BLOCKG1) && !(fuse & CONDENSA_NO_SAMPLING) && !reg_resident &&
                          (u64)pl.S > pl.cap && pl.S >= 8ll * N_SAMPLE;
    if (sampling && op == OP_BLOCK && pl.cap > (1ull << 20)) pl.cap = 1ull << 20;   // bounds the journal
    if (op == OP_BLOCKG1) {
        pl.jr_floats = (int)(sp.bs[0] * sp.bs[1]);
        const u64 cap_j = (16ull << 20) / (u64)pl.jr_floats;                        // journal of at most 64 MB
        if (sampling && pl.cap > cap_j) pl.cap = cap_j;
        sampling = sampling && (u64)pl.S > pl.cap && blockg_ring_config(pl, T);
    }
    const int journal_floats = sampling ? (op == OP_BLOCK ? 16 : op == OP_BLOCKG1 ? pl.jr_floats : 1) : 0;
    if (sampling && op == OP_BLOCKG1) {
        pl.tile_prefix.assign((size_t)T + 1, 0);
        for (int t = 0; t < T; ++t) {
            pl.td[t].tile_rows = blockg_fast_end(pl.td[t], pl.bt_arr) > 0 ? (int)blockg_rows_per_tile(pl.td[t], pl.bt_arr) : 0;
            for (long long j = 0; j < pl.prefix_b[t + 1] - pl.prefix_b[t]; ++j)
                if (!blockg_item_is_fast(pl.td[t], j, pl.bt_arr)) pl.edge_items.push_back(pl.prefix_b[t] + j);
            pl.tile_prefix[t + 1] = pl.tile_prefix[t] + blockg_tile_count(pl.td[t], pl.bt_arr);
        }
    } else if (sampling) {
        for (int t = 0; t < T; ++t)
            for (long long j = 0; j < pl.prefix_b[t + 1] - pl.prefix_b[t]; ++j) {
                const bool fast = op == OP_BLOCK ? block_item_is_fast(pl.td[t], j) : elem_item_is_fast(pl.td[t], j);
                if (!fast) pl.edge_items.push_back(pl.prefix_b[t] + j);
            }
        if (op == OP_BLOCK) {
            pl.tile_prefix.assign((size_t)T + 1, 0);
            for (int t = 0; t < T; ++t) {
                const TensorDesc &d = pl.td[t];
                const long long tiles = block_tile_count(d);
                pl.tile_prefix[t + 1] = pl.tile_prefix[t] + tiles;
            }
        }
    }
    return make_layout(T, pl, ranking, op == OP_FILTER || op == OP_BLOCKGEN, journal_floats);
}

int run_op(condensa_ctx *ctx, int op, const condensa_tensor *ts, int T, double sparsity, float mu,
           unsigned fuse, cudaStream_t stream, const HostSpec &sp = HostSpec())
{
    int rc = validate(ctx, op == OP_BLOCKGEN ? OP_BLOCK : op, ts, T, sparsity, mu, fuse);
    if (rc) return rc;
    if (op == OP_BLOCKGEN)
        for (int t = 0; t < T; ++t)
            for (int q = 0; q < ts[t].ndim; ++q)
                if (ts[t].ndim == sp.nd && ts[t].shape[q] > 0x7FFFFFFFll)
                    return fail(ctx, CONDENSA_ERR_UNSUPPORTED, "tensor %d: an extent above 2^31 - 1 cannot be cut into blocks", t);
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    Plan pl;
    bool ranking = false, sampling = false, small_prune = false;
    if (op == OP_PRUNE && !ctx->occ_prune_small) ctx->occ_prune_small = occupancy(k_prune_small);
    const long long small_items_max = (op == OP_PRUNE && ctx->occ_prune_small >= 2) ? 2ll * ctx->num_sms : 0;
    Layout L;
    bool planned = false;
    if (blockg_single_pass_candidate(op, sp, fuse)) {
        // bh x bw blocks of matrices by the L2 norm: the single-pass kernels, when the list is long
        // enough for a sample, at least one unit is kept and a block row fits the tile buffers
        L = plan_call(OP_BLOCKG1, ts, T, fuse, sp, pl, ranking, sampling, 0, nullptr);
        const long long Z = (long long)std::min<double>((double)pl.S, std::max(0.0, std::floor(sparsity * (double)pl.S + 0.5)));
        if (sampling && pl.S - Z > 0) {
            op = OP_BLOCKG1;
            planned = true;
        } else {
            pl = Plan();
        }
    }
    if (!planned) L = plan_call(op, ts, T, fuse, sp, pl, ranking, sampling, small_items_max, &small_prune);
    rc = ensure_workspace(ctx, L.total, stream);
    if (rc) return rc;
    char *ws = ctx->ws;
    rc = upload_desc(ctx, pl, T, ws + L.desc, L.desc_bytes, stream);
    if (rc) return rc;

    Params P;
    memset(&P, 0, sizeof(P));
    P.td = (const TensorDesc *)(ws + L.desc);
    const long long *pa = (const long long *)(ws + L.desc + sizeof(TensorDesc) * (size_t)T);
    const long long *pe = pa + (T + 1);                      // edge item list
    const long long *pb = pe + pl.edge_items.size();         // projection prefix, right behind it
    P.T = T;
    P.mu = mu;
    P.fuse = fuse & FUSE_KERNEL_BITS;
    if (op == OP_QUANTIZE && !(P.fuse & FUSE_QUANT)) P.fuse |= FUSE_FP16;
    if (op == OP_LAGRANGE) P.fuse &= ~FUSE_QUANT;
    P.ctl = (Ctl *)(ws + L.ctl);
    P.hist = (u64 *)(ws + L.hist);
    P.fin_key = (u64 *)(ws + L.fin_key);
    P.fin_id = (u64 *)(ws + L.fin_id);
    P.fin_idx = (u64 *)(ws + L.fin_idx);
    P.edge_items = pe;
    P.n_edge_items = (long long)pl.edge_items.size();
    P.tile_prefix = pb + (T + 1);
    P.n_tiles = pl.tile_prefix.empty() ? 0 : pl.tile_prefix[T];
    P.list_key = (u64 *)(ws + L.list_key);
    P.list_id = (u64 *)(ws + L.list_id);
    P.cap = pl.cap;
    P.arr_key = (u64 *)(ws + L.arr_key);
    P.partial = (double *)(ws + L.partial);
    P.S = pl.S;
    P.bits_key = (op == OP_PRUNE) ? 31 : 63;
    P.sample_key = (u64 *)(ws + L.sample);
    // a longer list pays for a larger sample: bracket and wrong provisional decisions shrink with its square root
    const bool big_sample = op == OP_PRUNE && pl.S >= SAMPLE_BIG_FROM;
    P.n_sample = big_sample ? N_SAMPLE_BIG : N_SAMPLE;
    P.jr_lam = (float *)(ws + L.journal);
    P.jr_floats = op == OP_BLOCKG1 ? pl.jr_floats : op == OP_BLOCK ? 16 : 1;
    P.bt_arr_bytes = pl.bt_arr;
    P.bt_stages = pl.bt_stages;
    P.onepass_cap = pl.cap;
    P.crit = sp.crit;
    P.seed = ctx->seed;
    {
        // a missed sample bracket can be repaired inside the call unless the first pass
        // has overwritten multipliers in place
        bool lam_in_place = false;
        if (fuse & CONDENSA_FUSE_LAMBDA)
            for (int t = 0; t < T; ++t) lam_in_place = lam_in_place || (ts[t].lambda != nullptr && ts[t].numel > 0);
        P.miss_fallback = lam_in_place ? 0 : 1;
    }
    bool need_h = (fuse & FUSE_QUANT) != 0;
    for (int t = 0; t < T; ++t) need_h = need_h || ts[t].theta_h != nullptr;
    ctx->ctl = P.ctl;
    // the workspace is shared by all calls of the context: a call on another stream
    // first waits for the previous call's kernels
    if (ctx->tail_recorded && ctx->last_stream != stream) CU_TRY(ctx, cudaStreamWaitEvent(stream, ctx->tail_ev, 0));
    ctx->last_stream = stream;

    if (!ctx->occ_stream) ctx->occ_stream = 3;

    bool applied_in_select = false;
    if (ranking && small_prune) {
        const long long Z = (long long)std::min<double>((double)pl.S, std::max(0.0, std::floor(sparsity * (double)pl.S + 0.5)));
        Sel init = initial_state(pl.S, pl.S - Z, P.bits_key);
        Params Ps = P;
        Ps.item_prefix = pb;
        Ps.n_items = pl.n_items_b;
        dim3 grid((unsigned)(2 * ctx->num_sms)), block(THREADS);
        void *args[] = {(void *)&Ps, (void *)&init};
        const int pa_ = prof_begin(ctx, "k_prune_small", stream);
        CU_TRY(ctx, cudaLaunchCooperativeKernel((const void *)k_prune_small, grid, block, args, 0, stream));
        ctx->launches += 1;
        prof_end(ctx, pa_, stream);
        ctx->has_result = true;
        if (cudaEventRecord(ctx->tail_ev, stream) == cudaSuccess) ctx->tail_recorded = true;
        return CONDENSA_OK;
    }
    if (ranking) {
        const long long Z = (long long)std::min<double>((double)pl.S, std::max(0.0, std::floor(sparsity * (double)pl.S + 0.5)));
        const long long k = pl.S - Z;
        Sel init = initial_state(pl.S, k, P.bits_key);
        const int do_list0 = (u64)pl.S <= pl.cap ? 1 : 0;
        // rankings of a short key array (filters, rows, general blocks) skip the grid-wide selection
        const bool small = (op == OP_FILTER || op == OP_BLOCKGEN) && pl.S <= SMALL_S_MAX &&
                           !(fuse & CONDENSA_NO_SAMPLING);

        // lists that stay in the L2 between the passes: one cooperative launch does
        // start, histogram passes, selection and projection
        const bool one_launch = (op == OP_PRUNE || op == OP_BLOCK) && !sampling && pl.N <= ONE_LAUNCH_MAX_N;

        Params Pa = P;
        Pa.item_prefix = pa;
        Pa.n_items = pl.n_items_a;
        if (op == OP_BLOCKGEN && pl.S > 0) {
            const int pa_ = prof_begin(ctx, "k_blockgen_norms", stream);
            k_blockgen_norms<<<stream_grid(ctx, pl.n_items_a, 8), THREADS, 0, stream>>>(Pa);
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pa_, stream);
        }
        if (op == OP_FILTER && pl.S > 0) {
            int pa_ = prof_begin(ctx, "k_filter_partial", stream);
            if (!ctx->occ_filter) ctx->occ_filter = occupancy(k_filter_partial);       // one wave of resident CTAs
            k_filter_partial<<<stream_grid(ctx, (pl.n_items_a + WARPS - 1) / WARPS, ctx->occ_filter), THREADS, 0, stream>>>(Pa);
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pa_, stream);
            if (!small) {           // the one-CTA selection forms the norms itself
                pa_ = prof_begin(ctx, "k_filter_combine", stream);
                k_filter_combine<<<stream_grid(ctx, (pl.S + THREADS - 1) / THREADS, 8), THREADS, 0, stream>>>(Pa);
                LAUNCH_CHECK(ctx);
                prof_end(ctx, pa_, stream);
            }
        }
        Params Pf = P;                      // single-pass kernel runs on the projection decomposition
        Pf.item_prefix = pb;
        Pf.n_items = pl.n_items_b;
        if (sampling) Pa.n_edge_items = 0;     // the single-pass kernels do their edge items themselves
        if (sampling && !init.done) {
            int pi_ = prof_begin(ctx, "k_sample", stream);
            if (op == OP_PRUNE && big_sample) k_sample<SRC_ELEM, SAMPLE_KEYS_PER_THREAD_BIG><<<SAMPLE_CTAS, SAMPLE_THREADS, 0, stream>>>(Pa, init);
            else if (op == OP_PRUNE) k_sample<SRC_ELEM, SAMPLE_KEYS_PER_THREAD><<<SAMPLE_CTAS, SAMPLE_THREADS, 0, stream>>>(Pa, init);
            else if (op == OP_BLOCKG1) k_sample<SRC_BLOCKG, SAMPLE_KEYS_PER_THREAD><<<SAMPLE_CTAS, SAMPLE_THREADS, 0, stream>>>(Pa, init);
            else k_sample<SRC_BLOCK, SAMPLE_KEYS_PER_THREAD><<<SAMPLE_CTAS, SAMPLE_THREADS, 0, stream>>>(Pa, init);
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pi_, stream);
            pi_ = prof_begin(ctx, op == OP_PRUNE ? "k_fused_elem" : op == OP_BLOCKG1 ? "k_fused_blockg" : "k_fused_block", stream);
            // block pruning: one CTA per WARPS warp tiles at least, and enough CTAs for the edge items
            const bool tiled = op == OP_BLOCK || op == OP_BLOCKG1;
            const long long work = tiled ? std::max<long long>(Pf.n_tiles, (long long)pl.edge_items.size()) : pl.n_items_b;
            const int gridf = stream_grid(ctx, work, tiled ? 1 : 3);
            const size_t dyn_g = op == OP_BLOCKG1 ? blockg_dyn_smem(pl.bt_arr, pl.bt_stages, pl.jr_floats) : 0;
            if (op == OP_BLOCKG1 && dyn_g > ctx->blockg_smem_set) {
                const int dyn = (int)dyn_g;
#define CS_X(BH, BW)                                                                                                          \
    CU_TRY(ctx, cudaFuncSetAttribute(k_fused_blockg<true, true, BH, BW>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));   \
    CU_TRY(ctx, cudaFuncSetAttribute(k_fused_blockg<true, false, BH, BW>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));  \
    CU_TRY(ctx, cudaFuncSetAttribute(k_fused_blockg<false, true, BH, BW>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));  \
    CU_TRY(ctx, cudaFuncSetAttribute(k_fused_blockg<false, false, BH, BW>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));
                CS_BLOCKG_SHAPES(CS_X)
#undef CS_X
                ctx->blockg_smem_set = dyn_g;
            }
            const bool need_g = (fuse & CONDENSA_FUSE_PENALTY) != 0;
            if (op == OP_BLOCK && !ctx->block_smem_set) {
                const int dyn = (int)BLOCK_FAST_DYN_SMEM;
                CU_TRY(ctx, cudaFuncSetAttribute(k_fused_block<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));
                CU_TRY(ctx, cudaFuncSetAttribute(k_fused_block<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));
                CU_TRY(ctx, cudaFuncSetAttribute(k_fused_block<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));
                CU_TRY(ctx, cudaFuncSetAttribute(k_fused_block<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn));
                ctx->block_smem_set = true;
            }
            // Programmatic dependent launch: the single-pass kernel may start while the sampler
            // still runs; it sets itself up (and the block kernel already fetches its first tiles)
            // and waits for the sampler's results with griddepcontrol.wait.
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cudaLaunchAttribute pdl;
            pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
            pdl.val.programmaticStreamSerializationAllowed = 1;
            cfg.gridDim = dim3((unsigned)gridf);
            cfg.blockDim = dim3((unsigned)(op == OP_PRUNE ? THREADS : op == OP_BLOCKG1 ? BG_THREADS : BT_THREADS));
            cfg.dynamicSmemBytes = op == OP_PRUNE ? 0 : op == OP_BLOCKG1 ? dyn_g : BLOCK_FAST_DYN_SMEM;
            cfg.stream = stream;
            cfg.attrs = &pdl;
            cfg.numAttrs = ctx->prof_on ? 0 : 1;       // with an event pair around every kernel there is nothing to overlap
#define CS_LAUNCH_FUSED(KERNEL)                                                                \
    do {                                                                                       \
        if (need_h && need_g) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, KERNEL<true, true>, Pf));   \
        else if (need_h) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, KERNEL<true, false>, Pf));       \
        else if (need_g) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, KERNEL<false, true>, Pf));       \
        else CU_TRY(ctx, cudaLaunchKernelEx(&cfg, KERNEL<false, false>, Pf));                  \
    } while (0)
            if (op == OP_PRUNE) CS_LAUNCH_FUSED(k_fused_elem);
            else if (op == OP_BLOCKG1) {
#define CS_X(BH, BW)                                                                                            \
    if (sp.bs[0] == BH && sp.bs[1] == BW) {                                                                     \
        if (need_h && need_g) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, k_fused_blockg<true, true, BH, BW>, Pf));    \
        else if (need_h) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, k_fused_blockg<true, false, BH, BW>, Pf));        \
        else if (need_g) CU_TRY(ctx, cudaLaunchKernelEx(&cfg, k_fused_blockg<false, true, BH, BW>, Pf));        \
        else CU_TRY(ctx, cudaLaunchKernelEx(&cfg, k_fused_blockg<false, false, BH, BW>, Pf));                   \
    }
                CS_BLOCKG_SHAPES(CS_X)
#undef CS_X
            } else CS_LAUNCH_FUSED(k_fused_block);
#undef CS_LAUNCH_FUSED
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pi_, stream);
        } else if (small) {
            // a few thousand structures: the whole selection in one CTA
            if (!ctx->small_smem_set) {
                CU_TRY(ctx, cudaFuncSetAttribute(k_select_small, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)(sizeof(u64) * SMALL_S_MAX)));
                ctx->small_smem_set = true;
            }
            const int pi_ = prof_begin(ctx, "k_select_small", stream);
            {
                PdlLaunch L2(ctx, 1, SMALL_THREADS, sizeof(u64) * (size_t)pl.S, stream);
                const int combine = op == OP_FILTER ? 1 : 0;
                CU_TRY(ctx, cudaLaunchKernelEx(&L2.cfg, k_select_small, Pa, init, combine));
            }
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pi_, stream);
        } else if (!one_launch) {
            int pi_ = prof_begin(ctx, "k_init", stream);
            k_init<<<8, THREADS, 0, stream>>>(P, init);
            LAUNCH_CHECK(ctx);
            prof_end(ctx, pi_, stream);
        }
        // with the single-pass path the fallback scan, if it is needed at all, runs inside k_select
        if (!init.done && !small && !sampling && !one_launch) {
            const int ps_ = prof_begin(ctx, op == OP_PRUNE ? "k_scan_elem" : op == OP_BLOCK ? "k_scan_block" : "k_scan_array", stream);
            if (op == OP_PRUNE) {
                k_scan<SRC_ELEM><<<stream_grid(ctx, pl.n_items_a, 4), THREADS, 0, stream>>>(Pa, do_list0);
            } else if (op == OP_BLOCK) {
                // with the single-pass path this launch only runs when the sample advised against it
                k_scan<SRC_BLOCK><<<stream_grid(ctx, pl.n_items_a, sampling ? 1 : 4), THREADS, 0, stream>>>(Pa, do_list0);
            } else {
                k_scan<SRC_ARRAY><<<stream_grid(ctx, (pl.S + THREADS - 1) / THREADS, 4), THREADS, 0, stream>>>(Pa, do_list0);
            }
            LAUNCH_CHECK(ctx);
            prof_end(ctx, ps_, stream);
        }
        // a call that went for the single pass needs no projection launch: after a fall-back k_select projects itself
        const int post_apply = ((sampling && !init.done) || one_launch) ? (need_h ? 2 : 1) : 0;
        applied_in_select = post_apply != 0;
        const int pre_scan = (sampling || one_launch) ? 1 : 0;
        const Sel *init_p = one_launch ? &init : nullptr;
        if (small) rc = CONDENSA_OK;
        else if (op == OP_PRUNE) rc = launch_select<SRC_ELEM>(ctx, Pa, do_list0, pre_scan, stream, pb, pl.n_items_b, post_apply, init_p);
        else if (op == OP_BLOCK) rc = launch_select<SRC_BLOCK>(ctx, Pa, do_list0, pre_scan, stream, pb, pl.n_items_b, post_apply, init_p);
        else if (op == OP_BLOCKG1) rc = launch_select<SRC_BLOCKG>(ctx, Pa, do_list0, pre_scan, stream, pb, pl.n_items_b, post_apply, init_p);
        else rc = launch_select<SRC_ARRAY>(ctx, Pa, do_list0, 0, stream);
        if (rc) return rc;
        ctx->has_result = true;
    }

    Params Pb = P;
    Pb.item_prefix = pb;
    Pb.n_items = pl.n_items_b;
    if (pl.n_items_b > 0 && !applied_in_select) {
        const int grid = stream_grid(ctx, pl.n_items_b, ctx->occ_stream);
        static const char *apply_names[7] = {"k_apply_prune", "k_apply_filter", "k_apply_block", "k_quantize", "k_lagrange", "k_apply_blockgen", "k_apply_blockgen"};
        const int pa_ = prof_begin(ctx, apply_names[op], stream);
        switch (op) {
        case OP_PRUNE:
            if (need_h) k_apply_linear<M_PRUNE, true><<<grid, THREADS, 0, stream>>>(Pb);
            else k_apply_linear<M_PRUNE, false><<<grid, THREADS, 0, stream>>>(Pb);
            break;
        case OP_FILTER: {
            PdlLaunch L2(ctx, grid, THREADS, 0, stream);
            if (need_h) CU_TRY(ctx, cudaLaunchKernelEx(&L2.cfg, k_apply_linear<M_FILTER, true>, Pb));
            else CU_TRY(ctx, cudaLaunchKernelEx(&L2.cfg, k_apply_linear<M_FILTER, false>, Pb));
            break;
        }
        case OP_BLOCK: k_apply_block<<<grid, THREADS, 0, stream>>>(Pb); break;
        case OP_BLOCKGEN:
            if (need_h) k_apply_linear<M_BLOCKGEN, true><<<grid, THREADS, 0, stream>>>(Pb);
            else k_apply_linear<M_BLOCKGEN, false><<<grid, THREADS, 0, stream>>>(Pb);
            break;
        case OP_QUANTIZE: k_apply_linear<M_KEEPALL, true><<<grid, THREADS, 0, stream>>>(Pb); break;
        default: k_apply_linear<M_LAGRANGE, false><<<grid, THREADS, 0, stream>>>(Pb); break;
        }
        LAUNCH_CHECK(ctx);
        prof_end(ctx, pa_, stream);
    }
    if (cudaEventRecord(ctx->tail_ev, stream) == cudaSuccess) ctx->tail_recorded = true;
    return CONDENSA_OK;
}

}  // namespace

// ---------------------------------------------------------------- C ABI
extern "C" {

int condensa_create(condensa_ctx **out, int device, size_t workspace_bytes)
{
    if (!out) return fail(nullptr, CONDENSA_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    int n = 0;
    cudaError_t e = cudaGetDeviceCount(&n);
    if (e != cudaSuccess || n == 0) {
        cudaGetLastError();
        return fail(nullptr, CONDENSA_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(e));
    }
    if (device < 0 || device >= n) return fail(nullptr, CONDENSA_ERR_INVALID_ARG, "device %d out of range", device);
    if ((e = cudaSetDevice(device)) != cudaSuccess) return fail(nullptr, CONDENSA_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(e));
    condensa_ctx *c = new condensa_ctx();
    c->device = device;
    int coop = 0;
    cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device);
    c->coop = coop != 0;
    if (!c->coop || c->num_sms <= 0) {
        delete c;
        return fail(nullptr, CONDENSA_ERR_UNSUPPORTED, "device lacks cooperative launch");
    }
    if ((e = cudaEventCreateWithFlags(&c->stage_ev, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&c->tail_ev, cudaEventDisableTiming)) != cudaSuccess) {
        if (c->stage_ev) cudaEventDestroy(c->stage_ev);
        delete c;
        return fail(nullptr, CONDENSA_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(e));
    }
    {
        // sample positions differ from context to context, so that no fixed input can be
        // built against them; condensa_set_seed() makes a run reproducible
        uint64_t z = 0x9E3779B97F4A7C15ull;
        try {
            std::random_device rd;
            z = ((uint64_t)rd() << 32) ^ (uint64_t)rd();
        } catch (...) {
            z ^= (uint64_t)(uintptr_t)c ^ ((uint64_t)std::hash<std::string>()(std::to_string((long long)clock())) << 1);
        }
        c->seed = z;
    }
    if (workspace_bytes) {
        int rc = ensure_workspace(c, workspace_bytes, nullptr, true);
        if (rc) {
            g_create_error = c->err;
            cudaEventDestroy(c->stage_ev);
            cudaEventDestroy(c->tail_ev);
            delete c;
            return rc;
        }
    }
    *out = c;
    return CONDENSA_OK;
}

int condensa_destroy(condensa_ctx *ctx)
{
    if (!ctx) return CONDENSA_OK;
    cudaSetDevice(ctx->device);
    if (ctx->last_stream) cudaStreamSynchronize(ctx->last_stream);
    cudaDeviceSynchronize();
    if (ctx->ws) cudaFree(ctx->ws);
    if (ctx->mirror.buf) cudaFree(ctx->mirror.buf);
    if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
    if (ctx->stage_ev) cudaEventDestroy(ctx->stage_ev);
    if (ctx->tail_ev) cudaEventDestroy(ctx->tail_ev);
    for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
    delete ctx;
    return CONDENSA_OK;
}

int condensa_workspace_bytes(int op, const condensa_tensor *tensors, int T, const condensa_structure_spec *spec,
                             unsigned fuse, size_t *bytes)
{
    if (!bytes || !tensors || T <= 0 || op < CONDENSA_OP_PRUNE || op > CONDENSA_OP_LAGRANGE)
        return fail(nullptr, CONDENSA_ERR_INVALID_ARG, "condensa_workspace_bytes: bad argument");
    HostSpec sp;
    int iop = op;
    if (op == CONDENSA_OP_FILTER || op == CONDENSA_OP_BLOCK) {
        if (spec) {
            sp.crit = spec->criterion;
            if (spec->kind == CONDENSA_SPEC_SLICES) { iop = OP_FILTER; sp.kinds = spec->kinds; }
            else {
                if (spec->ndim < 1 || spec->ndim > 4) return fail(nullptr, CONDENSA_ERR_INVALID_ARG, "blocks have 1 to 4 dimensions");
                sp.nd = spec->ndim;
                for (int q = 0; q < 4; ++q) sp.bs[q] = q < spec->ndim ? spec->block[q] : 1;
                const bool fast = sp.nd == 2 && sp.bs[0] == 4 && sp.bs[1] == 4 && sp.crit == CRIT_L2;
                iop = fast ? OP_BLOCK : OP_BLOCKGEN;
            }
        }
    }
    Plan pl;
    bool ranking = false, sampling = false;
    const Layout L = plan_call(iop, tensors, T, fuse, sp, pl, ranking, sampling);
    size_t total = L.total;
    if (blockg_single_pass_candidate(iop, sp, fuse)) {      // the call may take the single-pass kernels instead
        Plan pg;
        const Layout Lg = plan_call(OP_BLOCKG1, tensors, T, fuse, sp, pg, ranking, sampling);
        if (sampling) total = std::max(total, Lg.total);
    }
    *bytes = align_up(total + total / 4, 1 << 20);      // what a call of this shape makes the context hold
    return CONDENSA_OK;
}

int condensa_set_seed(condensa_ctx *ctx, uint64_t seed)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    ctx->seed = seed;
    return CONDENSA_OK;
}

int condensa_cstep_prune(condensa_ctx *ctx, const condensa_tensor *tensors, int T, double sparsity,
                         float mu, unsigned fuse, void *stream)
{
    return run_op(ctx, OP_PRUNE, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream);
}

int condensa_cstep_filter(condensa_ctx *ctx, const condensa_tensor *tensors, int T, double sparsity,
                          float mu, unsigned fuse, void *stream)
{
    return run_op(ctx, OP_FILTER, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream);
}

int condensa_cstep_structure(condensa_ctx *ctx, const condensa_tensor *tensors, int T, double sparsity,
                             float mu, int kinds, unsigned fuse, void *stream)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (kinds < 1 || kinds > (CONDENSA_STRUCT_FILTER | CONDENSA_STRUCT_NEURON))
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "kinds must be CONDENSA_STRUCT_FILTER and/or CONDENSA_STRUCT_NEURON");
    HostSpec sp;
    sp.kinds = kinds;
    return run_op(ctx, OP_FILTER, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream, sp);
}

int condensa_cstep_block(condensa_ctx *ctx, const condensa_tensor *tensors, int T, double sparsity,
                         float mu, int bh, int bw, unsigned fuse, void *stream)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (bh < 1 || bw < 1) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "block shape must be positive");
    if (bh > 4096 || bw > 4096) return fail(ctx, CONDENSA_ERR_UNSUPPORTED, "block sides above 4096 are not built");
    if (bh != 4 || bw != 4) {    // general shapes: norms per block, selection on the norm array, elementwise projection
        HostSpec sp;
        sp.nd = 2; sp.bs[0] = bh; sp.bs[1] = bw;
        return run_op(ctx, OP_BLOCKGEN, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream, sp);
    }
    return run_op(ctx, OP_BLOCK, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream);
}

int condensa_cstep_structured(condensa_ctx *ctx, const condensa_tensor *tensors, int T, double sparsity,
                              float mu, const condensa_structure_spec *spec, unsigned fuse, void *stream)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (!spec) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "spec is NULL");
    if (spec->criterion < CONDENSA_CRIT_L2 || spec->criterion > CONDENSA_CRIT_MAX)
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "criterion must be CONDENSA_CRIT_L2, _L1 or _MAX");
    HostSpec sp;
    sp.crit = spec->criterion;
    if (spec->kind == CONDENSA_SPEC_SLICES) {
        if (spec->kinds < 1 || spec->kinds > (CONDENSA_STRUCT_FILTER | CONDENSA_STRUCT_NEURON))
            return fail(ctx, CONDENSA_ERR_INVALID_ARG, "kinds must be CONDENSA_STRUCT_FILTER and/or CONDENSA_STRUCT_NEURON");
        sp.kinds = spec->kinds;
        return run_op(ctx, OP_FILTER, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream, sp);
    }
    if (spec->kind != CONDENSA_SPEC_BLOCKS) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "kind must be CONDENSA_SPEC_SLICES or CONDENSA_SPEC_BLOCKS");
    if (spec->ndim < 1 || spec->ndim > 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "blocks have 1 to 4 dimensions");
    sp.nd = spec->ndim;
    for (int q = 0; q < 4; ++q) sp.bs[q] = 1;
    for (int q = 0; q < spec->ndim; ++q) {
        if (spec->block[q] < 1) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "block extents must be positive");
        if (spec->block[q] > 4096) return fail(ctx, CONDENSA_ERR_UNSUPPORTED, "block extents above 4096 are not built");
        sp.bs[q] = spec->block[q];
    }
    // 4 x 4 blocks of matrices by the L2 norm take the single-pass kernels
    if (sp.nd == 2 && sp.bs[0] == 4 && sp.bs[1] == 4 && sp.crit == CRIT_L2)
        return run_op(ctx, OP_BLOCK, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream);
    return run_op(ctx, OP_BLOCKGEN, tensors, T, sparsity, mu, fuse, (cudaStream_t)stream, sp);
}

int condensa_cstep_quantize(condensa_ctx *ctx, const condensa_tensor *tensors, int T, float mu,
                            int dtype, unsigned fuse, void *stream)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (dtype < CONDENSA_DTYPE_FP16 || dtype > CONDENSA_DTYPE_FP8_E5M2)
        return fail(ctx, CONDENSA_ERR_UNSUPPORTED, "dtype must be one of CONDENSA_DTYPE_FP16 / BF16 / FP8_E4M3 / FP8_E5M2");
    if (fuse & FUSE_QUANT)
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "the type is given by dtype, not by fuse bits");
    if (dtype == CONDENSA_DTYPE_BF16) fuse |= CONDENSA_FUSE_BF16;
    if (dtype == CONDENSA_DTYPE_FP8_E4M3) fuse |= CONDENSA_FUSE_E4M3;
    if (dtype == CONDENSA_DTYPE_FP8_E5M2) fuse |= CONDENSA_FUSE_E5M2;
    return run_op(ctx, OP_QUANTIZE, tensors, T, 0.0, mu, fuse, (cudaStream_t)stream);
}

int condensa_cstep_lagrange_update(condensa_ctx *ctx, const condensa_tensor *tensors, int T, float mu,
                                   unsigned fuse, void *stream)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (!(fuse & (CONDENSA_FUSE_LAMBDA | CONDENSA_FUSE_PENALTY)))
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "nothing to do: set FUSE_LAMBDA and/or FUSE_PENALTY");
    return run_op(ctx, OP_LAGRANGE, tensors, T, 0.0, mu, fuse, (cudaStream_t)stream);
}

int condensa_lstep_update(condensa_ctx *ctx, const condensa_opt_tensor *ts, int T, float mu,
                          const condensa_opt *opt, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!ts || T <= 0 || T > (1 << 20) || !opt) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor list or optimizer is NULL");
    if (!(mu >= 0.0f) || !std::isfinite(mu)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "mu must be finite and >= 0");
    if (opt->kind != CONDENSA_OPT_SGD && opt->kind != CONDENSA_OPT_ADAM) return fail(ctx, CONDENSA_ERR_UNSUPPORTED, "unknown optimizer kind");
    if (!std::isfinite(opt->lr) || !std::isfinite(opt->momentum) || !std::isfinite(opt->weight_decay))
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "optimizer parameters must be finite");
    if (opt->kind == CONDENSA_OPT_ADAM &&
        (!(opt->beta1 >= 0.0f && opt->beta1 < 1.0f) || !(opt->beta2 >= 0.0f && opt->beta2 < 1.0f) || opt->step < 1 || !(opt->eps >= 0.0f)))
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "Adam needs 0 <= beta < 1, eps >= 0 and step >= 1");
    std::vector<Interval> iv;
    std::vector<OptDesc> td(T);
    std::vector<long long> prefix(T + 1, 0);
    for (int t = 0; t < T; ++t) {
        const condensa_opt_tensor &x = ts[t];
        if (x.numel < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: numel < 0", t);
        OptDesc d;
        memset(&d, 0, sizeof(d));
        d.numel = x.numel;
        if (x.numel > 0) {
            if (!x.w || !x.theta || !x.grad) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: w, theta and grad must not be NULL", t);
            const bool need_b1 = opt->kind == CONDENSA_OPT_ADAM || opt->momentum != 0.0f;
            if (need_b1 && !x.buf1) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: buf1 is NULL", t);
            if (opt->kind == CONDENSA_OPT_ADAM && !x.buf2) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: buf2 is NULL", t);
            const uintptr_t ptrs[6] = {(uintptr_t)x.w, (uintptr_t)x.theta, (uintptr_t)x.lambda, (uintptr_t)x.grad,
                                       (uintptr_t)(need_b1 ? x.buf1 : nullptr), (uintptr_t)(opt->kind == CONDENSA_OPT_ADAM ? x.buf2 : nullptr)};
            bool ok = true;
            for (int i = 0; i < 6; ++i) {
                if (ptrs[i] % 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: pointer not 4-byte aligned", t);
                if (ptrs[i] && ptrs[i] % 16 != ptrs[0] % 16) ok = false;
            }
            const size_t n4 = 4 * (size_t)x.numel;
            iv.push_back({ptrs[0], ptrs[0] + n4, true});
            iv.push_back({ptrs[1], ptrs[1] + n4, false});
            if (ptrs[2]) iv.push_back({ptrs[2], ptrs[2] + n4, false});
            iv.push_back({ptrs[3], ptrs[3] + n4, false});
            if (ptrs[4]) iv.push_back({ptrs[4], ptrs[4] + n4, true});
            if (ptrs[5]) iv.push_back({ptrs[5], ptrs[5] + n4, true});
            d.w = x.w; d.theta = x.theta; d.lam = x.lambda; d.grad = x.grad;
            d.buf1 = need_b1 ? x.buf1 : nullptr;
            d.buf2 = opt->kind == CONDENSA_OPT_ADAM ? x.buf2 : nullptr;
            d.vec_ok = ok ? 1 : 0;
            d.pad = ok ? (int)((ptrs[0] % 16) / 4) : 0;
        }
        td[t] = d;
        const long long groups = (x.numel + d.pad + 3) / 4;
        prefix[t + 1] = prefix[t] + (groups + GROUPS_PER_ITEM - 1) / GROUPS_PER_ITEM;
    }
    std::sort(iv.begin(), iv.end(), [](const Interval &a, const Interval &b) { return a.lo < b.lo; });
    uintptr_t reach = 0, reach_out = 0;
    for (size_t i = 0; i < iv.size(); ++i) {
        if (iv[i].lo < reach_out || (iv[i].out && iv[i].lo < reach))
            return fail(ctx, CONDENSA_ERR_INVALID_ARG, "an in/out buffer overlaps another buffer of the call");
        reach = std::max(reach, iv[i].hi);
        if (iv[i].out) reach_out = std::max(reach_out, iv[i].hi);
    }
    if (prefix[T] == 0) return CONDENSA_OK;
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    // descriptor image in the same workspace slot the C-step calls use
    Plan none;
    none.cap = 1;
    const Layout L = make_layout(0, none, false, false);
    const size_t bytes = sizeof(OptDesc) * (size_t)T + sizeof(long long) * (size_t)(T + 1);
    int rc = ensure_workspace(ctx, L.desc + align_up(bytes, 256), stream);
    if (rc) return rc;
    std::vector<char> img(bytes);
    memcpy(img.data(), td.data(), sizeof(OptDesc) * (size_t)T);
    memcpy(img.data() + sizeof(OptDesc) * (size_t)T, prefix.data(), sizeof(long long) * (size_t)(T + 1));
    rc = upload_image(ctx, img, ctx->ws + L.desc, stream);
    if (rc) return rc;
    OptParams P;
    memset(&P, 0, sizeof(P));
    P.td = (const OptDesc *)(ctx->ws + L.desc);
    P.item_prefix = (const long long *)(ctx->ws + L.desc + sizeof(OptDesc) * (size_t)T);
    P.T = T;
    P.n_items = prefix[T];
    P.mu = mu; P.lr = opt->lr; P.momentum = opt->momentum; P.wd = opt->weight_decay;
    P.beta1 = opt->beta1; P.beta2 = opt->beta2; P.eps = opt->eps;
    if (opt->kind == CONDENSA_OPT_ADAM) {
        volatile float c1 = 1.0f - opt->beta1, c2 = 1.0f - opt->beta2;
        P.c1 = c1; P.c2 = c2;
        const double bc1 = 1.0 - std::pow((double)opt->beta1, (double)opt->step);
        const double bc2 = 1.0 - std::pow((double)opt->beta2, (double)opt->step);
        P.step_size = (float)((double)opt->lr / bc1);
        P.sqrt_bc2 = (float)std::sqrt(bc2);
    }
    ctx->last_stream = stream;
    const int grid = stream_grid(ctx, P.n_items, 3);
    const int pa_ = prof_begin(ctx, opt->kind == CONDENSA_OPT_ADAM ? "k_lstep_adam" : "k_lstep_sgd", stream);
    if (opt->kind == CONDENSA_OPT_ADAM) k_lstep<OPT_ADAM><<<grid, THREADS, 0, stream>>>(P);
    else k_lstep<OPT_SGD><<<grid, THREADS, 0, stream>>>(P);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    return CONDENSA_OK;
}

// ---------------------------------------------------------------- thinning
int condensa_thin_flags(condensa_ctx *ctx, const float *theta, int64_t d0, int64_t d1, int64_t inner, int axis,
                        uint8_t *keep, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (d0 < 0 || d1 < 0 || inner < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "negative extent");
    if (axis != 0 && axis != 1) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "axis must be 0 or 1");
    const long long d = axis ? d1 : d0;
    if (d == 0) return CONDENSA_OK;
    if (!keep) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "keep is NULL");
    if ((double)d0 * (double)d1 * (double)inner > 9.0e18) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor too large");
    const long long n = d0 * d1 * inner;
    if (n > 0 && !theta) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "theta is NULL");
    if ((uintptr_t)theta % 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "theta is not 4-byte aligned");
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    CU_TRY(ctx, cudaMemsetAsync(keep, 0, (size_t)d, stream));
    ctx->last_stream = stream;
    if (n == 0) return CONDENSA_OK;
    const int pa_ = prof_begin(ctx, "k_thin_flags", stream);
    k_thin_flags<<<stream_grid(ctx, (n + THIN_ITEM - 1) / THIN_ITEM, 8), THREADS, 0, stream>>>(theta, d0, d1, inner, axis, keep);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    return CONDENSA_OK;
}

int condensa_thin_compact(condensa_ctx *ctx, const float *src, int64_t d0, int64_t d1, int64_t inner,
                          const uint8_t *keep0, const uint8_t *keep1, float *dst, int64_t *dims_out, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (d0 < 0 || d1 < 0 || inner < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "negative extent");
    if (!dims_out) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "dims_out is NULL");
    if (d0 > 0x7FFFFFFFll || d1 > 0x7FFFFFFFll || (double)d1 * (double)inner >= 2147483648.0)
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "d0, d1 and d1 * inner must be below 2^31");
    const long long n = d0 * d1 * inner;
    if (n > 0 && (!src || !dst)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "src or dst is NULL");
    if ((uintptr_t)src % 4 || (uintptr_t)dst % 4 || (uintptr_t)dims_out % 8)
        return fail(ctx, CONDENSA_ERR_INVALID_ARG, "misaligned pointer");
    if (n > 0) {
        const uintptr_t a = (uintptr_t)src, b = (uintptr_t)dst, bytes = (uintptr_t)n * 4;
        if (a < b + bytes && b < a + bytes) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "src and dst overlap");
    }
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    // index lists live in the descriptor area of the workspace
    Plan none;
    none.cap = 1;
    const Layout L = make_layout(0, none, false, false);
    const size_t bytes = align_up(sizeof(int) * (size_t)d0, 256) + align_up(sizeof(int) * (size_t)d1, 256);
    int rc = ensure_workspace(ctx, L.desc + bytes, stream);
    if (rc) return rc;
    ctx->last_upload.clear();           // a kernel overwrites the area: nothing is cached there any more
    ctx->last_upload_dst = nullptr;
    int *idx0 = (int *)(ctx->ws + L.desc);
    int *idx1 = (int *)(ctx->ws + L.desc + align_up(sizeof(int) * (size_t)d0, 256));
    ctx->last_stream = stream;
    int pa_ = prof_begin(ctx, "k_thin_index", stream);
    k_thin_index<<<1, THIN_INDEX_THREADS, 0, stream>>>(keep0, keep1, d0, d1, idx0, idx1, (long long *)dims_out);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    if (n == 0) return CONDENSA_OK;
    const long long L_in = d1 * inner;
    const long long tiles = d0 * ((L_in + 1023) / 1024);
    const bool vec = !keep1 && L_in % 4 == 0 && (uintptr_t)src % 16 == 0 && (uintptr_t)dst % 16 == 0;
    const int grid = stream_grid(ctx, tiles, 8);
    pa_ = prof_begin(ctx, "k_thin_gather", stream);
    if (vec) k_thin_gather<true><<<grid, THREADS, 0, stream>>>(src, dst, d1, inner, keep0 ? idx0 : nullptr, nullptr, (const long long *)dims_out);
    else k_thin_gather<false><<<grid, THREADS, 0, stream>>>(src, dst, d1, inner, keep0 ? idx0 : nullptr, keep1 ? idx1 : nullptr, (const long long *)dims_out);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    return CONDENSA_OK;
}

int condensa_thin_list(condensa_ctx *ctx, const condensa_thin_layer *layers, int L, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!layers || L <= 0 || L > 65535) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer list is empty, NULL or too long");
    std::vector<ThinLayerDesc> td((size_t)L);
    std::vector<long long> pre_f((size_t)L + 1, 0), pre_g((size_t)L + 1, 0);
    size_t idx_bytes = 0;
    std::vector<size_t> off0((size_t)L), off1((size_t)L);
    for (int l = 0; l < L; ++l) {
        const condensa_thin_layer &x = layers[l];
        if (x.d0 < 0 || x.d1 < 0 || x.inner < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: negative extent", l);
        if (x.d0 > 0x7FFFFFFFll || x.d1 > 0x7FFFFFFFll || (double)x.d1 * (double)x.inner >= 2147483648.0)
            return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: d0, d1 and d1 * inner must be below 2^31", l);
        const long long n = x.d0 * x.d1 * x.inner;
        if (!x.dims_out || (uintptr_t)x.dims_out % 8) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: dims_out is NULL or misaligned", l);
        if (n > 0 && (!x.src || !x.dst)) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: src or dst is NULL", l);
        if (x.d0 > 0 && !x.keep0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: keep0 is NULL", l);
        if ((uintptr_t)x.src % 4 || (uintptr_t)x.dst % 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: misaligned pointer", l);
        if (x.keep1_from >= L || (x.keep1_from >= 0 && layers[x.keep1_from].d0 != x.d1))
            return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: keep1_from must name a layer whose d0 equals this layer's d1", l);
        if (n > 0) {
            const uintptr_t a = (uintptr_t)x.src, b = (uintptr_t)x.dst, bytes = (uintptr_t)n * 4;
            if (a < b + bytes && b < a + bytes) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "layer %d: src and dst overlap", l);
        }
        ThinLayerDesc d;
        memset(&d, 0, sizeof(d));
        d.src = x.src; d.dst = x.dst; d.keep0 = x.keep0;
        d.keep1 = x.keep1_from >= 0 ? layers[x.keep1_from].keep0 : nullptr;
        d.dims_out = (long long *)x.dims_out;
        d.d0 = x.d0; d.d1 = x.d1; d.inner = x.inner;
        d.use_keep0 = x.remove_axis0 ? 1 : 0;
        td[l] = d;
        off0[l] = idx_bytes; idx_bytes += align_up(sizeof(int) * (size_t)x.d0, 256);
        off1[l] = idx_bytes; idx_bytes += align_up(sizeof(int) * (size_t)x.d1, 256);
        pre_f[l + 1] = pre_f[l] + x.d0;            // a slice without values still gets its flag (0)
        pre_g[l + 1] = pre_g[l] + (n > 0 ? x.d0 * ((x.d1 * x.inner + 1023) / 1024) : 0);
    }
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    Plan none;
    none.cap = 1;
    const Layout Lay = make_layout(0, none, false, false);
    const size_t desc_bytes = align_up(sizeof(ThinLayerDesc) * (size_t)L + 2 * sizeof(long long) * (size_t)(L + 1), 256);
    int rc = ensure_workspace(ctx, Lay.desc + desc_bytes + idx_bytes, stream);
    if (rc) return rc;
    char *base = ctx->ws + Lay.desc;
    for (int l = 0; l < L; ++l) {
        td[l].idx0 = (int *)(base + desc_bytes + off0[l]);
        td[l].idx1 = (int *)(base + desc_bytes + off1[l]);
    }
    std::vector<char> img(sizeof(ThinLayerDesc) * (size_t)L + 2 * sizeof(long long) * (size_t)(L + 1));
    memcpy(img.data(), td.data(), sizeof(ThinLayerDesc) * (size_t)L);
    memcpy(img.data() + sizeof(ThinLayerDesc) * (size_t)L, pre_f.data(), sizeof(long long) * (size_t)(L + 1));
    memcpy(img.data() + sizeof(ThinLayerDesc) * (size_t)L + sizeof(long long) * (size_t)(L + 1), pre_g.data(),
           sizeof(long long) * (size_t)(L + 1));
    rc = upload_image(ctx, img, base, stream);
    if (rc) return rc;
    const ThinLayerDesc *dtd = (const ThinLayerDesc *)base;
    const long long *dpf = (const long long *)(base + sizeof(ThinLayerDesc) * (size_t)L);
    const long long *dpg = dpf + (L + 1);
    ctx->last_stream = stream;
    int pa_ = prof_begin(ctx, "k_thin_list_flags", stream);
    if (pre_f[L] > 0) {
        k_thin_list_flags<<<stream_grid(ctx, (pre_f[L] + WARPS - 1) / WARPS, 8), THREADS, 0, stream>>>(dtd, dpf, L);
        LAUNCH_CHECK(ctx);
    }
    prof_end(ctx, pa_, stream);
    pa_ = prof_begin(ctx, "k_thin_list_index", stream);
    k_thin_list_index<<<L, THIN_INDEX_THREADS, 0, stream>>>(dtd);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    if (pre_g[L] > 0) {
        pa_ = prof_begin(ctx, "k_thin_list_gather", stream);
        k_thin_list_gather<<<stream_grid(ctx, pre_g[L], 8), THREADS, 0, stream>>>(dtd, dpg, L);
        LAUNCH_CHECK(ctx);
        prof_end(ctx, pa_, stream);
    }
    if (cudaEventRecord(ctx->tail_ev, stream) == cudaSuccess) ctx->tail_recorded = true;
    return CONDENSA_OK;
}

int condensa_count_nonzero(condensa_ctx *ctx, const float *const *arrays, const int64_t *numel, int T,
                           int64_t *counts, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!arrays || !numel || T <= 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "array list is empty or NULL");
    if (!counts || (uintptr_t)counts % 8) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "counts is NULL or misaligned");
    std::vector<CountDesc> td((size_t)T);
    std::vector<long long> prefix((size_t)T + 1, 0);
    for (int t = 0; t < T; ++t) {
        if (numel[t] < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "array %d: negative numel", t);
        if (numel[t] > 0 && !arrays[t]) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "array %d is NULL", t);
        if ((uintptr_t)arrays[t] % 4) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "array %d is not 4-byte aligned", t);
        td[t].x = arrays[t];
        td[t].numel = numel[t];
        prefix[t + 1] = prefix[t] + (numel[t] + THIN_ITEM - 1) / THIN_ITEM;
    }
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    Plan none;
    none.cap = 1;
    const Layout L = make_layout(0, none, false, false);
    const size_t bytes = sizeof(CountDesc) * (size_t)T + sizeof(long long) * (size_t)(T + 1);
    int rc = ensure_workspace(ctx, L.desc + align_up(bytes, 256), stream);
    if (rc) return rc;
    std::vector<char> img(bytes);
    memcpy(img.data(), td.data(), sizeof(CountDesc) * (size_t)T);
    memcpy(img.data() + sizeof(CountDesc) * (size_t)T, prefix.data(), sizeof(long long) * (size_t)(T + 1));
    rc = upload_image(ctx, img, ctx->ws + L.desc, stream);
    if (rc) return rc;
    CU_TRY(ctx, cudaMemsetAsync(counts, 0, sizeof(int64_t) * (size_t)(T + 1), stream));
    ctx->last_stream = stream;
    if (prefix[T] == 0) return CONDENSA_OK;
    const int pa_ = prof_begin(ctx, "k_count_nonzero", stream);
    k_count_nonzero<<<stream_grid(ctx, prefix[T], 8), THREADS, 0, stream>>>(
        (const CountDesc *)(ctx->ws + L.desc), (const long long *)(ctx->ws + L.desc + sizeof(CountDesc) * (size_t)T), T,
        prefix[T], (unsigned long long *)counts);
    LAUNCH_CHECK(ctx);
    prof_end(ctx, pa_, stream);
    return CONDENSA_OK;
}

int condensa_cstep_host(condensa_ctx *ctx, int op, const condensa_tensor *tensors, int T,
                        double sparsity, float mu, int bh, int bw, unsigned fuse, void *stream_)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    if (op < CONDENSA_OP_PRUNE || op > CONDENSA_OP_LAGRANGE) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "unknown op");
    if (!tensors || T <= 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor list is empty or NULL");
    cudaStream_t stream = (cudaStream_t)stream_;
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    // device mirror: w, lambda, theta, grad (fp32), theta_h (u16), mask (u8) per tensor
    size_t total = 0;
    std::vector<size_t> off(T);
    for (int t = 0; t < T; ++t) {
        if (tensors[t].numel < 0) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: numel < 0", t);
        off[t] = total;
        total += align_up((size_t)tensors[t].numel * 4, 256) * 4 + align_up((size_t)tensors[t].numel * 2, 256) +
                 align_up((size_t)tensors[t].numel, 256);
    }
    if (total > ctx->mirror.bytes) {
        CU_TRY(ctx, cudaStreamSynchronize(stream));
        if (ctx->mirror.buf) cudaFree(ctx->mirror.buf);
        ctx->mirror.buf = nullptr;
        ctx->mirror.bytes = 0;
        cudaError_t e = cudaMalloc((void **)&ctx->mirror.buf, total);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(ctx, CONDENSA_ERR_WORKSPACE, "cannot allocate %zu bytes of device mirror", total);
        }
        ctx->mirror.bytes = total;
    }
    std::vector<condensa_tensor> dev(tensors, tensors + T);
    for (int t = 0; t < T; ++t) {
        const condensa_tensor &h = tensors[t];
        const size_t n = (size_t)h.numel, a4 = align_up(n * 4, 256);
        char *base = ctx->mirror.buf + off[t];
        condensa_tensor &d = dev[t];
        d.w = (const float *)base;
        d.lambda = h.lambda ? (float *)(base + a4) : nullptr;
        d.theta = (float *)(base + 2 * a4);
        d.grad = h.grad ? (float *)(base + 3 * a4) : nullptr;
        d.theta_h = h.theta_h ? (uint16_t *)(base + 4 * a4) : nullptr;
        d.mask = h.mask ? (uint8_t *)(base + 4 * a4 + align_up(n * 2, 256)) : nullptr;
        if (n == 0) continue;
        if (!h.w || !h.theta) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "tensor %d: w and theta must not be NULL", t);
        CU_TRY(ctx, cudaMemcpyAsync((void *)d.w, h.w, n * 4, cudaMemcpyHostToDevice, stream));
        if (h.lambda) CU_TRY(ctx, cudaMemcpyAsync(d.lambda, h.lambda, n * 4, cudaMemcpyHostToDevice, stream));
        if (op == CONDENSA_OP_LAGRANGE) CU_TRY(ctx, cudaMemcpyAsync(d.theta, h.theta, n * 4, cudaMemcpyHostToDevice, stream));
    }
    int rc;
    switch (op) {
    case CONDENSA_OP_PRUNE: rc = condensa_cstep_prune(ctx, dev.data(), T, sparsity, mu, fuse, stream); break;
    case CONDENSA_OP_FILTER: rc = condensa_cstep_filter(ctx, dev.data(), T, sparsity, mu, fuse, stream); break;
    case CONDENSA_OP_BLOCK: rc = condensa_cstep_block(ctx, dev.data(), T, sparsity, mu, bh, bw, fuse, stream); break;
    case CONDENSA_OP_QUANTIZE: rc = condensa_cstep_quantize(ctx, dev.data(), T, mu, CONDENSA_DTYPE_FP16, fuse, stream); break;
    default: rc = condensa_cstep_lagrange_update(ctx, dev.data(), T, mu, fuse, stream); break;
    }
    if (rc) return rc;
    for (int t = 0; t < T; ++t) {
        const condensa_tensor &h = tensors[t];
        const condensa_tensor &d = dev[t];
        const size_t n = (size_t)h.numel;
        if (n == 0) continue;
        if (op != CONDENSA_OP_LAGRANGE) {
            CU_TRY(ctx, cudaMemcpyAsync(h.theta, d.theta, n * 4, cudaMemcpyDeviceToHost, stream));
            if (h.mask) CU_TRY(ctx, cudaMemcpyAsync(h.mask, d.mask, n, cudaMemcpyDeviceToHost, stream));
            if (h.theta_h) CU_TRY(ctx, cudaMemcpyAsync(h.theta_h, d.theta_h, n * 2, cudaMemcpyDeviceToHost, stream));
        }
        if (h.lambda && (fuse & CONDENSA_FUSE_LAMBDA))
            CU_TRY(ctx, cudaMemcpyAsync(h.lambda, d.lambda, n * 4, cudaMemcpyDeviceToHost, stream));
        if (h.grad && (fuse & CONDENSA_FUSE_PENALTY))
            CU_TRY(ctx, cudaMemcpyAsync(h.grad, d.grad, n * 4, cudaMemcpyDeviceToHost, stream));
    }
    CU_TRY(ctx, cudaStreamSynchronize(stream));
    return CONDENSA_OK;
}

int condensa_get_result(condensa_ctx *ctx, condensa_result *out)
{
    if (!ctx || !out) return CONDENSA_ERR_INVALID_ARG;
    if (!ctx->has_result || !ctx->ctl) return fail(ctx, CONDENSA_ERR_INVALID_ARG, "no ranking call has run on this context");
    CU_TRY(ctx, cudaSetDevice(ctx->device));
    CU_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    CU_TRY(ctx, cudaMemcpy(out, &ctx->ctl->res, sizeof(*out), cudaMemcpyDeviceToHost));
    {
        u64 rep = 0;
        CU_TRY(ctx, cudaMemcpy(&rep, &ctx->ctl->n_repaired, sizeof(rep), cudaMemcpyDeviceToHost));
        out->n_repaired = (int64_t)rep;
    }
    if (out->status == 0 && out->n_keep > 0) {
        // the index of the weakest kept unit as the kernels left it in the control block (the
        // register-resident route finds it by an atomic maximum when every tie is kept)
        u64 tid = 0;
        CU_TRY(ctx, cudaMemcpy(&tid, &ctx->ctl->tau_id, sizeof(tid), cudaMemcpyDeviceToHost));
        out->tau_id = (int64_t)tid;
    }
    if (out->status != 0) {
        int code = 0;
        cudaMemcpy(&code, &ctx->ctl->sel.error, sizeof(int), cudaMemcpyDeviceToHost);
        return fail(ctx, CONDENSA_ERR_INTERNAL, "device-side selection check failed (check %d)", code);
    }
    return CONDENSA_OK;
}

int condensa_profile_enable(condensa_ctx *ctx, int on)
{
    if (!ctx) return CONDENSA_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    if (ctx->prof_on) prof_collect(ctx);
    ctx->prof_on = on != 0;
    if (on) {
        std::fill(ctx->prof_ms.begin(), ctx->prof_ms.end(), 0.0);
        std::fill(ctx->prof_cnt.begin(), ctx->prof_cnt.end(), 0);
    }
    return CONDENSA_OK;
}

int condensa_profile_read(condensa_ctx *ctx, condensa_kernel_time *out, int max_entries, int *n_out)
{
    if (!ctx || !out || !n_out || max_entries < 0) return CONDENSA_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    prof_collect(ctx);
    int n = 0;
    for (size_t i = 0; i < ctx->prof_names.size() && n < max_entries; ++i) {
        if (!ctx->prof_cnt[i]) continue;
        memset(&out[n], 0, sizeof(out[n]));
        strncpy(out[n].name, ctx->prof_names[i].c_str(), sizeof(out[n].name) - 1);
        out[n].launches = ctx->prof_cnt[i];
        out[n].total_ms = ctx->prof_ms[i];
        ++n;
    }
    *n_out = n;
    return CONDENSA_OK;
}

int64_t condensa_launch_count(const condensa_ctx *ctx) { return ctx ? ctx->launches : 0; }

// ---------------------------------------------------------------- no-allocation variant
// Scratch of condensa_cstep_prune_noalloc(): selection state, histograms, the
// one-tensor descriptor and a candidate list for up to
// CONDENSA_NOALLOC_MAX_NUMEL elements. It is part of the loaded module, so
// every GPU that loads this library holds these bytes until the process exits.
constexpr size_t NOALLOC_SCRATCH_BYTES = 2304u * 1024u;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

namespace {

// Upper bound of make_layout() for one tensor of CONDENSA_NOALLOC_MAX_NUMEL elements:
// control block, three histograms, three final-buffer arrays, descriptor area, two
// list arrays of S / 8 entries, each rounded up to 256 bytes.
constexpr size_t noalloc_up(size_t x) { return (x + 255) / 256 * 256; }
constexpr size_t NOALLOC_LAYOUT_MAX =
    noalloc_up(sizeof(Ctl)) + noalloc_up(sizeof(u64) * 3 * NBINS) + 3 * noalloc_up(sizeof(u64) * FIN) +
    noalloc_up(sizeof(TensorDesc) + 4 * sizeof(long long)) + 2 * noalloc_up(sizeof(u64) * (CONDENSA_NOALLOC_MAX_NUMEL / 8));
static_assert(CONDENSA_NOALLOC_MAX_NUMEL / 8 >= 65536, "the list capacity rule of build_plan is S / 8 from this size on");
static_assert(NOALLOC_LAYOUT_MAX <= NOALLOC_SCRATCH_BYTES, "the built-in scratch must hold the largest accepted input");

constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;                          // guards the once-per-device set-up and the error text
unsigned char *g_noalloc_ptr[NOALLOC_MAX_DEVICES];   // device address of the scratch, per device
int g_noalloc_occ[NOALLOC_MAX_DEVICES];
int g_noalloc_occ_small[NOALLOC_MAX_DEVICES];
int g_noalloc_sms[NOALLOC_MAX_DEVICES];
size_t g_noalloc_ctl_off[NOALLOC_MAX_DEVICES];       // where the last call on the device put its control block
cudaStream_t g_noalloc_stream[NOALLOC_MAX_DEVICES];

// Writes the descriptor of the single tensor and its two work-item prefix
// arrays into the scratch (the regular path copies them from pinned memory).
__global__ void k_noalloc_setup(TensorDesc d, long long items, TensorDesc *td, long long *prefix)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *td = d;
        prefix[0] = 0; prefix[1] = items;     // scan decomposition
        prefix[2] = 0; prefix[3] = items;     // projection decomposition
    }
}

int noalloc_fail(int code, const char *text)
{
    std::lock_guard<std::mutex> lk(g_noalloc_mutex);
    g_create_error = text;
    return code;
}

}  // namespace

int condensa_cstep_prune_noalloc(const condensa_tensor *tensor, double sparsity, float mu,
                                 unsigned fuse, void *stream_)
{
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!tensor) return noalloc_fail(CONDENSA_ERR_INVALID_ARG, "tensor is NULL");
    if (tensor->numel > CONDENSA_NOALLOC_MAX_NUMEL)
        return noalloc_fail(CONDENSA_ERR_TOO_LARGE,
                            "condensa_cstep_prune_noalloc: numel exceeds CONDENSA_NOALLOC_MAX_NUMEL "
                            "(the built-in scratch is fixed); use condensa_cstep_prune with a context");
    {
        condensa_ctx checker;      // host-only object: collects the text of an argument error
        const int rc = validate(&checker, OP_PRUNE, tensor, 1, sparsity, mu, fuse);
        if (rc) return noalloc_fail(rc, checker.err.c_str());
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return noalloc_fail(CONDENSA_ERR_UNSUPPORTED, "device index too large");
    {
        std::unique_lock<std::mutex> lk(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            // Once per device, with that device current: the array's name is only a
            // host-side handle here; kernels need the address the runtime maps it to.
            unsigned char *p = nullptr;
            e = cudaGetSymbolAddress((void **)&p, g_noalloc_scratch);
            int sms = 0, coop = 0;
            if (e == cudaSuccess && p) {
                cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
                cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
            }
            if (e != cudaSuccess || !p || !coop || sms <= 0) {
                lk.unlock();
                return noalloc_fail(e != cudaSuccess || !p ? CONDENSA_ERR_CUDA : CONDENSA_ERR_UNSUPPORTED,
                                    e != cudaSuccess ? cudaGetErrorString(e) : "device lacks cooperative launch");
            }
            g_noalloc_occ[dev] = occupancy(k_select<SRC_ELEM>);
            g_noalloc_occ_small[dev] = occupancy(k_prune_small);
            g_noalloc_sms[dev] = sms;
            g_noalloc_ptr[dev] = p;
        }
    }
    Plan pl;
    build_plan(OP_PRUNE, tensor, 1, pl);
    const Layout L = make_layout(1, pl, true, false);
    if (L.total > NOALLOC_SCRATCH_BYTES) return noalloc_fail(CONDENSA_ERR_TOO_LARGE, "scratch layout exceeds the built-in array");
    unsigned char *ws = g_noalloc_ptr[dev];

    Params P;
    memset(&P, 0, sizeof(P));
    P.td = (const TensorDesc *)(ws + L.desc);
    long long *prefix = (long long *)(ws + L.desc + sizeof(TensorDesc));
    P.T = 1;
    P.mu = mu;
    P.fuse = fuse & FUSE_KERNEL_BITS;
    P.ctl = (Ctl *)(ws + L.ctl);
    P.hist = (u64 *)(ws + L.hist);
    P.fin_key = (u64 *)(ws + L.fin_key);
    P.fin_id = (u64 *)(ws + L.fin_id);
    P.fin_idx = (u64 *)(ws + L.fin_idx);
    P.list_key = (u64 *)(ws + L.list_key);
    P.list_id = (u64 *)(ws + L.list_id);
    P.cap = pl.cap;
    P.S = pl.S;
    P.bits_key = 31;
    P.item_prefix = prefix;
    P.n_items = pl.n_items_a;

    const long long Z = (long long)std::min<double>((double)pl.S, std::max(0.0, std::floor(sparsity * (double)pl.S + 0.5)));
    Sel init = initial_state(pl.S, pl.S - Z, 31);
    int do_list0 = (u64)pl.S <= pl.cap ? 1 : 0;
    const int sms = g_noalloc_sms[dev];

    k_noalloc_setup<<<1, 32, 0, stream>>>(pl.td[0], pl.n_items_a, (TensorDesc *)(ws + L.desc), prefix);
    if ((e = cudaGetLastError()) != cudaSuccess) return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    if (pl.n_items_b > 0 && pl.n_items_b <= 2ll * sms && g_noalloc_occ_small[dev] >= 2) {
        // at most one work item per resident CTA: the list stays in registers for the whole call
        P.item_prefix = prefix + 2;
        P.n_items = pl.n_items_b;
        dim3 grid((unsigned)(2 * sms)), block(THREADS);
        void *args[] = {(void *)&P, (void *)&init};
        e = cudaLaunchCooperativeKernel((const void *)k_prune_small, grid, block, args, 0, stream);
        if (e != cudaSuccess) return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    } else {
        // one cooperative launch: clears what the last call left in the scratch, ranks, projects
        dim3 grid((unsigned)(sms * std::min(g_noalloc_occ[dev], 2))), block(THREADS);
        int pre_scan = 1, post_apply = 2, do_init = 1;
        const long long *prefix_b = prefix + 2;
        long long items_b = pl.n_items_b;
        void *args[] = {(void *)&P, (void *)&do_list0, (void *)&pre_scan, (void *)&prefix_b, (void *)&items_b,
                        (void *)&post_apply, (void *)&do_init, (void *)&init};
        e = cudaLaunchCooperativeKernel((const void *)k_select<SRC_ELEM>, grid, block, args, 0, stream);
        if (e != cudaSuccess) return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    }
    {
        std::lock_guard<std::mutex> lk(g_noalloc_mutex);
        g_noalloc_ctl_off[dev] = L.ctl;
        g_noalloc_stream[dev] = stream;
    }
    return CONDENSA_OK;
}

int condensa_noalloc_status(void)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES || !g_noalloc_ptr[dev])
        return noalloc_fail(CONDENSA_ERR_INVALID_ARG, "condensa_cstep_prune_noalloc has not run on this device");
    if ((e = cudaStreamSynchronize(g_noalloc_stream[dev])) != cudaSuccess)
        return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    int status = 0;
    const Ctl *ctl = (const Ctl *)(g_noalloc_ptr[dev] + g_noalloc_ctl_off[dev]);
    if ((e = cudaMemcpy(&status, &ctl->res.status, sizeof(int), cudaMemcpyDeviceToHost)) != cudaSuccess)
        return noalloc_fail(CONDENSA_ERR_CUDA, cudaGetErrorString(e));
    if (status != 0) return noalloc_fail(CONDENSA_ERR_INTERNAL, "device-side selection check failed in the last allocation-free call");
    return CONDENSA_OK;
}

const char *condensa_last_error(const condensa_ctx *ctx)
{
    return ctx ? ctx->err.c_str() : g_create_error.c_str();
}

}  // extern "C"
