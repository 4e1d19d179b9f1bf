// Single-pass projection for bh x bw blocks of matrices (block shapes other than 4 x 4, which
// has its own kernel): the sample bracket, one pass that writes everything, the exact selection
// on the listed candidates. A block row - bh matrix rows - is one contiguous range of memory,
// so the pass moves whole block rows through shared memory exactly like the 4 x 4 kernel
// does; only the per-block arithmetic differs: unrolled at compile time for the shapes the
// kernel is built for, loops over the rows and columns that exist for a block of ragged width,
// always in row-major order (the order of the plain definition).
#pragma once
#include "fused_fast.cuh"

namespace cs {

// Shared memory of a CTA: `stages` tile buffers (w, lambda: `arr` bytes each; mask: arr / 4 + 16
// bytes, the tile's mask starts at the byte offset its global address has inside a 16-byte line,
// so that the aligned interior can leave by one bulk copy), then the candidate staging of each
// consumer group (BG_CAND keys, ids and blocks of jr_floats original multipliers; a candidate
// that finds it full goes to the list directly).
// The consumer warps may form several groups that work on different tiles at the same time
// (measured on 5 x 5 blocks of 1500-column matrices: two groups of ten warps at 80 registers
// were slower than one group of twelve at 128).
constexpr int BG_GROUPS = 1;
constexpr int BG_GWARPS = 12;                                   // warps of a group: 384 blocks of a tile at a time
constexpr int BG_CWARPS = BG_GROUPS * BG_GWARPS;                // consumer warps
constexpr int BG_THREADS = (BG_CWARPS + 1) * 32;                // + the producer warp
constexpr int BG_MAX_STAGES = 4;
// (The append stops the whole group for the round trip of one atomic on a word every CTA of the
// grid adds to - microseconds - so it should be rare: 64 / 24 entries instead of 144 / 104 cost
// 7 % of the kernel's time on 5 x 5 blocks. Two variants that take the wait off the group - the
// answer of the atomic picked up one tile later, or the copy done by one warp while the others
// go on - were measured slower: that warp is then late for the next tile's barriers.)
constexpr u32 BG_CAND = 144;        // staged candidates of a group
constexpr u32 BG_FLUSH = 104;       // ... appended to the list once there are more than this many

struct BlockGShared {
    u32 hist[NBINS];
    u64 red[BG_CWARPS];
    u64 flush_base[BG_GROUPS];
    u32 ccount[BG_GROUPS];                       // staged candidates of each group
    unsigned long long full_bar[BG_MAX_STAGES];  // bytes of a tile have arrived
    unsigned long long done_bar[BG_MAX_STAGES];  // every warp of the tile's group has finished with the buffer
    int abort;                                   // a bounded wait ran out somewhere in this CTA
    long long tile_prefix[BT_TD_CACHE + 1];
    TensorDesc td[BT_TD_CACHE];
};
__host__ __device__ inline size_t blockg_stage_bytes(int arr) { return (size_t)arr * 2 + (size_t)arr / 4 + 16; }
__host__ __device__ inline size_t blockg_cand_bytes(int jr_floats) { return (size_t)BG_CAND * (16 + 4 * (size_t)jr_floats); }
__host__ __device__ inline size_t blockg_dyn_smem(int arr, int stages, int jr_floats)
{
    return (size_t)stages * blockg_stage_bytes(arr) + (size_t)BG_GROUPS * blockg_cand_bytes(jr_floats);
}

// Block rows of one tile of tensor d: as many as fit a buffer, but no more blocks than the group
// has threads where one block row has fewer (the time of a tile is the time of the longest
// thread: a second block per thread costs as much as another tile).
__host__ __device__ inline long long blockg_rows_per_tile(const TensorDesc &d, int arr)
{
    const long long fit = (long long)arr / ((long long)d.bh * d.d1 * 4);       // >= 1 by blockg_fast_end
    const long long lanes = (long long)(BG_GWARPS * 32) / d.nbc;
    return lanes >= 1 && lanes < fit ? lanes : fit;
}

// Tiles of the aligned interior of tensor d.
__host__ __device__ inline long long blockg_tile_count(const TensorDesc &d, int arr)
{
    if (blockg_fast_end(d, arr) <= 0) return 0;
    const long long nbr = d.d0 / d.bh;
    const long long rpt = blockg_rows_per_tile(d, arr);
    return (nbr + rpt - 1) / rpt;
}

// Rounds of one block per thread that the tiles of tensor d take (what the kernel's time follows).
__host__ __device__ inline long long blockg_tile_rounds(const TensorDesc &d, int arr)
{
    if (blockg_fast_end(d, arr) <= 0) return 0;
    const long long per_tile = (blockg_rows_per_tile(d, arr) * d.nbc + BG_GWARPS * 32 - 1) / (BG_GWARPS * 32);
    return blockg_tile_count(d, arr) * per_tile;
}

struct TileG {
    int t;              // owning tensor
    u32 b0;             // first block (number inside the tensor); block q of the tile is b0 + q
    u32 nq;             // blocks in the tile
    u32 nrows;          // matrix rows in the tile
    u32 off0;           // element offset of the tile's first row
};

__device__ __forceinline__ TileG tile_geom_g(const long long *tile_prefix, const TensorDesc *td, int T, long long tile)
{
    TileG g;
    g.t = find_tensor(tile_prefix, T, tile);
    const TensorDesc &d = td[g.t];
    const u32 bh = (u32)d.bh, C = (u32)d.d1, nbc = (u32)d.nbc, nbr = (u32)d.d0 / bh;     // (fewer than 2^32 elements)
    const u32 local = (u32)(tile - tile_prefix[g.t]);
    const u32 rpt = (u32)d.tile_rows;               // = blockg_rows_per_tile(), worked out by the host
    const u32 brow0 = local * rpt;
    const u32 brows = nbr - brow0 < rpt ? nbr - brow0 : rpt;
    g.nq = brows * nbc;
    g.nrows = bh * brows;
    g.b0 = brow0 * nbc;
    g.off0 = bh * brow0 * C;
    return g;
}

__device__ __forceinline__ void bar_sync_named(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Candidate (key, id) with the original multipliers `lam` of its block (row-major, `n` floats):
// into the CTA's staging, or straight to the list when the staging is full.
struct CandStage {
    u64 *key, *id;
    float *lam;
    u32 *count;         // entries staged so far (may run past BG_CAND: those went to the list directly)
    u64 *base;          // scratch word of the flush
};
__device__ __forceinline__ CandStage blockg_stage_of(unsigned char *cand_buf, int jr_floats, BlockGShared &sh, int group)
{
    CandStage cs;
    cs.key = reinterpret_cast<u64 *>(cand_buf + (size_t)group * blockg_cand_bytes(jr_floats));
    cs.id = cs.key + BG_CAND;
    cs.lam = reinterpret_cast<float *>(cs.id + BG_CAND);
    cs.count = &sh.ccount[group];
    cs.base = &sh.flush_base[group];
    return cs;
}
__device__ __forceinline__ float *blockg_cand_slot(const Params &P, const CandStage &cs, u64 key, u64 id)
{
    const u32 J = (u32)P.jr_floats;
    const u32 slot = atomicAdd(cs.count, 1u);
    if (slot < BG_CAND) {
        cs.key[slot] = key;
        cs.id[slot] = id;
        return cs.lam + slot * J;
    }
    const u64 pos = atomicAdd(&P.ctl->list_count[0], 1ull);
    if (pos >= P.cap) return nullptr;            // (the selection reports the overflow)
    P.list_key[pos] = key;
    P.list_id[pos] = id;
    return P.jr_lam + pos * J;
}

// Appends the staged candidates to the list when there are more than `limit`: `nthreads` threads
// (numbered tid) call this together, synchronised by the named barrier `bar`. Every thread takes
// the same decision, and every call runs the same barriers whatever the outcome.
__device__ __forceinline__ void blockg_cta_flush(const Params &P, const CandStage &cs, int bar, int nthreads, int tid,
                                                 u32 limit)
{
    bar_sync_named(bar, nthreads);              // the staged entries are complete
    const u32 cnt = *cs.count;
    const u32 c = cnt < BG_CAND ? cnt : BG_CAND;
    bar_sync_named(bar, nthreads);              // everybody has read the count
    if (c <= limit) return;
    if (tid == 0) {
        *cs.base = atomicAdd(&P.ctl->list_count[0], (u64)c);
        *cs.count = 0;
    }
    bar_sync_named(bar, nthreads);
    const u64 base = *cs.base;
    for (u32 i = tid; i < c; i += nthreads) {
        const u64 pos = base + i;
        if (pos < P.cap) {
            P.list_key[pos] = cs.key[i];
            P.list_id[pos] = cs.id[i];
        }
    }
    const u32 J = (u32)P.jr_floats;
    for (u32 i = tid; i < c * J; i += nthreads) {
        const u64 pos = base + i / J;
        if (pos < P.cap) P.jr_lam[pos * J + (i % J)] = cs.lam[i];
    }
    bar_sync_named(bar, nthreads);              // the staging may be filled again
}

// One block of a tile in shared memory: norm, decision, outputs in place. BH x BW (when not 0)
// is the block shape at compile time: blocks of full width then run without loops or address
// arithmetic, with u kept in registers between the norm and the outputs.
struct BlockJob {
    u32 nc, bh, bw, C;              // columns that exist; block shape; row pitch (the matrix width)
    u32 base, goff;                 // element offset of the block in the tile; of the tile in the tensor
    u64 id;
    float *sw, *sl;
    unsigned char *sm;
    bool mstage, has_lam, upd;
};

template <bool H, bool G, int BH, int BW>
__device__ __forceinline__ u32 blockg_one(const Params &P, const TensorDesc &d, const BlockJob &jb, const Bracket &br,
                                          float mu, int fp16, u32 *hist, const CandStage &cs)
{
    if (BH > 0 && jb.nc == (u32)BW) {
        constexpr int RB = BH > 0 ? BH : 1, CB = BW > 0 ? BW : 1, N = RB * CB;
        float w[N], l[N], u[N];
        u32 nz = 0;
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int c = 0; c < CB; ++c) {
                const u32 o = jb.base + r * jb.C + c;
                w[r * CB + c] = jb.sw[o];
                l[r * CB + c] = jb.has_lam ? jb.sl[o] : 0.0f;
                nz |= __float_as_uint(l[r * CB + c]);
            }
        if (nz) {                       // one decision per block keeps the code free of branches per element
#pragma unroll
            for (int i = 0; i < N; ++i) u[i] = __fsub_rn(w[i], __fdiv_rn(l[i], mu));
        } else {                        // every lambda is +0: u is w, bit for bit
#pragma unroll
            for (int i = 0; i < N; ++i) u[i] = w[i];
        }
        double acc = 0.0;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const double x = (double)u[i];
            acc = __fma_rn(x, x, acc);
        }
        const u64 key = (u64)__double_as_longlong(acc);
        const bool keep = key >= br.guess;
        if (key >= br.lo && key <= br.hi) {
            float *jl = blockg_cand_slot(P, cs, key, jb.id);
            if (jl) {
#pragma unroll
                for (int i = 0; i < N; ++i) jl[i] = l[i];
            }
            atomicAdd(&hist[bracket_bin(br, key, jb.id)], 1u);
        }
        if (jb.mstage && jb.upd && !H && !G) {
            // the common case without side outputs: everything stays in shared memory
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int c = 0; c < CB; ++c) {
                    const int i = r * CB + c;
                    const u32 o = jb.base + r * jb.C + c;
                    const float th = keep ? u[i] : 0.0f;
                    jb.sw[o] = th;
                    jb.sl[o] = __fsub_rn(l[i], __fmul_rn(mu, __fsub_rn(w[i], th)));
                    jb.sm[o] = keep ? 1 : 0;
                }
            return key > br.hi ? 1u : 0u;
        }
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int c = 0; c < CB; ++c) {
                const int i = r * CB + c;
                const u32 o = jb.base + r * jb.C + c, go = jb.goff + jb.base + r * jb.C + c;
                const Out out = finish_lean<H>(w[i], l[i], u[i], keep, mu, fp16, jb.upd);
                jb.sw[o] = out.theta;
                if (jb.upd) jb.sl[o] = out.lam;
                if (jb.mstage) jb.sm[o] = out.m;
                else if (d.mask) d.mask[go] = out.m;
                if (H && d.theta_h) d.theta_h[go] = out.th;
                if (G && d.grad) d.grad[go] = out.grad;
            }
        return key > br.hi ? 1u : 0u;
    }
    // any shape, ragged width: loops over the rows and the columns that exist
    double acc = 0.0;
    for (u32 r = 0; r < jb.bh; ++r)
        for (u32 c = 0; c < jb.nc; ++c) {
            const u32 o = jb.base + r * jb.C + c;
            const double x = (double)form_u(jb.sw[o], jb.has_lam ? jb.sl[o] : 0.0f, mu, jb.has_lam);
            acc = __fma_rn(x, x, acc);
        }
    const u64 key = (u64)__double_as_longlong(acc);
    const bool keep = key >= br.guess;
    if (key >= br.lo && key <= br.hi) {
        float *jl = blockg_cand_slot(P, cs, key, jb.id);
        if (jl)
            for (u32 r = 0; r < jb.bh; ++r)
                for (u32 c = 0; c < jb.nc; ++c)
                    jl[r * jb.bw + c] = jb.has_lam ? jb.sl[jb.base + r * jb.C + c] : 0.0f;
        atomicAdd(&hist[bracket_bin(br, key, jb.id)], 1u);
    }
    for (u32 r = 0; r < jb.bh; ++r)
        for (u32 c = 0; c < jb.nc; ++c) {
            const u32 o = jb.base + r * jb.C + c, go = jb.goff + jb.base + r * jb.C + c;
            const float w = jb.sw[o], l = jb.has_lam ? jb.sl[o] : 0.0f;
            const Out out = finish_lean<H>(w, l, form_u(w, l, mu, jb.has_lam), keep, mu, fp16, jb.upd);
            jb.sw[o] = out.theta;
            if (jb.upd) jb.sl[o] = out.lam;
            if (jb.mstage) jb.sm[o] = out.m;
            else if (d.mask) d.mask[go] = out.m;
            if (H && d.theta_h) d.theta_h[go] = out.th;
            if (G && d.grad) d.grad[go] = out.grad;
        }
    return key > br.hi ? 1u : 0u;
}

template <bool H, bool G, int BH, int BW>
__global__ void __launch_bounds__(BG_THREADS, 1) k_fused_blockg(Params P)
{
    __shared__ BlockGShared sh;
    extern __shared__ __align__(128) unsigned char dyn_smem[];      // tile buffers, then the candidate staging
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int arr = P.bt_arr_bytes, n_stages = P.bt_stages;
    const size_t stage_bytes = blockg_stage_bytes(arr);
    unsigned char *tile_buf = dyn_smem;
    unsigned char *cand_buf = dyn_smem + (size_t)n_stages * stage_bytes;      // candidate staging of the CTA
    for (int i = threadIdx.x; i < NBINS; i += BG_THREADS) sh.hist[i] = 0;
    if (threadIdx.x < BG_GROUPS) sh.ccount[threadIdx.x] = 0;
    if (threadIdx.x == 0) sh.abort = 0;
    const bool cached = P.T <= BT_TD_CACHE;
    if (cached) {
        for (int i = threadIdx.x; i <= P.T; i += BG_THREADS) sh.tile_prefix[i] = P.tile_prefix[i];
        const int words = P.T * (int)(sizeof(TensorDesc) / sizeof(u32));
        const u32 *src = reinterpret_cast<const u32 *>(P.td);
        u32 *dst = reinterpret_cast<u32 *>(sh.td);
        for (int i = threadIdx.x; i < words; i += BG_THREADS) dst[i] = src[i];
    }
    if (threadIdx.x < n_stages) {
        mbar_init(smem_u32(&sh.full_bar[threadIdx.x]), 1);
        mbar_init(smem_u32(&sh.done_bar[threadIdx.x]), BG_GWARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const long long *tile_prefix = cached ? sh.tile_prefix : P.tile_prefix;
    const TensorDesc *td = cached ? sh.td : P.td;
    const int fp16 = quant_code(P.fuse);
    const float mu = P.mu;
    volatile int *abort_flag = &sh.abort;
    u64 na = 0;
    Bracket br;
    memset(&br, 0, sizeof(br));
    bool onepass = false;
    if (warp < BG_CWARPS) {
        pdl_wait();
        onepass = P.ctl->sel.onepass != 0;      // else the sampler advised against the single pass
        br = load_bracket(P.ctl->sel);
    }
    const u32 S_ = (u32)n_stages;

    if (warp == BG_CWARPS) {
        // ------------------------------------------------------------ producer (one lane)
        if (lane == 0) {
            u32 k = 0;
            bool ok = true, dep_seen = false, quiet = false;
            auto see_dependency = [&]() {       // before the first store and before leaving
                if (dep_seen) return;
                pdl_wait();
                dep_seen = true;
                if (!P.ctl->sel.onepass) { quiet = true; ok = false; }
            };
            auto store_tile = [&](long long tile, int stage) {
                const TileG g = tile_geom_g(tile_prefix, td, P.T, tile);
                const TensorDesc &d = td[g.t];
                const bool upd = (P.fuse & FUSE_LAMBDA) && d.lam != nullptr;
                const u32 bytes = g.nrows * (u32)d.d1 * 4u;
                unsigned char *sbp = tile_buf + (size_t)stage * stage_bytes;
                const u32 sb = smem_u32(sbp);
                bulk_store_1d(d.theta + g.off0, sb, bytes);
                if (upd) bulk_store_1d(d.lam + g.off0, sb + (u32)arr, bytes);
                if (d.mask && ((uintptr_t)d.mask & 15u) == 0) {
                    // the 16-byte aligned interior of the tile's mask by one bulk copy, the ragged ends byte by byte
                    const u32 n = bytes / 4u, m0 = g.off0, m1 = g.off0 + n;
                    const u32 a = (m0 + 15u) & ~15u, e = m1 & ~15u;
                    const unsigned char *smk = sbp + 2 * (size_t)arr + (m0 & 15u);     // mask byte of element m0
                    if (e > a) {
                        bulk_store_1d(d.mask + a, sb + 2u * (u32)arr + (m0 & 15u) + (a - m0), e - a);
                        for (u32 i = m0; i < a; ++i) d.mask[i] = smk[i - m0];
                        for (u32 i = e; i < m1; ++i) d.mask[i] = smk[i - m0];
                    } else {
                        for (u32 i = m0; i < m1; ++i) d.mask[i] = smk[i - m0];
                    }
                }
                bulk_commit();
            };
            long long tile = blockIdx.x;
#pragma unroll 1
            for (; tile < P.n_tiles && ok; tile += gridDim.x, ++k) {
                const int stage = (int)(k % S_);
                if (k >= S_) {
                    see_dependency();
                    if (!ok) break;
                    ok = mbar_wait_bounded(smem_u32(&sh.done_bar[stage]), ((k / S_) - 1u) & 1u, abort_flag);
                    if (!ok) break;
                    store_tile(tile - (long long)S_ * gridDim.x, stage);
                    bulk_wait_read_all();               // shared memory has been read: the buffer is free
                }
                if (*abort_flag) { ok = false; break; }
                const TileG g = tile_geom_g(tile_prefix, td, P.T, tile);
                const TensorDesc &d = td[g.t];
                const bool has_lam = d.lam != nullptr;
                const u32 bytes = g.nrows * (u32)d.d1 * 4u;
                const u32 bar = smem_u32(&sh.full_bar[stage]);
                const u32 sb = smem_u32(tile_buf + (size_t)stage * stage_bytes);
                mbar_arrive_expect_tx(bar, (has_lam ? 2u : 1u) * bytes);
                bulk_load_1d(sb, d.w + g.off0, bytes, bar);
                if (has_lam) bulk_load_1d(sb + (u32)arr, d.lam + g.off0, bytes, bar);
            }
            const u32 issued = k;                       // tiles whose loads have been issued
            see_dependency();
            if (ok) {                                   // drain: the last tiles still sit in their buffers
                const u32 first = issued > S_ ? issued - S_ : 0u;
                for (u32 j = first; j < issued && ok; ++j) {
                    const int stage = (int)(j % S_);
                    ok = mbar_wait_bounded(smem_u32(&sh.done_bar[stage]), (j / S_) & 1u, abort_flag);
                    if (ok) store_tile((long long)blockIdx.x + (long long)j * gridDim.x, stage);
                }
            }
            if (!ok) {
                // a wait ran out (or the single pass is off: `quiet`): the loads still in flight get the
                // same bounded time, so that none lands in shared memory after this CTA has gone
                *abort_flag = 1;
                if (!quiet) atomicExch(&P.ctl->async_error, 1);
                const u32 first = issued > S_ ? issued - S_ : 0u;
                for (u32 j = first; j < issued; ++j)
                    (void)mbar_wait_bounded(smem_u32(&sh.full_bar[j % S_]), (j / S_) & 1u, nullptr);
            }
            bulk_wait_all();                            // every store has left shared memory and is performed
        }
    } else {
        // ------------------------------------------------------------ consumers
        // Group `grp` takes the tiles k = grp, grp + BG_GROUPS, ... of this CTA. Every warp of a
        // group runs every iteration and every barrier of its loop, also after a wait has run
        // out (it then only skips the work): the flush below synchronises the group.
        const int grp = warp / BG_GWARPS, gw = warp - grp * BG_GWARPS;
        const int gtid = gw * 32 + lane, gthreads = BG_GWARPS * 32;
        const CandStage cs = blockg_stage_of(cand_buf, P.jr_floats, sh, grp);
        u32 n_above = 0;
        bool ok = true;
#pragma unroll 1
        for (u32 k = (u32)grp; onepass && (long long)blockIdx.x + (long long)k * gridDim.x < P.n_tiles; k += (u32)BG_GROUPS) {
            const long long tile = (long long)blockIdx.x + (long long)k * gridDim.x;
            const int stage = (int)(k % S_);
            if (ok && (*abort_flag || !mbar_wait_bounded(smem_u32(&sh.full_bar[stage]), (k / S_) & 1u, abort_flag))) {
                ok = false;
                if (lane == 0 && !*abort_flag) {
                    *abort_flag = 1;
                    atomicExch(&P.ctl->async_error, 1);
                }
            }
            if (ok) {
                const TileG g = tile_geom_g(tile_prefix, td, P.T, tile);
                const TensorDesc &d = td[g.t];
                const bool has_lam = d.lam != nullptr;
                const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
                const bool mstage = d.mask && ((uintptr_t)d.mask & 15u) == 0;      // the producer stores the mask
                const u32 C = (u32)d.d1, bh = (u32)d.bh, bw = (u32)d.bw, nbc = (u32)d.nbc;
                unsigned char *sbp = tile_buf + (size_t)stage * stage_bytes;
                float *sw = reinterpret_cast<float *>(sbp);
                float *sl = reinterpret_cast<float *>(sbp + arr);
                unsigned char *sm = sbp + 2 * (size_t)arr + (g.off0 & 15u);
#pragma unroll 1
                for (u32 q = (u32)gtid; q < g.nq; q += (u32)gthreads) {
                    BlockJob jb;
                    const u32 brl = q / nbc, bcol = q - brl * nbc;
                    const u32 c0 = bcol * bw;
                    jb.nc = C - c0 < bw ? C - c0 : bw;
                    jb.bh = bh; jb.bw = bw; jb.C = C;
                    jb.base = brl * bh * C + c0;
                    jb.goff = g.off0;
                    jb.id = (u64)d.unit_prefix + g.b0 + q;
                    jb.sw = sw; jb.sl = sl; jb.sm = sm;
                    jb.mstage = mstage; jb.has_lam = has_lam; jb.upd = upd;
                    n_above += blockg_one<H, G, BH, BW>(P, d, jb, br, mu, fp16, sh.hist, cs);
                }
                fence_proxy_async();                    // the bulk stores of the producer read these writes
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.done_bar[stage]));
            }
            blockg_cta_flush(P, cs, 1 + grp, gthreads, gtid, BG_FLUSH);
        }
        blockg_cta_flush(P, cs, 1 + grp, gthreads, gtid, 0);
        na = n_above;
    }
    __syncthreads();
    pdl_wait();
    if (!P.ctl->sel.onepass) return;         // (the same for every thread)
    // the blocks outside the aligned interior (ragged last block rows, unaligned or too wide
    // tensors) and the tensors that pass through: work items listed by the host, generic code
    if (P.n_edge_items > 0) {
        const CandStage cs = blockg_stage_of(cand_buf, P.jr_floats, sh, 0);
        for (long long i = blockIdx.x; i < P.n_edge_items; i += gridDim.x) {
            const long long item = P.edge_items[i];
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc g = P.td[t];
            const long long local = item - P.item_prefix[t];
            if (!g.ranked) {
                if (threadIdx.x < THREADS) process_linear_item<M_KEEPALL>(P, g, local, 0, 0);
                continue;
            }
            const long long b = local * BLOCKS_PER_ITEM + warp * 32 + lane;         // 8 warps x 32 blocks make one item
            if (warp < BLOCKS_PER_ITEM / 32 && b < g.n_units && b >= blockg_fast_end(g, arr)) {
                const u64 key = blockg_key_global(g, b, mu);
                const u64 id = (u64)(g.unit_prefix + b);
                na += key > br.hi ? 1 : 0;
                if (key >= br.lo && key <= br.hi) {
                    float *jl = blockg_cand_slot(P, cs, key, id);
                    const BlockExt e = blockg_ext(g, b);
                    if (jl)
                        for (int r = 0; r < e.nr; ++r)
                            for (int c = 0; c < e.nc; ++c)
                                jl[r * g.bw + c] = g.lam ? g.lam[(e.r0 + r) * g.d1 + e.c0 + c] : 0.0f;
                    atomicAdd(&sh.hist[bracket_bin(br, key, id)], 1u);
                }
                blockg_write_global(P, g, b, key >= br.guess, nullptr, 0, 1);
            }
            blockg_cta_flush(P, cs, 1 + BG_GROUPS, BG_THREADS, threadIdx.x, 0);
        }
    }
    if (warp < BG_CWARPS) {
        for (int o = 16; o > 0; o >>= 1) na += __shfl_xor_sync(0xffffffffu, na, o);
        if (lane == 0) sh.red[warp] = na;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < BG_CWARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += BG_THREADS) {
        const u32 hc = sh.hist[i];
        if (hc) atomicAdd(&P.hist[i], (u64)hc);
    }
}

}  // namespace cs
