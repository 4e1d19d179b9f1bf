// Aligned interior work items of the single-pass projection: the kernels that
// move almost all of the bytes. No CTA-wide barrier inside the item loop:
// candidates are staged per warp in shared memory and flushed to the list with
// one global atomic per flush.
#pragma once
#include "common.cuh"
#include "fused.cuh"

namespace cs {

// ---------------------------------------------------------------- unstructured
constexpr int ESTG = 64;        // staged candidates per warp

struct ElemFastShared {
    u32 hist[NBINS];            // the first four members mirror FusedShared (edge items reuse them)
    u32 cnt[2];
    u64 base[2];
    u64 red[WARPS];
    u32 wcount[WARPS];
    u64 id[WARPS][ESTG];
    u32 key[WARPS][ESTG];
    float lam[WARPS][ESTG];
};

// The journal entry is written for every staged candidate: entries staged by an
// earlier item of this CTA may belong to another tensor (one with multipliers)
// than the item that triggers the flush; tensors without multipliers stage 0.
__device__ __forceinline__ void elem_flush(const Params &P, ElemFastShared &sh, u32 limit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncwarp();
    u32 c = sh.wcount[warp];
    if (c > limit) {
        if (c > ESTG) c = ESTG;        // entries past the staging area went straight to the list
        u64 base = 0;
        if (lane == 0) base = atomicAdd(&P.ctl->list_count[0], (u64)c);
        base = __shfl_sync(0xffffffffu, base, 0);
        for (u32 i = lane; i < c; i += 32) {
            const u64 pos = base + i;
            if (pos < P.cap) {
                P.list_key[pos] = (u64)sh.key[warp][i];
                P.list_id[pos] = sh.id[warp][i];
                P.jr_lam[pos] = sh.lam[warp][i];
            }
        }
        __syncwarp();
        if (lane == 0) sh.wcount[warp] = 0;
    }
    __syncwarp();
}

template <bool H, bool G>
__global__ void __launch_bounds__(THREADS, 3) k_fused_elem(Params P)
{
    __shared__ ElemFastShared sh;
    for (int i = threadIdx.x; i < NBINS; i += THREADS) sh.hist[i] = 0;
    if (threadIdx.x < WARPS) sh.wcount[threadIdx.x] = 0;
    pdl_wait();                     // the sampler's bracket and cleared counters are needed from here on
    if (!P.ctl->sel.onepass) return;
    const Bracket br = load_bracket(P.ctl->sel);
    __syncthreads();
    const int fp16 = quant_code(P.fuse);     // quantisation of theta
    const u32 lo = (u32)br.lo, range = (u32)br.hi - (u32)br.lo, guess = (u32)br.guess;
    const float mu = P.mu;
    const int warp = threadIdx.x >> 5;
    u32 n_above = 0;
    long long t_first = 0, t_end = -1, fast_lo = 0, fast_hi = 0;
    struct { const float *w; float *lam, *theta, *grad; uint8_t *mask; uint16_t *theta_h; long long elem_prefix; int pad; } d;
    d.w = nullptr; d.lam = d.theta = d.grad = nullptr; d.mask = nullptr; d.theta_h = nullptr;
    d.elem_prefix = 0; d.pad = 0;
    for (long long item = blockIdx.x; item < P.n_items; item += gridDim.x) {
        if (item >= t_end) {        // look the tensor up only when the items leave it
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc &g = P.td[t];
            t_first = P.item_prefix[t];
            t_end = P.item_prefix[t + 1];
            // fast items form a range of local indices (same rule as elem_item_is_fast)
            fast_lo = g.pad ? 1 : 0;
            fast_hi = g.vec_ok ? (g.numel + g.pad) / (4 * GROUPS_PER_ITEM) : 0;
            d.w = g.w; d.lam = g.lam; d.theta = g.theta; d.grad = g.grad; d.mask = g.mask; d.theta_h = g.theta_h;
            d.elem_prefix = g.elem_prefix; d.pad = g.pad;
        }
        const long long local = item - t_first;
        if (local < fast_lo || local >= fast_hi) continue;
        const long long e_base = 4 * (local * GROUPS_PER_ITEM) - d.pad;
        const bool has_lam = d.lam != nullptr;
        const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
        const float4 *wp = reinterpret_cast<const float4 *>(d.w + e_base) + threadIdx.x;
        float4 wv[LIN_UNROLL], lv[LIN_UNROLL];
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) wv[it] = __ldg(wp + it * THREADS);
        if (has_lam) {
            const float4 *lp = reinterpret_cast<const float4 *>(d.lam + e_base) + threadIdx.x;
#pragma unroll
            for (int it = 0; it < LIN_UNROLL; ++it) lv[it] = lp[it * THREADS];
        } else {
#pragma unroll
            for (int it = 0; it < LIN_UNROLL; ++it) lv[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        u32 nkeep = 0, candm = 0;       // candm bit 4*it+j: element lies in the bracket
#pragma unroll
        for (int it = 0; it < LIN_UNROLL; ++it) {
            const float w[4] = {wv[it].x, wv[it].y, wv[it].z, wv[it].w};
            const float l[4] = {lv[it].x, lv[it].y, lv[it].z, lv[it].w};
            float u[4], th[4], ln[4], g[4];
            form_u4(w, l, mu, has_lam, u);
            u32 m = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const u32 key = __float_as_uint(u[j]) & 0x7FFFFFFFu;
                const bool keep = key >= guess;
                th[j] = keep ? u[j] : 0.0f;
                m |= keep ? (1u << (8 * j)) : 0u;
                candm |= (key - lo <= range) ? (1u << (4 * it + j)) : 0u;
            }
            nkeep += __popc(m);
            unsigned short h[4];
            if (H) {
                half4(th, h, fp16 ? fp16 : 1);     // 16-bit code of theta (zeroed entries give +0)
                if (fp16) widen4(h, th, th, fp16);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float p = __fmul_rn(mu, __fsub_rn(w[j], th[j]));
                ln[j] = upd ? __fsub_rn(l[j], p) : l[j];
                g[j] = __fsub_rn(p, ln[j]);
            }
            const long long go = it * THREADS + threadIdx.x;      // group offset inside the item
            reinterpret_cast<float4 *>(d.theta + e_base)[go] = make_float4(th[0], th[1], th[2], th[3]);
            if (d.mask) reinterpret_cast<u32 *>(d.mask + e_base)[go] = m;
            if (H && d.theta_h) reinterpret_cast<uint2 *>(d.theta_h + e_base)[go] =
                make_uint2((u32)h[0] | ((u32)h[1] << 16), (u32)h[2] | ((u32)h[3] << 16));
            if (upd) reinterpret_cast<float4 *>(d.lam + e_base)[go] = make_float4(ln[0], ln[1], ln[2], ln[3]);
            if (G && d.grad) reinterpret_cast<float4 *>(d.grad + e_base)[go] = make_float4(g[0], g[1], g[2], g[3]);
        }
        // the few elements inside the bracket: once per item, from the lambda still in registers
        u32 ncandkeep = 0;
        while (candm) {
            const int qb = __ffs(candm) - 1;
            candm &= candm - 1;
            float ll = 0.0f;
#pragma unroll
            for (int a = 0; a < LIN_UNROLL; ++a) {      // select without indexing the registers
                if (qb == 4 * a + 0) ll = lv[a].x;
                if (qb == 4 * a + 1) ll = lv[a].y;
                if (qb == 4 * a + 2) ll = lv[a].z;
                if (qb == 4 * a + 3) ll = lv[a].w;
            }
            const u32 eo = 4u * (u32)((qb >> 2) * THREADS + threadIdx.x) + (u32)(qb & 3);
            const float ww = __ldg(d.w + e_base + eo);
            // same operations as above: the key comes out bit-identical
            const float uu = (has_lam && __float_as_uint(ll) != 0u) ? __fsub_rn(ww, __fdiv_rn(ll, mu)) : ww;
            const u32 key = __float_as_uint(uu) & 0x7FFFFFFFu;
            const u64 id = (u64)(d.elem_prefix + e_base) + eo;
            ncandkeep += key >= guess ? 1u : 0u;
            atomicAdd(&sh.hist[bracket_bin(br, (u64)key, id)], 1u);
            const u32 slot = atomicAdd(&sh.wcount[warp], 1u);
            if (slot < ESTG) {
                sh.key[warp][slot] = key;
                sh.id[warp][slot] = id;
                sh.lam[warp][slot] = ll;
            } else {
                const u64 pos = atomicAdd(&P.ctl->list_count[0], 1ull);
                if (pos < P.cap) {
                    P.list_key[pos] = (u64)key;
                    P.list_id[pos] = id;
                    if (has_lam) P.jr_lam[pos] = ll;
                }
            }
        }
        n_above += nkeep - ncandkeep;      // keeps that are not candidates lie above the bracket
        elem_flush(P, sh, ESTG / 2);
    }
    elem_flush(P, sh, 0);
    __syncthreads();
    u64 na = n_above;
    // the items outside the aligned fast path (tensor heads and tails, unaligned
    // tensors), listed by the host
    if (P.n_edge_items > 0) {
        FusedShared &fs = reinterpret_cast<FusedShared &>(sh);
        if (threadIdx.x < 2) fs.cnt[threadIdx.x] = 0;
        __syncthreads();
        const long long *prefix_b = P.edge_items + P.n_edge_items;      // [T+1] projection items per tensor
        int par = 0;
        for (long long i = blockIdx.x; i < P.n_edge_items; i += gridDim.x) {
            const long long item = P.edge_items[i];
            const int t = find_tensor(prefix_b, P.T, item);
            const TensorDesc g = P.td[t];
            fused_elem_item_generic<H>(P, g, item - prefix_b[t], fs, br, par, na, fp16);
            par ^= 1;
        }
        __syncthreads();
    }
    // totals of this CTA
    for (int o = 16; o > 0; o >>= 1) na += __shfl_xor_sync(0xffffffffu, na, o);
    if ((threadIdx.x & 31) == 0) sh.red[warp] = na;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < WARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += THREADS) {
        const u32 hc = sh.hist[i];
        if (hc) atomicAdd(&P.hist[i], (u64)hc);
    }
}

// ---------------------------------------------------------------- 4x4 blocks
// The aligned interior of block pruning: all complete block rows of a tensor whose
// arrays are 16-byte aligned, with C % 4 == 0 and fewer than 2^32 elements
// (block_fast_end). The four matrix rows of a block row - and consecutive block
// rows - are one contiguous range of memory, so a CTA takes whole block rows and
// moves them the way a plain copy would:
//
//   producer warp   one-dimensional bulk copies (cp.async.bulk, completion on an
//                   mbarrier; no multicast, no cluster) bring the rows of w and of
//                   lambda of a tile into one of BT_STAGES buffers in shared
//                   memory; when the consumers are done with a buffer, bulk copies
//                   write theta, the updated lambda and the mask, which the
//                   consumers left in the buffer, back to global memory;
//   consumer warps  one lane per block: its four rows from shared memory, the fp64
//                   sum of squares in row-major order, one decision, the outputs
//                   into the same places (16-bit codes and gradient, where asked
//                   for, by ordinary stores), candidates staged per warp.
//
// A tile is as many whole block rows as hold at most BT_BLOCKS blocks (one copy per
// array and direction), or, for matrices wider than that, a column chunk of one block
// row (four copies). Global memory therefore sees long contiguous reads and writes,
// the bytes in flight are set by the ring and not by registers, and no CTA-wide
// barrier sits in the loop: consumers wait for `full[stage]`, the producer for
// `done[stage]`. Every wait is bounded; if one runs out the call ends with an error
// status.
constexpr int BT_CWARPS = 12;                            // consumer warps
constexpr int BT_THREADS = (BT_CWARPS + 1) * 32;         // + the producer warp
constexpr int BT_BLOCKS = BT_CWARPS * 32;                // blocks of one tile at most (384)
constexpr int BT_STAGES = 3;                             // tile buffers of a CTA
constexpr int BT_ARRAY_BYTES = BT_BLOCKS * 64;           // w (or lambda) of one tile
constexpr int BT_MASK_BYTES = BT_BLOCKS * 16;
constexpr int BT_STAGE_BYTES = 2 * BT_ARRAY_BYTES + BT_MASK_BYTES;
constexpr int BT_TD_CACHE = 16;                          // tensors whose descriptors are cached in shared memory
constexpr u32 BT_WAIT_POLLS = 1u << 22;                  // bound of every wait (then the call reports an error)
constexpr int BSTG = 40;        // staged candidate blocks per warp (a warp adds at most 32 per tile)

struct BlockCand {              // candidates staged by one consumer warp
    u64 key[BSTG];
    u64 id[BSTG];
    float4 lam[BSTG][4];
};
constexpr size_t BLOCK_FAST_DYN_SMEM = (size_t)BT_STAGES * BT_STAGE_BYTES + (size_t)BT_CWARPS * sizeof(BlockCand);

struct BlockFastShared {
    u32 hist[NBINS];
    u64 red[BT_CWARPS];
    u32 wcount[BT_CWARPS];
    unsigned long long full_bar[BT_STAGES];      // bytes of a tile have arrived
    unsigned long long done_bar[BT_STAGES];      // every consumer warp has finished with the buffer
    int abort;                                   // a bounded wait ran out somewhere in this CTA
    long long tile_prefix[BT_TD_CACHE + 1];
    TensorDesc td[BT_TD_CACHE];
};

__device__ __forceinline__ u32 smem_u32(const void *p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(u32 bar, u32 count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u32 bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(u32 bar, u32 bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u32 bar, u32 parity)
{
    u32 ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits for the phase `parity` of the barrier; gives up after BT_WAIT_POLLS polls, or
// earlier when another warp of the CTA has given up (`abort_flag`, may be NULL).
__device__ __forceinline__ bool mbar_wait_bounded(u32 bar, u32 parity, volatile int *abort_flag)
{
    for (u32 i = 0; i < BT_WAIT_POLLS; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && abort_flag && *abort_flag) return false;
        __nanosleep(64);        // a tight polling loop takes issue slots and pipe time from the warps that work
    }
    return false;
}
// One-dimensional bulk copies; both addresses 16-byte aligned, `bytes` a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(u32 dst, const void *src, u32 bytes, u32 bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store_1d(void *dst, u32 src, u32 bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders this thread's ordinary shared-memory writes before later bulk copies that read them.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Appends the candidates a consumer warp has staged to the list (one global atomic per flush).
__device__ __forceinline__ void block_flush(const Params &P, BlockFastShared &sh, BlockCand &cd, int cw, u32 limit)
{
    const int lane = threadIdx.x & 31;
    __syncwarp();
    const u32 c = sh.wcount[cw];
    if (c > limit) {
        u64 base = 0;
        if (lane == 0) base = atomicAdd(&P.ctl->list_count[0], (u64)c);
        base = __shfl_sync(0xffffffffu, base, 0);
        for (u32 i = lane; i < c; i += 32) {
            const u64 pos = base + i;
            if (pos < P.cap) {
                P.list_key[pos] = cd.key[i];
                P.list_id[pos] = cd.id[i];
            }
        }
        for (u32 i = lane; i < 4 * c; i += 32) {      // journal rows, 16 bytes each
            const u64 pos = base + (i >> 2);
            if (pos < P.cap) reinterpret_cast<float4 *>(P.jr_lam + pos * 16)[i & 3] = cd.lam[i >> 2][i & 3];
        }
        __syncwarp();
        if (lane == 0) sh.wcount[cw] = 0;
    }
    __syncwarp();
}

// Tiles of the aligned interior of tensor d (host and device use the same rule).
__host__ __device__ inline long long block_tile_count(const TensorDesc &d)
{
    if (block_fast_end(d) <= 0) return 0;
    const long long nbr = d.d0 >> 2;
    if (d.nbc <= BT_BLOCKS) {
        const long long rpt = BT_BLOCKS / d.nbc;        // whole block rows per tile
        return (nbr + rpt - 1) / rpt;
    }
    return nbr * ((d.nbc + BT_BLOCKS - 1) / BT_BLOCKS);  // column chunks of one block row
}

// Geometry of tile `tile` (global tile number).
struct TileGeom {
    int t;              // owning tensor
    u32 b0;             // first block (number inside the tensor); the tile's blocks are b0 .. b0 + nq - 1
    u32 nq;             // blocks in the tile
    u32 nbpr;           // blocks per row piece
    u32 nrows;          // matrix rows in the tile (4 per block row)
    u32 off0;           // element offset of the first row piece
    bool whole;         // whole block rows: one contiguous range
};

__device__ __forceinline__ TileGeom tile_geom(const long long *tile_prefix, const TensorDesc *td, int T, long long tile)
{
    TileGeom g;
    g.t = find_tensor(tile_prefix, T, tile);
    const TensorDesc &d = td[g.t];
    const u32 nbc = (u32)d.nbc, nbr = (u32)(d.d0 >> 2), C = (u32)d.d1;
    const u32 local = (u32)(tile - tile_prefix[g.t]);
    g.whole = nbc <= (u32)BT_BLOCKS;
    if (g.whole) {
        const u32 rpt = (u32)BT_BLOCKS / nbc;
        const u32 brow0 = local * rpt;
        const u32 brows = nbr - brow0 < rpt ? nbr - brow0 : rpt;
        g.nbpr = nbc;
        g.nq = brows * nbc;
        g.nrows = 4u * brows;
        g.b0 = brow0 * nbc;
        g.off0 = 4u * brow0 * C;
    } else {
        const u32 cpr = (nbc + BT_BLOCKS - 1) / BT_BLOCKS;
        const u32 brow = local / cpr, chunk = local - brow * cpr;
        const u32 bc0 = chunk * BT_BLOCKS;
        g.nbpr = nbc - bc0 < (u32)BT_BLOCKS ? nbc - bc0 : (u32)BT_BLOCKS;
        g.nq = g.nbpr;
        g.nrows = 4u;
        g.b0 = brow * nbc + bc0;
        g.off0 = 4u * brow * C + 4u * bc0;
    }
    return g;
}

// May the mask of this tile be written by bulk copies (16-byte rule on addresses and sizes)?
__device__ __forceinline__ bool tile_mask_bulk(const TensorDesc &d, const TileGeom &g)
{
    if (!d.mask || ((uintptr_t)d.mask & 15u)) return false;
    return g.whole || ((d.d1 & 15) == 0 && (g.nbpr & 3u) == 0);
}

template <bool H, bool G>
__global__ void __launch_bounds__(BT_THREADS, 1) k_fused_block(Params P)
{
    __shared__ BlockFastShared sh;
    extern __shared__ __align__(128) unsigned char dyn_smem[];      // tile buffers, then the candidate staging
    // The kernel may have been launched while the sampler ahead of it still runs (programmatic
    // dependent launch): until pdl_wait() nothing the sampler writes is read - the set-up below and
    // the first tile loads need only w, lambda and the descriptors.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char *tile_buf = dyn_smem;
    BlockCand *cands = reinterpret_cast<BlockCand *>(dyn_smem + (size_t)BT_STAGES * BT_STAGE_BYTES);
    for (int i = threadIdx.x; i < NBINS; i += BT_THREADS) sh.hist[i] = 0;
    if (threadIdx.x < BT_CWARPS) sh.wcount[threadIdx.x] = 0;
    if (threadIdx.x == 0) sh.abort = 0;
    const bool cached = P.T <= BT_TD_CACHE;
    if (cached) {
        for (int i = threadIdx.x; i <= P.T; i += BT_THREADS) sh.tile_prefix[i] = P.tile_prefix[i];
        const int words = P.T * (int)(sizeof(TensorDesc) / sizeof(u32));
        const u32 *src = reinterpret_cast<const u32 *>(P.td);
        u32 *dst = reinterpret_cast<u32 *>(sh.td);
        for (int i = threadIdx.x; i < words; i += BT_THREADS) dst[i] = src[i];
    }
    if (threadIdx.x < BT_STAGES) {
        mbar_init(smem_u32(&sh.full_bar[threadIdx.x]), 1);
        mbar_init(smem_u32(&sh.done_bar[threadIdx.x]), BT_CWARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const long long *tile_prefix = cached ? sh.tile_prefix : P.tile_prefix;
    const TensorDesc *td = cached ? sh.td : P.td;
    const int fp16 = quant_code(P.fuse);     // quantisation of theta
    const float mu = P.mu;
    volatile int *abort_flag = &sh.abort;
    u64 na = 0;
    Bracket br;
    memset(&br, 0, sizeof(br));
    bool onepass = false;
    if (warp < BT_CWARPS) {
        pdl_wait();
        onepass = P.ctl->sel.onepass != 0;      // else the sampler advised against the single pass: nothing to do here
        br = load_bracket(P.ctl->sel);
    }

    if (warp == BT_CWARPS) {
        // ------------------------------------------------------------ producer (one lane)
        if (lane == 0) {
            u32 k = 0;
            bool ok = true, dep_seen = false, quiet = false;
            // before the first store, and before leaving: the sampler must have finished and
            // must have said that the single pass is on
            auto see_dependency = [&]() {
                if (dep_seen) return;
                pdl_wait();
                dep_seen = true;
                if (!P.ctl->sel.onepass) { quiet = true; ok = false; }
            };
            // writes the outputs of the tile that used buffer `stage` (tile number `tile`) back
            auto store_tile = [&](long long tile, int stage) {
                const TileGeom g = tile_geom(tile_prefix, td, P.T, tile);
                const TensorDesc &d = td[g.t];
                const bool upd = (P.fuse & FUSE_LAMBDA) && d.lam != nullptr;
                const bool mbulk = tile_mask_bulk(d, g);
                const u32 C = (u32)d.d1, pitch = g.nbpr * 16u;
                const u32 sb = smem_u32(tile_buf + (size_t)stage * BT_STAGE_BYTES);
                if (g.whole) {
                    const u32 bytes = g.nrows * pitch;
                    bulk_store_1d(d.theta + g.off0, sb, bytes);
                    if (upd) bulk_store_1d(d.lam + g.off0, sb + BT_ARRAY_BYTES, bytes);
                    if (mbulk) bulk_store_1d(d.mask + g.off0, sb + 2 * BT_ARRAY_BYTES, bytes / 4u);
                } else {
#pragma unroll
                    for (u32 i = 0; i < 4; ++i) {
                        bulk_store_1d(d.theta + g.off0 + i * C, sb + i * pitch, pitch);
                        if (upd) bulk_store_1d(d.lam + g.off0 + i * C, sb + BT_ARRAY_BYTES + i * pitch, pitch);
                        if (mbulk) bulk_store_1d(d.mask + g.off0 + i * C, sb + 2 * BT_ARRAY_BYTES + i * (pitch / 4u), pitch / 4u);
                    }
                }
                bulk_commit();
            };
            long long tile = blockIdx.x;
#pragma unroll 1
            for (; tile < P.n_tiles && ok; tile += gridDim.x, ++k) {
                const int stage = (int)(k % BT_STAGES);
                if (k >= (u32)BT_STAGES) {
                    see_dependency();
                    if (!ok) break;
                    // the consumers have left theta / lambda / mask of the tile before in this buffer
                    ok = mbar_wait_bounded(smem_u32(&sh.done_bar[stage]), ((k / BT_STAGES) - 1u) & 1u, abort_flag);
                    if (!ok) break;
                    store_tile(tile - (long long)BT_STAGES * gridDim.x, stage);
                    bulk_wait_read_all();               // shared memory has been read: the buffer is free
                }
                if (*abort_flag) { ok = false; break; }
                const TileGeom g = tile_geom(tile_prefix, td, P.T, tile);
                const TensorDesc &d = td[g.t];
                const bool has_lam = d.lam != nullptr;
                const u32 C = (u32)d.d1, pitch = g.nbpr * 16u;
                const u32 bar = smem_u32(&sh.full_bar[stage]);
                const u32 sb = smem_u32(tile_buf + (size_t)stage * BT_STAGE_BYTES);
                mbar_arrive_expect_tx(bar, (has_lam ? 2u : 1u) * g.nrows * pitch);
                if (g.whole) {
                    bulk_load_1d(sb, d.w + g.off0, g.nrows * pitch, bar);
                    if (has_lam) bulk_load_1d(sb + BT_ARRAY_BYTES, d.lam + g.off0, g.nrows * pitch, bar);
                } else {
#pragma unroll
                    for (u32 i = 0; i < 4; ++i) {
                        bulk_load_1d(sb + i * pitch, d.w + g.off0 + i * C, pitch, bar);
                        if (has_lam) bulk_load_1d(sb + BT_ARRAY_BYTES + i * pitch, d.lam + g.off0 + i * C, pitch, bar);
                    }
                }
            }
            // drain: the last tiles still sit in their buffers
            const u32 issued = k;                       // tiles whose loads have been issued
            see_dependency();
            if (ok) {
                const u32 first = issued > (u32)BT_STAGES ? issued - BT_STAGES : 0u;
                for (u32 j = first; j < issued && ok; ++j) {
                    const int stage = (int)(j % BT_STAGES);
                    ok = mbar_wait_bounded(smem_u32(&sh.done_bar[stage]), (j / BT_STAGES) & 1u, abort_flag);
                    if (ok) store_tile((long long)blockIdx.x + (long long)j * gridDim.x, stage);
                }
            }
            if (!ok) {
                // A wait ran out: report it (the selection kernels turn it into an error status) and
                // give the loads still in flight the same bounded time, so that none lands in shared
                // memory after this CTA has gone. The consumers see the flag and stop. (`quiet`: no
                // error, the single pass is simply off; the loads fetched ahead are waited for too.)
                *abort_flag = 1;
                if (!quiet) atomicExch(&P.ctl->async_error, 1);
                const u32 first = issued > (u32)BT_STAGES ? issued - BT_STAGES : 0u;
                for (u32 j = first; j < issued; ++j)
                    (void)mbar_wait_bounded(smem_u32(&sh.full_bar[j % BT_STAGES]), (j / BT_STAGES) & 1u, nullptr);
            }
            bulk_wait_all();                            // every store has left shared memory and is performed
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int cw = warp;
        BlockCand &cd = cands[cw];
        u32 n_above = 0, k = 0;
        bool ok = true;
#pragma unroll 1
        for (long long tile = blockIdx.x; onepass && tile < P.n_tiles; tile += gridDim.x, ++k) {
            const int stage = (int)(k % BT_STAGES);
            const TileGeom g = tile_geom(tile_prefix, td, P.T, tile);
            const TensorDesc &d = td[g.t];
            const bool has_lam = d.lam != nullptr;
            const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
            const bool mbulk = tile_mask_bulk(d, g);
            const u32 C = (u32)d.d1, pitch = g.nbpr * 16u;
            if (*abort_flag || !mbar_wait_bounded(smem_u32(&sh.full_bar[stage]), (k / BT_STAGES) & 1u, abort_flag)) { ok = false; break; }
            const u32 q = (u32)(cw * 32 + lane);                    // block of this lane inside the tile
            if (q < g.nq) {
                const u32 brl = g.whole ? q / g.nbpr : 0u;          // block row inside the tile
                const u32 bcol = q - brl * g.nbpr;
                unsigned char *sw = tile_buf + (size_t)stage * BT_STAGE_BYTES + (size_t)(4u * brl) * pitch + (size_t)bcol * 16;
                unsigned char *sl = sw + BT_ARRAY_BYTES;
                unsigned char *sm = tile_buf + (size_t)stage * BT_STAGE_BYTES + 2 * BT_ARRAY_BYTES +
                                    (size_t)(4u * brl) * (pitch / 4u) + (size_t)bcol * 4;
                float4 w4[4], l4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    w4[i] = *reinterpret_cast<const float4 *>(sw + i * pitch);
                    l4[i] = has_lam ? *reinterpret_cast<const float4 *>(sl + i * pitch) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float w[16], l[16], u[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    w[4 * i] = w4[i].x; w[4 * i + 1] = w4[i].y; w[4 * i + 2] = w4[i].z; w[4 * i + 3] = w4[i].w;
                    l[4 * i] = l4[i].x; l[4 * i + 1] = l4[i].y; l[4 * i + 2] = l4[i].z; l[4 * i + 3] = l4[i].w;
                }
                u32 nz = 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) nz |= __float_as_uint(l[i]);
                if (nz) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) u[i] = __fsub_rn(w[i], __fdiv_rn(l[i], mu));
                } else {                    // every lambda is +0: u is w, bit for bit
#pragma unroll
                    for (int i = 0; i < 16; ++i) u[i] = w[i];
                }
                double acc = 0.0;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const double x = (double)u[i];
                    acc = __fma_rn(x, x, acc);
                }
                const u64 key = (u64)__double_as_longlong(acc);
                const bool keep = key >= br.guess;
                n_above += key > br.hi ? 1u : 0u;
                if (key >= br.lo && key <= br.hi) {
                    const u64 id = (u64)d.unit_prefix + g.b0 + q;
                    const u32 slot = atomicAdd(&sh.wcount[cw], 1u);
                    cd.key[slot] = key;
                    cd.id[slot] = id;
#pragma unroll
                    for (int i = 0; i < 4; ++i) cd.lam[slot][i] = l4[i];
                    atomicAdd(&sh.hist[bracket_bin(br, key, id)], 1u);
                }
                const u32 off0 = g.off0 + 4u * brl * C + 4u * bcol;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float th[4], ln[4], gr[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) th[j] = keep ? u[4 * i + j] : 0.0f;
                    unsigned short h[4];
                    if (H) {
                        half4(th, h, fp16 ? fp16 : 1);
                        if (fp16) widen4(h, th, th, fp16);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float p = __fmul_rn(mu, __fsub_rn(w[4 * i + j], th[j]));
                        ln[j] = upd ? __fsub_rn(l[4 * i + j], p) : l[4 * i + j];
                        gr[j] = __fsub_rn(p, ln[j]);
                    }
                    *reinterpret_cast<float4 *>(sw + i * pitch) = make_float4(th[0], th[1], th[2], th[3]);
                    if (upd) *reinterpret_cast<float4 *>(sl + i * pitch) = make_float4(ln[0], ln[1], ln[2], ln[3]);
                    const u32 off = off0 + i * C;
                    if (mbulk) *reinterpret_cast<u32 *>(sm + i * (pitch / 4u)) = keep ? 0x01010101u : 0u;
                    else if (d.mask) *reinterpret_cast<u32 *>(d.mask + off) = keep ? 0x01010101u : 0u;
                    if (H && d.theta_h) *reinterpret_cast<uint2 *>(d.theta_h + off) =
                        make_uint2((u32)h[0] | ((u32)h[1] << 16), (u32)h[2] | ((u32)h[3] << 16));
                    if (G && d.grad) *reinterpret_cast<float4 *>(d.grad + off) = make_float4(gr[0], gr[1], gr[2], gr[3]);
                }
                fence_proxy_async();                    // the bulk stores of the producer read these writes
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.done_bar[stage]));
            block_flush(P, sh, cd, cw, BSTG - 32);
        }
        if (!ok && lane == 0 && !*abort_flag) {
            *abort_flag = 1;
            atomicExch(&P.ctl->async_error, 1);
        }
        block_flush(P, sh, cd, cw, 0);
        na = n_above;
    }
    __syncthreads();
    pdl_wait();
    if (!P.ctl->sel.onepass) return;         // (the same for every thread)
    // the blocks outside the aligned interior (ragged last block rows, unaligned tensors) and
    // the tensors that pass through: work items listed by the host, done by generic code
    if (P.n_edge_items > 0) {
        for (long long i = blockIdx.x; i < P.n_edge_items; i += gridDim.x) {
            const long long item = P.edge_items[i];
            const int t = find_tensor(P.item_prefix, P.T, item);
            const TensorDesc g = P.td[t];
            const long long local = item - P.item_prefix[t];
            if (!g.ranked) {
                if (threadIdx.x < THREADS) process_linear_item<M_KEEPALL>(P, g, local, 0, 0);
                continue;
            }
            if (warp >= BLOCKS_PER_ITEM / 32) continue;             // 8 warps x 32 blocks make one item
            const int cw = warp;
            BlockCand &cd = cands[cw];
            const bool has_lam = g.lam != nullptr;
            const bool upd = (P.fuse & FUSE_LAMBDA) && has_lam;
            const bool wr_grad = (P.fuse & FUSE_PENALTY) && g.grad != nullptr;
            const long long b = local * BLOCKS_PER_ITEM + warp * 32 + lane;
            if (b < g.n_units && b >= block_fast_end(g)) {
                BlockData bd;
                float u[16];
                load_block(g, b, bd);
                const u64 key = block_key(bd, mu, has_lam, u);
                const u64 id = (u64)(g.unit_prefix + b);
                na += key > br.hi ? 1 : 0;
                if (key >= br.lo && key <= br.hi) {
                    const u32 slot = atomicAdd(&sh.wcount[cw], 1u);
                    cd.key[slot] = key;
                    cd.id[slot] = id;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        cd.lam[slot][q] = make_float4(bd.l[4 * q], bd.l[4 * q + 1], bd.l[4 * q + 2], bd.l[4 * q + 3]);
                    atomicAdd(&sh.hist[bracket_bin(br, key, id)], 1u);
                }
                store_block_lean<H>(g, bd, u, key >= br.guess, mu, fp16, upd, wr_grad);
            }
            block_flush(P, sh, cd, cw, 0);
        }
    }
    if (warp < BT_CWARPS) {
        for (int o = 16; o > 0; o >>= 1) na += __shfl_xor_sync(0xffffffffu, na, o);
        if (lane == 0) sh.red[warp] = na;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 tot = 0;
        for (int i = 0; i < BT_CWARPS; ++i) tot += sh.red[i];
        if (tot) atomicAdd(&P.ctl->scan_above[0], tot);
    }
    for (int i = threadIdx.x; i < NBINS; i += BT_THREADS) {
        const u32 hc = sh.hist[i];
        if (hc) atomicAdd(&P.hist[i], (u64)hc);
    }
}

}  // namespace cs
