// Network thinning on the device (paper, Implementation: "Network Thinning"):
// finding the zero structures that structure pruning leaves in a tensor and
// removing them, plus the non-zero count behind the memory-footprint objective
// (Evaluation, Objective 1). The dependency analysis between layers stays with
// the caller: it decides which axis flags of which tensor apply to which other
// tensor; these kernels do the per-tensor data movement.
//
// A tensor is seen as a 3-D view [d0][d1][inner], row-major: a conv weight
// F x C x kh x kw has d0 = F, d1 = C, inner = kh*kw; a matrix R x C has
// d0 = R, d1 = C, inner = 1; a bias has d0 = n, d1 = inner = 1.
#pragma once
#include "common.cuh"

namespace cs {

constexpr int THIN_ITEM = 4096;          // elements per work item (16 per thread)
constexpr int THIN_INDEX_THREADS = 1024;

__device__ __forceinline__ bool is_nonzero(float x) { return (__float_as_uint(x) & 0x7FFFFFFFu) != 0u; }

// keep[i] = 1 iff slice i along `axis` (0 or 1) holds a non-zero value. `keep`
// was cleared before the launch; threads only ever store 1.
__global__ void __launch_bounds__(THREADS) k_thin_flags(const float *__restrict__ x, long long d0, long long d1,
                                                        long long inner, int axis, uint8_t *keep)
{
    const long long n = d0 * d1 * inner;
    const long long n_items = (n + THIN_ITEM - 1) / THIN_ITEM;
    const long long L = d1 * inner;
    const bool small = n < 0xFFFFFFFFll;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const long long base = item * THIN_ITEM + threadIdx.x;
        float v[THIN_ITEM / THREADS];
#pragma unroll
        for (int k = 0; k < THIN_ITEM / THREADS; ++k) {
            const long long e = base + (long long)k * THREADS;
            v[k] = e < n ? __ldg(x + e) : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < THIN_ITEM / THREADS; ++k) {
            if (!is_nonzero(v[k])) continue;
            const long long e = base + (long long)k * THREADS;
            long long idx;
            if (small) {
                const u32 e32 = (u32)e;
                idx = axis == 0 ? e32 / (u32)L : (e32 / (u32)inner) % (u32)d1;
            } else {
                idx = axis == 0 ? e / L : (e / inner) % d1;
            }
            if (!keep[idx]) keep[idx] = 1;
        }
    }
}

// Ascending positions of the non-zero flags of each axis (identity when the
// flag array is NULL) and the two kept extents. One CTA.
__global__ void __launch_bounds__(THIN_INDEX_THREADS) k_thin_index(const uint8_t *keep0, const uint8_t *keep1,
                                                                   long long d0, long long d1, int *idx0, int *idx1,
                                                                   long long *dims_out)
{
    __shared__ int wsum[THIN_INDEX_THREADS / 32];
    __shared__ int carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int ax = 0; ax < 2; ++ax) {
        const uint8_t *keep = ax ? keep1 : keep0;
        const long long d = ax ? d1 : d0;
        int *idx = ax ? idx1 : idx0;
        if (!keep) {
            if (threadIdx.x == 0) dims_out[ax] = d;
            continue;
        }
        if (threadIdx.x == 0) carry = 0;
        __syncthreads();
        for (long long c0 = 0; c0 < d; c0 += THIN_INDEX_THREADS) {
            const long long i = c0 + threadIdx.x;
            const int f = (i < d && keep[i]) ? 1 : 0;
            int s = f;                                   // inclusive scan inside the warp
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += y;
            }
            if (lane == 31) wsum[warp] = s;
            __syncthreads();
            if (warp == 0) {
                int t = wsum[lane];
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, t, o);
                    if (lane >= o) t += y;
                }
                wsum[lane] = t;
            }
            __syncthreads();
            const int before = carry + (warp ? wsum[warp - 1] : 0) + s - f;
            if (f) idx[before] = (int)i;
            __syncthreads();
            if (threadIdx.x == 0) carry += wsum[THIN_INDEX_THREADS / 32 - 1];
            __syncthreads();
        }
        if (threadIdx.x == 0) dims_out[ax] = carry;
        __syncthreads();
    }
}

// dst[i'][j'][r] = src[idx0[i']][idx1[j']][r]. A work item is 1024 consecutive
// elements of one output row i' (length d1' * inner). VEC: both rows are copied
// whole (no axis-1 removal) with 128-bit accesses.
template <bool VEC>
__global__ void __launch_bounds__(THREADS) k_thin_gather(const float *__restrict__ src, float *__restrict__ dst,
                                                         long long d1, long long inner, const int *idx0,
                                                         const int *idx1, const long long *dims)
{
    const long long n0 = dims[0], n1 = dims[1];
    const long long L_in = d1 * inner, L_out = n1 * inner;
    const long long tiles_per_row = (L_out + 1023) / 1024;
    const long long n_tiles = n0 * tiles_per_row;
    const u32 inner32 = (u32)inner;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const long long io = tile / tiles_per_row;
        const long long c = tile - io * tiles_per_row;
        const long long ii = idx0 ? (long long)idx0[io] : io;
        const float *s = src + ii * L_in;
        float *o = dst + io * L_out;
        const u32 r0 = (u32)(c * 1024) + 4u * threadIdx.x;
        if (VEC) {
            if (r0 < (u32)L_out)
                *reinterpret_cast<float4 *>(o + r0) = __ldg(reinterpret_cast<const float4 *>(s + r0));
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const u32 r = (u32)(c * 1024) + (u32)q * THREADS + threadIdx.x;
                if (r < (u32)L_out) {
                    u32 sr = r;
                    if (idx1) {
                        const u32 jo = r / inner32;
                        sr = (u32)idx1[jo] * inner32 + (r - jo * inner32);
                    }
                    o[r] = __ldg(s + sr);
                }
            }
        }
    }
}

// Non-zero values per array of a list and in total (the footprint objective
// multiplies by the bytes of a stored value).
struct CountDesc {
    const float *x;
    long long numel;
};

__global__ void __launch_bounds__(THREADS) k_count_nonzero(const CountDesc *td, const long long *item_prefix, int T,
                                                           long long n_items, unsigned long long *counts)
{
    __shared__ u32 red[WARPS];
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int t = find_tensor(item_prefix, T, item);
        const CountDesc d = td[t];
        const long long base = (item - item_prefix[t]) * THIN_ITEM + threadIdx.x;
        float v[THIN_ITEM / THREADS];
#pragma unroll
        for (int k = 0; k < THIN_ITEM / THREADS; ++k) {
            const long long e = base + (long long)k * THREADS;
            v[k] = e < d.numel ? __ldg(d.x + e) : 0.0f;
        }
        u32 c = 0;
#pragma unroll
        for (int k = 0; k < THIN_ITEM / THREADS; ++k) c += is_nonzero(v[k]) ? 1u : 0u;
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = c;
        __syncthreads();
        if (threadIdx.x == 0) {
            u32 tot = 0;
            for (int i = 0; i < WARPS; ++i) tot += red[i];
            if (tot) {
                atomicAdd(&counts[t], (unsigned long long)tot);
                atomicAdd(&counts[T], (unsigned long long)tot);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------- a whole list of layers at once
// The same three steps for a list of tensors in three launches instead of three per tensor
// (thinning a network is dozens of small tensors: launch latency, not bandwidth).
struct ThinLayerDesc {
    const float *src;
    float *dst;
    uint8_t *keep0;            // out: axis-0 flags of this tensor (d0 bytes), written 0 / 1
    const uint8_t *keep1;      // in : flags that remove axis-1 slices (another tensor's keep0), or NULL
    long long *dims_out;       // out: d0', d1'
    int *idx0, *idx1;          // scratch: ascending positions of the kept slices
    long long d0, d1, inner;
    int use_keep0;             // remove the axis-0 slices whose flag is 0
    int pad;
};

// keep0[i] = 1 iff slice [i][:][:] of its tensor holds a non-zero value; one warp per slice.
// Work items: slices, numbered through the list (`prefix[l]` = first slice of layer l).
__global__ void __launch_bounds__(THREADS) k_thin_list_flags(const ThinLayerDesc *td, const long long *prefix, int L)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long n = prefix[L];
    for (long long base = (long long)blockIdx.x * WARPS; base < n; base += (long long)gridDim.x * WARPS) {
        const long long item = base + warp;
        if (item >= n) continue;
        const int l = find_tensor(prefix, L, item);
        const ThinLayerDesc &d = td[l];
        const long long i = item - prefix[l], len = d.d1 * d.inner;
        const float *x = d.src + i * len;
        bool nz = false;
        for (long long j = lane; j < len && !nz; j += 32) nz = is_nonzero(__ldg(x + j));
        nz = __any_sync(0xffffffffu, nz);
        if (lane == 0) d.keep0[i] = nz ? 1 : 0;
    }
}

// Index lists and kept extents of every layer: CTA l does layer l.
__global__ void __launch_bounds__(THIN_INDEX_THREADS) k_thin_list_index(const ThinLayerDesc *td)
{
    const ThinLayerDesc &d = td[blockIdx.x];
    __shared__ int wsum[THIN_INDEX_THREADS / 32];
    __shared__ int carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int ax = 0; ax < 2; ++ax) {
        const uint8_t *keep = ax ? d.keep1 : (d.use_keep0 ? d.keep0 : nullptr);
        const long long n = ax ? d.d1 : d.d0;
        int *idx = ax ? d.idx1 : d.idx0;
        if (!keep) {
            if (threadIdx.x == 0) d.dims_out[ax] = n;
            continue;
        }
        if (threadIdx.x == 0) carry = 0;
        __syncthreads();
        for (long long c0 = 0; c0 < n; c0 += THIN_INDEX_THREADS) {
            const long long i = c0 + threadIdx.x;
            const int f = (i < n && keep[i]) ? 1 : 0;
            int sc = f;
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, sc, o);
                if (lane >= o) sc += y;
            }
            if (lane == 31) wsum[warp] = sc;
            __syncthreads();
            if (warp == 0) {
                int t = wsum[lane];
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, t, o);
                    if (lane >= o) t += y;
                }
                wsum[lane] = t;
            }
            __syncthreads();
            const int before = carry + (warp ? wsum[warp - 1] : 0) + sc - f;
            if (f) idx[before] = (int)i;
            __syncthreads();
            if (threadIdx.x == 0) carry += wsum[THIN_INDEX_THREADS / 32 - 1];
            __syncthreads();
        }
        if (threadIdx.x == 0) d.dims_out[ax] = carry;
        __syncthreads();
    }
}

// dst = src without the removed slices, for every layer. Work items: 1024 consecutive elements of
// one INPUT row position (an upper bound of the output rows; `prefix[l]` = first item of layer l).
__global__ void __launch_bounds__(THREADS) k_thin_list_gather(const ThinLayerDesc *td, const long long *prefix, int L)
{
    const long long n = prefix[L];
    for (long long item = blockIdx.x; item < n; item += gridDim.x) {
        const int l = find_tensor(prefix, L, item);
        const ThinLayerDesc &d = td[l];
        const long long n0 = d.dims_out[0], n1 = d.dims_out[1];
        const long long L_in = d.d1 * d.inner, L_out = n1 * d.inner;
        const long long tiles_per_row = (L_in + 1023) / 1024;        // of the input row: the bound the host used
        const long long local = item - prefix[l];
        const long long io = local / tiles_per_row, c = local - io * tiles_per_row;
        if (io >= n0 || c * 1024 >= L_out) continue;
        const bool rm0 = d.use_keep0 != 0;
        const long long ii = rm0 ? (long long)d.idx0[io] : io;
        const float *s = d.src + ii * L_in;
        float *o = d.dst + io * L_out;
        const u32 inner32 = (u32)d.inner;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const u32 r = (u32)(c * 1024) + (u32)q * THREADS + threadIdx.x;
            if (r < (u32)L_out) {
                u32 sr = r;
                if (d.keep1) {
                    const u32 jo = r / inner32;
                    sr = (u32)d.idx1[jo] * inner32 + (r - jo * inner32);
                }
                o[r] = __ldg(s + sr);
            }
        }
    }
}

}  // namespace cs
