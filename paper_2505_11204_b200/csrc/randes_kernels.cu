// sm_100a kernels of the RanDeS hot path: retrieve, and accumulate
// (compress / add_model / remove_model).  HBM-bound streaming kernels:
// 128-bit loads, fp32 arithmetic with one rounding per operation, sign bits
// generated in registers from Philox4x32-10 and never stored to memory, the
// per-task layer permutation resolved per unit of work from small index tables.
//
// Work decomposition.  A CTA (8 warps) walks a list of units; a unit is a block
// of rows x up to 8 column blocks of 128 columns of one layer.  A warp owns one
// column block (lane = 4 adjacent columns, so one Philox block of 128 bits is
// exactly the warp's sign bits) and walks down the rows: the sign bits are
// computed once per unit and reused for every row.  Every output element is
// written by exactly one thread, tasks are summed in a fixed order: results are
// bit-reproducible.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_internal.h"

namespace randes {
namespace {

typedef __nv_bfloat16 bf16;

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter (c0..c3), key (k0,k1).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The four sign bits of this lane's columns (bit j = column 4*lane + j of the
// warp's 128-column block) out of the block's four words.
__device__ __forceinline__ uint32_t lane_nibble(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, int lane)
{
    const int q = lane >> 3;
    const uint32_t w = q == 0 ? w0 : (q == 1 ? w1 : (q == 2 ? w2 : w3));
    return (w >> ((lane & 7) * 4)) & 0xFu;
}

__device__ __forceinline__ float flip(float x, uint32_t mask) { return __uint_as_float(__float_as_uint(x) ^ mask); }

// ---- element access: fp32 and bf16 storage, 4 columns per lane -------------------------
template <typename T> struct Io;

template <> struct Io<float> {
    static constexpr uintptr_t kVecAlign = 16;
    static __device__ __forceinline__ float4 load4_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ float4 load4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ float load1(const float* p) { return __ldg(p); }
    static __device__ __forceinline__ void store4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};

template <> struct Io<bf16> {
    static constexpr uintptr_t kVecAlign = 8;
    static __device__ __forceinline__ float4 widen(uint2 raw)
    {
        float4 f;
        f.x = __uint_as_float(raw.x << 16);
        f.y = __uint_as_float(raw.x & 0xFFFF0000u);
        f.z = __uint_as_float(raw.y << 16);
        f.w = __uint_as_float(raw.y & 0xFFFF0000u);
        return f;
    }
    static __device__ __forceinline__ float4 load4_stream(const bf16* p) { return widen(__ldcs(reinterpret_cast<const uint2*>(p))); }
    static __device__ __forceinline__ float4 load4(const bf16* p) { return widen(__ldg(reinterpret_cast<const uint2*>(p))); }
    static __device__ __forceinline__ float load1(const bf16* p)
    {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    static __device__ __forceinline__ void store4(bf16* p, float4 v)
    {
        // round to nearest even, two values per conversion
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 raw;
        raw.x = *reinterpret_cast<const uint32_t*>(&lo);
        raw.y = *reinterpret_cast<const uint32_t*>(&hi);
        __stcs(reinterpret_cast<uint2*>(p), raw);
    }
    static __device__ __forceinline__ void store1(bf16* p, float v) { *p = __float2bfloat16_rn(v); }
};

template <typename T>
__device__ __forceinline__ bool vec_aligned(const void* p)
{
    return (reinterpret_cast<uintptr_t>(p) & (Io<T>::kVecAlign - 1)) == 0;
}

// geometry of this warp inside a unit
struct WarpTile {
    uint32_t cb;      // column block (128 columns) of the layer
    uint32_t c;       // first of this lane's 4 columns
    uint32_t r0;      // first row of this warp
    uint32_t r_end;   // one past the last row of the unit
    uint32_t rstep;   // row stride between this warp's rows
};

__device__ __forceinline__ WarpTile warp_tile(const DevUnit& un, int warp, int lane)
{
    WarpTile t;
    const uint32_t nbc = un.nbc;
    t.cb = un.cb0 + (warp & (nbc - 1));
    t.c = t.cb * kColsPerWarp + lane * 4;
    t.rstep = kWarpsPerCta / nbc;
    t.r0 = un.row0 + warp / nbc;
    t.r_end = un.row0 + un.nrows;
    return t;
}

// =========================================================================================
// retrieve:  out[p] = fma(lambda, s_t(l, c) * M[l], W_0[p]),  l = sigma_t^-1(p)
// (Section 4, second display; Section 4.4, second display.)  The sign is folded
// into lambda: fma(+-lambda, m, w) is bit-identical to fma(lambda, +-m, w).
// =========================================================================================
template <typename ST, typename OT, bool VEC>
__device__ __forceinline__ void retrieve_rows(const WarpTile& t, uint32_t cols, const float* __restrict__ mp,
                                              const ST* __restrict__ wp, OT* __restrict__ op, const float (&lam)[4])
{
    constexpr int U = 4;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep * U) {
        float4 m[U], w[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint32_t rr = r + j * t.rstep;
            if (rr < t.r_end) {
                const size_t off = static_cast<size_t>(rr) * cols + t.c;
                if (VEC) {
                    m[j] = __ldcs(reinterpret_cast<const float4*>(mp + off));
                    w[j] = Io<ST>::load4_stream(wp + off);
                } else {
                    float mm[4] = {0.f, 0.f, 0.f, 0.f}, ww[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (t.c + e < cols) { mm[e] = mp[off + e]; ww[e] = Io<ST>::load1(wp + off + e); }
                    m[j] = make_float4(mm[0], mm[1], mm[2], mm[3]);
                    w[j] = make_float4(ww[0], ww[1], ww[2], ww[3]);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint32_t rr = r + j * t.rstep;
            if (rr < t.r_end) {
                const size_t off = static_cast<size_t>(rr) * cols + t.c;
                float4 y;
                y.x = __fmaf_rn(lam[0], m[j].x, w[j].x);
                y.y = __fmaf_rn(lam[1], m[j].y, w[j].y);
                y.z = __fmaf_rn(lam[2], m[j].z, w[j].z);
                y.w = __fmaf_rn(lam[3], m[j].w, w[j].w);
                if (VEC) {
                    Io<OT>::store4(op + off, y);
                } else {
                    const float yy[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (t.c + e < cols) Io<OT>::store1(op + off + e, yy[e]);
                }
            }
        }
    }
}

template <typename ST, typename OT>
__global__ void __launch_bounds__(kThreadsPerCta) retrieve_kernel(const RetrieveArgs a)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;                       // layer position being rebuilt
        const DevLayer lp = a.layers[p];
        const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[p] : p;   // sigma^-1
        const unsigned long long m_off = slot == p ? lp.m_off : a.layers[slot].m_off;
        const WarpTile t = warp_tile(un, warp, lane);
        if (t.c >= lp.cols || t.r0 >= t.r_end) continue;

        uint32_t nib = 0;
        if (lp.flags & kFlagFlip) {
            uint32_t blk[4];
            philox4x32_10(t.cb, slot, kTagSign, a.task.id, a.task.key0, a.task.key1, blk);
            nib = lane_nibble(blk[0], blk[1], blk[2], blk[3], lane);
        }
        float lam[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) lam[e] = flip(a.lambda, ((nib >> e) & 1u) << 31);

        const ST* wp = static_cast<const ST*>(a.base[p]);
        OT* op = static_cast<OT*>(a.out[p]);
        const float* mp = a.M + m_off;
        const bool vec = (lp.cols & 3u) == 0 && vec_aligned<ST>(wp) && vec_aligned<OT>(op);
        if (vec) retrieve_rows<ST, OT, true>(t, lp.cols, mp, wp, op, lam);
        else retrieve_rows<ST, OT, false>(t, lp.cols, mp, wp, op, lam);
    }
}

// =========================================================================================
// accumulate:  M[l] (=|+=|-=) sum_i s_i(l, c) * ( W_i[sigma_i(l)] - W_0[sigma_i(l)] )
// compress (Section 4, first display): all registered tasks, from +0, in plan order.
// add / remove (Section 5.7): one task, starting from M, sign negated for remove.
// A warp keeps the resolved source pointers and the Philox sign blocks of up to
// kTaskChunk tasks in its private shared-memory scratch: lane i prepares task i.
// =========================================================================================
struct WarpScratch {
    const void* pw[kTaskChunk];
    const void* pb[kTaskChunk];
    uint4 sign[kTaskChunk];
};

template <typename ST, bool VEC>
__device__ __forceinline__ float4 load_tile(const ST* p, size_t off, uint32_t c, uint32_t cols, bool stream)
{
    if (VEC) return stream ? Io<ST>::load4_stream(p + off) : Io<ST>::load4(p + off);
    float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int e = 0; e < 4; ++e)
        if (c + e < cols) v[e] = Io<ST>::load1(p + off + e);
    return make_float4(v[0], v[1], v[2], v[3]);
}

template <typename ST, bool VEC>
__device__ __forceinline__ void accumulate_rows(const WarpTile& t, uint32_t cols, const WarpScratch& ws, int lane,
                                                uint32_t nt, bool init, bool has_base, bool per_task_base,
                                                uint32_t negate_nib, float* __restrict__ mp)
{
    constexpr int U = 2;
    const int q = lane >> 3, sh = (lane & 7) * 4;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep * U) {
        float4 acc[U], w0[U];
        size_t off[U];
        bool on[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint32_t rr = r + j * t.rstep;
            on[j] = rr < t.r_end;
            off[j] = static_cast<size_t>(rr) * cols + t.c;
            acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            w0[j] = acc[j];
            if (on[j]) {
                if (init) {
                    if (VEC) {
                        acc[j] = *reinterpret_cast<const float4*>(mp + off[j]);
                    } else {
                        float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (t.c + e < cols) v[e] = mp[off[j] + e];
                        acc[j] = make_float4(v[0], v[1], v[2], v[3]);
                    }
                }
                // without a shuffle every task subtracts the same W_0 tile: fetch it once
                if (has_base && !per_task_base)
                    w0[j] = load_tile<ST, VEC>(static_cast<const ST*>(ws.pb[0]), off[j], t.c, cols, true);
            }
        }
#pragma unroll 4
        for (uint32_t i = 0; i < nt; ++i) {
            const ST* pw = static_cast<const ST*>(ws.pw[i]);
            const ST* pb = static_cast<const ST*>(ws.pb[i]);
            const uint4 sw = ws.sign[i];
            const uint32_t word = q == 0 ? sw.x : (q == 1 ? sw.y : (q == 2 ? sw.z : sw.w));
            const uint32_t nib = ((word >> sh) & 0xFu) ^ negate_nib;
            const uint32_t m0 = (nib & 1u) << 31, m1 = (nib & 2u) << 30, m2 = (nib & 4u) << 29, m3 = (nib & 8u) << 28;
#pragma unroll
            for (int j = 0; j < U; ++j) {
                if (!on[j]) continue;
                float4 d = load_tile<ST, VEC>(pw, off[j], t.c, cols, true);
                if (has_base) {
                    const float4 b = per_task_base ? load_tile<ST, VEC>(pb, off[j], t.c, cols, false) : w0[j];
                    d.x = __fsub_rn(d.x, b.x);
                    d.y = __fsub_rn(d.y, b.y);
                    d.z = __fsub_rn(d.z, b.z);
                    d.w = __fsub_rn(d.w, b.w);
                }
                acc[j].x = __fadd_rn(acc[j].x, flip(d.x, m0));
                acc[j].y = __fadd_rn(acc[j].y, flip(d.y, m1));
                acc[j].z = __fadd_rn(acc[j].z, flip(d.z, m2));
                acc[j].w = __fadd_rn(acc[j].w, flip(d.w, m3));
            }
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            if (!on[j]) continue;
            if (VEC) {
                *reinterpret_cast<float4*>(mp + off[j]) = acc[j];
            } else {
                const float v[4] = {acc[j].x, acc[j].y, acc[j].z, acc[j].w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (t.c + e < cols) mp[off[j] + e] = v[e];
            }
        }
    }
}

template <typename ST>
__global__ void __launch_bounds__(kThreadsPerCta) accumulate_kernel(const AccumulateArgs a)
{
    __shared__ WarpScratch scratch[kWarpsPerCta];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WarpScratch& ws = scratch[warp];
    const uint32_t L = a.n_layers;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const WarpTile t = warp_tile(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * kColsPerWarp >= ls.cols) continue;   // warp-uniform: nothing for this warp
        const bool lane_on = t.c < ls.cols;
        const bool shuffled = (ls.flags & kFlagShuffle) != 0;
        const bool flipped = (ls.flags & kFlagFlip) != 0;
        float* mp = a.M + ls.m_off;

        for (uint32_t chunk0 = 0; chunk0 < a.n_tasks; chunk0 += kTaskChunk) {
            const uint32_t nt = min(static_cast<uint32_t>(kTaskChunk), a.n_tasks - chunk0);
            __syncwarp();   // the previous chunk's readers are done with the scratch
            bool ok = true;
            if (lane < nt) {
                const uint32_t ti = chunk0 + lane;
                const uint32_t src = shuffled ? a.src_of_slot[static_cast<size_t>(ti) * L + slot] : slot;   // sigma_i(l)
                const void* pw = a.task_ptrs[static_cast<size_t>(ti) * L + src];
                const void* pb = a.has_base ? a.base[src] : nullptr;
                ws.pw[lane] = pw;
                ws.pb[lane] = pb;
                ok = vec_aligned<ST>(pw) && vec_aligned<ST>(pb);
                uint32_t blk[4] = {0u, 0u, 0u, 0u};
                if (flipped) {
                    const DevTask tk = a.tasks[ti];
                    philox4x32_10(t.cb, slot, kTagSign, tk.id, tk.key0, tk.key1, blk);
                }
                ws.sign[lane] = make_uint4(blk[0], blk[1], blk[2], blk[3]);
            }
            const bool vec = (ls.cols & 3u) == 0 && __all_sync(0xFFFFFFFFu, ok);
            __syncwarp();
            if (lane_on) {
                const bool init = a.init_from_m != 0 || chunk0 > 0;
                const uint32_t neg = a.negate ? 0xFu : 0u;
                if (vec)
                    accumulate_rows<ST, true>(t, ls.cols, ws, lane, nt, init, a.has_base != 0, shuffled, neg, mp);
                else
                    accumulate_rows<ST, false>(t, ls.cols, ws, lane, nt, init, a.has_base != 0, shuffled, neg, mp);
            }
        }
    }
}

template <typename K>
int ctas_per_sm(K kernel)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreadsPerCta, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

}  // namespace

int launch_retrieve(int storage_dtype, int out_dtype, const RetrieveArgs& a, int grid, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (storage_dtype == 0 && out_dtype == 0) retrieve_kernel<float, float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else if (storage_dtype == 0 && out_dtype == 1) retrieve_kernel<float, bf16><<<grid, kThreadsPerCta, 0, s>>>(a);
    else if (storage_dtype == 1 && out_dtype == 0) retrieve_kernel<bf16, float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else retrieve_kernel<bf16, bf16><<<grid, kThreadsPerCta, 0, s>>>(a);
    return static_cast<int>(cudaGetLastError());
}

int launch_accumulate(int storage_dtype, const AccumulateArgs& a, int grid, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (storage_dtype == 0) accumulate_kernel<float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else accumulate_kernel<bf16><<<grid, kThreadsPerCta, 0, s>>>(a);
    return static_cast<int>(cudaGetLastError());
}

int retrieve_ctas_per_sm(int storage_dtype, int out_dtype)
{
    if (storage_dtype == 0 && out_dtype == 0) return ctas_per_sm(retrieve_kernel<float, float>);
    if (storage_dtype == 0 && out_dtype == 1) return ctas_per_sm(retrieve_kernel<float, bf16>);
    if (storage_dtype == 1 && out_dtype == 0) return ctas_per_sm(retrieve_kernel<bf16, float>);
    return ctas_per_sm(retrieve_kernel<bf16, bf16>);
}

int accumulate_ctas_per_sm(int storage_dtype)
{
    return storage_dtype == 0 ? ctas_per_sm(accumulate_kernel<float>) : ctas_per_sm(accumulate_kernel<bf16>);
}

}  // namespace randes
