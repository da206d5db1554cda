// Superposition and retrieval with a general diagonal context matrix: the "RD" ablation of
// Section 5.5, where the per-column +-1 of Section 4.4 is replaced by a (nearly) standard normal
// deviate g_i(l, c).  Such a D is not orthogonal: compress multiplies by it, retrieval divides.
//
//   compress / add / remove:  M[l][r,c] (+|-)= g_i(l,c) * ( W_i[sigma_i(l)][r,c] - W_0[sigma_i(l)][r,c] )
//   retrieve:                 out[p][r,c] = fma(lambda, M[l][r,c] / g_t(l,c), W_0[p][r,c]),  l = sigma_t^-1(p)
//
// A plan with such a group runs ALL its layers through these kernels; layers with a +-1 context or
// none use g = +-1 or 1, for which the arithmetic below gives the bits of the streaming kernels
// (x * +-1 and x / +-1 are exact).  Every operation is an explicitly rounded fp32 intrinsic, in the
// order of the definition, so results are bit-identical to a scalar evaluation.
//
// g: the paper names no generator.  Sum of twelve uniforms minus six: the twelve words of Philox
// blocks 3c, 3c+1, 3c+2 of the (slot, task) stream tagged "GAUS", each reduced to
// u = (word >> 8) * 2^-24 (exact) and added left to right; a zero is replaced by one.
//
// The factors cost three Philox blocks per (task, column), far more than one sign bit, so they are
// not recomputed per tile: context_fill_kernel writes them once per registered task into a table in
// the plan's workspace (one float per task and column of every slot; +-1 and 1 for the other
// layers, so the kernels below never branch on the kind of context), and the kernels read them
// from there (the table stays in L2: 4 bytes per task and column against 4 bytes per task and
// ELEMENT of weight traffic).  A thread owns four neighbouring columns of a unit and walks down its rows.  Compress sums
// four tasks per pass over the unit, the rows travelling through a per-thread cp.async ring (three rows in flight);
// further tasks take further passes over the unit's part of M, which is still in L2 then.  The units are those of the
// streaming kernels, in their order (all slots of a group at one tile offset adjacent), so the W_0 tiles that several
// slots read under a shuffle are served by L2 as well -- helped by eviction priorities on the copies (task weights:
// evict first; W_0: evict last), without which a fifth of the W_0 reads and the second write of M went to DRAM.
// Add / remove (one task) and retrieve keep eight and four rows of plain loads in flight per thread instead.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;


__device__ __forceinline__ float gauss_entry(const DevTask& tk, uint32_t slot, uint32_t col)
{
    float sum = 0.0f;
#pragma unroll
    for (uint32_t b = 0; b < 3; ++b) {
        const uint4 blk = philox4x32_10(3u * col + b, slot, kTagGauss, tk.id, tk.key0, tk.key1);
        sum = __fadd_rn(sum, __fmul_rn(__uint2float_rn(blk.x >> 8), 0x1p-24f));
        sum = __fadd_rn(sum, __fmul_rn(__uint2float_rn(blk.y >> 8), 0x1p-24f));
        sum = __fadd_rn(sum, __fmul_rn(__uint2float_rn(blk.z >> 8), 0x1p-24f));
        sum = __fadd_rn(sum, __fmul_rn(__uint2float_rn(blk.w >> 8), 0x1p-24f));
    }
    const float g = __fsub_rn(sum, 6.0f);
    return g == 0.0f ? 1.0f : g;
}

// diagonal entry of the slot's context for (task, column): Gaussian-like, +-1, or 1
__device__ __forceinline__ float context_entry(uint32_t flags, const DevTask& tk, uint32_t slot, uint32_t col)
{
    if (flags & kFlagGauss) return gauss_entry(tk, slot, col);
    if (flags & kFlagFlip) {
        const uint4 blk = philox4x32_10(col >> 7, slot, kTagSign, tk.id, tk.key0, tk.key1);
        const uint32_t q = (col >> 5) & 3u;
        const uint32_t w = q == 0 ? blk.x : (q == 1 ? blk.y : (q == 2 ? blk.z : blk.w));
        return ((w >> (col & 31u)) & 1u) ? -1.0f : 1.0f;
    }
    return 1.0f;
}

// table[row][off[slot] + c] = g_row(slot, c) for the task rows first_row .. first_row + n_rows - 1
// grid: x over columns, y over slots, z over task rows (y and z wrap when the plan has more than the grid holds)
__global__ void __launch_bounds__(kThreadsPerCta) context_fill_kernel(float* table, const uint32_t* off, uint32_t stride, const DevLayer* layers,
                                                                        uint32_t n_layers, const DevTask* tasks, uint32_t first_row, uint32_t n_rows)
{
    for (uint32_t i = blockIdx.z; i < n_rows; i += gridDim.z) {
        const uint32_t row = first_row + i;
        const DevTask tk = tasks[row];
        for (uint32_t slot = blockIdx.y; slot < n_layers; slot += gridDim.y) {
            const DevLayer ls = layers[slot];
            float* dst = table + static_cast<size_t>(row) * stride + off[slot];
            for (uint32_t c = blockIdx.x * kThreadsPerCta + threadIdx.x; c < ls.cols; c += gridDim.x * kThreadsPerCta)
                dst[c] = context_entry(ls.flags, tk, slot, c);
        }
    }
}

template <typename T> __device__ __forceinline__ float load_elem(const void* p, size_t i);
template <> __device__ __forceinline__ float load_elem<float>(const void* p, size_t i) { return static_cast<const float*>(p)[i]; }
template <> __device__ __forceinline__ float load_elem<bf16>(const void* p, size_t i)
{
    return __uint_as_float(static_cast<uint32_t>(static_cast<const unsigned short*>(p)[i]) << 16);
}

// four neighbouring elements of a row
template <typename T> __device__ __forceinline__ void load_quad(const void* p, size_t i, float (&v)[4]);
template <> __device__ __forceinline__ void load_quad<float>(const void* p, size_t i, float (&v)[4])
{
    const float4 x = *reinterpret_cast<const float4*>(static_cast<const float*>(p) + i);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
template <> __device__ __forceinline__ void load_quad<bf16>(const void* p, size_t i, float (&v)[4])
{
    const uint2 x = *reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(p) + i);
    v[0] = __uint_as_float(x.x << 16); v[1] = __uint_as_float(x.x & 0xFFFF0000u);
    v[2] = __uint_as_float(x.y << 16); v[3] = __uint_as_float(x.y & 0xFFFF0000u);
}
template <typename T> __device__ __forceinline__ bool quad_aligned(const void* p)
{
    return (reinterpret_cast<uintptr_t>(p) & (4 * sizeof(T) - 1)) == 0;
}
__device__ __forceinline__ void store_quad(float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
__device__ __forceinline__ void store_quad(bf16* p, const float (&v)[4])
{
    *reinterpret_cast<uint2*>(p) = make_uint2(Out<bf16>::pack(v[0], v[1]), Out<bf16>::pack(v[2], v[3]));
}

// One pass over a unit for the tasks chunk0 .. chunk0 + nt - 1 (nt <= CH), four neighbouring columns per thread, RU rows
// per trip: the 2 CH RU loads of a trip (W_i and W_0 of every task and row) are issued before the first use.
template <typename ST, int CH, int RU>
__device__ __forceinline__ void accumulate_quads(const AccumulateArgs& a, const DevUnit& un, uint32_t cols, uint32_t c_begin, uint32_t c_end, float* mp,
                                                 const float* gchunk, uint32_t gstride, uint32_t nt, const void* const (&pw)[CH],
                                                 const void* const (&pb)[CH], bool from_m)
{
    for (uint32_t c = c_begin + 4 * threadIdx.x; c < c_end; c += 4 * kThreadsPerCta) {
        float g[CH][4];
#pragma unroll
        for (int k = 0; k < CH; ++k)
            if (static_cast<uint32_t>(k) < nt) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(gchunk + static_cast<size_t>(k) * gstride + c));
                g[k][0] = a.negate ? -t.x : t.x; g[k][1] = a.negate ? -t.y : t.y;   // remove: M - x = M + (-g) d, exactly
                g[k][2] = a.negate ? -t.z : t.z; g[k][3] = a.negate ? -t.w : t.w;
            }
        const uint32_t r_end = un.row0 + un.nrows;
        for (uint32_t r0 = un.row0; r0 < r_end; r0 += RU) {
            float w[RU][CH][4], b[RU][CH][4], acc[RU][4];
#pragma unroll
            for (int j = 0; j < RU; ++j)
                if (r0 + j < r_end) {
                    const size_t idx = static_cast<size_t>(r0 + j) * cols + c;
#pragma unroll
                    for (int k = 0; k < CH; ++k)
                        if (static_cast<uint32_t>(k) < nt) {
                            load_quad<ST>(pw[k], idx, w[j][k]);
                            if (pb[k]) load_quad<ST>(pb[k], idx, b[j][k]);
                        }
                    if (from_m) load_quad<float>(mp, idx, acc[j]);
                    else acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
                }
#pragma unroll
            for (int j = 0; j < RU; ++j)
                if (r0 + j < r_end) {
#pragma unroll
                    for (int k = 0; k < CH; ++k)
                        if (static_cast<uint32_t>(k) < nt) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float d = pb[k] ? __fsub_rn(w[j][k][e], b[j][k][e]) : w[j][k][e];
                                acc[j][e] = __fadd_rn(acc[j][e], __fmul_rn(d, g[k][e]));
                            }
                        }
                    store_quad(mp + static_cast<size_t>(r0 + j) * cols + c, acc[j]);
                }
        }
    }
}

// The same pass with the rows travelling through a per-thread cp.async ring in shared memory (a thread reads back only
// what it copied: no barrier): a stage holds one row -- the four columns of W_i and of W_0 for each of the CH tasks, and
// of M when the sum continues from it -- and kContextStages rows are in flight while one is summed, which the register
// form above (loads of a trip issued, awaited, used, then the next trip) cannot keep up.
constexpr int kContextStages = 3;
template <int CH> struct ContextRing {
    static constexpr int kSlots = 2 * CH + 1;
    static constexpr uint32_t kStageBytes = kSlots * kSlotBytes;
    static constexpr size_t kSmem = static_cast<size_t>(kContextStages) * kStageBytes;
};
// copies with an L2 eviction priority: the task weights stream through once (evict first), the W_0 tiles are read again by
// the other slots of the group under a shuffle (evict last)
template <typename T> __device__ __forceinline__ void copy_quad(uint32_t dst, const void* p, size_t i, uint64_t pol);
template <> __device__ __forceinline__ void copy_quad<float>(uint32_t dst, const void* p, size_t i, uint64_t pol)
{
    cp_async16_hint(dst, static_cast<const float*>(p) + i, pol);
}
template <> __device__ __forceinline__ void copy_quad<bf16>(uint32_t dst, const void* p, size_t i, uint64_t pol)
{
    asm volatile("cp.async.ca.shared.global.L2::cache_hint [%0], [%1], 8, %2;" ::"r"(dst), "l"(static_cast<const unsigned short*>(p) + i), "l"(pol) : "memory");
}
template <typename T> __device__ __forceinline__ void read_quad(uint32_t src, float (&v)[4]);
template <> __device__ __forceinline__ void read_quad<float>(uint32_t src, float (&v)[4])
{
    const uint4 x = lds128(src);
    v[0] = __uint_as_float(x.x); v[1] = __uint_as_float(x.y); v[2] = __uint_as_float(x.z); v[3] = __uint_as_float(x.w);
}
template <> __device__ __forceinline__ void read_quad<bf16>(uint32_t src, float (&v)[4])
{
    const uint4 x = lds128(src);      // the low 8 bytes hold the four bf16 values
    v[0] = __uint_as_float(x.x << 16); v[1] = __uint_as_float(x.x & 0xFFFF0000u);
    v[2] = __uint_as_float(x.y << 16); v[3] = __uint_as_float(x.y & 0xFFFF0000u);
}

template <typename ST, int CH>
__device__ __forceinline__ void accumulate_quads_ring(const AccumulateArgs& a, const DevUnit& un, uint32_t cols, uint32_t c_begin, uint32_t c_end,
                                                      float* mp, const float* gchunk, uint32_t gstride, uint32_t nt, const void* const (&pw)[CH],
                                                      const void* const (&pb)[CH], bool from_m, uint32_t ring)
{
    typedef ContextRing<CH> R;
    const uint64_t pol_stream = l2_evict_first_policy(), pol_keep = l2_evict_last_policy();
    for (uint32_t c = c_begin + 4 * threadIdx.x; c < c_end; c += 4 * kThreadsPerCta) {
        float g[CH][4];
#pragma unroll
        for (int k = 0; k < CH; ++k)
            if (static_cast<uint32_t>(k) < nt) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(gchunk + static_cast<size_t>(k) * gstride + c));
                g[k][0] = a.negate ? -t.x : t.x; g[k][1] = a.negate ? -t.y : t.y;   // remove: M - x = M + (-g) d, exactly
                g[k][2] = a.negate ? -t.z : t.z; g[k][3] = a.negate ? -t.w : t.w;
            }
        // one commit group per row, empty past the last row, so that "all but the newest kContextStages - 1 groups have
        // landed" always means "row i has landed"
        auto issue = [&](uint32_t i) {
            if (i < un.nrows) {
                const size_t idx = static_cast<size_t>(un.row0 + i) * cols + c;
                const uint32_t st = ring + (i % kContextStages) * R::kStageBytes;
#pragma unroll
                for (int k = 0; k < CH; ++k)
                    if (static_cast<uint32_t>(k) < nt) {
                        copy_quad<ST>(st + (2 * k) * kSlotBytes, pw[k], idx, pol_stream);
                        if (pb[k]) copy_quad<ST>(st + (2 * k + 1) * kSlotBytes, pb[k], idx, pol_keep);
                    }
                if (from_m) cp_async16(st + (2 * CH) * kSlotBytes, mp + idx);
            }
            cp_async_commit();
        };
#pragma unroll
        for (int i = 0; i < kContextStages - 1; ++i) issue(i);
        for (uint32_t i = 0; i < un.nrows; ++i) {
            issue(i + kContextStages - 1);      // into the stage that row i - 1 has left
            cp_async_wait<kContextStages - 1>();
            const uint32_t st = ring + (i % kContextStages) * R::kStageBytes;
            float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (from_m) read_quad<float>(st + (2 * CH) * kSlotBytes, acc);
#pragma unroll
            for (int k = 0; k < CH; ++k)
                if (static_cast<uint32_t>(k) < nt) {
                    float w[4], b[4];
                    read_quad<ST>(st + (2 * k) * kSlotBytes, w);
                    if (pb[k]) read_quad<ST>(st + (2 * k + 1) * kSlotBytes, b);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float d = pb[k] ? __fsub_rn(w[e], b[e]) : w[e];
                        acc[e] = __fadd_rn(acc[e], __fmul_rn(d, g[k][e]));
                    }
                }
            store_quad(mp + static_cast<size_t>(un.row0 + i) * cols + c, acc);
        }
        cp_async_wait<0>();                      // (only empty groups are left)
    }
    __threadfence_block();                       // this pass's stores to M before the next pass's copies from it
}

// CH tasks per pass over a unit; RU > 0: rows per trip of the register form (one task: eight rows), RU = 0: the ring form
template <typename ST, int CH, int RU>
__global__ void __launch_bounds__(kThreadsPerCta, 2) context_accumulate_kernel(const AccumulateArgs a, const ContextArgs x)
{
    constexpr uint32_t WC = 32 * Store<ST>::CPL;          // columns of one column block of the unit list
    extern __shared__ __align__(16) unsigned char ring_smem[];
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(ring_smem)) + threadIdx.x * 16;
    const uint32_t L = a.n_layers;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const uint32_t cols = ls.cols;
        const uint32_t c_begin = un.cb0 * WC, c_end = min(cols, (un.cb0 + un.nbc) * WC);
        float* mp = static_cast<float*>(a.M) + ls.m_off;
        const float* grow = x.table + x.off[slot];        // + task row * stride + column
        for (uint32_t chunk0 = 0; chunk0 < a.n_tasks; chunk0 += CH) {
            const uint32_t nt = min(static_cast<uint32_t>(CH), a.n_tasks - chunk0);
            const void* pw[CH];
            const void* pb[CH];
            bool vec = cols % 4 == 0;
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                pw[k] = pb[k] = nullptr;
                if (static_cast<uint32_t>(k) < nt) {
                    const uint32_t ti = chunk0 + k;
                    const uint32_t src = (ls.flags & kFlagShuffle) ? a.src_of_slot[static_cast<size_t>(ti) * L + slot] : slot;   // sigma_i(l)
                    pw[k] = a.task_ptrs[static_cast<size_t>(ti) * L + src];
                    pb[k] = a.has_base ? a.base[src] : nullptr;
                    vec = vec && quad_aligned<ST>(pw[k]) && (!pb[k] || quad_aligned<ST>(pb[k]));
                }
            }
            const bool from_m = chunk0 > 0 || a.init_from_m;
            const float* gchunk = grow + static_cast<size_t>(chunk0) * x.stride;
            // the same thread owns an element of M in every pass: no barrier between the passes
            if (vec) {
                if constexpr (RU > 0) accumulate_quads<ST, CH, RU>(a, un, cols, c_begin, c_end, mp, gchunk, x.stride, nt, pw, pb, from_m);
                else accumulate_quads_ring<ST, CH>(a, un, cols, c_begin, c_end, mp, gchunk, x.stride, nt, pw, pb, from_m, ring);
                continue;
            }
            for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += kThreadsPerCta) {
                float g[CH];
#pragma unroll
                for (int k = 0; k < CH; ++k)
                    if (static_cast<uint32_t>(k) < nt) {
                        const float t = gchunk[static_cast<size_t>(k) * x.stride + c];
                        g[k] = a.negate ? -t : t;
                    }
                for (uint32_t r = un.row0; r < un.row0 + un.nrows; ++r) {
                    const size_t idx = static_cast<size_t>(r) * cols + c;
                    float acc = from_m ? mp[idx] : 0.0f;
#pragma unroll
                    for (int k = 0; k < CH; ++k) {
                        if (static_cast<uint32_t>(k) < nt) {
                            float d = load_elem<ST>(pw[k], idx);
                            if (pb[k]) d = __fsub_rn(d, load_elem<ST>(pb[k], idx));
                            acc = __fadd_rn(acc, __fmul_rn(d, g[k]));
                        }
                    }
                    mp[idx] = acc;
                }
            }
        }
    }
}

template <typename ST, typename OT>
__global__ void __launch_bounds__(kThreadsPerCta) context_retrieve_kernel(const RetrieveArgs a, const ContextArgs x)
{
    constexpr uint32_t WC = 32 * Store<ST>::CPL;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;
        const DevLayer lp = a.layers[p];
        const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[p] : p;   // sigma^-1
        const float* mp = static_cast<const float*>(a.M) + a.layers[slot].m_off;
        const float* grow = x.table + x.off[slot];        // this task's row of the table, this slot's columns
        const void* wp = a.base[p];
        OT* op = static_cast<OT*>(a.out[p]);
        const uint32_t cols = lp.cols;
        const uint32_t c_begin = un.cb0 * WC, c_end = min(cols, (un.cb0 + un.nbc) * WC);
        if (cols % 4 == 0 && quad_aligned<ST>(wp) && quad_aligned<OT>(op)) {
            for (uint32_t c = c_begin + 4 * threadIdx.x; c < c_end; c += 4 * kThreadsPerCta) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(grow + c));
                const float g[4] = {t.x, t.y, t.z, t.w};
                for (uint32_t r0 = un.row0; r0 < un.row0 + un.nrows; r0 += 4) {
                    float m[4][4], w[4][4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (r0 + j < un.row0 + un.nrows) {
                            const size_t idx = static_cast<size_t>(r0 + j) * cols + c;
                            load_quad<float>(mp, idx, m[j]);
                            load_quad<ST>(wp, idx, w[j]);
                        }
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (r0 + j < un.row0 + un.nrows) {
                            float y[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) y[e] = __fmaf_rn(a.lambda, __fdiv_rn(m[j][e], g[e]), w[j][e]);
                            store_quad(op + static_cast<size_t>(r0 + j) * cols + c, y);
                        }
                }
            }
            continue;
        }
        for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += kThreadsPerCta) {
            const float g = grow[c];
            for (uint32_t r = un.row0; r < un.row0 + un.nrows; ++r) {
                const size_t idx = static_cast<size_t>(r) * cols + c;
                const float t = __fdiv_rn(mp[idx], g);      // D^-1 of a diagonal D divides (+-1: exact)
                Out<OT>::store1(op + idx, __fmaf_rn(a.lambda, t, load_elem<ST>(wp, idx)));
            }
        }
    }
}

}  // namespace

int launch_context_fill(const ContextArgs& x, const DevLayer* layers, uint32_t n_layers, uint32_t max_cols, const DevTask* tasks,
                        uint32_t first_row, uint32_t n_rows, void* stream)
{
    if (n_rows == 0 || n_layers == 0 || max_cols == 0) return static_cast<int>(cudaSuccess);
    const dim3 grid((max_cols + kThreadsPerCta - 1) / kThreadsPerCta, n_layers < 65535u ? n_layers : 65535u, n_rows < 65535u ? n_rows : 65535u);
    context_fill_kernel<<<grid, kThreadsPerCta, 0, static_cast<cudaStream_t>(stream)>>>(const_cast<float*>(x.table), x.off, x.stride, layers, n_layers,
                                                                                            tasks, first_row, n_rows);
    return static_cast<int>(cudaGetLastError());
}

// One CTA per unit (the block scheduler deals the units out as SMs come free; measured 5 - 15 % faster than a resident
// loop on the small sets, equal on the large ones).
template <typename K> int launch_accumulate_form(K kernel, size_t smem, const AccumulateArgs& a, const ContextArgs& x, cudaStream_t s)
{
    if (smem) {
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) { (void)cudaGetLastError(); return static_cast<int>(e); }
    }
    const int grid = static_cast<int>(min(static_cast<unsigned long long>(a.n_units), 0x7FFFFFFFull));
    kernel<<<grid, kThreadsPerCta, smem, s>>>(a, x);
    return static_cast<int>(cudaGetLastError());
}

int launch_context_accumulate(int storage_dtype, const AccumulateArgs& a, const ContextArgs& x, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // one task (add / remove): eight rows per trip in registers; several: four tasks per pass through the ring
    // (six or eight tasks per pass leave room for one CTA per SM only and measured 50 - 80 % slower)
    if (a.n_tasks == 1)
        return storage_dtype == 0 ? launch_accumulate_form(context_accumulate_kernel<float, 1, 8>, 0, a, x, s)
                                  : launch_accumulate_form(context_accumulate_kernel<bf16, 1, 8>, 0, a, x, s);
    return storage_dtype == 0 ? launch_accumulate_form(context_accumulate_kernel<float, 4, 0>, ContextRing<4>::kSmem, a, x, s)
                              : launch_accumulate_form(context_accumulate_kernel<bf16, 4, 0>, ContextRing<4>::kSmem, a, x, s);
}

int launch_context_retrieve(int storage_dtype, int out_dtype, const RetrieveArgs& a, const ContextArgs& x, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid = static_cast<int>(min(static_cast<unsigned long long>(a.n_units), 0x7FFFFFFFull));   // one CTA per unit
    if (storage_dtype == 0 && out_dtype == 0) context_retrieve_kernel<float, float><<<grid, kThreadsPerCta, 0, s>>>(a, x);
    else if (storage_dtype == 0) context_retrieve_kernel<float, bf16><<<grid, kThreadsPerCta, 0, s>>>(a, x);
    else if (out_dtype == 0) context_retrieve_kernel<bf16, float><<<grid, kThreadsPerCta, 0, s>>>(a, x);
    else context_retrieve_kernel<bf16, bf16><<<grid, kThreadsPerCta, 0, s>>>(a, x);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace randes
