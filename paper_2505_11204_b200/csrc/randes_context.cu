// Superposition and retrieval with a general diagonal context matrix: the "RD" ablation of
// Section 5.5, where the per-column +-1 of Section 4.4 is replaced by a (nearly) standard normal
// deviate g_i(l, c).  Such a D is not orthogonal: compress multiplies by it, retrieval divides.
//
//   compress / add / remove:  M[l][r,c] (+|-)= g_i(l,c) * ( W_i[sigma_i(l)][r,c] - W_0[sigma_i(l)][r,c] )
//   retrieve:                 out[p][r,c] = fma(lambda, M[l][r,c] / g_t(l,c), W_0[p][r,c]),  l = sigma_t^-1(p)
//
// A plan with such a group runs ALL its layers through these kernels; layers with a +-1 context or
// none use g = +-1 or 1, for which the arithmetic below gives the bits of the streaming kernels
// (x * +-1 and x / +-1 are exact).  This is an ablation the paper itself discards (it interferes
// more), so the kernels are plain: a thread takes four neighbouring columns and walks the rows of a
// unit, with the loads of all tasks of a row issued before the first use; no staging, no tuning
// beyond that (a third to under a half of the streaming kernels' speed).  Every operation is an
// explicitly rounded fp32 intrinsic, in the order of the definition, so results are bit-identical
// to a scalar evaluation.
//
// g: the paper names no generator.  Sum of twelve uniforms minus six: the twelve words of Philox
// blocks 3c, 3c+1, 3c+2 of the (slot, task) stream tagged "GAUS", each reduced to
// u = (word >> 8) * 2^-24 (exact) and added left to right; a zero is replaced by one.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

constexpr int kContextChunk = 8;                                  // tasks whose factors a CTA keeps at once
constexpr int kContextSpan = kWarpsPerCta * 32 * 8;               // widest unit: 8 column blocks of 256 columns
constexpr size_t kContextSmem = static_cast<size_t>(kContextChunk) * kContextSpan * sizeof(float);

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

template <typename ST>
__global__ void __launch_bounds__(kThreadsPerCta) context_accumulate_kernel(const AccumulateArgs a)
{
    constexpr uint32_t WC = 32 * Store<ST>::CPL;          // columns of one column block of the unit list
    extern __shared__ __align__(16) float gtab[];         // [kContextChunk][kContextSpan]
    const uint32_t L = a.n_layers;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const uint32_t cols = ls.cols;
        const uint32_t c_begin = un.cb0 * WC, c_end = min(cols, (un.cb0 + un.nbc) * WC);
        float* mp = static_cast<float*>(a.M) + ls.m_off;
        for (uint32_t chunk0 = 0; chunk0 < a.n_tasks; chunk0 += kContextChunk) {
            const uint32_t nt = min(static_cast<uint32_t>(kContextChunk), a.n_tasks - chunk0);
            const void* pw[kContextChunk];
            const void* pb[kContextChunk];
#pragma unroll
            for (int k = 0; k < kContextChunk; ++k) {
                pw[k] = pb[k] = nullptr;
                if (static_cast<uint32_t>(k) < nt) {
                    const uint32_t ti = chunk0 + k;
                    const uint32_t src = (ls.flags & kFlagShuffle) ? a.src_of_slot[static_cast<size_t>(ti) * L + slot] : slot;   // sigma_i(l)
                    pw[k] = a.task_ptrs[static_cast<size_t>(ti) * L + src];
                    pb[k] = a.has_base ? a.base[src] : nullptr;
                    const DevTask tk = a.tasks[ti];
                    for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += kThreadsPerCta) {
                        const float g = context_entry(ls.flags, tk, slot, c);
                        gtab[k * kContextSpan + (c - c_begin)] = a.negate ? -g : g;   // remove: M - x = M + (-g) d, exactly
                    }
                }
            }
            const bool from_m = chunk0 > 0 || a.init_from_m;
            bool vec = cols % 4 == 0;
#pragma unroll
            for (int k = 0; k < kContextChunk; ++k)
                if (static_cast<uint32_t>(k) < nt) vec = vec && quad_aligned<ST>(pw[k]) && (!pb[k] || quad_aligned<ST>(pb[k]));
            if (vec) {
                // a thread owns columns 4q .. 4q+3, q = its index + 256 j; the factors of those columns were written
                // by threads 4q .. 4q+3 of the same pass (column c by thread (c - c_begin) % 256)
                __syncthreads();
                for (uint32_t r = un.row0; r < un.row0 + un.nrows; ++r) {
                    for (uint32_t c = c_begin + 4 * threadIdx.x; c < c_end; c += 4 * kThreadsPerCta) {
                        const size_t idx = static_cast<size_t>(r) * cols + c;
                        float w[kContextChunk][4], b[kContextChunk][4], acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int k = 0; k < kContextChunk; ++k)
                            if (static_cast<uint32_t>(k) < nt) {
                                load_quad<ST>(pw[k], idx, w[k]);
                                if (pb[k]) load_quad<ST>(pb[k], idx, b[k]);
                            }
                        if (from_m) load_quad<float>(mp, idx, acc);
#pragma unroll
                        for (int k = 0; k < kContextChunk; ++k)
                            if (static_cast<uint32_t>(k) < nt) {
                                const float4 g = *reinterpret_cast<const float4*>(&gtab[k * kContextSpan + (c - c_begin)]);
                                const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float d = pb[k] ? __fsub_rn(w[k][e], b[k][e]) : w[k][e];
                                    acc[e] = __fadd_rn(acc[e], __fmul_rn(d, gv[e]));
                                }
                            }
                        store_quad(mp + idx, acc);
                    }
                }
                __syncthreads();   // the table is rewritten by the next pass
                continue;
            }
            // element-wise: each thread reads back only the columns it wrote: no barrier
            for (uint32_t r = un.row0; r < un.row0 + un.nrows; ++r) {
                for (uint32_t c = c_begin + threadIdx.x; c < c_end; c += kThreadsPerCta) {
                    const size_t idx = static_cast<size_t>(r) * cols + c;
                    float acc = from_m ? mp[idx] : 0.0f;
#pragma unroll
                    for (int k = 0; k < kContextChunk; ++k) {
                        if (static_cast<uint32_t>(k) < nt) {
                            float d = load_elem<ST>(pw[k], idx);
                            if (pb[k]) d = __fsub_rn(d, load_elem<ST>(pb[k], idx));
                            acc = __fadd_rn(acc, __fmul_rn(d, gtab[k * kContextSpan + (c - c_begin)]));
                        }
                    }
                    mp[idx] = acc;
                }
            }
        }
    }
}

template <typename ST, typename OT>
__global__ void __launch_bounds__(kThreadsPerCta) context_retrieve_kernel(const RetrieveArgs a)
{
    constexpr uint32_t WC = 32 * Store<ST>::CPL;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;
        const DevLayer lp = a.layers[p];
        const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[p] : p;   // sigma^-1
        const float* mp = static_cast<const float*>(a.M) + a.layers[slot].m_off;
        const void* wp = a.base[p];
        OT* op = static_cast<OT*>(a.out[p]);
        const uint32_t cols = lp.cols;
        const uint32_t c_begin = un.cb0 * WC, c_end = min(cols, (un.cb0 + un.nbc) * WC);
        if (cols % 4 == 0 && quad_aligned<ST>(wp) && quad_aligned<OT>(op)) {
            for (uint32_t c = c_begin + 4 * threadIdx.x; c < c_end; c += 4 * kThreadsPerCta) {
                float g[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) g[e] = context_entry(lp.flags, a.task, slot, c + e);
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
            const float g = context_entry(lp.flags, a.task, slot, c);
            for (uint32_t r = un.row0; r < un.row0 + un.nrows; ++r) {
                const size_t idx = static_cast<size_t>(r) * cols + c;
                const float t = __fdiv_rn(mp[idx], g);      // D^-1 of a diagonal D divides (+-1: exact)
                Out<OT>::store1(op + idx, __fmaf_rn(a.lambda, t, load_elem<ST>(wp, idx)));
            }
        }
    }
}

}  // namespace

int launch_context_accumulate(int storage_dtype, const AccumulateArgs& a, int sm_count, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid = static_cast<int>(min(static_cast<unsigned long long>(sm_count) * 4ull, static_cast<unsigned long long>(a.n_units)));
    cudaError_t e;
    if (storage_dtype == 0) {
        e = cudaFuncSetAttribute(context_accumulate_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kContextSmem));
        if (e == cudaSuccess) context_accumulate_kernel<float><<<grid, kThreadsPerCta, kContextSmem, s>>>(a);
    } else {
        e = cudaFuncSetAttribute(context_accumulate_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kContextSmem));
        if (e == cudaSuccess) context_accumulate_kernel<bf16><<<grid, kThreadsPerCta, kContextSmem, s>>>(a);
    }
    if (e != cudaSuccess) { (void)cudaGetLastError(); return static_cast<int>(e); }
    return static_cast<int>(cudaGetLastError());
}

int launch_context_retrieve(int storage_dtype, int out_dtype, const RetrieveArgs& a, int sm_count, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid = static_cast<int>(min(static_cast<unsigned long long>(sm_count) * 8ull, static_cast<unsigned long long>(a.n_units)));
    if (storage_dtype == 0 && out_dtype == 0) context_retrieve_kernel<float, float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else if (storage_dtype == 0) context_retrieve_kernel<float, bf16><<<grid, kThreadsPerCta, 0, s>>>(a);
    else if (out_dtype == 0) context_retrieve_kernel<bf16, float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else context_retrieve_kernel<bf16, bf16><<<grid, kThreadsPerCta, 0, s>>>(a);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace randes
