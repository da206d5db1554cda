// Diagnostics of the superposition: the Gram matrix of the transformed deltas,
//
//     G[i][j] = < T_i d_i , T_j d_j >,   d_i = W_i - W_0,   summed over every parameter,
//
// from which follow the quantities the paper analyses: the pairwise cosines among
// the deltas that interfere when one task is retrieved (its figures on cosine
// similarity during retrieval) and the interference norm of Section 3,
// || lambda * sum_{j != t} T_t^-1 T_j d_j || = lambda * sqrt( sum_{j,l != t} G[j][l] )
// (T_t is orthogonal, so it drops out of every inner product).
//
// One pass over the weights.  G = X X^T with X = [tasks x parameters] is a contraction, and it has
// to be exact in its products (fp32 x fp32 fits fp64) and fixed in its order: it runs on the fp64
// tensor-core instruction mma.m8n8k4.  A warp owns a tile (rows x one warp-wide column block) of a
// slot and walks it in chunks of 16 columns: lane (g, k) = (lane / 4, lane % 4) loads the four
// elements 4k .. 4k+3 of the chunk for tasks g, 8 + g, 16 + g, 24 + g (64 contiguous bytes per
// task and chunk), forms x = +-(W_i - W_0) in fp32 exactly as compress does, widens to fp64, and
// holds one A fragment per block of 8 tasks -- which is also that block's B fragment, because
// B[k][j] = X[j][k].  Four mma steps per chunk (step m contracts elements m, 4 + m, 8 + m, 12 + m)
// update the blocks (bi <= bj) of the upper triangle; the lower one is mirrored at the end.
// Accumulators stay in registers for the whole kernel, are added over the warps of a CTA in warp
// order, and over CTAs in index order by a second kernel: the result does not depend on timing.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

constexpr int kFrag = 64;                     // doubles of one 8 x 8 block: lane holds [lane / 4][2 (lane % 4) + {0, 1}]
constexpr int kMaxBlocks = kGramBlocks;       // upper-triangle blocks of a 32 x 32 matrix

__device__ __forceinline__ void dmma(double (&c)[2], double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c[0]), "+d"(c[1])
                 : "d"(a), "d"(b));
}

// four consecutive elements of a row as fp32 (vector load when the tensor allows it); elements past the row's end are zero
template <typename ST> __device__ __forceinline__ void load4(const ST* p, size_t off, uint32_t c, uint32_t cols, bool vec, float (&v)[4]);
template <> __device__ __forceinline__ void load4<float>(const float* p, size_t off, uint32_t c, uint32_t cols, bool vec, float (&v)[4])
{
    if (vec) {
        const float4 x = __ldcs(reinterpret_cast<const float4*>(p + off));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = c + e < cols ? __ldg(p + off + e) : 0.f;
    }
}
template <> __device__ __forceinline__ void load4<bf16>(const bf16* p, size_t off, uint32_t c, uint32_t cols, bool vec, float (&v)[4])
{
    if (vec) {
        const uint2 x = __ldcs(reinterpret_cast<const uint2*>(p + off));
        v[0] = __uint_as_float(x.x << 16); v[1] = __uint_as_float(x.x & 0xFFFF0000u);
        v[2] = __uint_as_float(x.y << 16); v[3] = __uint_as_float(x.y & 0xFFFF0000u);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = c + e < cols ? Store<bf16>::load1(p + off + e) : 0.f;
    }
}

// NB = blocks of 8 tasks (1 .. 4)
template <typename ST, int NB>
__global__ void __launch_bounds__(kThreadsPerCta, 2) gram_kernel(const GramArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    constexpr uint32_t SPAN = 32 * CPL;          // columns of a warp-wide column block of the unit list
    constexpr int HB = CPL / 4;                  // Philox blocks (128 columns each) under it
    constexpr int NBLK = NB * (NB + 1) / 2;
    __shared__ double red[kWarpsPerCta][NBLK][kFrag];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t g = lane >> 2, kk = lane & 3;
    const uint32_t L = a.n_layers, n = a.n_tasks;
    double acc[NBLK][2];
#pragma unroll
    for (int q = 0; q < NBLK; ++q) acc[q][0] = acc[q][1] = 0.0;

    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const uint32_t cols = ls.cols;
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        const uint32_t c_warp = t.cb * SPAN;
        if (t.r0 >= t.r_end || c_warp >= cols) continue;   // warp-uniform
        // this lane's tasks g, 8 + g, ...: source tensors through sigma_i, and the sign bits of its columns:
        // nibble q of sel[b][h] = signs of columns 128 h + 16 q + 4 kk .. + 3 of the warp's span
        const ST* pw[NB];
        const ST* pb[NB];
        uint32_t sel[NB][HB];
        bool vec[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const uint32_t i = 8 * b + g;
            pw[b] = pb[b] = nullptr;
            vec[b] = false;
#pragma unroll
            for (int h = 0; h < HB; ++h) sel[b][h] = 0;
            if (i < n) {
                const uint32_t src = (ls.flags & kFlagShuffle) ? a.src_of_slot[static_cast<size_t>(i) * L + slot] : slot;   // sigma_i(l)
                pw[b] = static_cast<const ST*>(a.task_ptrs[static_cast<size_t>(i) * L + src]);
                pb[b] = a.has_base ? static_cast<const ST*>(a.base[src]) : nullptr;
                constexpr uintptr_t kAlign = 4 * sizeof(ST) - 1;
                vec[b] = cols % 4 == 0 && (reinterpret_cast<uintptr_t>(pw[b]) & kAlign) == 0 && (reinterpret_cast<uintptr_t>(pb[b]) & kAlign) == 0;
                if (ls.flags & kFlagFlip) {
                    const DevTask tk = a.tasks[i];
#pragma unroll
                    for (int h = 0; h < HB; ++h) {
                        const uint4 blk = philox4x32_10(t.cb * HB + h, slot, kTagSign, tk.id, tk.key0, tk.key1);
                        const uint32_t w[4] = {blk.x, blk.y, blk.z, blk.w};
                        uint32_t s = 0;
#pragma unroll
                        for (int q = 0; q < 8; ++q) s |= ((w[q >> 1] >> (16 * (q & 1) + 4 * kk)) & 0xFu) << (4 * q);
                        sel[b][h] = s;
                    }
                }
            }
        }
        for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
            const size_t row = static_cast<size_t>(r) * cols;
#pragma unroll 2
            for (uint32_t q = 0; q < SPAN / 16; ++q) {
                const uint32_t c = c_warp + 16 * q + 4 * kk;
                if (c_warp + 16 * q >= cols) break;                // warp-uniform: the rest of the span lies past the row
                double x[NB][4];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    float w[4] = {0.f, 0.f, 0.f, 0.f}, b0[4] = {0.f, 0.f, 0.f, 0.f};
                    if (pw[b] != nullptr && c < cols) {
                        load4<ST>(pw[b], row + c, c, cols, vec[b], w);
                        if (pb[b] != nullptr) load4<ST>(pb[b], row + c, c, cols, vec[b], b0);
                    }
                    const uint32_t bits = sel[b][HB == 1 ? 0 : (q >> 3)] >> (4 * (q & 7));
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float d = pb[b] != nullptr ? __fsub_rn(w[e], b0[e]) : w[e];     // the fp32 value compress sums
                        x[b][e] = static_cast<double>(flip(d, ((bits >> e) & 1u) << 31));
                    }
                }
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    int blk = 0;
#pragma unroll
                    for (int bi = 0; bi < NB; ++bi)
#pragma unroll
                        for (int bj = bi; bj < NB; ++bj, ++blk) dmma(acc[blk], x[bi][m], x[bj][m]);
                }
            }
        }
    }
    // over the warps of the CTA, in warp order
#pragma unroll
    for (int q = 0; q < NBLK; ++q) {
        red[warp][q][2 * lane] = acc[q][0];
        red[warp][q][2 * lane + 1] = acc[q][1];
    }
    __syncthreads();
    double* out = a.partial + static_cast<size_t>(blockIdx.x) * (kMaxBlocks * kFrag);
    for (int idx = threadIdx.x; idx < NBLK * kFrag; idx += kThreadsPerCta) {
        double s = 0.0;
        for (int w = 0; w < kWarpsPerCta; ++w) s += red[w][idx / kFrag][idx % kFrag];
        out[idx] = s;
    }
}

// G[i][j] for i <= j = sum over CTAs, in index order, of the CTA sums; the lower triangle is its mirror image
__global__ void gram_reduce_kernel(const double* partial, uint32_t n_ctas, double* gram, uint32_t n, uint32_t nb)
{
    const uint32_t nblk = nb * (nb + 1) / 2;
    for (uint32_t idx = threadIdx.x; idx < nblk * kFrag; idx += blockDim.x) {
        uint32_t blk = idx / kFrag, bi = 0;
        while (blk >= nb - bi) { blk -= nb - bi; ++bi; }        // blocks are listed row by row: (0,0) (0,1) .. (1,1) ..
        const uint32_t bj = bi + blk;
        const uint32_t f = idx % kFrag, i = 8 * bi + (f >> 3), j = 8 * bj + (f & 7);
        if (i >= n || j >= n) continue;
        double s = 0.0;
        for (uint32_t r = 0; r < n_ctas; ++r) s += partial[static_cast<size_t>(r) * (kMaxBlocks * kFrag) + idx];
        if (bi == bj && j < i) continue;                          // written from its mirror image
        gram[static_cast<size_t>(i) * n + j] = s;
        gram[static_cast<size_t>(j) * n + i] = s;
    }
}

template <typename ST, typename F> int with_blocks(uint32_t nb, F&& f)
{
    switch (nb) {
        case 1: return f(gram_kernel<ST, 1>);
        case 2: return f(gram_kernel<ST, 2>);
        case 3: return f(gram_kernel<ST, 3>);
        default: return f(gram_kernel<ST, 4>);
    }
}

}  // namespace

int gram_ctas_per_sm(int storage_dtype)
{
    int n = 0;
    cudaError_t e = storage_dtype == 0 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gram_kernel<float, 4>, kThreadsPerCta, 0)
                                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gram_kernel<__nv_bfloat16, 4>, kThreadsPerCta, 0);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

int launch_gram(int storage_dtype, const GramArgs& a, int grid, double* gram, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t nb = (a.n_tasks + 7) / 8;
    auto go = [&](auto kernel) {
        kernel<<<grid, kThreadsPerCta, 0, s>>>(a);
        return static_cast<int>(cudaGetLastError());
    };
    const int e = storage_dtype == 0 ? with_blocks<float>(nb, go) : with_blocks<__nv_bfloat16>(nb, go);
    if (e) return e;
    gram_reduce_kernel<<<1, 640, 0, s>>>(a.partial, static_cast<uint32_t>(grid), gram, a.n_tasks, nb);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace randes
