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
// Products of two fp32 values are exact in fp64; they are accumulated in fp64, per
// lane over a tile, then across the warp by a fixed shuffle tree, then per warp over
// its tiles in a fixed order, then over warps and CTAs by a second kernel in index
// order: the result does not depend on timing.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

constexpr int GA = kGramAnchors;   // anchor tasks (rows of G) per pass
constexpr int JB = 4;              // partner tasks whose sums are kept in registers at a time

struct GramScratch {
    const void* pw[kTaskChunk];
    const void* pb[kTaskChunk];
    unsigned char bits[kTaskChunk][32];   // [task][lane]
    double acc[GA][kTaskChunk];           // this warp's running sums for the pass
};

// the lane's CPL values of the transformed delta of task i at element offset `off`
template <typename ST, bool VEC>
__device__ __forceinline__ void load_x(const GramScratch& ws, uint32_t i, int lane, size_t off, uint32_t c, uint32_t cols, bool on,
                                       bool has_base, float (&x)[Store<ST>::CPL])
{
    constexpr int CPL = Store<ST>::CPL;
#pragma unroll
    for (int e = 0; e < CPL; ++e) x[e] = 0.f;
    if (!on) return;
    const ST* pw = static_cast<const ST*>(ws.pw[i]);
    const ST* pb = static_cast<const ST*>(ws.pb[i]);
    float b[CPL];
    if (VEC) {
        Store<ST>::widen(__ldg(reinterpret_cast<const uint4*>(pw + off)), x);
        if (has_base) Store<ST>::widen(__ldg(reinterpret_cast<const uint4*>(pb + off)), b);
    } else {
#pragma unroll
        for (int e = 0; e < CPL; ++e) {
            b[e] = 0.f;
            if (c + e < cols) {
                x[e] = Store<ST>::load1(pw + off + e);
                if (has_base) b[e] = Store<ST>::load1(pb + off + e);
            }
        }
    }
    const uint32_t bits = ws.bits[i][lane];
#pragma unroll
    for (int e = 0; e < CPL; ++e) {
        if (has_base) x[e] = __fsub_rn(x[e], b[e]);
        x[e] = flip(x[e], ((bits >> e) & 1u) << 31);
    }
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

template <typename ST, bool VEC>
__device__ __forceinline__ void gram_rows(const WarpTile& t, uint32_t cols, GramScratch& ws, int lane, uint32_t n, uint32_t a0,
                                          uint32_t na, bool lane_on, bool has_base)
{
    constexpr int CPL = Store<ST>::CPL;
    for (uint32_t j0 = 0; j0 < n; j0 += JB) {
        double s[GA][JB];
#pragma unroll
        for (int a = 0; a < GA; ++a)
#pragma unroll
            for (int b = 0; b < JB; ++b) s[a][b] = 0.0;
        for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
            const size_t off = static_cast<size_t>(r) * cols + t.c;
            float xa[GA][CPL];
#pragma unroll
            for (int a = 0; a < GA; ++a) load_x<ST, VEC>(ws, a0 + (a < static_cast<int>(na) ? a : 0), lane, off, t.c, cols, lane_on, has_base, xa[a]);
#pragma unroll
            for (int b = 0; b < JB; ++b) {
                if (j0 + b < n) {
                    float xj[CPL];
                    load_x<ST, VEC>(ws, j0 + b, lane, off, t.c, cols, lane_on, has_base, xj);
#pragma unroll
                    for (int a = 0; a < GA; ++a)
#pragma unroll
                        for (int e = 0; e < CPL; ++e) s[a][b] = fma(static_cast<double>(xa[a][e]), static_cast<double>(xj[e]), s[a][b]);
                }
            }
        }
#pragma unroll
        for (int a = 0; a < GA; ++a)
#pragma unroll
            for (int b = 0; b < JB; ++b) {
                const double v = warp_sum(s[a][b]);
                if (lane == 0 && a < static_cast<int>(na) && j0 + b < n) ws.acc[a][j0 + b] += v;
            }
    }
}

template <typename ST>
__global__ void __launch_bounds__(kThreadsPerCta, 4) gram_kernel(const GramArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    __shared__ GramScratch scratch[kWarpsPerCta];
    __shared__ uint4 block_table[2][kWarpsPerCta][kTaskChunk];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    GramScratch& ws = scratch[warp];
    const uint32_t L = a.n_layers, n = a.n_tasks;
    for (int g = 0; g < GA; ++g) ws.acc[g][lane] = 0.0;
    __syncwarp();
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * 32 * CPL >= ls.cols) continue;   // warp-uniform
        const bool lane_on = t.c < ls.cols;
        const bool shuffled = (ls.flags & kFlagShuffle) != 0;
        const bool flipped = (ls.flags & kFlagFlip) != 0;
        __syncwarp();
        bool ok = true;
        if (lane < n) {
            const uint32_t src = shuffled ? a.src_of_slot[static_cast<size_t>(lane) * L + slot] : slot;   // sigma_i(l)
            const void* pw = a.task_ptrs[static_cast<size_t>(lane) * L + src];
            const void* pb = a.has_base ? a.base[src] : nullptr;
            ws.pw[lane] = pw;
            ws.pb[lane] = pb;
            ok = aligned16(pw) && aligned16(pb);
            if (flipped) {
                const DevTask tk = a.tasks[lane];
#pragma unroll
                for (int h = 0; h < CPL / 4; ++h)
                    block_table[h][warp][lane] = philox4x32_10(t.cb * (CPL / 4) + h, slot, kTagSign, tk.id, tk.key0, tk.key1);
            }
        }
        const bool vec = ls.cols % CPL == 0 && __all_sync(0xFFFFFFFFu, ok);
        __syncwarp();
        for (uint32_t i = 0; i < n; ++i)
            ws.bits[i][lane] = flipped ? static_cast<unsigned char>(lane_bits<CPL>(block_table[CPL == 8 ? (lane >> 4) : 0][warp][i], lane)) : 0;
        __syncwarp();
        if (vec) gram_rows<ST, true>(t, ls.cols, ws, lane, n, a.a0, a.na, lane_on, a.has_base != 0);
        else gram_rows<ST, false>(t, ls.cols, ws, lane, n, a.a0, a.na, lane_on, a.has_base != 0);
    }
    __syncwarp();
    double* out = a.partial + (static_cast<size_t>(blockIdx.x) * kWarpsPerCta + warp) * (GA * kTaskChunk);
    for (int g = 0; g < GA; ++g) out[g * kTaskChunk + lane] = ws.acc[g][lane];
}

// G[a0 + g][j] = sum over (CTA, warp) in index order of the per-warp sums
__global__ void gram_reduce_kernel(const double* partial, uint32_t n_rows, double* gram, uint32_t a0, uint32_t na, uint32_t n)
{
    const uint32_t g = threadIdx.x / kTaskChunk, j = threadIdx.x % kTaskChunk;
    if (g >= na || j >= n) return;
    double s = 0.0;
    for (uint32_t r = 0; r < n_rows; ++r) s += partial[static_cast<size_t>(r) * (GA * kTaskChunk) + g * kTaskChunk + j];
    gram[static_cast<size_t>(a0 + g) * n + j] = s;
}

}  // namespace

int gram_ctas_per_sm(int storage_dtype)
{
    int n = 0;
    cudaError_t e = storage_dtype == 0 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gram_kernel<float>, kThreadsPerCta, 0)
                                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gram_kernel<__nv_bfloat16>, kThreadsPerCta, 0);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

int launch_gram_pass(int storage_dtype, const GramArgs& a, int grid, double* gram, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (storage_dtype == 0) gram_kernel<float><<<grid, kThreadsPerCta, 0, s>>>(a);
    else gram_kernel<__nv_bfloat16><<<grid, kThreadsPerCta, 0, s>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return static_cast<int>(e);
    gram_reduce_kernel<<<1, GA * kTaskChunk, 0, s>>>(a.partial, static_cast<uint32_t>(grid) * kWarpsPerCta, gram, a.a0, a.na, a.n_tasks);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace randes
