// Batched retrieve: several tasks rebuilt in one pass over W_0.
//
//   out_b[p] = fma(lambda, s_b(l_b, c) * M[l_b], W_0[p]),   l_b = sigma_b^-1(p),   b = 0 .. n-1
//
// (Section 4, second display, applied to n tasks at once: the serving case of the
// paper's introduction, where many fine-tuned models are wanted from one store.)
// W_0 is read once instead of n times; every task reads the slot of M its own
// permutation points at, and the tile list keeps the slots of a group adjacent
// in time so that slots wanted by several tasks are served by L2.
// Results are bit-identical to n single retrieves.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

// per warp: what lane i resolved for task i, and every lane's own sign bits per task
struct BatchScratch {
    const void* m[kTaskChunk];       // M slot of task i for this layer
    void* out[kTaskChunk];           // output tensor of task i for this layer
    uint4 block[2][kTaskChunk];      // Philox blocks of task i (second one only for 256-column warps)
    unsigned short bits[kTaskChunk][32];
};

template <typename ST, typename OT, typename MT>
__global__ void __launch_bounds__(kThreadsPerCta, 2) retrieve_batch_kernel(const RetrieveBatchArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    constexpr int U = CPL == 4 ? 2 : 1;     // rows per trip
    constexpr int TB = 4;                   // tasks whose loads are issued together
    __shared__ BatchScratch scratch[kWarpsPerCta];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    BatchScratch& ws = scratch[warp];
    const uint32_t L = a.n_layers, n = a.n_tasks;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;
        const DevLayer lp = a.layers[p];
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * 32 * CPL >= lp.cols) continue;   // warp-uniform
        const bool flipped = (lp.flags & kFlagFlip) != 0;
        const ST* wp = static_cast<const ST*>(a.base[p]);

        __syncwarp();
        bool ok = aligned16(wp);
        if (lane < n) {
            const uint32_t row = a.task_rows[lane];
            const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[static_cast<size_t>(row) * L + p] : p;   // sigma^-1
            ws.m[lane] = static_cast<const MT*>(a.M) + a.layers[slot].m_off;
            void* o = a.out[static_cast<size_t>(lane) * L + p];
            ws.out[lane] = o;
            ok = ok && Out<OT>::template aligned<CPL>(o);
            if (flipped) {
                const DevTask tk = a.tasks[row];
#pragma unroll
                for (int h = 0; h < CPL / 4; ++h)
                    ws.block[h][lane] = philox4x32_10(t.cb * (CPL / 4) + h, slot, kTagSign, tk.id, tk.key0, tk.key1);
            }
        }
        const bool vec = lp.cols % CPL == 0 && __all_sync(0xFFFFFFFFu, ok);
        __syncwarp();
        for (uint32_t i = 0; i < n; ++i)
            ws.bits[i][lane] = flipped ? static_cast<unsigned short>(lane_bits<CPL>(ws.block[CPL == 8 ? (lane >> 4) : 0][i], lane)) : 0;
        __syncwarp();
        if (t.c >= lp.cols) continue;

        if (!vec) {
            for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
                const size_t off = static_cast<size_t>(r) * lp.cols + t.c;
                for (int e = 0; e < CPL; ++e) {
                    if (t.c + e >= lp.cols) break;
                    const float w = Store<ST>::load1(wp + off + e);
                    for (uint32_t i = 0; i < n; ++i) {
                        const float lam = flip(a.lambda, ((static_cast<uint32_t>(ws.bits[i][lane]) >> e) & 1u) << 31);
                        Out<OT>::store1(static_cast<OT*>(ws.out[i]) + off + e, __fmaf_rn(lam, MTile<MT, CPL>::load1(static_cast<const MT*>(ws.m[i]) + off + e), w));
                    }
                }
            }
            continue;
        }

        const uint32_t row_stride = t.rstep * lp.cols;
        uint32_t off = t.r0 * lp.cols + t.c;
        for (uint32_t r = t.r0; r < t.r_end; r += t.rstep * U, off += row_stride * U) {
            float wv[U][CPL];
            bool on[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                on[j] = r + j * t.rstep < t.r_end;
                if (on[j]) Store<ST>::widen(__ldcs(reinterpret_cast<const uint4*>(wp + off + j * row_stride)), wv[j]);
            }
            for (uint32_t i0 = 0; i0 < n; i0 += TB) {
                float m[TB][U][CPL];
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    if (i0 + b < n) {
                        const MT* mp = static_cast<const MT*>(ws.m[i0 + b]);
#pragma unroll
                        for (int j = 0; j < U; ++j)
                            if (on[j]) MTile<MT, CPL>::template load<false>(mp + off + j * row_stride, m[b][j]);
                    }
                }
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    if (i0 + b < n) {
                        const uint32_t bits = ws.bits[i0 + b][lane];
                        float lam[CPL];
#pragma unroll
                        for (int e = 0; e < CPL; ++e) lam[e] = flip(a.lambda, ((bits >> e) & 1u) << 31);
                        OT* op = static_cast<OT*>(ws.out[i0 + b]);
#pragma unroll
                        for (int j = 0; j < U; ++j)
                            if (on[j]) {
                                float y[CPL];
#pragma unroll
                                for (int e = 0; e < CPL; ++e) y[e] = __fmaf_rn(lam[e], m[b][j][e], wv[j][e]);
                                Out<OT>::template store<CPL>(op + off + j * row_stride, y);
                            }
                    }
                }
            }
        }
    }
}

template <typename K> int occupancy(K kernel)
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreadsPerCta, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

template <typename T> struct Tag { typedef T type; };
template <typename F> int with_type(int dtype, F&& f) { return dtype == 0 ? f(Tag<float>{}) : f(Tag<__nv_bfloat16>{}); }

}  // namespace

int launch_retrieve_batch(int storage_dtype, int out_dtype, int m_dtype, const RetrieveBatchArgs& a, int grid, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return with_type(storage_dtype, [&](auto st) {
        return with_type(out_dtype, [&](auto ot) {
            return with_type(m_dtype, [&](auto mt) {
                retrieve_batch_kernel<typename decltype(st)::type, typename decltype(ot)::type, typename decltype(mt)::type>
                    <<<grid, kThreadsPerCta, 0, s>>>(a);
                return static_cast<int>(cudaGetLastError());
            });
        });
    });
}

int retrieve_batch_ctas_per_sm(int storage_dtype, int out_dtype, int m_dtype)
{
    return with_type(storage_dtype, [&](auto st) {
        return with_type(out_dtype, [&](auto ot) {
            return with_type(m_dtype, [&](auto mt) {
                return occupancy(retrieve_batch_kernel<typename decltype(st)::type, typename decltype(ot)::type, typename decltype(mt)::type>);
            });
        });
    });
}

}  // namespace randes
