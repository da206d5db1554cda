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

#include <algorithm>

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
        if (!checked(p < a.n_layers, 5, kCheckLayer, u)) continue;
        const DevLayer lp = a.layers[p];
        if (!checked(un.row0 + un.nrows <= lp.rows, 5, kCheckRows, u)) continue;
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * 32 * CPL >= lp.cols) continue;   // warp-uniform
        const bool flipped = (lp.flags & kFlagFlip) != 0;
        const ST* wp = static_cast<const ST*>(a.base[p]);

        __syncwarp();
        bool ok = aligned16(wp);
        if (lane < n) {
            const uint32_t row = a.task_rows[lane];
            uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[static_cast<size_t>(row) * L + p] : p;   // sigma^-1
            if (!checked(slot < L, 5, kCheckPermuted, u)) slot = p;   // (checked build: recorded; the tile reads its own slot)
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
        if constexpr (CPL == 8 && sizeof(MT) == 4) {
            // bf16 weights, fp32 M: with 8 neighbouring columns per lane the 32-byte M tiles and fp32 outputs of a warp are
            // requests whose lanes sit 32 bytes apart.  When widths and alignment allow, a lane takes columns 4 lane ..
            // 4 lane + 3 of BOTH 128-column halves of the warp's block instead (as retrieve_kernel does): every request is
            // contiguous across the warp, and each half reads its own Philox block like an fp32 warp.
            if (vec) {
                for (uint32_t i = 0; i < n; ++i)
                    ws.bits[i][lane] = flipped ? static_cast<unsigned short>(lane_bits<4>(ws.block[0][i], lane) | (lane_bits<4>(ws.block[1][i], lane) << 4)) : 0;
                __syncwarp();
                const uint32_t c0 = t.cb * 256u + lane * 4u;
                const bool on[2] = {c0 < lp.cols, c0 + 128u < lp.cols};
                const uint32_t row_stride = t.rstep * lp.cols;
                uint32_t off = t.r0 * lp.cols + c0;
                for (uint32_t r = t.r0; r < t.r_end; r += t.rstep, off += row_stride) {
                    float wv[2][4];
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        if (on[h]) {
                            const uint2 w = __ldcs(reinterpret_cast<const uint2*>(wp + off + h * 128u));
                            wv[h][0] = __uint_as_float(w.x << 16); wv[h][1] = __uint_as_float(w.x & 0xFFFF0000u);
                            wv[h][2] = __uint_as_float(w.y << 16); wv[h][3] = __uint_as_float(w.y & 0xFFFF0000u);
                        }
                    for (uint32_t i0 = 0; i0 < n; i0 += TB) {
                        float4 m[TB][2];
#pragma unroll
                        for (int b = 0; b < TB; ++b)
                            if (i0 + b < n) {
                                const float* mp = static_cast<const float*>(ws.m[i0 + b]);
#pragma unroll
                                for (int h = 0; h < 2; ++h)
                                    if (on[h]) m[b][h] = __ldg(reinterpret_cast<const float4*>(mp + off + h * 128u));
                            }
#pragma unroll
                        for (int b = 0; b < TB; ++b)
                            if (i0 + b < n) {
                                const uint32_t bits = ws.bits[i0 + b][lane];
                                OT* op = static_cast<OT*>(ws.out[i0 + b]);
#pragma unroll
                                for (int h = 0; h < 2; ++h)
                                    if (on[h]) {
                                        const float mv[4] = {m[b][h].x, m[b][h].y, m[b][h].z, m[b][h].w};
                                        float y[4];
#pragma unroll
                                        for (int e = 0; e < 4; ++e)
                                            y[e] = __fmaf_rn(flip(a.lambda, ((bits >> (4 * h + e)) & 1u) << 31), mv[e], wv[h][e]);
                                        Out<OT>::template store<4>(op + off + h * 128u, y);
                                    }
                            }
                    }
                }
                continue;
            }
        }
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

// Batched retrieve of a shuffled group, fp32 weights and superposition.  Task b needs, for layer
// position p, the slot M[sigma_b^-1(p)]: every slot of the group is wanted by several tasks.  A
// CTA takes a group unit (a few rows x one warp-wide column block of every member), copies the M
// tiles of all slots and the W_0 tiles of all positions into shared memory once, and resolves
// one record per (position, task) -- output tensor, which member the wanted slot is, Philox block
// of sign bits -- in parallel over its threads.  After that the row loop only reads shared memory
// and streams 16-byte stores: the call is bound by HBM writes, as it should be.
// (Measured against this form and slower by 1 - 4 %: tables built once per chunk of units of one column block;
// the next unit's tiles prefetched into L2 during the row loop; stashes double-buffered by halves with the next
// step's tiles in flight while a step is written.  What limits the kernel is the stream of stores itself.)
constexpr uint32_t kBatchRecBytes = 32;   // {out pointer, slot member, pad, Philox block}

__device__ __forceinline__ void store_plain(float* p, const float (&y)[4])
{
    *reinterpret_cast<float4*>(p) = make_float4(y[0], y[1], y[2], y[3]);
}
__device__ __forceinline__ void store_plain(__nv_bfloat16* p, const float (&y)[4])
{
    *reinterpret_cast<uint2*>(p) = make_uint2(Out<__nv_bfloat16>::pack(y[0], y[1]), Out<__nv_bfloat16>::pack(y[2], y[3]));
}

template <typename OT>
__global__ void __launch_bounds__(kThreadsPerCta, 2) retrieve_batch_group_kernel(const RetrieveBatchArgs a)
{
    constexpr int CPL = 4;
    extern __shared__ __align__(16) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
    const uint32_t m_stash = smem_s, w_stash = smem_s + kStashBytes, s_rec = smem_s + 2 * kStashBytes;
    const uint32_t L = a.n_layers, n = a.n_tasks;
    const uint32_t sign_word = 16 + (lane >> 3) * 4u, sign_shift = (lane & 7) * 4u;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t* mem = a.members + un.layer;
#ifdef RANDES_CHECKED
        {   // every member, every permuted slot and the unit's rows must lie inside the plan; else the unit is skipped
            bool sound = checked(mem[0] < L, 6, kCheckLayer, u);
            const uint32_t G_claimed = sound ? a.layers[mem[0]].group_size : 0;
            for (uint32_t m = 0; sound && m < G_claimed; ++m) {
                sound = checked(mem[m] < L, 6, kCheckLayer, u);
                for (uint32_t b = 0; sound && b < n; ++b)
                    sound = checked(!(a.layers[mem[m]].flags & kFlagShuffle) || a.slot_of_pos[static_cast<size_t>(a.task_rows[b]) * L + mem[m]] < L, 6,
                                    kCheckPermuted, u);
            }
            sound = sound && checked(un.row0 + un.nrows <= a.layers[mem[0]].rows, 6, kCheckRows, u);
            if (!sound) continue;       // (uniform over the CTA: every thread evaluates the same tables)
        }
#endif
        const DevLayer l0 = a.layers[mem[0]];
        const uint32_t G = l0.group_size, cols = l0.cols, Rn = un.nrows;
        const uint32_t c = (un.cb0 * 32u + lane) * CPL;
        const bool lane_on = c < cols;
        const uint32_t off0 = un.row0 * cols + c;          // layers hold < 2^32 elements

        if (lane_on) {
            const uint32_t ntiles = G * Rn;
            for (uint32_t q = warp; q < ntiles; q += kWarpsPerCta) {
                const uint32_t m = q / Rn, r = q - m * Rn;
                const uint32_t layer = mem[m];
                const uint32_t off = off0 + r * cols;
                cp_async16(m_stash + q * kStashTileBytes + lane * 16, static_cast<const float*>(a.M) + a.layers[layer].m_off + off);
                cp_async16(w_stash + q * kStashTileBytes + lane * 16, static_cast<const float*>(a.base[layer]) + off);
            }
        }
        cp_async_commit();
        const uint32_t npairs = G * n;
        for (uint32_t p = threadIdx.x; p < npairs; p += kThreadsPerCta) {
            const uint32_t mp = p / n, b = p - mp * n;
            const uint32_t pos = mem[mp];
            const uint32_t fl = a.layers[pos].flags;
            const uint32_t row = a.task_rows[b];
            const uint32_t slot = (fl & kFlagShuffle) ? a.slot_of_pos[static_cast<size_t>(row) * L + pos] : pos;   // sigma_b^-1(p)
            sts_ptrs(s_rec + p * kBatchRecBytes, a.out[static_cast<size_t>(b) * L + pos],
                     reinterpret_cast<const void*>(static_cast<uintptr_t>(a.layers[slot].member)));
            uint4 blk = make_uint4(0, 0, 0, 0);
            if (fl & kFlagFlip) {
                const DevTask tk = a.tasks[row];
                blk = philox4x32_10(un.cb0, slot, kTagSign, tk.id, tk.key0, tk.key1);
            }
            sts128(s_rec + p * kBatchRecBytes + 16, blk);
        }
        cp_async_wait<0>();
        __syncthreads();   // stashes and records are complete and visible to every warp

        if (lane_on) {
            const uint32_t n_chunks = (Rn + kItemRows - 1) / kItemRows;
            const uint32_t n_items = G * n_chunks;
            for (uint32_t item = warp; item < n_items; item += kWarpsPerCta) {
                const uint32_t mp = item / n_chunks;
                const uint32_t r0 = (item - mp * n_chunks) * kItemRows;
                const uint32_t nr = min(kItemRows, Rn - r0);
                float wv[kItemRows][CPL];
#pragma unroll
                for (int r = 0; r < static_cast<int>(kItemRows); ++r)
                    if (r < static_cast<int>(nr)) Store<float>::widen(lds128(w_stash + (mp * Rn + r0 + r) * kStashTileBytes + lane * 16), wv[r]);
                const uint32_t off = off0 + r0 * cols;
                uint32_t rec = s_rec + mp * n * kBatchRecBytes;
                for (uint32_t b = 0; b < n; ++b, rec += kBatchRecBytes) {
                    OT* op = reinterpret_cast<OT*>(const_cast<char*>(lds_ptr(rec))) + off;
                    const uint32_t member = lds_u32(rec + 8);
                    const uint32_t bits = lds_u32(rec + sign_word) >> sign_shift;
                    float lam[CPL];
#pragma unroll
                    for (int e = 0; e < CPL; ++e) lam[e] = flip(a.lambda, ((bits >> e) & 1u) << 31);
                    const uint32_t mb = m_stash + (member * Rn + r0) * kStashTileBytes + lane * 16;
#pragma unroll
                    for (int r = 0; r < static_cast<int>(kItemRows); ++r) {
                        if (r < static_cast<int>(nr)) {
                            float m[CPL], y[CPL];
                            Store<float>::widen(lds128(mb + r * kStashTileBytes), m);
#pragma unroll
                            for (int e = 0; e < CPL; ++e) y[e] = __fmaf_rn(lam[e], m[e], wv[r][e]);
                            store_plain(op + static_cast<size_t>(r) * cols, y);
                        }
                    }
                }
            }
        }
        __syncthreads();   // every warp is done with the stashes and records before the next unit overwrites them
    }
}

size_t batch_group_smem(uint32_t pairs) { return 2 * static_cast<size_t>(kStashBytes) + static_cast<size_t>(pairs) * kBatchRecBytes; }

template <typename T> struct Tag { typedef T type; };
template <typename F> int with_type(int dtype, F&& f) { return dtype == 0 ? f(Tag<float>{}) : f(Tag<__nv_bfloat16>{}); }

}  // namespace

RANDES_VIOLATION_READER(violation_in_batch_kernels)

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

int retrieve_batch_group_prepare()
{
    cudaError_t e = cudaFuncSetAttribute(retrieve_batch_group_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(retrieve_batch_group_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) (void)cudaGetLastError();
    return static_cast<int>(e);
}

bool retrieve_batch_group_fits(uint32_t max_group, uint32_t n_tasks)
{
    return max_group >= 1 && max_group * kStashTileBytes <= kStashBytes && batch_group_smem(max_group * n_tasks) <= 227 * 1024;
}

int launch_retrieve_batch_groups(int out_dtype, const RetrieveBatchArgs& a, uint32_t max_group, int sm_count, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t smem = batch_group_smem(max_group * a.n_tasks);
    return with_type(out_dtype, [&](auto ot) {
        typedef typename decltype(ot)::type OT;
        // One CTA per unit, not a resident loop: the block scheduler hands the next unit to whichever SM has room.
        // This kernel is bound by its stores, and SMs do not drain stores at equal rates; with the units dealt out
        // evenly in advance the slowest SM set the time (measured: 5.1 -> 4.6 ms for 20 ViT-L/14-shaped models).
        const int grid = static_cast<int>(std::min<uint64_t>(a.n_units, 0x7FFFFFFFull));
        (void)sm_count;
        retrieve_batch_group_kernel<OT><<<grid, kThreadsPerCta, smem, s>>>(a);
        return static_cast<int>(cudaGetLastError());
    });
}

}  // namespace randes
