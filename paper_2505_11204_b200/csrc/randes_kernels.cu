// sm_100a kernels of the RanDeS hot path: retrieve, and accumulate
// (compress / add_model / remove_model).  HBM-bound streaming kernels: every
// lane moves 16 bytes of a weight tensor per request, arithmetic is fp32 with
// one rounding per operation, sign bits are generated in registers from
// Philox4x32-10 and never stored to global memory, the per-task layer
// permutation is resolved per unit of work from small index tables.
//
// Work decomposition.  A CTA (8 warps) walks a list of units; a unit is a block
// of rows x up to 8 warp-wide column blocks of one layer.  A warp owns one
// column block (32 lanes x 16 bytes: 128 fp32 or 256 bf16 columns, i.e. one or
// two Philox blocks of sign bits) and walks down the rows: the sign bits are
// computed once per unit and reused for every row.  Every output element is
// written by exactly one thread and tasks are summed in a fixed order, so
// results are bit-reproducible.
//
// The accumulate kernel keeps its weight streams in flight with cp.async into a
// per-thread ring in shared memory (each lane reads back only what it copied,
// so no barrier is needed): the number of bytes in flight is set by shared
// memory, not by registers.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

// =========================================================================================
// retrieve:  out[p] = fma(lambda, s_t(l, c) * M[l], W_0[p]),  l = sigma_t^-1(p)
// (Section 4, second display; Section 4.4, second display.)  The sign is folded
// into lambda: fma(+-lambda, m, w) is bit-identical to fma(lambda, +-m, w).
// =========================================================================================

// Vector path: U rows per trip, all loads issued before the first use.
template <typename ST, typename OT, typename MT>
__device__ __forceinline__ void retrieve_rows(const WarpTile& t, uint32_t cols, const MT* __restrict__ mp,
                                              const ST* __restrict__ wp, OT* __restrict__ op,
                                              const float (&lam)[Store<ST>::CPL])
{
    constexpr int CPL = Store<ST>::CPL;
    // rows per trip, measured best per type pair: bf16 weights with fp32 output move 80 B per lane
    // and row and are fastest one row at a time; bf16 -> bf16 (48 B) wants four
    constexpr int U = CPL == 4 ? 4 : (sizeof(OT) == 4 ? 1 : 4);
    const uint32_t row_stride = t.rstep * cols;
    uint32_t off = t.r0 * cols + t.c;               // layers hold < 2^32 elements
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep * U, off += row_stride * U) {
        float m[U][CPL];
        uint4 w[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            if (r + j * t.rstep < t.r_end) {
                const uint32_t o = off + j * row_stride;
                MTile<MT, CPL>::load(mp + o, m[j]);
                w[j] = __ldcs(reinterpret_cast<const uint4*>(wp + o));
            }
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            if (r + j * t.rstep < t.r_end) {
                const uint32_t o = off + j * row_stride;
                float wv[CPL], y[CPL];
                Store<ST>::widen(w[j], wv);
#pragma unroll
                for (int e = 0; e < CPL; ++e) y[e] = __fmaf_rn(lam[e], m[j][e], wv[e]);
                Out<OT>::template store<CPL>(op + o, y);
            }
        }
    }
}

// Element-at-a-time path for ragged widths and unaligned tensors; out of line so
// that it does not set the register budget of the vector path.
template <typename ST, typename OT, typename MT>
__device__ __noinline__ void retrieve_rows_scalar(WarpTile t, uint32_t cols, const MT* mp, const ST* wp, OT* op, float lambda,
                                                  uint32_t bits)
{
    constexpr int CPL = Store<ST>::CPL;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
        const size_t off = static_cast<size_t>(r) * cols + t.c;
        for (int e = 0; e < CPL; ++e) {
            if (t.c + e >= cols) break;
            const float lam = flip(lambda, ((bits >> e) & 1u) << 31);
            Out<OT>::store1(op + off + e, __fmaf_rn(lam, MTile<MT, CPL>::load1(mp + off + e), Store<ST>::load1(wp + off + e)));
        }
    }
}

// bf16 weights with an fp32 superposition.  In the layout above a lane owns 8 neighbouring columns, so its M tile
// and its fp32 output are 32 bytes: two requests whose lanes sit 32 bytes apart, each using half of every sector it
// touches.  Here a lane owns 4 + 4 columns instead -- columns 4 lane .. 4 lane + 3 of both 128-column halves of the
// warp's block -- so that every request of the warp is contiguous (512 bytes of M or fp32 output, 256 bytes of
// weights), and each half has its own Philox block, read like an fp32 warp would.  The rows travel through a
// per-thread cp.async ring (per row: the two M tiles and the 8 + 8 bytes of W_0), thirteen rows ahead of their use:
// 156 KiB, one CTA per SM.  Measured on the ViT-L/14- / GPT-2-shaped sets: 0.465 / 0.195 ms per model, against
// 0.482 / 0.203 ms with register loads two rows per trip and two CTAs per SM; 6 stages are slower than registers,
// 10 to 16 within 1 % of each other, 18 slower again.
constexpr int kRetHStages = 13;
constexpr uint32_t kRetHStageBytes = 3 * kSlotBytes;     // per row: M half 0, M half 1, W_0 (8 + 8 bytes)
template <typename ST, typename MT> struct RetrieveHalvesRing { static constexpr bool value = sizeof(ST) == 2 && sizeof(MT) == 4; };

template <typename OT>
__device__ __forceinline__ void retrieve_rows_halves_ring(const WarpTile& t, uint32_t cols, int lane, const float* __restrict__ mp,
                                                          const bf16* __restrict__ wp, OT* __restrict__ op, float lambda,
                                                          uint32_t bits0, uint32_t bits1, uint32_t ring)
{
    constexpr int NSTAGE = kRetHStages;
    const uint32_t c0 = t.cb * 256u + lane * 4u;
    const bool on[2] = {c0 < cols, c0 + 128u < cols};
    if (!on[0]) return;
    float lam[2][4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        lam[0][e] = flip(lambda, ((bits0 >> e) & 1u) << 31);
        lam[1][e] = flip(lambda, ((bits1 >> e) & 1u) << 31);
    }
    const uint32_t row_stride = t.rstep * cols;
    const uint32_t N = (t.r_end - t.r0 + t.rstep - 1) / t.rstep;
    const uint32_t ring_end = ring + NSTAGE * kRetHStageBytes;
    uint32_t off_i = t.r0 * cols + c0, off_c = off_i, issued = 0, stage_i = ring, stage_c = ring;
    auto issue = [&]() {
#pragma unroll
        for (int h = 0; h < 2; ++h)
            if (on[h]) {
                cp_async16(stage_i + h * kSlotBytes, mp + off_i + h * 128u);
                cp_async8(stage_i + 2 * kSlotBytes + h * 8, wp + off_i + h * 128u);
            }
        off_i += row_stride;
        stage_i += kRetHStageBytes;
        if (stage_i == ring_end) stage_i = ring;
        ++issued;
    };
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (issued < N) issue();
        cp_async_commit();
    }
    for (uint32_t it = 0; it < N; ++it, off_c += row_stride) {
        if (issued < N) issue();
        cp_async_commit();
        cp_async_wait<NSTAGE - 1>();
        const uint4 w = lds128(stage_c + 2 * kSlotBytes);
#pragma unroll
        for (int h = 0; h < 2; ++h)
            if (on[h]) {
                const uint4 m = lds128(stage_c + h * kSlotBytes);
                const uint32_t wx = h ? w.z : w.x, wy = h ? w.w : w.y;
                const float wv[4] = {__uint_as_float(wx << 16), __uint_as_float(wx & 0xFFFF0000u), __uint_as_float(wy << 16), __uint_as_float(wy & 0xFFFF0000u)};
                const float mv[4] = {__uint_as_float(m.x), __uint_as_float(m.y), __uint_as_float(m.z), __uint_as_float(m.w)};
                float y[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) y[e] = __fmaf_rn(lam[h][e], mv[e], wv[e]);
                Out<OT>::template store<4>(op + off_c + h * 128u, y);
            }
        stage_c += kRetHStageBytes;
        if (stage_c == ring_end) stage_c = ring;
    }
    cp_async_wait<0>();
}

template <typename ST, typename OT, typename MT>
__global__ void __launch_bounds__(kThreadsPerCta, 2) retrieve_kernel(const RetrieveArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    extern __shared__ __align__(16) unsigned char ring_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(ring_smem)) + threadIdx.x * 16;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;                       // layer position being rebuilt
        if (!checked(p < a.n_layers, 1, kCheckLayer, u)) continue;
        const DevLayer lp = a.layers[p];
        const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[p] : p;   // sigma^-1
        if (!checked(slot < a.n_layers, 1, kCheckPermuted, u) || !checked(un.row0 + un.nrows <= lp.rows, 1, kCheckRows, u)) continue;
        const unsigned long long m_off = slot == p ? lp.m_off : a.layers[slot].m_off;
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if constexpr (CPL == 8 && sizeof(MT) == 4) {
            // bf16 weights, fp32 M: the lane mapping with contiguous requests, when widths and alignment allow
            const bf16* wp8 = static_cast<const bf16*>(a.base[p]);
            OT* op8 = static_cast<OT*>(a.out[p]);
            if (lp.cols % 8 == 0 && aligned16(wp8) && (reinterpret_cast<uintptr_t>(op8) & 15) == 0) {
                if (t.r0 >= t.r_end || t.cb * 256u >= lp.cols) continue;   // warp-uniform
                uint32_t b0 = 0, b1 = 0;
                if (lp.flags & kFlagFlip) {
                    b0 = lane_bits<4>(philox4x32_10(t.cb * 2, slot, kTagSign, a.task.id, a.task.key0, a.task.key1), lane);
                    b1 = lane_bits<4>(philox4x32_10(t.cb * 2 + 1, slot, kTagSign, a.task.id, a.task.key0, a.task.key1), lane);
                }
                retrieve_rows_halves_ring<OT>(t, lp.cols, lane, static_cast<const float*>(a.M) + m_off, wp8, op8, a.lambda, b0, b1, ring);
                continue;
            }
        }
        if (t.c >= lp.cols || t.r0 >= t.r_end) continue;

        uint32_t bits = 0;
        if (lp.flags & kFlagFlip) {
            const uint4 blk = philox4x32_10(lane_block<CPL>(t.cb, lane), slot, kTagSign, a.task.id, a.task.key0, a.task.key1);
            bits = lane_bits<CPL>(blk, lane);
        }
        const ST* wp = static_cast<const ST*>(a.base[p]);
        OT* op = static_cast<OT*>(a.out[p]);
        const MT* mp = static_cast<const MT*>(a.M) + m_off;
        const bool vec = lp.cols % CPL == 0 && aligned16(wp) && Out<OT>::template aligned<CPL>(op);   // M slots are 256-byte aligned
        if (vec) {
            float lam[CPL];
#pragma unroll
            for (int e = 0; e < CPL; ++e) lam[e] = flip(a.lambda, ((bits >> e) & 1u) << 31);
            retrieve_rows<ST, OT, MT>(t, lp.cols, mp, wp, op, lam);
        } else {
            retrieve_rows_scalar<ST, OT, MT>(t, lp.cols, mp, wp, op, a.lambda, bits);
        }
    }
}

// =========================================================================================
// accumulate:  M[l] (=|+=|-=) sum_i s_i(l, c) * ( W_i[sigma_i(l)] - W_0[sigma_i(l)] )
// compress (Section 4, first display): all registered tasks, from +0, in plan order.
// add / remove (Section 5.7): one task, starting from M, sign negated for remove.
//
// Per unit a warp first resolves, for up to MAXT tasks, the source pointers
// (lane i looks up sigma_i(l) for task i) and the sign bits (lane i runs Philox
// for task i; every lane then gathers its own columns' bits of NB tasks into one
// word per batch).  The row loop is then a software pipeline over (U rows, batch
// of NB tasks): W_i tiles travel through a per-thread cp.async ring in shared
// memory, several stages ahead of their use.  Arithmetic uses the packed fp32x2
// instructions: d = W_i - W_0 (one rounding per half), acc = fma(d, +-1, acc)
// (the product is exact, so this is acc + (+-d) with one rounding).
// =========================================================================================

// How W_0 enters the difference W_i - W_0.
constexpr int kNoBase = 0;        // the task tensors already hold deltas
constexpr int kSharedBase = 1;    // no shuffle: every task subtracts the same W_0 tile, fetched once per row
constexpr int kPerTaskBase = 2;   // shuffle: task i subtracts W_0[sigma_i(l)]; tiles repeat across slots and hit in L2

// Shared memory of the accumulate kernel, per CTA:
//   ring     kRingSlots slots x (256 threads x 16 B), cut into stages whose layout
//            depends on how W_0 comes in (StageGeom)
//   per warp ptrs[MAXT] = {W_i layer, W_0 layer} resolved through sigma_i, 16 B each
//            bits[MAXT/NB][32 lanes] 16-bit words: bit k*CPL + e = sign of column e for task k
constexpr int kRingSlots = 24;    // 16-byte slots per thread: 96 KiB per CTA, two CTAs per SM

template <typename ST, bool SINGLE> struct AccConfig {
    static constexpr int CPL = Store<ST>::CPL;
    // measured best: fp32 weights 2 rows x 2 tasks per stage, bf16 weights 1 row x 2 tasks, add / remove 1 row
    static constexpr int U = (SINGLE || CPL == 8) ? 1 : 2;   // rows per stage
    static constexpr int NB = SINGLE ? 1 : 2;                // tasks per stage
    static constexpr int MAXT = SINGLE ? 1 : kTaskChunk;
    static constexpr bool kAsyncInit = SINGLE;        // add / remove start from M
    static constexpr uint32_t kRingBytes = kRingSlots * kSlotBytes;
    static constexpr int kBatches = (MAXT + NB - 1) / NB;
    static constexpr uint32_t kPtrBytes = MAXT * 16;
    static constexpr uint32_t kWarpBytes = kPtrBytes + kBatches * 64;
    static constexpr size_t kSmemBytes = kRingBytes + kWarpsPerCta * kWarpBytes;
    static_assert(NB * CPL <= 16, "a batch's sign bits must fit a 16-bit word");
};

// Stage layout for one way of bringing W_0 in (slot-major across the CTA's threads):
//   [0, U*NB)                 W_i tiles, slot u*NB + k = row u, task k of the batch
//   kPerTaskBase: next U*NB   W_0[sigma_i(l)] tiles, same order (L2 hits, staged as deep as the W_i)
//   kSharedBase:  next U      W_0 tile of row u, filled with the rows' first batch
//   add / remove: next U*CPL/4  M tiles of the rows, filled likewise
template <typename ST, bool SINGLE, int BASE, typename MT> struct StageGeom {
    typedef AccConfig<ST, SINGLE> C;
    static constexpr int kW = 0;
    static constexpr int kB = C::U * C::NB;
    static constexpr int kM = kB + (BASE == kPerTaskBase ? C::U * C::NB : (BASE == kSharedBase ? C::U : 0));
    // A lane's M tile (CPL elements) is 8, 16 or 32 bytes.  Up to 16 bytes it travels through the
    // ring, one slot per row.  32 bytes (fp32 M under bf16 weights) could only be fetched by two
    // 16-byte copies with a 32-byte stride between lanes, which cp.async handles badly: there M is
    // prefetched into L2 and loaded into registers one step ahead.
    static constexpr int kMBytes = static_cast<int>(sizeof(MT)) * C::CPL;
    static constexpr bool kInitViaRing = C::kAsyncInit && kMBytes <= 16;
    static constexpr bool kInitViaRegs = C::kAsyncInit && kMBytes == 32;
    static constexpr int SLOTS = kM + (kInitViaRing ? C::U : 0);
    static constexpr int NSTAGE = (kRingSlots / SLOTS) > 8 ? 8 : (kRingSlots / SLOTS);
    static constexpr uint32_t kStageBytes = SLOTS * kSlotBytes;
    static_assert(NSTAGE >= 2, "ring too small");
};

template <typename ST, bool SINGLE, int BASE, bool FULL, typename MT>
__device__ __forceinline__ void accumulate_rows_async(const WarpTile& t, uint32_t cols, uint32_t nt, bool init_plain, bool init_async,
                                                      MT* __restrict__ mp, uint32_t ring, uint32_t sptr, uint32_t sbits)
{
    typedef AccConfig<ST, SINGLE> C;
    typedef StageGeom<ST, SINGLE, BASE, MT> G;
    typedef MTile<MT, C::CPL> MTl;
    constexpr int CPL = C::CPL, U = C::U, NB = C::NB, NSTAGE = G::NSTAGE;
    constexpr uint32_t ES = sizeof(ST);
    const uint32_t nrows = (t.r_end - t.r0 + t.rstep - 1) / t.rstep;
    const uint32_t nbat = (nt + NB - 1) / NB;
    const uint32_t N = ((nrows + U - 1) / U) * nbat;
    const uint32_t row_stride = t.rstep * cols;          // elements between this warp's rows
    const uint32_t off0 = t.r0 * cols + t.c;             // element offset of the first tile (layers hold < 2^32 elements)

    // two cursors over the same (row group, batch) sequence: copies issued, stages consumed
    uint32_t off_i = off0, b_i = 0, left_i = nrows;
    uint32_t off_c = off0, b_c = 0, left_c = nrows;
    uint32_t issued = 0;
    uint32_t stage_c = ring, stage_i = ring;
    const uint32_t ring_end = ring + NSTAGE * G::kStageBytes;

    // Under a shuffle without staging (more than 32 tasks, several models added at once) every W_0 tile is read by
    // several slots of its group and the repeats are meant to hit in L2: the W_0 copies ask L2 to keep their lines, the
    // task weights, which pass through once, to drop theirs first (2 - 3 % on those paths).
    uint64_t pol_stream = 0, pol_keep = 0;
    if (BASE == kPerTaskBase) {
        pol_stream = l2_evict_first_policy();
        pol_keep = l2_evict_last_policy();
    }
    auto issue = [&]() {
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const uint32_t i = b_i * NB + k;
            if (FULL || i < nt) {
                const char* pw = lds_ptr(sptr + i * 16);
                const char* pb = BASE == kPerTaskBase ? lds_ptr(sptr + i * 16 + 8) : nullptr;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (u == 0 || left_i > u) {
                        const size_t byte_off = static_cast<size_t>(off_i + u * row_stride) * ES;
                        if (BASE == kPerTaskBase) {
                            cp_async16_hint(stage_i + (G::kW + u * NB + k) * kSlotBytes, pw + byte_off, pol_stream);
                            cp_async16_hint(stage_i + (G::kB + u * NB + k) * kSlotBytes, pb + byte_off, pol_keep);
                        } else {
                            cp_async16(stage_i + (G::kW + u * NB + k) * kSlotBytes, pw + byte_off);
                        }
                    }
                }
            }
        }
        if (b_i == 0 && (BASE == kSharedBase || (C::kAsyncInit && init_async))) {
            const char* pb0 = BASE == kSharedBase ? lds_ptr(sptr + 8) : nullptr;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (u == 0 || left_i > u) {
                    const uint32_t off = off_i + u * row_stride;
                    if (BASE == kSharedBase) cp_async16(stage_i + (G::kB + u) * kSlotBytes, pb0 + static_cast<size_t>(off) * ES);
                    if (G::kInitViaRing && init_async) {
                        if (G::kMBytes == 16) cp_async16(stage_i + (G::kM + u) * kSlotBytes, mp + off);
                        else cp_async8(stage_i + (G::kM + u) * kSlotBytes, mp + off);
                    }
                    if (G::kInitViaRegs && init_async) prefetch_l2(mp + off);
                }
            }
        }
        if (++b_i == nbat) { b_i = 0; off_i += U * row_stride; left_i -= U; }
        stage_i += G::kStageBytes;
        if (stage_i == ring_end) stage_i = ring;
        ++issued;
    };

#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (issued < N) issue();
        cp_async_commit();
    }

    f32x2 acc[U][CPL / 2], w0row[U][CPL / 2];
    const uint32_t one = 0x3F800000u;

    // M tiles of the next row group, when they come through registers
    uint4 m_next[U][2];
    uint32_t off_m = off0, left_m = nrows;
    auto load_m_next = [&]() {
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (u == 0 || left_m > u) {
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    m_next[u][h] = reinterpret_cast<const uint4*>(mp + off_m + u * row_stride)[h];
            }
        off_m += U * row_stride;
        left_m -= U;
    };
    if (G::kInitViaRegs && init_async && N > 0) load_m_next();

    for (uint32_t it = 0; it < N; ++it) {
        if (issued < N) issue();
        cp_async_commit();
        cp_async_wait<NSTAGE - 1>();   // everything but the newest NSTAGE-1 groups has landed: stage_c is ready

        if (b_c == 0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int e = 0; e < CPL / 2; ++e) { acc[u][e] = 0ull; w0row[u][e] = 0ull; }
                if (u == 0 || left_c > u) {
                    bool have = false;
                    float mv[CPL];
                    if (G::kInitViaRing && init_async) {
                        const uint4 raw[1] = {lds128(stage_c + (G::kM + u) * kSlotBytes)};
                        MTile<MT, CPL>::unpack(reinterpret_cast<const uint4(&)[(G::kMBytes + 15) / 16]>(raw), mv);
                        have = true;
                    } else if (G::kInitViaRegs && init_async) {
                        MTile<MT, CPL>::unpack(reinterpret_cast<const uint4(&)[(G::kMBytes + 15) / 16]>(m_next[u]), mv);
                        have = true;
                    } else if (init_plain) {
                        // a sum that starts from M (several models added at once; a later chunk of a
                        // long compress): the next row group's M tile is pulled into L2 meanwhile
                        MTl::load(mp + off_c + u * row_stride, mv);
                        if (left_c > U + u) prefetch_l2(mp + off_c + (U + u) * row_stride);
                        have = true;
                    }
                    if (have) {
#pragma unroll
                        for (int e = 0; e < CPL / 2; ++e) acc[u][e] = pack2(__float_as_uint(mv[2 * e]), __float_as_uint(mv[2 * e + 1]));
                    }
                    if (BASE == kSharedBase) Store<ST>::widen2(lds128(stage_c + (G::kB + u) * kSlotBytes), w0row[u]);
                }
            }
        }
        if (G::kInitViaRegs && init_async && b_c == 0 && left_m > 0 && left_m <= nrows) load_m_next();
        const uint32_t pack = lds_u16(sbits + b_c * 64);
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            if (FULL || b_c * NB + k < nt) {
                // +-1.0f per column, shared by the U rows
                f32x2 sg[CPL / 2];
#pragma unroll
                for (int e = 0; e < CPL / 2; ++e)
                    sg[e] = pack2(((pack << (31 - (k * CPL + 2 * e))) & 0x80000000u) | one,
                                  ((pack << (31 - (k * CPL + 2 * e + 1))) & 0x80000000u) | one);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (u == 0 || left_c > u) {
                        f32x2 d[CPL / 2];
                        Store<ST>::widen2(lds128(stage_c + (G::kW + u * NB + k) * kSlotBytes), d);
                        if (BASE == kPerTaskBase) {
                            f32x2 b[CPL / 2];
                            Store<ST>::widen2(lds128(stage_c + (G::kB + u * NB + k) * kSlotBytes), b);
#pragma unroll
                            for (int e = 0; e < CPL / 2; ++e) d[e] = sub2(d[e], b[e]);
                        } else if (BASE == kSharedBase) {
#pragma unroll
                            for (int e = 0; e < CPL / 2; ++e) d[e] = sub2(d[e], w0row[u][e]);
                        }
#pragma unroll
                        for (int e = 0; e < CPL / 2; ++e) acc[u][e] = fma2(d[e], sg[e], acc[u][e]);
                    }
                }
            }
        }
        if (b_c + 1 == nbat) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (u == 0 || left_c > u) {
                    float v[CPL];
#pragma unroll
                    for (int e = 0; e < CPL / 2; ++e) unpack2(acc[u][e], v[2 * e], v[2 * e + 1]);
                    MTl::store(mp + off_c + u * row_stride, v);
                }
            }
            b_c = 0;
            off_c += U * row_stride;
            left_c -= U;
        } else {
            ++b_c;
        }
        stage_c += G::kStageBytes;
        if (stage_c == ring_end) stage_c = ring;
    }
    cp_async_wait<0>();
}

// Element-at-a-time path for layers whose width is not a multiple of the lane
// width or whose tensors are not 16-byte aligned.  Kept out of line: it is rare
// and must not set the register budget of the vector path.
template <typename ST, int NB, typename MT>
__device__ __noinline__ void accumulate_rows_scalar(WarpTile t, uint32_t cols, uint32_t nt, bool init, MT* mp, int base_mode,
                                                    uint32_t sptr, uint32_t sbits)
{
    constexpr int CPL = Store<ST>::CPL;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
        const size_t off = static_cast<size_t>(r) * cols + t.c;
        for (int e = 0; e < CPL; ++e) {
            if (t.c + e >= cols) break;
            float acc = init ? MTile<MT, CPL>::load1(mp + off + e) : 0.f;
            for (uint32_t i = 0; i < nt; ++i) {
                float d = Store<ST>::load1(reinterpret_cast<const ST*>(lds_ptr(sptr + i * 16)) + off + e);
                if (base_mode != kNoBase) d = __fsub_rn(d, Store<ST>::load1(reinterpret_cast<const ST*>(lds_ptr(sptr + i * 16 + 8)) + off + e));
                const uint32_t bit = (lds_u16(sbits + (i / NB) * 64) >> ((i % NB) * CPL + e)) & 1u;
                acc = __fadd_rn(acc, flip(d, bit << 31));
            }
            MTile<MT, CPL>::store1(mp + off + e, acc);
        }
    }
}

// SINGLE: one task per launch (add / remove): a deep ring of single rows, M staged
// with the weights.  Otherwise (compress): 2 rows x 2 tasks per stage.
template <typename ST, bool SINGLE, typename MT>
__global__ void __launch_bounds__(kThreadsPerCta, 2) accumulate_kernel(const AccumulateArgs a)
{
    typedef AccConfig<ST, SINGLE> C;
    constexpr int CPL = C::CPL, NB = C::NB, MAXT = C::MAXT;
    extern __shared__ __align__(16) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
    const uint32_t ring = smem_s + threadIdx.x * 16;
    // between units the ring is idle: its first slots double as the warp's table of Philox blocks
    const uint32_t blocks = smem_s + warp * 512;
    const uint32_t sptr = smem_s + C::kRingBytes + warp * C::kWarpBytes;
    const uint32_t sbits = sptr + C::kPtrBytes + lane * 2;
    const uint32_t L = a.n_layers;
    const uint32_t negate_bits = a.negate ? 0xFFFFu : 0u;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        if (!checked(slot < a.n_layers, 2, kCheckLayer, u)) continue;
        const DevLayer ls = a.layers[slot];
        if (!checked(un.row0 + un.nrows <= ls.rows, 2, kCheckRows, u)) continue;
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * 32 * CPL >= ls.cols) continue;   // warp-uniform: nothing for this warp
        const bool lane_on = t.c < ls.cols;
        const bool shuffled = (ls.flags & kFlagShuffle) != 0;
        const bool flipped = (ls.flags & kFlagFlip) != 0;
        MT* mp = static_cast<MT*>(a.M) + ls.m_off;
        const int base_mode = !a.has_base ? kNoBase : ((shuffled && !SINGLE) ? kPerTaskBase : kSharedBase);

        for (uint32_t chunk0 = 0; chunk0 < a.n_tasks; chunk0 += MAXT) {
            const uint32_t nt = min(static_cast<uint32_t>(MAXT), a.n_tasks - chunk0);
            __syncwarp();   // the previous chunk's readers are done with the scratch
            bool ok = true;
            if (lane < nt) {
                const uint32_t ti = chunk0 + lane;
                uint32_t src = shuffled ? a.src_of_slot[static_cast<size_t>(ti) * L + slot] : slot;   // sigma_i(l)
                if (!checked(src < L, 2, kCheckPermuted, u)) src = slot;   // (checked build: recorded; the tile reads its own layer)
                const void* pw = a.task_ptrs[static_cast<size_t>(ti) * L + src];
                const void* pb = a.has_base ? a.base[src] : nullptr;
                sts_ptrs(sptr + lane * 16, pw, pb);
                ok = aligned16(pw) && aligned16(pb);
                if (flipped) {
                    const DevTask tk = a.tasks[ti];
#pragma unroll
                    for (int h = 0; h < CPL / 4; ++h)
                        sts128(blocks + h * kSlotBytes + lane * 16,
                               philox4x32_10(t.cb * (CPL / 4) + h, slot, kTagSign, tk.id, tk.key0, tk.key1));
                }
            }
            const bool vec = ls.cols % CPL == 0 && __all_sync(0xFFFFFFFFu, ok);
            __syncwarp();
            // every lane gathers the bits of its own columns, NB tasks to a word
            const uint32_t nbat = (nt + NB - 1) / NB;
            for (uint32_t b = 0; b < nbat; ++b) {
                uint32_t pack = 0;
                if (flipped) {
#pragma unroll
                    for (int k = 0; k < NB; ++k) {
                        const uint32_t i = b * NB + k;
                        if (i < nt)
                            pack |= lane_bits<CPL>(lds128(blocks + (CPL == 8 ? (lane >> 4) : 0) * kSlotBytes + i * 16), lane) << (k * CPL);
                    }
                }
                sts_u16(sbits + b * 64, pack ^ negate_bits);
            }
            __syncwarp();   // the block table is free again before any lane's copies land in the ring
            if (lane_on) {
                const bool init_plain = chunk0 > 0 || (!SINGLE && a.init_from_m);
                const bool init_async = SINGLE && chunk0 == 0 && a.init_from_m;
                const bool full = nt % NB == 0;
                if (!vec)
                    accumulate_rows_scalar<ST, NB, MT>(t, ls.cols, nt, init_plain || a.init_from_m, mp, base_mode, sptr, sbits);
                else if (base_mode == kNoBase) {
                    if (full) accumulate_rows_async<ST, SINGLE, kNoBase, true, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                    else accumulate_rows_async<ST, SINGLE, kNoBase, false, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                } else if (base_mode == kSharedBase) {
                    if (full) accumulate_rows_async<ST, SINGLE, kSharedBase, true, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                    else accumulate_rows_async<ST, SINGLE, kSharedBase, false, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                } else {
                    if (full) accumulate_rows_async<ST, SINGLE, kPerTaskBase, true, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                    else accumulate_rows_async<ST, SINGLE, kPerTaskBase, false, MT>(t, ls.cols, nt, init_plain, init_async, mp, ring, sptr, sbits);
                }
            }
        }
    }
}

// add / remove for bf16 weights and an fp32 superposition, with the lane mapping of retrieve_rows_halves: a lane
// owns columns 4 lane .. 4 lane + 3 of both 128-column halves of the warp's block, so the 32 bytes of M it reads
// and writes per row are two requests that are contiguous across the warp.  The rows travel through a per-thread
// cp.async ring in shared memory, as in the fp32 kernel: per row a lane copies its two 16-byte M tiles and the 8 + 8
// bytes of W_j (and of W_0) of both halves, ten rows ahead of their use (160 KiB, one CTA per SM: measured best; with
// plain register loads, two rows per trip and three CTAs per SM the same kernel ran 4 - 5 % slower).  Used when every
// layer has a width that is a multiple of 8 and 16-byte aligned tensors; the result is the same as
// accumulate_kernel's: d = W_j - W_0 (one rounding), M +- s d (one rounding).
constexpr int kAddHStages = 10;
template <bool HAS_BASE> struct AddHalvesRing {
    static constexpr int kSlots = HAS_BASE ? 4 : 3;                       // M half 0, M half 1, W_j (8 + 8 bytes), W_0 (8 + 8 bytes)
    static constexpr uint32_t kStageBytes = kSlots * kSlotBytes;
    static constexpr size_t kSmem = static_cast<size_t>(kAddHStages) * kStageBytes;
};

template <bool HAS_BASE>
__global__ void __launch_bounds__(kThreadsPerCta, 1) add_halves_kernel(const AccumulateArgs a)
{
    typedef AddHalvesRing<HAS_BASE> R;
    constexpr int NSTAGE = kAddHStages;
    extern __shared__ __align__(16) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + threadIdx.x * 16;
    const uint32_t ring_end = ring + NSTAGE * R::kStageBytes;
    const DevTask tk = a.tasks[0];
    const uint32_t neg = a.negate ? 0xFu : 0u;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        if (!checked(slot < a.n_layers, 3, kCheckLayer, u)) continue;
        const DevLayer ls = a.layers[slot];
        if (!checked(un.row0 + un.nrows <= ls.rows, 3, kCheckRows, u)) continue;
        const WarpTile t = warp_tile<8>(un, warp, lane);
        const uint32_t cols = ls.cols;
        if (t.r0 >= t.r_end || t.cb * 256u >= cols) continue;   // warp-uniform
        const uint32_t src = (ls.flags & kFlagShuffle) ? a.src_of_slot[slot] : slot;   // sigma_j(l)
        if (!checked(src < a.n_layers, 3, kCheckPermuted, u)) continue;
        const bf16* wp = static_cast<const bf16*>(a.task_ptrs[src]);
        const bf16* bp = HAS_BASE ? static_cast<const bf16*>(a.base[src]) : nullptr;
        float* mp = static_cast<float*>(a.M) + ls.m_off;
        uint32_t bits[2] = {neg, neg};
        if (ls.flags & kFlagFlip) {
            bits[0] ^= lane_bits<4>(philox4x32_10(t.cb * 2, slot, kTagSign, tk.id, tk.key0, tk.key1), lane);
            bits[1] ^= lane_bits<4>(philox4x32_10(t.cb * 2 + 1, slot, kTagSign, tk.id, tk.key0, tk.key1), lane);
        }
        const uint32_t c0 = t.cb * 256u + lane * 4u;
        const bool on[2] = {c0 < cols, c0 + 128u < cols};
        if (!on[0]) continue;
        const uint32_t row_stride = t.rstep * cols;
        const uint32_t N = (t.r_end - t.r0 + t.rstep - 1) / t.rstep;
        uint32_t off_i = t.r0 * cols + c0, off_c = off_i, issued = 0, stage_i = ring, stage_c = ring;
        auto issue = [&]() {
#pragma unroll
            for (int h = 0; h < 2; ++h)
                if (on[h]) {
                    const uint32_t o = off_i + h * 128u;
                    cp_async16(stage_i + h * kSlotBytes, mp + o);
                    cp_async8(stage_i + 2 * kSlotBytes + h * 8, wp + o);
                    if (HAS_BASE) cp_async8(stage_i + 3 * kSlotBytes + h * 8, bp + o);
                }
            off_i += row_stride;
            stage_i += R::kStageBytes;
            if (stage_i == ring_end) stage_i = ring;
            ++issued;
        };
#pragma unroll
        for (int s = 0; s < NSTAGE - 1; ++s) {
            if (issued < N) issue();
            cp_async_commit();
        }
        for (uint32_t it = 0; it < N; ++it, off_c += row_stride) {
            if (issued < N) issue();
            cp_async_commit();
            cp_async_wait<NSTAGE - 1>();
            const uint4 w = lds128(stage_c + 2 * kSlotBytes);
            uint4 b = make_uint4(0, 0, 0, 0);
            if (HAS_BASE) b = lds128(stage_c + 3 * kSlotBytes);
#pragma unroll
            for (int h = 0; h < 2; ++h)
                if (on[h]) {
                    const uint4 m = lds128(stage_c + h * kSlotBytes);
                    const uint32_t wx = h ? w.z : w.x, wy = h ? w.w : w.y, bx = h ? b.z : b.x, by = h ? b.w : b.y;
                    const float wv[4] = {__uint_as_float(wx << 16), __uint_as_float(wx & 0xFFFF0000u), __uint_as_float(wy << 16), __uint_as_float(wy & 0xFFFF0000u)};
                    const float bv[4] = {__uint_as_float(bx << 16), __uint_as_float(bx & 0xFFFF0000u), __uint_as_float(by << 16), __uint_as_float(by & 0xFFFF0000u)};
                    const float mv[4] = {__uint_as_float(m.x), __uint_as_float(m.y), __uint_as_float(m.z), __uint_as_float(m.w)};
                    float y[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float d = HAS_BASE ? __fsub_rn(wv[e], bv[e]) : wv[e];
                        y[e] = __fadd_rn(mv[e], flip(d, ((bits[h] >> e) & 1u) << 31));
                    }
                    *reinterpret_cast<float4*>(mp + off_c + h * 128u) = make_float4(y[0], y[1], y[2], y[3]);
                }
            stage_c += R::kStageBytes;
            if (stage_c == ring_end) stage_c = ring;
        }
        cp_async_wait<0>();
    }
}

template <typename K> int ctas_per_sm(K kernel, size_t smem)
{
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreadsPerCta, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

}  // namespace

// dtype code -> element type, for the launch and occupancy dispatch below
template <typename T> struct Tag { typedef T type; };
template <typename F> int with_type(int dtype, F&& f) { return dtype == 0 ? f(Tag<float>{}) : f(Tag<bf16>{}); }

int launch_retrieve(int storage_dtype, int out_dtype, int m_dtype, const RetrieveArgs& a, int grid, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return with_type(storage_dtype, [&](auto st) {
        return with_type(out_dtype, [&](auto ot) {
            return with_type(m_dtype, [&](auto mt) {
                typedef typename decltype(st)::type ST;
                typedef typename decltype(mt)::type MT;
                const size_t smem = RetrieveHalvesRing<ST, MT>::value ? static_cast<size_t>(kRetHStages) * kRetHStageBytes : 0;
                retrieve_kernel<ST, typename decltype(ot)::type, MT><<<grid, kThreadsPerCta, smem, s>>>(a);
                return static_cast<int>(cudaGetLastError());
            });
        });
    });
}

int launch_add_halves(const AccumulateArgs& a, int sm_count, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t smem = a.has_base ? AddHalvesRing<true>::kSmem : AddHalvesRing<false>::kSmem;
    // resident CTAs per SM, asked once per device and kernel (the query also opts the kernel into its shared memory)
    static std::mutex mutex;
    static int resident[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return static_cast<int>(cudaErrorInvalidDevice);
    int per_sm;
    {
        std::lock_guard<std::mutex> lock(mutex);
        int& slot = resident[dev][a.has_base ? 1 : 0];
        if (slot == 0) slot = a.has_base ? ctas_per_sm(add_halves_kernel<true>, smem) : ctas_per_sm(add_halves_kernel<false>, smem);
        per_sm = slot;
    }
    if (per_sm <= 0) return static_cast<int>(cudaErrorInvalidConfiguration);
    const unsigned long long want = static_cast<unsigned long long>(sm_count) * per_sm;
    const int grid = static_cast<int>(want < a.n_units ? want : a.n_units);
    if (a.has_base) add_halves_kernel<true><<<grid, kThreadsPerCta, smem, s>>>(a);
    else add_halves_kernel<false><<<grid, kThreadsPerCta, smem, s>>>(a);
    return static_cast<int>(cudaGetLastError());
}

int launch_accumulate(int storage_dtype, int m_dtype, const AccumulateArgs& a, int resident_grid, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool single = a.n_tasks == 1;
    return with_type(storage_dtype, [&](auto st) {
        return with_type(m_dtype, [&](auto mt) {
            typedef typename decltype(st)::type ST;
            typedef typename decltype(mt)::type MT;
            // fp32 weights: one CTA per unit, so that the block scheduler deals the units out as SMs come free (add / remove
            // 3 - 4 % faster than the resident loop: a quarter of their traffic is stores, which SMs drain at unequal
            // rates); bf16 weights: the resident loop, which measured 1 % faster there
            const int grid = sizeof(ST) == 4 ? static_cast<int>(std::min<unsigned long long>(a.n_units, 0x7FFFFFFFull)) : resident_grid;
            if (single) accumulate_kernel<ST, true, MT><<<grid, kThreadsPerCta, AccConfig<ST, true>::kSmemBytes, s>>>(a);
            else accumulate_kernel<ST, false, MT><<<grid, kThreadsPerCta, AccConfig<ST, false>::kSmemBytes, s>>>(a);
            return static_cast<int>(cudaGetLastError());
        });
    });
}

// ---- retrieve without a caller-provided workspace ---------------------------------------------
// The tables the retrieve kernel reads (layers, units, sigma^-1, pointer arrays) are
// placed in this fixed array instead of a workspace the caller would have to allocate.
// Every GPU that loads the library holds the array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device
int g_static_grid[kMaxDevices][2][2][2] = {};    // persistent grid size [storage][out dtype][M dtype], per device
// Host image of the tables of the call being enqueued, one per device, kept for the life of the library:
// the five tables are laid out here and reach the device array in ONE copy.
std::vector<unsigned char> g_static_host[kMaxDevices];
size_t align256(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

size_t retrieve_static_bytes(uint32_t n_layers, uint32_t n_units)
{
    return align256(n_layers * sizeof(DevLayer)) + align256(n_units * sizeof(DevUnit)) + align256(n_layers * sizeof(uint32_t)) +
           2 * align256(n_layers * sizeof(void*));
}

int launch_retrieve_static(int storage_dtype, int out_dtype, int m_dtype, const DevLayer* layers, uint32_t n_layers, const DevUnit* units,
                           uint32_t n_units, const uint32_t* slot_of_pos, const void* const* base, void* const* out,
                           const void* M, const DevTask& task, float lambda, void* stream)
{
    const size_t need = retrieve_static_bytes(n_layers, n_units);
    if (need > kStaticScratchBytes) return -1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return static_cast<int>(e);
    if (dev < 0 || dev >= kMaxDevices) return static_cast<int>(cudaErrorInvalidDevice);
    RetrieveArgs a;
    int grid = 0;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            // once per device, with that device current: the array's name is only a host-side
            // handle here; the kernel needs the address the symbol has on this device
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess) return static_cast<int>(e);
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return static_cast<int>(e);
            for (int st = 0; st < 2; ++st)
                for (int od = 0; od < 2; ++od)
                    for (int md = 0; md < 2; ++md) {
                        const int occ = retrieve_ctas_per_sm(st, od, md);
                        if (occ <= 0) return static_cast<int>(cudaErrorInvalidDeviceFunction);
                        g_static_grid[dev][st][od][md] = sms * occ;
                    }
            g_static_host[dev].resize(kStaticScratchBytes);
            g_static_ptr[dev] = static_cast<unsigned char*>(p);
        }
        unsigned char* scratch = g_static_ptr[dev];
        unsigned char* image = g_static_host[dev].data();
        grid = g_static_grid[dev][storage_dtype][out_dtype][m_dtype];
        size_t off = 0;
        auto put = [&](const void* src, size_t bytes) -> unsigned char* {
            unsigned char* dst = scratch + off;
            if (bytes) std::memcpy(image + off, src, bytes);
            off += align256(bytes);
            return dst;
        };
        a.layers = reinterpret_cast<const DevLayer*>(put(layers, n_layers * sizeof(DevLayer)));
        a.units = reinterpret_cast<const DevUnit*>(put(units, n_units * sizeof(DevUnit)));
        a.slot_of_pos = reinterpret_cast<const uint32_t*>(put(slot_of_pos, n_layers * sizeof(uint32_t)));
        a.base = reinterpret_cast<const void* const*>(put(base, n_layers * sizeof(void*)));
        a.out = reinterpret_cast<void* const*>(put(out, n_layers * sizeof(void*)));
        // one copy for all five tables; the image is ordinary host memory, so the call returns once the
        // driver has taken its contents, and the next call may overwrite it
        if (off) e = cudaMemcpyAsync(scratch, image, off, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return static_cast<int>(e);
    }
    a.n_units = n_units;
    a.n_layers = n_layers;
    a.M = M;
    a.task = task;
    a.lambda = lambda;
    if (n_units == 0) return 0;
    return launch_retrieve(storage_dtype, out_dtype, m_dtype, a, grid < static_cast<int>(n_units) ? grid : static_cast<int>(n_units), stream);
}

RANDES_VIOLATION_READER(violation_in_streaming_kernels)

int retrieve_ctas_per_sm(int storage_dtype, int out_dtype, int m_dtype)
{
    return with_type(storage_dtype, [&](auto st) {
        return with_type(out_dtype, [&](auto ot) {
            return with_type(m_dtype, [&](auto mt) {
                typedef typename decltype(st)::type ST;
                typedef typename decltype(mt)::type MT;
                return ctas_per_sm(retrieve_kernel<ST, typename decltype(ot)::type, MT>, RetrieveHalvesRing<ST, MT>::value ? static_cast<size_t>(kRetHStages) * kRetHStageBytes : 0);
            });
        });
    });
}

int accumulate_ctas_per_sm(int storage_dtype, int m_dtype, bool single)
{
    return with_type(storage_dtype, [&](auto st) {
        return with_type(m_dtype, [&](auto mt) {
            typedef typename decltype(st)::type ST;
            typedef typename decltype(mt)::type MT;
            return single ? ctas_per_sm(accumulate_kernel<ST, true, MT>, AccConfig<ST, true>::kSmemBytes)
                          : ctas_per_sm(accumulate_kernel<ST, false, MT>, AccConfig<ST, false>::kSmemBytes);
        });
    });
}

}  // namespace randes
