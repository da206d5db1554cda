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

#include "randes_internal.h"

namespace randes {
namespace {

typedef __nv_bfloat16 bf16;

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter (c0..c3), key (k0,k1).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1)
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
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ float flip(float x, uint32_t mask) { return __uint_as_float(__float_as_uint(x) ^ mask); }

// ---- storage types: a lane's 16 bytes hold CPL columns -------------------------------------
template <typename T> struct Store;

template <> struct Store<float> {
    static constexpr int CPL = 4;
    static __device__ __forceinline__ void widen(const uint4& raw, float (&v)[4])
    {
        v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
        v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
    }
    static __device__ __forceinline__ float load1(const float* p) { return __ldg(p); }
};

template <> struct Store<bf16> {
    static constexpr int CPL = 8;
    static __device__ __forceinline__ void widen(const uint4& raw, float (&v)[8])
    {
        v[0] = __uint_as_float(raw.x << 16); v[1] = __uint_as_float(raw.x & 0xFFFF0000u);
        v[2] = __uint_as_float(raw.y << 16); v[3] = __uint_as_float(raw.y & 0xFFFF0000u);
        v[4] = __uint_as_float(raw.z << 16); v[5] = __uint_as_float(raw.z & 0xFFFF0000u);
        v[6] = __uint_as_float(raw.w << 16); v[7] = __uint_as_float(raw.w & 0xFFFF0000u);
    }
    static __device__ __forceinline__ float load1(const bf16* p)
    {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
};

// ---- output types: CPL consecutive values ---------------------------------------------------
template <typename T> struct Out;

template <> struct Out<float> {
    template <int CPL> static __device__ __forceinline__ void store(float* p, const float (&y)[CPL])
    {
#pragma unroll
        for (int j = 0; j < CPL / 4; ++j)
            __stcs(reinterpret_cast<float4*>(p) + j, make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]));
    }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
    template <int CPL> static __device__ __forceinline__ bool aligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
};

template <> struct Out<bf16> {
    // round to nearest even, two values per conversion
    static __device__ __forceinline__ uint32_t pack(float lo, float hi)
    {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
    template <int CPL> static __device__ __forceinline__ void store(bf16* p, const float (&y)[CPL])
    {
        if (CPL == 4) {
            __stcs(reinterpret_cast<uint2*>(p), make_uint2(pack(y[0], y[1]), pack(y[2], y[3])));
        } else {
            __stcs(reinterpret_cast<uint4*>(p),
                   make_uint4(pack(y[0], y[1]), pack(y[2], y[3]), pack(y[4 % CPL], y[5 % CPL]), pack(y[6 % CPL], y[7 % CPL])));
        }
    }
    static __device__ __forceinline__ void store1(bf16* p, float v) { *p = __float2bfloat16_rn(v); }
    template <int CPL> static __device__ __forceinline__ bool aligned(const void* p)
    {
        return (reinterpret_cast<uintptr_t>(p) & (2 * CPL - 1)) == 0;
    }
};

__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The sign bits of this lane's CPL columns (bit e = column c + e), out of the
// Philox block that covers them.
template <int CPL> __device__ __forceinline__ uint32_t lane_bits(const uint4& blk, int lane)
{
    if (CPL == 4) {
        const int q = lane >> 3;
        const uint32_t w = q == 0 ? blk.x : (q == 1 ? blk.y : (q == 2 ? blk.z : blk.w));
        return (w >> ((lane & 7) * 4)) & 0xFu;
    }
    const int q = (lane & 15) >> 2;
    const uint32_t w = q == 0 ? blk.x : (q == 1 ? blk.y : (q == 2 ? blk.z : blk.w));
    return (w >> ((lane & 3) * 8)) & 0xFFu;
}

// Which 128-column Philox block holds this lane's columns.
template <int CPL> __device__ __forceinline__ uint32_t lane_block(uint32_t cb, int lane)
{
    return CPL == 4 ? cb : cb * 2 + (lane >> 4);
}

// geometry of this warp inside a unit
struct WarpTile {
    uint32_t cb;      // warp-wide column block of the layer
    uint32_t c;       // first of this lane's CPL columns
    uint32_t r0;      // first row of this warp
    uint32_t r_end;   // one past the last row of the unit
    uint32_t rstep;   // row stride between this warp's rows
};

template <int CPL> __device__ __forceinline__ WarpTile warp_tile(const DevUnit& un, int warp, int lane)
{
    WarpTile t;
    const uint32_t nbc = un.nbc;
    t.cb = un.cb0 + (warp & (nbc - 1));
    t.c = (t.cb * 32 + lane) * CPL;
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
                                              const ST* __restrict__ wp, OT* __restrict__ op,
                                              const float (&lam)[Store<ST>::CPL])
{
    constexpr int CPL = Store<ST>::CPL;
    constexpr int U = CPL == 4 ? 4 : 2;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep * U) {
        float4 m[U][CPL / 4];
        uint4 w[U];
        float ms[U][CPL], wsc[U][CPL];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint32_t rr = r + j * t.rstep;
            if (rr < t.r_end) {
                const size_t off = static_cast<size_t>(rr) * cols + t.c;
                if (VEC) {
#pragma unroll
                    for (int h = 0; h < CPL / 4; ++h) m[j][h] = __ldcs(reinterpret_cast<const float4*>(mp + off) + h);
                    w[j] = __ldcs(reinterpret_cast<const uint4*>(wp + off));
                } else {
#pragma unroll
                    for (int e = 0; e < CPL; ++e) {
                        ms[j][e] = 0.f; wsc[j][e] = 0.f;
                        if (t.c + e < cols) { ms[j][e] = mp[off + e]; wsc[j][e] = Store<ST>::load1(wp + off + e); }
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const uint32_t rr = r + j * t.rstep;
            if (rr < t.r_end) {
                const size_t off = static_cast<size_t>(rr) * cols + t.c;
                float mv[CPL], wv[CPL], y[CPL];
                if (VEC) {
#pragma unroll
                    for (int h = 0; h < CPL / 4; ++h) {
                        mv[4 * h] = m[j][h].x; mv[4 * h + 1] = m[j][h].y; mv[4 * h + 2] = m[j][h].z; mv[4 * h + 3] = m[j][h].w;
                    }
                    Store<ST>::widen(w[j], wv);
                } else {
#pragma unroll
                    for (int e = 0; e < CPL; ++e) { mv[e] = ms[j][e]; wv[e] = wsc[j][e]; }
                }
#pragma unroll
                for (int e = 0; e < CPL; ++e) y[e] = __fmaf_rn(lam[e], mv[e], wv[e]);
                if (VEC) {
                    Out<OT>::template store<CPL>(op + off, y);
                } else {
#pragma unroll
                    for (int e = 0; e < CPL; ++e)
                        if (t.c + e < cols) Out<OT>::store1(op + off + e, y[e]);
                }
            }
        }
    }
}

template <typename ST, typename OT>
__global__ void __launch_bounds__(kThreadsPerCta) retrieve_kernel(const RetrieveArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t p = un.layer;                       // layer position being rebuilt
        const DevLayer lp = a.layers[p];
        const uint32_t slot = (lp.flags & kFlagShuffle) ? a.slot_of_pos[p] : p;   // sigma^-1
        const unsigned long long m_off = slot == p ? lp.m_off : a.layers[slot].m_off;
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.c >= lp.cols || t.r0 >= t.r_end) continue;

        uint32_t bits = 0;
        if (lp.flags & kFlagFlip) {
            const uint4 blk = philox4x32_10(lane_block<CPL>(t.cb, lane), slot, kTagSign, a.task.id, a.task.key0, a.task.key1);
            bits = lane_bits<CPL>(blk, lane);
        }
        float lam[CPL];
#pragma unroll
        for (int e = 0; e < CPL; ++e) lam[e] = flip(a.lambda, ((bits >> e) & 1u) << 31);

        const ST* wp = static_cast<const ST*>(a.base[p]);
        OT* op = static_cast<OT*>(a.out[p]);
        const float* mp = a.M + m_off;
        const bool vec = lp.cols % CPL == 0 && aligned16(wp) && Out<OT>::template aligned<CPL>(op);
        if (vec) retrieve_rows<ST, OT, true>(t, lp.cols, mp, wp, op, lam);
        else retrieve_rows<ST, OT, false>(t, lp.cols, mp, wp, op, lam);
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
// word per batch).  The row loop is then a software pipeline over (row, batch of
// NB tasks): W_i tiles travel through a per-thread cp.async ring in shared
// memory, several stages ahead of their use.
// =========================================================================================

// How W_0 enters the difference W_i - W_0.
constexpr int kNoBase = 0;        // the task tensors already hold deltas
constexpr int kSharedBase = 1;    // no shuffle: every task subtracts the same W_0 tile, fetched once per row
constexpr int kPerTaskBase = 2;   // shuffle: task i subtracts W_0[sigma_i(l)]; tiles repeat across slots and hit in L2

constexpr int kInitZero = 0;      // start from +0
constexpr int kInitAsync = 1;     // start from M written by an earlier launch: staged like the weights
constexpr int kInitPlain = 2;     // start from M written earlier by this thread: plain load

constexpr uint32_t kSlotBytes = kThreadsPerCta * 16;   // one 16-byte slot of every thread of the CTA

template <int NB, int MAXT> struct WarpScratch {
    const void* pw[MAXT];
    const void* pb[MAXT];
    uint32_t bits[(MAXT + NB - 1) / NB][32];   // [batch][lane]: bit k*CPL + e = sign of column e for task k of the batch
};

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t saddr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t saddr, const uint4& v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Ring of one thread: NSTAGE stages x SLOTS 16-byte slots, slot-major across the
// CTA's threads (consecutive lanes are contiguous: conflict-free).  Per stage:
//   slots [0, NB)            W_i tiles of the batch
//   slot  NB                 W_0 tile of the row (kSharedBase), filled with the row's first batch
//   slots NB+1 .. NB+CPL/4   M tile of the row (kInitAsync), filled with the row's first batch
template <int CPL, int NB> struct RingGeom {
    static constexpr int SLOTS = NB + 1 + CPL / 4;
    static constexpr uint32_t kStageBytes = SLOTS * kSlotBytes;
};

template <typename ST, int BASE, int NB, int NSTAGE, int MAXT, bool FULL>
__device__ __forceinline__ void accumulate_rows_async(const WarpTile& t, uint32_t cols, const WarpScratch<NB, MAXT>& ws, int lane,
                                                      uint32_t nt, int init_mode, float* __restrict__ mp, uint32_t ring)
{
    constexpr int CPL = Store<ST>::CPL;
    typedef RingGeom<CPL, NB> G;
    static_assert(NB * CPL <= 32, "a batch's sign bits must fit one word");
    const uint32_t nrows = (t.r_end - t.r0 + t.rstep - 1) / t.rstep;
    const uint32_t nbat = (nt + NB - 1) / NB;
    const uint32_t N = nrows * nbat;
    const uint32_t row_stride = t.rstep * cols;          // elements between this warp's rows
    const uint32_t off0 = t.r0 * cols + t.c;             // element offset of the first tile (layers hold < 2^32 elements)

    // three cursors over the same (row, batch) sequence: copies issued, W_0 prefetched, consumed
    uint32_t off_i = off0, b_i = 0, off_p = off0, b_p = 0, off_c = off0, b_c = 0;

    auto issue = [&](uint32_t stage) {
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const uint32_t i = b_i * NB + k;
            if (FULL || i < nt) cp_async16(stage + k * kSlotBytes, static_cast<const ST*>(ws.pw[i]) + off_i);
        }
        if (b_i == 0) {
            if (BASE == kSharedBase) cp_async16(stage + NB * kSlotBytes, static_cast<const ST*>(ws.pb[0]) + off_i);
            if (init_mode == kInitAsync) {
#pragma unroll
                for (int h = 0; h < CPL / 4; ++h) cp_async16(stage + (NB + 1 + h) * kSlotBytes, mp + off_i + 4 * h);
            }
        }
        if (++b_i == nbat) { b_i = 0; off_i += row_stride; }
    };

    // W_0 tiles under a shuffle come from L2 (each is shared by several slots): they
    // are fetched into registers one batch ahead instead of occupying the ring.
    uint4 w0_next[NB];
    auto prefetch_base = [&]() {
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            const uint32_t i = b_p * NB + k;
            if (FULL || i < nt) w0_next[k] = __ldg(reinterpret_cast<const uint4*>(static_cast<const ST*>(ws.pb[i]) + off_p));
        }
        if (++b_p == nbat) { b_p = 0; off_p += row_stride; }
    };

    uint32_t issued = 0;
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (issued < N) { issue(ring + s * G::kStageBytes); ++issued; }
        cp_async_commit();
    }
    if (BASE == kPerTaskBase) prefetch_base();

    float acc[CPL], w0row[CPL];
    uint32_t stage_c = ring, stage_i = ring + (NSTAGE - 1) * G::kStageBytes;
    const uint32_t ring_end = ring + NSTAGE * G::kStageBytes;
    for (uint32_t it = 0; it < N; ++it) {
        if (issued < N) { issue(stage_i); ++issued; }
        cp_async_commit();
        stage_i += G::kStageBytes;
        if (stage_i == ring_end) stage_i = ring;

        uint4 w0_cur[NB];
        if (BASE == kPerTaskBase) {
#pragma unroll
            for (int k = 0; k < NB; ++k) w0_cur[k] = w0_next[k];
            if (it + 1 < N) prefetch_base();
        }
        cp_async_wait<NSTAGE - 1>();   // everything but the newest NSTAGE-1 groups has landed: stage_c is ready

        if (b_c == 0) {
#pragma unroll
            for (int e = 0; e < CPL; ++e) { acc[e] = 0.f; w0row[e] = 0.f; }
            if (init_mode == kInitAsync) {
#pragma unroll
                for (int h = 0; h < CPL / 4; ++h) {
                    const uint4 raw = lds128(stage_c + (NB + 1 + h) * kSlotBytes);
                    acc[4 * h] = __uint_as_float(raw.x); acc[4 * h + 1] = __uint_as_float(raw.y);
                    acc[4 * h + 2] = __uint_as_float(raw.z); acc[4 * h + 3] = __uint_as_float(raw.w);
                }
            } else if (init_mode == kInitPlain) {
#pragma unroll
                for (int h = 0; h < CPL / 4; ++h) {
                    const float4 v = *reinterpret_cast<const float4*>(mp + off_c + 4 * h);
                    acc[4 * h] = v.x; acc[4 * h + 1] = v.y; acc[4 * h + 2] = v.z; acc[4 * h + 3] = v.w;
                }
            }
            if (BASE == kSharedBase) Store<ST>::widen(lds128(stage_c + NB * kSlotBytes), w0row);
        }
        const uint32_t pack = ws.bits[b_c][lane];
#pragma unroll
        for (int k = 0; k < NB; ++k) {
            if (FULL || b_c * NB + k < nt) {
                float d[CPL];
                Store<ST>::widen(lds128(stage_c + k * kSlotBytes), d);
                if (BASE == kPerTaskBase) {
                    float s[CPL];
                    Store<ST>::widen(w0_cur[k], s);
#pragma unroll
                    for (int e = 0; e < CPL; ++e) d[e] = __fsub_rn(d[e], s[e]);
                } else if (BASE == kSharedBase) {
#pragma unroll
                    for (int e = 0; e < CPL; ++e) d[e] = __fsub_rn(d[e], w0row[e]);
                }
#pragma unroll
                for (int e = 0; e < CPL; ++e)
                    acc[e] = __fadd_rn(acc[e], flip(d[e], (pack << (31 - (k * CPL + e))) & 0x80000000u));
            }
        }
        if (b_c + 1 == nbat) {
#pragma unroll
            for (int h = 0; h < CPL / 4; ++h)
                *reinterpret_cast<float4*>(mp + off_c + 4 * h) = make_float4(acc[4 * h], acc[4 * h + 1], acc[4 * h + 2], acc[4 * h + 3]);
            b_c = 0;
            off_c += row_stride;
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
template <typename ST, int NB, int MAXT>
__device__ __noinline__ void accumulate_rows_scalar(WarpTile t, uint32_t cols, const WarpScratch<NB, MAXT>* wsp, int lane,
                                                    uint32_t nt, int init_mode, float* mp, int base_mode)
{
    constexpr int CPL = Store<ST>::CPL;
    const WarpScratch<NB, MAXT>& ws = *wsp;
    for (uint32_t r = t.r0; r < t.r_end; r += t.rstep) {
        const size_t off = static_cast<size_t>(r) * cols + t.c;
        for (int e = 0; e < CPL; ++e) {
            if (t.c + e >= cols) break;
            float acc = init_mode == kInitZero ? 0.f : mp[off + e];
            for (uint32_t i = 0; i < nt; ++i) {
                float d = Store<ST>::load1(static_cast<const ST*>(ws.pw[i]) + off + e);
                if (base_mode != kNoBase) d = __fsub_rn(d, Store<ST>::load1(static_cast<const ST*>(ws.pb[i]) + off + e));
                const uint32_t bit = (ws.bits[i / NB][lane] >> ((i % NB) * CPL + e)) & 1u;
                acc = __fadd_rn(acc, flip(d, bit << 31));
            }
            mp[off + e] = acc;
        }
    }
}

#ifndef RANDES_COMPRESS_NB
#define RANDES_COMPRESS_NB 4
#endif
#ifndef RANDES_COMPRESS_NSTAGE_F32
#define RANDES_COMPRESS_NSTAGE_F32 4
#endif
#ifndef RANDES_COMPRESS_NSTAGE_BF16
#define RANDES_COMPRESS_NSTAGE_BF16 3
#endif
#ifndef RANDES_SINGLE_NSTAGE_F32
#define RANDES_SINGLE_NSTAGE_F32 8
#endif
#ifndef RANDES_SINGLE_NSTAGE_BF16
#define RANDES_SINGLE_NSTAGE_BF16 6
#endif

template <typename ST, bool SINGLE> struct AccConfig {
    static constexpr int CPL = Store<ST>::CPL;
    static constexpr int NB = SINGLE ? 1 : RANDES_COMPRESS_NB;
    static constexpr int MAXT = SINGLE ? 1 : kTaskChunk;
    static constexpr int NSTAGE = SINGLE ? (CPL == 4 ? RANDES_SINGLE_NSTAGE_F32 : RANDES_SINGLE_NSTAGE_BF16)
                                         : (CPL == 4 ? RANDES_COMPRESS_NSTAGE_F32 : RANDES_COMPRESS_NSTAGE_BF16);
    typedef WarpScratch<NB, MAXT> Scratch;
    static constexpr size_t kRingBytes = static_cast<size_t>(NSTAGE) * RingGeom<CPL, NB>::kStageBytes;
    static constexpr size_t kSmemBytes = kRingBytes + kWarpsPerCta * sizeof(Scratch);
};

// SINGLE: one task per launch (add / remove): a deep ring of rows.  Otherwise
// (compress): NB tasks per stage.
template <typename ST, bool SINGLE>
__global__ void __launch_bounds__(kThreadsPerCta, 2) accumulate_kernel(const AccumulateArgs a)
{
    typedef AccConfig<ST, SINGLE> Cfg;
    constexpr int CPL = Cfg::CPL, NB = Cfg::NB, MAXT = Cfg::MAXT, NS = Cfg::NSTAGE;
    extern __shared__ __align__(16) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + threadIdx.x * 16;
    // between units the ring is idle: its first slots double as the warp's table of Philox blocks
    const uint32_t blocks = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + warp * 512;
    typename Cfg::Scratch& ws = reinterpret_cast<typename Cfg::Scratch*>(smem + Cfg::kRingBytes)[warp];
    const uint32_t L = a.n_layers;
    const uint32_t negate_bits = a.negate ? 0xFFFFFFFFu : 0u;
    for (uint32_t u = blockIdx.x; u < a.n_units; u += gridDim.x) {
        const DevUnit un = a.units[u];
        const uint32_t slot = un.layer;
        const DevLayer ls = a.layers[slot];
        const WarpTile t = warp_tile<CPL>(un, warp, lane);
        if (t.r0 >= t.r_end || t.cb * 32 * CPL >= ls.cols) continue;   // warp-uniform: nothing for this warp
        const bool lane_on = t.c < ls.cols;
        const bool shuffled = (ls.flags & kFlagShuffle) != 0;
        const bool flipped = (ls.flags & kFlagFlip) != 0;
        float* mp = a.M + ls.m_off;
        const int base_mode = !a.has_base ? kNoBase : ((shuffled && !SINGLE) ? kPerTaskBase : kSharedBase);

        for (uint32_t chunk0 = 0; chunk0 < a.n_tasks; chunk0 += MAXT) {
            const uint32_t nt = min(static_cast<uint32_t>(MAXT), a.n_tasks - chunk0);
            __syncwarp();   // the previous chunk's readers are done with the scratch
            bool ok = true;
            if (lane < nt) {
                const uint32_t ti = chunk0 + lane;
                const uint32_t src = shuffled ? a.src_of_slot[static_cast<size_t>(ti) * L + slot] : slot;   // sigma_i(l)
                const void* pw = a.task_ptrs[static_cast<size_t>(ti) * L + src];
                const void* pb = a.has_base ? a.base[src] : nullptr;
                ws.pw[lane] = pw;
                ws.pb[lane] = pb;
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
                ws.bits[b][lane] = pack ^ negate_bits;
            }
            __syncwarp();   // the block table is free again before any lane's copies land in the ring
            if (lane_on) {
                const int init_mode = chunk0 > 0 ? kInitPlain : (a.init_from_m ? kInitAsync : kInitZero);
                const bool full = nt % NB == 0;
                if (!vec)
                    accumulate_rows_scalar<ST, NB, MAXT>(t, ls.cols, &ws, lane, nt, init_mode, mp, base_mode);
                else if (base_mode == kNoBase) {
                    if (full) accumulate_rows_async<ST, kNoBase, NB, NS, MAXT, true>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                    else accumulate_rows_async<ST, kNoBase, NB, NS, MAXT, false>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                } else if (base_mode == kSharedBase) {
                    if (full) accumulate_rows_async<ST, kSharedBase, NB, NS, MAXT, true>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                    else accumulate_rows_async<ST, kSharedBase, NB, NS, MAXT, false>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                } else {
                    if (full) accumulate_rows_async<ST, kPerTaskBase, NB, NS, MAXT, true>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                    else accumulate_rows_async<ST, kPerTaskBase, NB, NS, MAXT, false>(t, ls.cols, ws, lane, nt, init_mode, mp, ring);
                }
            }
        }
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
    const bool single = a.n_tasks == 1;
    if (storage_dtype == 0) {
        if (single) accumulate_kernel<float, true><<<grid, kThreadsPerCta, AccConfig<float, true>::kSmemBytes, s>>>(a);
        else accumulate_kernel<float, false><<<grid, kThreadsPerCta, AccConfig<float, false>::kSmemBytes, s>>>(a);
    } else {
        if (single) accumulate_kernel<bf16, true><<<grid, kThreadsPerCta, AccConfig<bf16, true>::kSmemBytes, s>>>(a);
        else accumulate_kernel<bf16, false><<<grid, kThreadsPerCta, AccConfig<bf16, false>::kSmemBytes, s>>>(a);
    }
    return static_cast<int>(cudaGetLastError());
}

int retrieve_ctas_per_sm(int storage_dtype, int out_dtype)
{
    if (storage_dtype == 0 && out_dtype == 0) return ctas_per_sm(retrieve_kernel<float, float>, 0);
    if (storage_dtype == 0 && out_dtype == 1) return ctas_per_sm(retrieve_kernel<float, bf16>, 0);
    if (storage_dtype == 1 && out_dtype == 0) return ctas_per_sm(retrieve_kernel<bf16, float>, 0);
    return ctas_per_sm(retrieve_kernel<bf16, bf16>, 0);
}

int accumulate_ctas_per_sm(int storage_dtype, bool single)
{
    if (storage_dtype == 0)
        return single ? ctas_per_sm(accumulate_kernel<float, true>, AccConfig<float, true>::kSmemBytes)
                      : ctas_per_sm(accumulate_kernel<float, false>, AccConfig<float, false>::kSmemBytes);
    return single ? ctas_per_sm(accumulate_kernel<bf16, true>, AccConfig<bf16, true>::kSmemBytes)
                  : ctas_per_sm(accumulate_kernel<bf16, false>, AccConfig<bf16, false>::kSmemBytes);
}

}  // namespace randes
