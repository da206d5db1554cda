// Device-side helpers shared by the kernels of the RanDeS library: Philox4x32-10,
// packed fp32x2 arithmetic, element access for fp32 / bf16 storage and output,
// the lane <-> column mapping and the geometry of a warp inside a unit of work.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "randes_internal.h"

namespace randes {
namespace device {


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

// Checked build (-DRANDES_CHECKED): before a thread block touches a tile, the indices that every later address of the
// tile is derived from -- the unit's layer, the permuted layer, the unit's rows -- are compared with the plan's
// bounds; a tile that fails is skipped and the first failure is recorded in a device word (kernel, what, unit) that
// randes_debug_violation() reads.  In the ordinary build checked() is the constant true and costs nothing.
enum { kCheckLayer = 1, kCheckPermuted = 2, kCheckRows = 3 };
#ifdef RANDES_CHECKED
static __device__ unsigned long long g_violation;     // of the kernels of this translation unit
__device__ __forceinline__ bool checked(bool ok, uint32_t kernel_id, uint32_t what, uint32_t unit)
{
    if (ok) return true;
    atomicCAS(&g_violation, 0ull, (1ull << 63) | (static_cast<unsigned long long>(kernel_id) << 48) |
                                      (static_cast<unsigned long long>(what) << 40) | unit);
    return false;
}
#define RANDES_VIOLATION_READER(name)                                                              \
    unsigned long long name()                                                                      \
    {                                                                                              \
        unsigned long long w = 0;                                                                  \
        if (cudaMemcpyFromSymbol(&w, device::g_violation, sizeof w) != cudaSuccess) w = ~0ull;     \
        return w;                                                                                  \
    }
#else
__device__ __forceinline__ constexpr bool checked(bool, uint32_t, uint32_t, uint32_t) { return true; }
#define RANDES_VIOLATION_READER(name) \
    unsigned long long name() { return 0; }
#endif

__device__ __forceinline__ float flip(float x, uint32_t mask) { return __uint_as_float(__float_as_uint(x) ^ mask); }

// Two fp32 values in one 64-bit register, for the packed add / sub / fma of sm_100.
// Each half is rounded to nearest even exactly like the scalar instruction.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(uint32_t lo, uint32_t hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi)
{
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b)
{
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// ---- storage types: a lane's 16 bytes hold CPL columns -------------------------------------
template <typename T> struct Store;

template <> struct Store<float> {
    static constexpr int CPL = 4;
    static __device__ __forceinline__ void widen(const uint4& raw, float (&v)[4])
    {
        v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
        v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
    }
    static __device__ __forceinline__ void widen2(const uint4& raw, f32x2 (&v)[2])
    {
        v[0] = pack2(raw.x, raw.y);
        v[1] = pack2(raw.z, raw.w);
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
    static __device__ __forceinline__ void widen2(const uint4& raw, f32x2 (&v)[4])
    {
        v[0] = pack2(raw.x << 16, raw.x & 0xFFFF0000u);
        v[1] = pack2(raw.y << 16, raw.y & 0xFFFF0000u);
        v[2] = pack2(raw.z << 16, raw.z & 0xFFFF0000u);
        v[3] = pack2(raw.w << 16, raw.w & 0xFFFF0000u);
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


// ---- a lane's CPL consecutive elements of the superposition M (fp32 or bf16) ------------------
template <typename MT, int CPL> struct MTile;

template <int CPL> struct MTile<float, CPL> {
    static constexpr int kBytes = 4 * CPL;
    // STREAM: the tile is read once (evict-first); otherwise other CTAs will want it from L2
    template <bool STREAM = true> static __device__ __forceinline__ void load(const float* p, float (&v)[CPL])
    {
#pragma unroll
        for (int h = 0; h < CPL / 4; ++h) {
            const float4 m = STREAM ? __ldcs(reinterpret_cast<const float4*>(p) + h) : __ldg(reinterpret_cast<const float4*>(p) + h);
            v[4 * h] = m.x; v[4 * h + 1] = m.y; v[4 * h + 2] = m.z; v[4 * h + 3] = m.w;
        }
    }
    static __device__ __forceinline__ void store(float* p, const float (&v)[CPL])
    {
#pragma unroll
        for (int h = 0; h < CPL / 4; ++h)
            reinterpret_cast<float4*>(p)[h] = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
    }
    // from 16-byte words as they sit in memory (word h = elements 4h .. 4h+3)
    static __device__ __forceinline__ void unpack(const uint4 (&raw)[(kBytes + 15) / 16], float (&v)[CPL])
    {
#pragma unroll
        for (int h = 0; h < CPL / 4; ++h) {
            v[4 * h] = __uint_as_float(raw[h].x); v[4 * h + 1] = __uint_as_float(raw[h].y);
            v[4 * h + 2] = __uint_as_float(raw[h].z); v[4 * h + 3] = __uint_as_float(raw[h].w);
        }
    }
    static __device__ __forceinline__ float load1(const float* p) { return *p; }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};

template <int CPL> struct MTile<__nv_bfloat16, CPL> {
    static constexpr int kBytes = 2 * CPL;
    static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);   // round to nearest even
        return *reinterpret_cast<const uint32_t*>(&v);
    }
    template <bool STREAM = true> static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[CPL])
    {
        if (CPL == 4) {
            const uint2 m = STREAM ? __ldcs(reinterpret_cast<const uint2*>(p)) : __ldg(reinterpret_cast<const uint2*>(p));
            v[0] = lo(m.x); v[1] = hi(m.x); v[2] = lo(m.y); v[3] = hi(m.y);
        } else {
            const uint4 m = STREAM ? __ldcs(reinterpret_cast<const uint4*>(p)) : __ldg(reinterpret_cast<const uint4*>(p));
            v[0] = lo(m.x); v[1] = hi(m.x); v[2] = lo(m.y); v[3] = hi(m.y);
            v[4 % CPL] = lo(m.z); v[5 % CPL] = hi(m.z); v[6 % CPL] = lo(m.w); v[7 % CPL] = hi(m.w);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[CPL])
    {
        if (CPL == 4) *reinterpret_cast<uint2*>(p) = make_uint2(pack(v[0], v[1]), pack(v[2], v[3]));
        else *reinterpret_cast<uint4*>(p) = make_uint4(pack(v[0], v[1]), pack(v[2], v[3]), pack(v[4 % CPL], v[5 % CPL]), pack(v[6 % CPL], v[7 % CPL]));
    }
    static __device__ __forceinline__ void unpack(const uint4 (&raw)[1], float (&v)[CPL])
    {
        v[0] = lo(raw[0].x); v[1] = hi(raw[0].x); v[2] = lo(raw[0].y); v[3] = hi(raw[0].y);
        if (CPL == 8) { v[4 % CPL] = lo(raw[0].z); v[5 % CPL] = hi(raw[0].z); v[6 % CPL] = lo(raw[0].w); v[7 % CPL] = hi(raw[0].w); }
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16* p)
    {
        return __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(p)) << 16);
    }
    static __device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// ---- asynchronous copies into shared memory and 32-bit shared-window accesses ----------------
constexpr uint32_t kSlotBytes = kThreadsPerCta * 16;   // one 16-byte slot of every thread of the CTA

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
// the same copy with an L2 eviction priority (a policy word made by one of the two functions below)
__device__ __forceinline__ void cp_async16_hint(uint32_t smem_dst, const void* gmem_src, uint64_t policy)
{
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gmem_src), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_evict_last_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void cp_async8(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* gmem) { asm volatile("prefetch.global.L2 [%0];" ::"l"(gmem)); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t saddr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
    return v;
}
__device__ __forceinline__ const char* lds_ptr(uint32_t saddr)
{
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(saddr));
    return reinterpret_cast<const char*>(v);
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t saddr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t saddr)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(saddr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t saddr, const uint4& v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts_u16(uint32_t saddr, uint32_t v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(saddr), "h"(static_cast<unsigned short>(v)) : "memory");
}
__device__ __forceinline__ void sts_ptrs(uint32_t saddr, const void* a, const void* b)
{
    asm volatile("st.shared.v2.u64 [%0], {%1, %2};" ::"r"(saddr), "l"(a), "l"(b) : "memory");
}

}  // namespace device
}  // namespace randes
