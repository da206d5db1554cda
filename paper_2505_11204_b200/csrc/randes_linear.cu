// A linear layer on a retrieved weight that is never written to memory:
//
//   y[b][r] = sum_c x[b][c] * ( W_0[p][r,c] + lambda * s_t(l,c) * M[l][r,c] ),     l = sigma_t^-1(p)
//           = ( x W_0[p]^T )[b][r] + lambda * ( (x D_t) M[l]^T )[b][r]
//
// (Section 4, second display, put inside y = x What^T; D_t is the sign diagonal of Section 4.4,
// so the inverse transform becomes a sign flip on the activations' columns, and the inverse
// shuffle of Section 4.3 is the choice of the slot l.)  Two bf16 GEMMs that share the activation
// tile, on the fifth-generation tensor cores:
//
//   * operands are staged in shared memory by TMA (128-byte swizzle), three or four stages deep:
//     x tile [128 or 256 tokens x 64], W_0 tile [128 features x 64], M tile [128 features x 64];
//   * (x D) M^T = x (M D)^T: four warps flip, in place, the sign bits of the M tile's 64 columns
//     (bf16 sign bit XOR: exact), Philox bits generated in registers -- no second buffer;
//   * the W_0 tile and the flipped M tile lie back to back in shared memory and form one
//     [256 x 64] operand: one thread issues tcgen05.mma with M = 128, N = 256, K = 16, which fills
//     both fp32 accumulators of a block of 128 tokens in tensor memory (columns 0-127: x W_0^T,
//     128-255: x (M D)^T) and reads the x tile once; with 256 tokens per CTA each weight tile
//     feeds two such products (1.5 x the flops per byte staged);
//   * the epilogue reads the accumulators with tcgen05.ld and stores fma(lambda, acc1, acc0).
//
// lambda stays in fp32 and is applied once per output, so the operands keep their stored bits.
// Every wait is bounded in time (the global nanosecond timer; one second unless the caller gives
// another limit): a CTA whose wait runs out raises a shared flag, every role leaves its loop,
// copies already issued are waited for, tensor memory is freed, nothing is written to y, and a
// device counter records the event.  The gated form of the call makes every CTA wait first for a
// word in device memory to become non-zero; a gate that nothing opens is the one wait of this
// kernel that can run out in a healthy program.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {

static __device__ unsigned int g_linear_giveups;   // CTAs that gave up waiting (0 in a healthy run)

namespace {

using namespace device;

constexpr int kBM = 128;          // tokens per block of accumulators (the M of one tcgen05.mma)
constexpr int kBN = 128;          // output features per CTA tile
constexpr int kBK = 64;           // bf16 columns per stage: one 128-byte swizzle row
constexpr int kTileBytes = kBM * kBK * 2;                    // 16 KiB, also for the kBN x kBK tiles
constexpr int kLinearThreads = 192;                          // warp 0 TMA, warp 1 MMA, warps 2-5 flip + epilogue
constexpr int kFlipThreads = 128;
constexpr uint32_t kSpinLimit = 1u << 22;                    // iteration cap of the clean-up waits after a give-up
constexpr unsigned long long kDefaultWaitNs = 1000000000ull; // one second
constexpr int kMaxStages = 4;

// HALVES = blocks of 128 tokens per CTA (1 or 2)
template <int HALVES> struct LinearGeom {
    static constexpr int kStages = HALVES == 1 ? 4 : 3;
    static constexpr int kStageBytes = (HALVES + 2) * kTileBytes;            // x block(s), W_0, M
    static constexpr uint32_t kTmemCols = HALVES * 2 * kBN;                  // two accumulators per token block
    static constexpr size_t kSmem = 1024 + kStages * kStageBytes + 256;      // alignment slack + stages + barriers
};

struct LinearArgs {
    uint32_t n_tokens, rows, cols;
    uint32_t token0;               // first token of this launch (a call may cover its tokens with two launches)
    float lambda;
    uint32_t flip;                 // 0: no sign flip on this slot
    uint32_t slot;                 // l = sigma_t^-1(p): counter word 1 of the sign stream
    DevTask task;
    void* y;                       // [n_tokens, rows], fp32 or bf16
    uint32_t y_bf16;
    const uint32_t* gate;          // NULL, or a device word the CTA waits on (non-zero = go) before its first copy
    unsigned long long wait_ns;    // limit of every wait of a CTA, measured from its start
};

// ---- mbarrier, TMA, tcgen05 wrappers --------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// The CTA gives up: the first thread to say so counts it.
__device__ __forceinline__ void give_up(volatile uint32_t* abort_flag)
{
    if (atomicExch(const_cast<uint32_t*>(abort_flag), 1u) == 0u) atomicAdd(&g_linear_giveups, 1u);
}
// Wait bounded by `deadline` (global timer, ns).  Returns false when the CTA has given up (here or in another role).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, unsigned long long deadline)
{
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_ns() > deadline) break;
        }
    }
    give_up(abort_flag);
    return false;
}
// Wait, bounded likewise, for a word in device memory to become non-zero.
__device__ __forceinline__ bool gate_wait(const uint32_t* gate, volatile uint32_t* abort_flag, unsigned long long deadline)
{
    for (;;) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(gate) : "memory");
        if (v) {
            asm volatile("fence.proxy.async.global;" ::: "memory");   // what the gate's writer stored is read by TMA next
            return true;
        }
        if (*abort_flag) return false;
        if (global_ns() > deadline) break;
        __nanosleep(200);
    }
    give_up(abort_flag);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_load32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a [128 rows x 64 bf16] K-major tile written by TMA with the
// 128-byte swizzle: rows are 128 bytes apart, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr)
{
    return static_cast<uint64_t>((saddr >> 4) & 0x3FFFu)      // start address, 16-byte units
           | (1ull << 16)                                     // leading byte offset: unused with this layout
           | (static_cast<uint64_t>(1024 >> 4) << 32)         // stride byte offset: 8 rows x 128 bytes
           | (1ull << 46)                                     // descriptor version of this architecture
           | (2ull << 61);                                    // 128-byte swizzle
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 2 kBN (both accumulators at once).
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>((2 * kBN) >> 3) << 17) | (static_cast<uint32_t>(kBM >> 4) << 24);

template <int HALVES>
__global__ void __launch_bounds__(kLinearThreads, 1)
linear_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
              const __grid_constant__ CUtensorMap map_m, const LinearArgs a)
{
    typedef LinearGeom<HALVES> Geo;
    constexpr int kStages = Geo::kStages;
    constexpr int kStageBytes = Geo::kStageBytes;
    constexpr int kOffW = HALVES * kTileBytes, kOffM = kOffW + kTileBytes;   // inside a stage: x block(s), W_0, M
    extern __shared__ unsigned char smem_raw[];
    const uint32_t smem_base = (static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw)) + 1023u) & ~1023u;
    const uint32_t bars = smem_base + kStages * kStageBytes;
    // barriers: full[s], flipped[s], empty[s] (kMaxStages each), then acc_full; then the tensor-memory address and the give-up flag
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_flipped = [&](int s) { return bars + 8u * (kMaxStages + s); };
    auto bar_empty = [&](int s) { return bars + 8u * (2 * kMaxStages + s); };
    const uint32_t bar_acc = bars + 8u * (3 * kMaxStages);
    const uint32_t tmem_slot = bar_acc + 8;
    unsigned char* gen_base = smem_raw + (smem_base - static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw)));
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(gen_base + kStages * kStageBytes + 8 * (3 * kMaxStages + 1));
    volatile uint32_t* abort_flag = tmem_ptr + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * kBN, m0 = a.token0 + blockIdx.y * (HALVES * kBM);
    const uint32_t n_k = (a.cols + kBK - 1) / kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_flipped(s), kFlipThreads);
            mbar_init(bar_empty(s), 1);
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(Geo::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_ptr;
    const unsigned long long deadline = global_ns() + a.wait_ns;

    if (warp == 0) {
        // ---- TMA producer
        if (lane == 0) {
            uint32_t issued = 0;
            const bool open = a.gate == nullptr || gate_wait(a.gate, abort_flag, deadline);
            for (uint32_t kk = 0; open && kk < n_k; ++kk) {
                const int s = kk % kStages;
                const uint32_t ph = (kk / kStages) & 1u;
                if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, deadline)) break;
                const uint32_t st = smem_base + s * kStageBytes;
                mbar_expect_tx(bar_full(s), kStageBytes);
                tma_load_2d(st, &map_x, bar_full(s), kk * kBK, m0);             // HALVES x 128 tokens in one box
                tma_load_2d(st + kOffW, &map_w, bar_full(s), kk * kBK, n0);
                tma_load_2d(st + kOffM, &map_m, bar_full(s), kk * kBK, n0);
                issued = kk + 1;
            }
            if (*abort_flag) {
                // gave up: let the copies already issued land before the CTA's shared memory is released
                const uint32_t first = issued > static_cast<uint32_t>(kStages) ? issued - kStages : 0;
                for (uint32_t kk = first; kk < issued; ++kk)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar_full(kk % kStages), (kk / kStages) & 1u); ++it) {}
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer
        if (lane == 0) {
            bool ok = true;
            for (uint32_t kk = 0; kk < n_k && ok; ++kk) {
                const int s = kk % kStages;
                const uint32_t ph = (kk / kStages) & 1u;
                ok = mbar_wait(bar_full(s), ph, abort_flag, deadline);
                if (!ok) break;
                tc_fence_after();
                if (a.flip) {
                    ok = mbar_wait(bar_flipped(s), ph, abort_flag, deadline);
                    if (!ok) break;
                    tc_fence_after();
                }
                // The W_0 tile and the (flipped) M tile lie back to back: one [256 x 64] B operand, so ONE product
                // x [W_0; M D]^T with N = 256 fills both accumulators (columns 0-127 and 128-255) and reads the x tile once.
                const uint32_t st = smem_base + s * kStageBytes;
                const uint64_t dwm = smem_desc_sw128(st + kOffW);
#pragma unroll
                for (int h = 0; h < HALVES; ++h) {
                    const uint64_t dx = smem_desc_sw128(st + h * kTileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)   // 16 bf16 columns = 32 bytes = 2 units of the descriptor's start address
                        tc_mma_bf16(tmem + h * 2 * kBN, dx + 2 * k, dwm + 2 * k, kIdesc, (kk | k) ? 1u : 0u);
                }
                tc_commit(bar_empty(s));     // the stage is free once these products have read it
            }
            tc_commit(bar_acc);              // the accumulators are final (or, after giving up, quiescent)
            if (!ok) {
                for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar_acc, 0); ++it) {}
            }
        }
    } else {
        // ---- warps 2-5: sign flip of the M tile's columns, in place; then the epilogue
        const int t = threadIdx.x - 64;                       // 0 .. 127
        bool ok = true;
        if (a.flip) {
            // 16-byte chunk q = t + 128 j of the tile sits in row q / 8 at physical position q % 8, which the
            // 128-byte swizzle maps to logical chunk (q % 8) ^ (row % 8): the same for all j of a thread
            const uint32_t lc = static_cast<uint32_t>((t & 7) ^ ((t >> 3) & 7));   // columns 8 lc .. 8 lc + 7 of the stage
            uint4 blk = make_uint4(0, 0, 0, 0);
            for (uint32_t kk = 0; kk < n_k; ++kk) {
                const int s = kk % kStages;
                const uint32_t ph = (kk / kStages) & 1u;
                if ((kk & 1u) == 0) blk = philox4x32_10(kk >> 1, a.slot, kTagSign, a.task.id, a.task.key0, a.task.key1);
                // column c = 64 kk + 8 lc: word (c >> 5) & 3 of the block, bits (c & 31) .. + 7
                const uint32_t wsel = (kk & 1u) * 2u + (lc >> 2);
                const uint32_t word = wsel == 0 ? blk.x : (wsel == 1 ? blk.y : (wsel == 2 ? blk.z : blk.w));
                const uint32_t bits = (word >> ((lc & 3u) * 8u)) & 0xFFu;
                uint32_t mask[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) mask[j] = (((bits >> (2 * j)) & 1u) << 15) | (((bits >> (2 * j + 1)) & 1u) << 31);
                ok = mbar_wait(bar_full(s), ph, abort_flag, deadline);
                if (!ok) break;
                const uint32_t tile = smem_base + s * kStageBytes + kOffM + t * 16;
                uint4 v[kTileBytes / (16 * kFlipThreads)];
#pragma unroll
                for (int j = 0; j < kTileBytes / (16 * kFlipThreads); ++j) v[j] = lds128(tile + j * kFlipThreads * 16);
#pragma unroll
                for (int j = 0; j < kTileBytes / (16 * kFlipThreads); ++j) {
                    v[j].x ^= mask[0]; v[j].y ^= mask[1]; v[j].z ^= mask[2]; v[j].w ^= mask[3];
                    sts128(tile + j * kFlipThreads * 16, v[j]);
                }
                fence_proxy_async();          // the tensor core reads the tile through the async proxy
                mbar_arrive(bar_flipped(s));
            }
        }
        if (ok) ok = mbar_wait(bar_acc, 0, abort_flag, deadline);
        if (ok && *abort_flag) ok = false;   // the issuer also arrives on this barrier when it gives up: nothing to store then
        if (ok) {
            // The accumulators hold one token per tensor-memory lane, i.e. per thread; stored like that, a warp's
            // store would touch 32 rows of y at once.  Each warp therefore turns its [32 tokens x 128 features]
            // block through shared memory (the operand ring is idle now: every product has completed) and writes
            // whole 512-byte rows.  Row pitch 528 bytes: the 16-byte writes of a quarter-warp fall into distinct banks.
            tc_fence_after();
            const int quarter = warp & 3;                     // tensor-memory lanes 32 q .. 32 q + 31
            const uint32_t tlane = static_cast<uint32_t>(quarter * 32) << 16;
            constexpr uint32_t kPitch = kBN * 4 + 16;
            const uint32_t stage = smem_base + quarter * (32 * kPitch);
            const uint32_t esz = a.y_bf16 ? 2u : 4u;
            const bool vec = (a.rows & 3u) == 0 && (reinterpret_cast<uintptr_t>(a.y) & (4 * esz - 1)) == 0;
            const uint32_t f0 = n0 + lane * 4;                // this lane's four features when rows are written
#pragma unroll 1
            for (int h = 0; h < HALVES; ++h) {
#pragma unroll 1
                for (int cchunk = 0; cchunk < kBN / 32; ++cchunk) {
                    uint32_t v0[32], v1[32];
                    tc_load32(tmem + tlane + h * 2 * kBN + cchunk * 32, v0);
                    tc_load32(tmem + tlane + h * 2 * kBN + kBN + cchunk * 32, v1);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        uint4 o;
                        o.x = __float_as_uint(__fmaf_rn(a.lambda, __uint_as_float(v1[j]), __uint_as_float(v0[j])));
                        o.y = __float_as_uint(__fmaf_rn(a.lambda, __uint_as_float(v1[j + 1]), __uint_as_float(v0[j + 1])));
                        o.z = __float_as_uint(__fmaf_rn(a.lambda, __uint_as_float(v1[j + 2]), __uint_as_float(v0[j + 2])));
                        o.w = __float_as_uint(__fmaf_rn(a.lambda, __uint_as_float(v1[j + 3]), __uint_as_float(v0[j + 3])));
                        sts128(stage + lane * kPitch + (cchunk * 32 + j) * 4, o);
                    }
                }
                __syncwarp();
                const uint32_t token0 = m0 + h * kBM + quarter * 32;
#pragma unroll 4
                for (int i = 0; i < 32; ++i) {
                    const uint32_t token = token0 + i;
                    if (token >= a.n_tokens) break;               // warp-uniform
                    const uint4 o = lds128(stage + i * kPitch + lane * 16);
                    const size_t y0 = static_cast<size_t>(token) * a.rows + f0;
                    const float of[4] = {__uint_as_float(o.x), __uint_as_float(o.y), __uint_as_float(o.z), __uint_as_float(o.w)};
                    if (a.y_bf16) {     // rounded to nearest even, once
                        bf16* yh = static_cast<bf16*>(a.y) + y0;
                        if (vec && f0 + 3 < a.rows) {
                            *reinterpret_cast<uint2*>(yh) = make_uint2(Out<bf16>::pack(of[0], of[1]), Out<bf16>::pack(of[2], of[3]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (f0 + e < a.rows) yh[e] = __float2bfloat16_rn(of[e]);
                        }
                    } else {
                        float* yp = static_cast<float*>(a.y) + y0;
                        if (vec && f0 + 3 < a.rows) {
                            *reinterpret_cast<float4*>(yp) = make_float4(of[0], of[1], of[2], of[3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (f0 + e < a.rows) yp[e] = of[e];
                        }
                    }
                }
                __syncwarp();   // the block is reused for the next 128 tokens
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(Geo::kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_encode_mutex;
EncodeTiledFn g_encode = nullptr;

EncodeTiledFn encode_fn()
{
    std::lock_guard<std::mutex> lock(g_encode_mutex);
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult st;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &st) != cudaSuccess || st != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    return g_encode;
}

// row-major [outer, inner] bf16 matrix, tiles of [box_outer, 64] with the 128-byte swizzle; out-of-range elements read as zero
bool make_map(EncodeTiledFn enc, CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_outer)
{
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {inner * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK), box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int linear_prepare()
{
    cudaError_t e = cudaFuncSetAttribute(linear_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(LinearGeom<1>::kSmem));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(linear_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(LinearGeom<2>::kSmem));
    if (e != cudaSuccess) (void)cudaGetLastError();
    return static_cast<int>(e);
}

int launch_linear(const void* x, uint32_t n_tokens, const void* w0, const void* m_slot, uint32_t rows, uint32_t cols, bool flip,
                  uint32_t slot, const DevTask& task, float lambda, void* y, bool y_bf16, const uint32_t* gate,
                  unsigned long long wait_ns, void* stream, int* n_launched)
{
    *n_launched = 0;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return static_cast<int>(cudaErrorNotSupported);
    // 128 or 256 tokens per CTA (with 256 each staged weight tile feeds two products)
    int dev = 0, sms = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (ce != cudaSuccess) return static_cast<int>(ce);
    // measured: a 128-token tile takes about 3/4 of the time of a 256-token tile (half the products, but each staged
    // weight tile then feeds one product instead of two). The first `lead` tokens (a multiple of 256) go to a launch of
    // 256-token tiles, the rest to a launch of 128-token tiles in the same stream; the split whose
    // (waves over the SMs) x (cost of a tile), summed over the two launches, is lowest wins, ties going to the larger lead.
    const uint64_t feature_tiles = (rows + kBN - 1) / kBN;
    const uint32_t blocks256 = (n_tokens + 2 * kBM - 1) / (2 * kBM);
    uint32_t lead = 0;
    uint64_t best = ~0ull;
    for (uint32_t b = 0; b <= blocks256; ++b) {
        const uint32_t covered = b * 2u * kBM;
        const uint64_t rest = covered >= n_tokens ? 0 : (n_tokens - covered + kBM - 1) / kBM;
        const uint64_t cost = (feature_tiles * b + sms - 1) / sms * 4 + (feature_tiles * rest + sms - 1) / sms * 3;
        if (cost <= best) {
            best = cost;
            lead = covered < n_tokens ? covered : n_tokens;
        }
    }
    CUtensorMap mx, mw, mm;
    if (!make_map(enc, &mw, w0, cols, rows, kBN) || !make_map(enc, &mm, m_slot, cols, rows, kBN)) return static_cast<int>(cudaErrorInvalidValue);
    LinearArgs a;
    a.n_tokens = n_tokens;
    a.rows = rows;
    a.cols = cols;
    a.lambda = lambda;
    a.flip = flip ? 1u : 0u;
    a.slot = slot;
    a.task = task;
    a.y = y;
    a.y_bf16 = y_bf16 ? 1u : 0u;
    a.gate = gate;
    a.wait_ns = wait_ns ? wait_ns : kDefaultWaitNs;
    if (lead) {
        if (!make_map(enc, &mx, x, cols, n_tokens, 2 * kBM)) return static_cast<int>(cudaErrorInvalidValue);
        a.token0 = 0;
        const dim3 grid(static_cast<unsigned>(feature_tiles), (lead + 2 * kBM - 1) / (2 * kBM));
        linear_kernel<2><<<grid, kLinearThreads, LinearGeom<2>::kSmem, static_cast<cudaStream_t>(stream)>>>(mx, mw, mm, a);
        const cudaError_t le = cudaGetLastError();
        if (le != cudaSuccess) return static_cast<int>(le);
        ++*n_launched;
    }
    if (lead < n_tokens) {
        if (!make_map(enc, &mx, x, cols, n_tokens, kBM)) return static_cast<int>(cudaErrorInvalidValue);
        a.token0 = lead;
        const dim3 grid(static_cast<unsigned>(feature_tiles), (n_tokens - lead + kBM - 1) / kBM);
        linear_kernel<1><<<grid, kLinearThreads, LinearGeom<1>::kSmem, static_cast<cudaStream_t>(stream)>>>(mx, mw, mm, a);
        const cudaError_t le = cudaGetLastError();
        if (le != cudaSuccess) return static_cast<int>(le);
        ++*n_launched;
    }
    return static_cast<int>(cudaSuccess);
}

int linear_giveups(unsigned int* count)
{
    return static_cast<int>(cudaMemcpyFromSymbol(count, g_linear_giveups, sizeof(unsigned int)));
}

}  // namespace randes
