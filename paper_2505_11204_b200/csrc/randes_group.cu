// Compress under a layer shuffle, one group of same-shape layers at a time.
//
//   M[l] = sum_i s_i(l, c) * ( W_i[sigma_i(l)] - W_0[sigma_i(l)] )        (Section 4, first display;
//                                                                           Section 4.3 for sigma, 4.4 for s)
//
// Under a shuffle slot l needs W_0[sigma_i(l)] for every task i: each W_0 tile of a
// group is wanted by every slot of the group and K times per slot.  A CTA therefore takes a
// group unit -- a few rows x one warp-wide column block of EVERY member of the group --,
// copies the W_0 tiles of all members into a shared-memory stash once, and resolves, for all
// (slot, task) pairs of the unit at once and in parallel over its threads, the source tensor
// sigma_i(l) and the Philox block of sign bits.  After that only the task tensors stream from
// HBM, through a per-thread cp.async ring (each lane reads back only what it copied, so the
// row loop needs no barrier), and W_0 and the signs come from shared memory.
//
// A warp takes (slot, block of rows) items in turn and runs ONE software pipeline over all its
// items: stage = one task x two rows (fp32 weights, items of four rows) or one task x three rows
// (bf16 weights, items of three rows: the sign decode is shared by more rows).  Sums run in task order, every output
// element is written by one thread: results are bit-reproducible and equal to the per-layer
// kernel's.  (Measured and not kept: the W_0 tiles of the CTA's next unit prefetched into L2 during the
// row loop -- slower by 3 - 5 %; the warps' copy pipelines running on across unit boundaries, with
// the first stages of the next unit in flight during the barrier and the stash refill -- no gain.)
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <type_traits>

#include "randes_device.cuh"
#include "randes_internal.h"

namespace randes {
namespace {

using namespace device;

constexpr uint32_t kMaxGroup = kStashBytes / kStashTileBytes;   // members whose tiles fit the largest stash at one row each
constexpr uint32_t kOffTableBytes = kMaxGroup * 16;             // per member: first element of its slot in M, its W_0 tensor

// rows per stage (SR), rows per item (IR) and stash size per weight type
template <typename ST> struct GroupGeom;
template <> struct GroupGeom<float> {
    static constexpr uint32_t SR = 2, IR = item_rows(0), kStash = stash_bytes(0);
};
template <> struct GroupGeom<__nv_bfloat16> {
    static constexpr uint32_t SR = 3, IR = item_rows(1), kStash = stash_bytes(1);
};
constexpr uint32_t stage_rows(int storage_dtype) { return storage_dtype == 1 ? 3u : 2u; }

__device__ __forceinline__ unsigned long long lds_u64(uint32_t saddr)
{
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(saddr));
    return v;
}

// Per (slot, task) pair of a unit, in shared memory: the task's source tensor W_i[sigma_i(l)],
// which member of the group that source layer is (-> its W_0 tile in the stash), and the
// Philox blocks with the sign bits of the unit's columns.
template <int HB> struct PairRecord {
    static constexpr uint32_t kBytes = 16 + 16 * HB;
    static constexpr uint32_t kPtr = 0, kMember = 8, kBlocks = 16;
};

// Position of a warp in its sequence of stages: item (slot, block of rows) -> row pair -> task.
// Everything a stage needs is kept incrementally so that the common step (next task of the
// same row pair) is one addition and one comparison.
struct Cursor {
    uint32_t rec;        // shared address of the current pair's record
    uint32_t rec_begin;  // record of task 0 of the current slot
    uint32_t rec_end;    // one past the record of the last task
    uint32_t off;        // element offset of the row pair's first row inside a layer (+ this lane's column)
    uint32_t row;        // that row, relative to the unit (-> stash)
    uint32_t rows_left;  // rows of the item from `row` on
    uint32_t item;       // index of the (slot, block of rows) item
    uint32_t m_off;      // shared address of the slot's offset in M
};

template <uint32_t REC, uint32_t IR>
__device__ __forceinline__ void cursor_set(Cursor& c, uint32_t item, uint32_t n_chunks, uint32_t Rn, uint32_t nt, uint32_t s_rec,
                                           uint32_t off0, uint32_t cols)
{
    c.item = item;
    const uint32_t ms = item / n_chunks;
    c.m_off = s_rec - kOffTableBytes + ms * 16;
    const uint32_t chunk = item - ms * n_chunks;
    c.row = chunk * IR;
    c.rows_left = min(IR, Rn - c.row);
    c.off = off0 + c.row * cols;
    c.rec_begin = c.rec = s_rec + ms * nt * REC;
    c.rec_end = c.rec_begin + nt * REC;
}

template <uint32_t REC, uint32_t IR, uint32_t SR>
__device__ __forceinline__ void cursor_next(Cursor& c, uint32_t n_chunks, uint32_t Rn, uint32_t nt, uint32_t s_rec, uint32_t off0,
                                            uint32_t cols)
{
    c.rec += REC;
    if (c.rec != c.rec_end) return;
    if (c.rows_left > SR) {         // next rows of the same slot
        c.rec = c.rec_begin;
        c.row += SR;
        c.rows_left -= SR;
        c.off += SR * cols;
    } else {                        // next item; may run past the last one: never used then
        cursor_set<REC, IR>(c, c.item + kWarpsPerCta, n_chunks, Rn, nt, s_rec, off0, cols);
    }
}

template <typename ST, typename MT, int NSTAGE>
__global__ void __launch_bounds__(kThreadsPerCta, 2) compress_group_kernel(const CompressGroupArgs a)
{
    constexpr int CPL = Store<ST>::CPL;
    constexpr int HB = CPL / 4;                          // Philox blocks under a warp-wide column block
    typedef PairRecord<HB> Rec;
    constexpr uint32_t REC = Rec::kBytes;
    constexpr uint32_t ES = sizeof(ST);
    constexpr uint32_t SR = GroupGeom<ST>::SR;             // rows per stage
    constexpr uint32_t IR = GroupGeom<ST>::IR;             // rows per item
    constexpr uint32_t kStash = GroupGeom<ST>::kStash;
    constexpr uint32_t kRingBytes = NSTAGE * SR * kSlotBytes;
    constexpr uint32_t kStageBytes = SR * kSlotBytes;
    typedef MTile<MT, CPL> MTl;
    extern __shared__ __align__(16) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
    const uint32_t ring = smem_s + threadIdx.x * 16;
    const uint32_t ring_end = ring + kRingBytes;
    const uint32_t stash = smem_s + kRingBytes;
    const uint32_t s_off = stash + kStash;               // per member: first element of its slot in M
    const uint32_t s_rec = s_off + kOffTableBytes;       // per (slot, task): PairRecord
    const uint32_t L = a.n_layers, nt = a.n_tasks;
    // where this lane's sign bits sit inside a record
    const uint32_t sign_word = Rec::kBlocks + (CPL == 4 ? (lane >> 3) * 4u : (lane >> 4) * 16u + ((lane & 15) >> 2) * 4u);
    const uint32_t sign_shift = CPL == 4 ? (lane & 7) * 4u : (lane & 3) * 8u;
    const uint32_t one = 0x3F800000u;

    // The unit list keeps kUnitChunk units of one (group, column block) next to each other (consecutive blocks of
    // rows), and a CTA takes whole chunks (see the loop): the tables below depend on the group, the column block and the tasks only,
    // so they are built once per chunk and every further unit of the chunk just refills the stash.
    uint32_t key_group = 0xFFFFFFFFu, key_cb = 0xFFFFFFFFu;
    uint32_t G = 0, cols = 0, c = 0;
    bool lane_on = false;
    // Whole rounds of chunks first (round r: CTA b takes chunk r * grid + b); what is left -- fewer than grid chunks --
    // is dealt out unit by unit, so that the last round is as short as one unit instead of one chunk.
    const uint32_t chunk_rounds = a.n_units / (kUnitChunk * gridDim.x);
    const uint32_t chunked_units = chunk_rounds * gridDim.x * kUnitChunk;
    const uint32_t my_chunked = chunk_rounds * kUnitChunk;
    const uint32_t my_units = my_chunked + (a.n_units - chunked_units > blockIdx.x ? (a.n_units - chunked_units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u);
    auto unit_at = [&](uint32_t t) {
        return t < my_chunked ? ((t / kUnitChunk) * gridDim.x + blockIdx.x) * kUnitChunk + t % kUnitChunk
                              : chunked_units + blockIdx.x + (t - my_chunked) * gridDim.x;
    };
    for (uint32_t t = 0; t < my_units; ++t) {
        const DevUnit un = a.units[unit_at(t)];
        const uint32_t Rn = un.nrows, row0 = un.row0;
        if (un.layer != key_group || un.cb0 != key_cb) {
            // ---- tables, all threads: per (slot, task) pair the source tensor and the sign bits; per member its slot's
            //      place in M and its W_0 tensor
            const uint32_t* mem = a.members + un.layer;
#ifdef RANDES_CHECKED
            // every member and every permuted source layer of the chunk must be a layer of the plan
            bool sound = checked(mem[0] < L, 4, kCheckLayer, unit_at(t));
            const uint32_t G_claimed = sound ? a.layers[mem[0]].group_size : 0;
            for (uint32_t ms = 0; sound && ms < G_claimed; ++ms) {
                sound = checked(mem[ms] < L, 4, kCheckLayer, unit_at(t));
                for (uint32_t i = 0; sound && i < nt; ++i)
                    sound = checked(!(a.layers[mem[ms]].flags & kFlagShuffle) || a.src_of_slot[static_cast<size_t>(i) * L + mem[ms]] < L, 4,
                                    kCheckPermuted, unit_at(t));
            }
            if (!sound) {       // nothing is copied, summed or stored for this chunk
                G = cols = 0;
                lane_on = false;
                key_group = un.layer;
                key_cb = un.cb0;
                continue;
            }
#endif
            const DevLayer l0 = a.layers[mem[0]];
            G = l0.group_size;
            cols = l0.cols;
            c = (un.cb0 * 32u + lane) * CPL;
            lane_on = c < cols;
            const uint32_t npairs = G * nt;
            for (uint32_t p = threadIdx.x; p < npairs; p += kThreadsPerCta) {
                const uint32_t ms = p / nt, i = p - ms * nt;
                const uint32_t slot = mem[ms];
                const uint32_t fl = a.layers[slot].flags;
                const uint32_t src = (fl & kFlagShuffle) ? a.src_of_slot[static_cast<size_t>(i) * L + slot] : slot;   // sigma_i(l)
                const void* pw = a.task_ptrs[static_cast<size_t>(i) * L + src];
                sts_ptrs(s_rec + p * REC + Rec::kPtr, pw, reinterpret_cast<const void*>(static_cast<uintptr_t>(a.layers[src].member)));
                const DevTask tk = a.tasks[i];
#pragma unroll
                for (int h = 0; h < HB; ++h) {
                    uint4 blk = make_uint4(0, 0, 0, 0);
                    if (fl & kFlagFlip) blk = philox4x32_10(un.cb0 * HB + h, slot, kTagSign, tk.id, tk.key0, tk.key1);
                    sts128(s_rec + p * REC + Rec::kBlocks + h * 16, blk);
                }
            }
            for (uint32_t ms = threadIdx.x; ms < G; ms += kThreadsPerCta)
                sts_ptrs(s_off + ms * 16, reinterpret_cast<const void*>(static_cast<uintptr_t>(a.layers[mem[ms]].m_off)), a.base[mem[ms]]);
            key_group = un.layer;
            key_cb = un.cb0;
            __syncthreads();   // the tables are complete and visible to every warp
        }
        const uint32_t off0 = row0 * cols + c;           // layers hold < 2^32 elements
#ifdef RANDES_CHECKED
        if (G == 0) continue;                            // a chunk that failed its check above
        const bool rows_ok = checked(row0 + Rn <= a.layers[a.members[un.layer]].rows, 4, kCheckRows, unit_at(t));
#else
        constexpr bool rows_ok = true;
#endif

        // ---- W_0 tiles of every member into the stash
        if (lane_on && rows_ok) {
            const uint32_t ntiles = G * Rn;
            for (uint32_t q = warp; q < ntiles; q += kWarpsPerCta) {
                const uint32_t m = q / Rn, r = q - m * Rn;
                const char* pb = lds_ptr(s_off + m * 16 + 8);
                cp_async16(stash + q * kStashTileBytes + lane * 16, pb + static_cast<size_t>(off0 + r * cols) * ES);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();   // the stash is complete and visible to every warp

        if (lane_on && rows_ok) {
            const uint32_t n_chunks = (Rn + IR - 1) / IR;
            const uint32_t n_items = G * n_chunks;
            uint32_t N = 0;   // stages of this warp
            for (uint32_t item = warp; item < n_items; item += kWarpsPerCta) {
                const uint32_t chunk = item % n_chunks;
                N += (min(IR, Rn - chunk * IR) + SR - 1) / SR * nt;
            }
            Cursor ci, cc;
            cursor_set<REC, IR>(ci, warp, n_chunks, Rn, nt, s_rec, off0, cols);
            cc = ci;
            uint32_t to_issue = N, stage_i = ring, stage_c = ring;
            const uint32_t stash_lane = stash + lane * 16;
            const uint32_t member_bytes = Rn * kStashTileBytes;
            const size_t row_bytes = static_cast<size_t>(cols) * ES;

            auto issue = [&]() {
                const char* src = lds_ptr(ci.rec + Rec::kPtr) + static_cast<size_t>(ci.off) * ES;
#pragma unroll
                for (uint32_t r = 0; r < SR; ++r)
                    if (r == 0 || ci.rows_left > r) cp_async16(stage_i + r * kSlotBytes, src + r * row_bytes);
                cursor_next<REC, IR, SR>(ci, n_chunks, Rn, nt, s_rec, off0, cols);
                stage_i += kStageBytes;
                if (stage_i == ring_end) stage_i = ring;
                --to_issue;
            };

#pragma unroll
            for (int s = 0; s < NSTAGE - 1; ++s) {
                if (to_issue) issue();
                cp_async_commit();
            }
            f32x2 acc[SR][CPL / 2];
            for (uint32_t it = 0; it < N; ++it) {
                if (to_issue) issue();
                cp_async_commit();
                cp_async_wait<NSTAGE - 1>();   // all but the newest NSTAGE-1 groups have landed: stage_c is ready
                if (cc.rec == cc.rec_begin) {
#pragma unroll
                    for (uint32_t r = 0; r < SR; ++r)
#pragma unroll
                        for (int e = 0; e < CPL / 2; ++e) acc[r][e] = 0ull;
                }
                const uint32_t member = lds_u32(cc.rec + Rec::kMember);
                const uint32_t bits = lds_u32(cc.rec + sign_word) >> sign_shift;
                f32x2 sg[CPL / 2];   // +-1.0f per column
#pragma unroll
                for (int e = 0; e < CPL / 2; ++e)
                    sg[e] = pack2(((bits << (31 - 2 * e)) & 0x80000000u) | one, ((bits << (30 - 2 * e)) & 0x80000000u) | one);
                const uint32_t b0 = stash_lane + member * member_bytes + cc.row * kStashTileBytes;
                const uint32_t rows_here = cc.rows_left;
#pragma unroll
                for (uint32_t r = 0; r < SR; ++r) {
                    if (r == 0 || rows_here > r) {
                        f32x2 d[CPL / 2], b[CPL / 2];
                        Store<ST>::widen2(lds128(stage_c + r * kSlotBytes), d);
                        Store<ST>::widen2(lds128(b0 + r * kStashTileBytes), b);
#pragma unroll
                        for (int e = 0; e < CPL / 2; ++e) acc[r][e] = fma2(sub2(d[e], b[e]), sg[e], acc[r][e]);
                    }
                }
                if (cc.rec + REC == cc.rec_end) {   // last task: the rows of this slot are complete
                    MT* mp = static_cast<MT*>(a.M) + lds_u64(cc.m_off) + cc.off;
#pragma unroll
                    for (uint32_t r = 0; r < SR; ++r) {
                        if (r == 0 || rows_here > r) {
                            float v[CPL];
#pragma unroll
                            for (int e = 0; e < CPL / 2; ++e) unpack2(acc[r][e], v[2 * e], v[2 * e + 1]);
                            MTl::store(mp + static_cast<size_t>(r) * cols, v);
                        }
                    }
                }
                cursor_next<REC, IR, SR>(cc, n_chunks, Rn, nt, s_rec, off0, cols);
                stage_c += kStageBytes;
                if (stage_c == ring_end) stage_c = ring;
            }
            cp_async_wait<0>();
        }
        __syncthreads();   // every warp is done with the stash and the tables before the next unit overwrites them
    }
}

template <typename T> struct Tag { typedef T type; };
template <typename F> int with_type(int dtype, F&& f) { return dtype == 0 ? f(Tag<float>{}) : f(Tag<bf16>{}); }
template <typename F> int with_stages(int nstage, F&& f)
{
    return nstage >= 6 ? f(std::integral_constant<int, 6>{})
                       : (nstage == 5 ? f(std::integral_constant<int, 5>{})
                                      : (nstage == 4 ? f(std::integral_constant<int, 4>{}) : f(std::integral_constant<int, 3>{})));
}

constexpr size_t kMaxDynamicSmem = 227 * 1024;
constexpr size_t kTwoCtaSmem = (228 * 1024 - 2 * 1024) / 2;   // two CTAs per SM, 1 KiB reserved for each

size_t group_smem_bytes(int storage_dtype, int nstage, uint32_t pair_cap)
{
    const size_t hb = storage_dtype == 1 ? 2 : 1;
    return static_cast<size_t>(nstage) * stage_rows(storage_dtype) * kSlotBytes + stash_bytes(storage_dtype) + kOffTableBytes +
           static_cast<size_t>(pair_cap) * (16 + 16 * hb);
}
// ring depths tried, deepest first.  fp32 weights: at most 6 stages of 2 rows.  bf16 weights: 4 stages of 3 rows fit beside the
// records of 20 tasks x 24 members; with fewer pairs the ring grows to 6 stages (72 KiB), which measured 1 % faster at 7 - 8 tasks
int max_stages(int storage_dtype) { (void)storage_dtype; return 6; }
int min_stages(int storage_dtype) { return storage_dtype == 1 ? 3 : 4; }

}  // namespace

RANDES_VIOLATION_READER(violation_in_group_kernel)

int compress_group_prepare(int storage_dtype, int m_dtype)
{
    return with_type(storage_dtype, [&](auto st) {
        return with_type(m_dtype, [&](auto mt) {
            typedef typename decltype(st)::type ST;
            typedef typename decltype(mt)::type MT;
            cudaError_t e = cudaFuncSetAttribute(compress_group_kernel<ST, MT, 6>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxDynamicSmem));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(compress_group_kernel<ST, MT, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxDynamicSmem));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(compress_group_kernel<ST, MT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxDynamicSmem));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(compress_group_kernel<ST, MT, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxDynamicSmem));
            if (e != cudaSuccess) (void)cudaGetLastError();
            return static_cast<int>(e);
        });
    });
}

bool compress_group_fits(int storage_dtype, uint32_t max_group, uint32_t n_tasks)
{
    return max_group >= 1 && max_group * kStashTileBytes <= stash_bytes(storage_dtype) &&
           group_smem_bytes(storage_dtype, min_stages(storage_dtype), max_group * n_tasks) <= kMaxDynamicSmem;
}

int launch_compress_groups(int storage_dtype, int m_dtype, const CompressGroupArgs& a, uint32_t max_group, int sm_count, void* stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t pair_cap = max_group * a.n_tasks;
    // the deepest ring that still leaves room for two CTAs per SM; failing that, the deepest ring with one
    int nstage = 0;
    for (int n = max_stages(storage_dtype); n >= min_stages(storage_dtype) && !nstage; --n)
        if (group_smem_bytes(storage_dtype, n, pair_cap) <= kTwoCtaSmem) nstage = n;
    for (int n = max_stages(storage_dtype); n >= min_stages(storage_dtype) && !nstage; --n)
        if (group_smem_bytes(storage_dtype, n, pair_cap) <= kMaxDynamicSmem) nstage = n;
    if (!nstage) return static_cast<int>(cudaErrorInvalidConfiguration);
    const size_t smem = group_smem_bytes(storage_dtype, nstage, pair_cap);
    return with_type(storage_dtype, [&](auto st) {
        return with_type(m_dtype, [&](auto mt) {
            return with_stages(nstage, [&](auto ns) {
                typedef typename decltype(st)::type ST;
                typedef typename decltype(mt)::type MT;
                constexpr int NS = decltype(ns)::value;
                int per_sm = 0;
                cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compress_group_kernel<ST, MT, NS>, kThreadsPerCta, smem);
                if (e != cudaSuccess) { (void)cudaGetLastError(); return static_cast<int>(e); }
                if (per_sm <= 0) return static_cast<int>(cudaErrorInvalidConfiguration);
                const int grid = static_cast<int>(std::min<uint64_t>(static_cast<uint64_t>(sm_count) * per_sm, a.n_units));
                compress_group_kernel<ST, MT, NS><<<grid, kThreadsPerCta, smem, s>>>(a);
                return static_cast<int>(cudaGetLastError());
            });
        });
    });
}

}  // namespace randes
