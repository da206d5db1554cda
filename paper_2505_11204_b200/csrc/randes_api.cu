// Host side of the RanDeS library: the C ABI, the plan (layer table, unit list,
// per-task permutation tables drawn from seeds), argument validation and the
// staging of pointer tables into the caller's device workspace.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#ifdef RANDES_NVTX
#include <nvtx3/nvToolsExt.h>
#endif

#include "../../include/randes.h"
#include "randes_internal.h"

using namespace randes;

namespace {

thread_local std::string g_error;
std::atomic<uint64_t> g_launches{0};

int fail(int code, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_error = buf;
    return code;
}

int fail_cuda(cudaError_t e, const char* what)
{
    return fail(RANDES_CUDA_ERROR, "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
}

// ---- random streams ----------------------------------------------------------------------
// Philox4x32-10 as published (SC'11): a 4-word counter is mixed by ten rounds;
// round = two 32x32->64 products whose halves are crossed with the other two
// counter words and the key; the key advances by a Weyl sequence per round.
struct Philox {
    uint32_t key[2];
    explicit Philox(uint64_t seed) { key[0] = static_cast<uint32_t>(seed); key[1] = static_cast<uint32_t>(seed >> 32); }
    void block(uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t out[4]) const
    {
        uint32_t x[4] = {a, b, c, d};
        uint32_t k[2] = {key[0], key[1]};
        for (int round = 0; round < 10; ++round) {
            const uint64_t left = 0xD2511F53ull * x[0];
            const uint64_t right = 0xCD9E8D57ull * x[2];
            const uint32_t y[4] = {static_cast<uint32_t>(right >> 32) ^ x[1] ^ k[0], static_cast<uint32_t>(right),
                                   static_cast<uint32_t>(left >> 32) ^ x[3] ^ k[1], static_cast<uint32_t>(left)};
            std::memcpy(x, y, sizeof x);
            k[0] += 0x9E3779B9u;
            k[1] += 0xBB67AE85u;
        }
        std::memcpy(out, x, sizeof x);
    }
};

// sigma ~ S_G for (task, group): Fisher-Yates from the last position down; the
// r-th random word of the (group, task) stream picks j in [0, k] as (word*(k+1)) >> 32.
void draw_sigma(uint64_t seed, uint32_t task_id, uint32_t group, uint32_t G, std::vector<uint32_t>& sigma)
{
    sigma.resize(G);
    for (uint32_t k = 0; k < G; ++k) sigma[k] = k;
    const Philox rng(seed);
    uint32_t words[4];
    uint32_t drawn = 0;
    for (uint32_t k = G; k > 1; --k) {
        if ((drawn & 3u) == 0) rng.block(drawn >> 2, group, kTagPerm, task_id, words);
        const uint32_t word = words[drawn & 3u];
        ++drawn;
        const uint32_t j = static_cast<uint32_t>((static_cast<uint64_t>(word) * k) >> 32);
        std::swap(sigma[k - 1], sigma[j]);
    }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct TaskEntry {
    uint32_t id;
    uint64_t seed;
    std::vector<uint32_t> src_of_slot;   // sigma over the whole layer list
    std::vector<uint32_t> slot_of_pos;   // sigma^-1
};

struct WorkspaceLayout {
    size_t layers, units, tasks, src_of_slot, slot_of_pos, base_ptrs, out_ptrs, task_ptrs, members, staged_units, total;
    size_t ctx_off = 0, ctx_table = 0;   // plans with a general diagonal context only (appended after `total` is first set)
};

// floats per task row of the context table: every layer's columns, each span padded to a multiple of four
size_t context_stride(const randes_layer_t* layers, uint32_t n_layers)
{
    size_t n = 0;
    for (uint32_t l = 0; l < n_layers; ++l) n += align_up(static_cast<size_t>(layers[l].cols), 4);
    return n;
}

// append the column offsets and the factor table of a general diagonal context to a layout
void layout_context(WorkspaceLayout& w, const randes_layer_t* layers, uint32_t n_layers, size_t max_tasks)
{
    size_t off = align_up(w.total, 256);
    w.ctx_off = off;
    off = align_up(off + n_layers * sizeof(uint32_t), 256);
    w.ctx_table = off;
    off = align_up(off + max_tasks * context_stride(layers, n_layers) * sizeof(float), 256);
    w.total = off;
}

WorkspaceLayout layout_workspace(size_t n_layers, size_t n_units, size_t n_staged_units, size_t max_tasks)
{
    WorkspaceLayout w;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    w.layers = take(n_layers * sizeof(DevLayer));
    w.units = take(n_units * sizeof(DevUnit));
    w.tasks = take(max_tasks * sizeof(DevTask));
    w.src_of_slot = take(max_tasks * n_layers * sizeof(uint32_t));
    w.slot_of_pos = take(max_tasks * n_layers * sizeof(uint32_t));
    w.base_ptrs = take(n_layers * sizeof(void*));
    w.out_ptrs = take(n_layers * sizeof(void*));
    w.task_ptrs = take(max_tasks * n_layers * sizeof(void*));
    w.members = take(n_layers * sizeof(uint32_t));
    w.staged_units = take(n_staged_units * sizeof(DevUnit));
    w.total = off;
    return w;
}

// Units in group order; inside a group, all members at one (row block, column
// chunk) are adjacent, so that tiles of W_0 which several slots read (under a
// shuffle) are touched close together in time and stay in L2.
//
// With `staged` (one flag per group) the flagged groups are cut into group units
// instead: one unit = a few rows x one warp-wide column block of every member,
// whose W_0 tiles the CTA stages in shared memory (`member_base[g]` = index of
// the group's first entry in the member table).  `which` selects the groups that
// are listed at all.  `per_group`, if given, receives the number of units of each
// group (indexed by group id).
enum { kAllGroups = 0, kStagedGroups = 1, kOtherGroups = 2 };
void build_units(const randes_layer_t* layers, uint32_t n_layers, int storage, std::vector<DevUnit>& units,
                 const std::vector<char>* staged = nullptr, const std::vector<uint32_t>* member_base = nullptr,
                 int which = kAllGroups, std::vector<size_t>* per_group = nullptr, uint32_t rows_per_warp = kRowsPerWarp)
{
    const uint32_t wcols = cols_per_warp(storage);
    units.clear();
    std::vector<char> done(n_layers, 0);
    std::vector<uint32_t> members;
    for (uint32_t first = 0; first < n_layers; ++first) {
        if (done[first]) continue;
        const uint32_t g = layers[first].group;
        members.clear();
        for (uint32_t l = first; l < n_layers; ++l)
            if (!done[l] && layers[l].group == g) { members.push_back(l); done[l] = 1; }
        const uint32_t rows = layers[first].rows, cols = layers[first].cols;
        if (rows == 0 || cols == 0) continue;
        const bool is_staged = staged && (*staged)[g];
        if ((which == kStagedGroups && !is_staged) || (which == kOtherGroups && is_staged)) continue;
        const size_t before = units.size();
        const uint32_t nb = (cols + wcols - 1) / wcols;
        if (is_staged) {
            // kUnitChunk consecutive blocks of rows of one column block lie next to each other (a CTA takes them together
            // and builds its per-(group, column block) tables once); the column blocks of such a band of rows follow, so
            // that CTAs working side by side read neighbouring pieces of the same rows
            const uint32_t R = group_unit_rows(static_cast<uint32_t>(members.size()), storage);
            const uint32_t band = R * kUnitChunk;
            for (uint32_t band0 = 0; band0 < rows; band0 += band)
                for (uint32_t cb0 = 0; cb0 < nb; ++cb0)
                    for (uint32_t r0 = band0; r0 < std::min(rows, band0 + band); r0 += R) {
                        DevUnit u;
                        u.layer = (*member_base)[g];
                        u.row0 = r0;
                        u.nrows = std::min(R, rows - r0);
                        u.cb0 = static_cast<uint16_t>(cb0);
                        u.nbc = 0;
                        units.push_back(u);
                    }
        } else {
            uint32_t nbc = 1;
            while (nbc < static_cast<uint32_t>(kWarpsPerCta) && nb % (nbc * 2) == 0) nbc *= 2;
            const uint32_t rows_per_unit = rows_per_warp * (kWarpsPerCta / nbc);
            for (uint32_t r0 = 0; r0 < rows; r0 += rows_per_unit)
                for (uint32_t cb0 = 0; cb0 < nb; cb0 += nbc)
                    for (uint32_t l : members) {
                        DevUnit u;
                        u.layer = l;
                        u.row0 = r0;
                        u.nrows = std::min(rows_per_unit, rows - r0);
                        u.cb0 = static_cast<uint16_t>(cb0);
                        u.nbc = static_cast<uint16_t>(nbc);
                        units.push_back(u);
                    }
        }
        if (per_group) {
            if (per_group->size() <= g) per_group->resize(g + 1, 0);
            (*per_group)[g] += units.size() - before;
        }
    }
}

// Could group g (of `size` members, `cols` wide) be cut into group units at all?
bool group_fits_stash(size_t size, uint32_t cols, int storage)
{
    return size >= 1 && cols % cols_per_lane(storage) == 0 && group_unit_rows(static_cast<uint32_t>(size), storage) >= 1;
}

// Upper bound of the length of a unit list in which any subset of the groups is staged.
size_t max_mixed_units(const randes_layer_t* layers, uint32_t n_layers, int storage)
{
    uint32_t n_groups = 0;
    for (uint32_t l = 0; l < n_layers; ++l) n_groups = std::max(n_groups, layers[l].group + 1);
    std::vector<size_t> size(n_groups, 0);
    std::vector<uint32_t> cols(n_groups, 0), base(n_groups, 0);
    for (uint32_t l = 0; l < n_layers; ++l) { ++size[layers[l].group]; cols[layers[l].group] = layers[l].cols; }
    std::vector<char> staged(n_groups, 0);
    for (uint32_t g = 0; g < n_groups; ++g) staged[g] = group_fits_stash(size[g], cols[g], storage);
    std::vector<DevUnit> units;
    std::vector<size_t> plain(n_groups, 0), mixed(n_groups, 0);
    build_units(layers, n_layers, storage, units, nullptr, nullptr, kAllGroups, &plain);
    build_units(layers, n_layers, storage, units, &staged, &base, kAllGroups, &mixed);
    size_t total = 0;
    for (uint32_t g = 0; g < n_groups; ++g) total += std::max(g < plain.size() ? plain[g] : 0, g < mixed.size() ? mixed[g] : 0);
    return total;
}

int check_layers(const randes_layer_t* layers, uint32_t n_layers)
{
    if (!layers || n_layers == 0) return fail(RANDES_INVALID_ARGUMENT, "layers is NULL or empty");
    for (uint32_t l = 0; l < n_layers; ++l)
    {
        if (layers[l].cols > 65535u * 128u)
            return fail(RANDES_INVALID_ARGUMENT, "layer %u: cols %u exceeds the supported %u", l, layers[l].cols,
                        65535u * 128u);
        // the kernels index inside a layer with 32-bit element offsets
        if (static_cast<unsigned long long>(layers[l].rows) * layers[l].cols > 0xFFFFFFFFull)
            return fail(RANDES_INVALID_ARGUMENT, "layer %u: %u x %u elements exceed the supported 2^32 - 1 per layer", l,
                        layers[l].rows, layers[l].cols);
    }
    return RANDES_OK;
}

}  // namespace

struct randes_plan_s {
    uint32_t n_layers = 0, n_groups = 0, max_tasks = 0;
    int storage = RANDES_F32;
    int m_dtype = RANDES_F32;                     // element type of the superposition arena
    std::vector<randes_layer_t> layers;
    std::vector<uint32_t> gflags;
    bool has_gauss = false;                       // some group carries the Gaussian-like context: every call takes the plain kernels
    uint32_t ctx_stride = 0, max_cols = 0;        // has_gauss: floats per task row of the factor table; widest layer
    std::vector<std::vector<uint32_t>> members;   // per group, in layer order
    std::vector<DevLayer> dev_layers;
    std::vector<DevUnit> units;
    // compress: the shuffled groups cut into group units (their W_0 tiles are staged in shared
    // memory), the other groups as in `units`; both empty when no group qualifies.
    // member table = layers of every group, group after group
    std::vector<DevUnit> group_units, other_units;
    std::vector<char> group_staged;
    std::vector<uint32_t> member_table;
    uint32_t max_staged_group = 0;
    std::vector<size_t> m_off_bytes;
    size_t m_bytes = 0;
    std::vector<TaskEntry> tasks;                 // summation order
    // device side
    char* ws = nullptr;
    WorkspaceLayout lay{};
    int sm_count = 0;
    int grid_acc[2] = {0, 0};   // [0] compress, [1] one task (add / remove)
    int grid_ret[2] = {0, 0};
    int grid_gram = 0;
    // host mirrors of what the device pointer tables currently hold
    std::vector<const void*> h_base, h_out, h_tasks;
    std::vector<DevTask> h_dev_tasks;
    bool base_valid = false, out_valid = false;
    size_t tasks_valid = 0;
    const void* checked_m = nullptr;              // M and output element size of the last retrieve whose tensors were found disjoint
    size_t checked_out_elem = 0;

    template <typename T> T* dev(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace {

// the members of group g that the skip rate selects (every k-th, in layer order)
std::vector<uint32_t> participants(const randes_plan_t& p, uint32_t g)
{
    const uint32_t k = std::max<uint32_t>(1, (p.gflags[g] >> 8) & 0xFFu);
    std::vector<uint32_t> out;
    for (size_t j = 0; j < p.members[g].size(); j += k) out.push_back(p.members[g][j]);
    return out;
}

void make_task_tables(const randes_plan_t& p, TaskEntry& t)
{
    t.src_of_slot.resize(p.n_layers);
    t.slot_of_pos.resize(p.n_layers);
    for (uint32_t l = 0; l < p.n_layers; ++l) t.src_of_slot[l] = t.slot_of_pos[l] = l;
    std::vector<uint32_t> sigma;
    for (uint32_t g = 0; g < p.n_groups; ++g) {
        const std::vector<uint32_t> mem = participants(p, g);
        if (mem.size() < 2) continue;
        const uint32_t n = static_cast<uint32_t>(mem.size());
        if (p.gflags[g] & RANDES_SHUFFLE) {
            draw_sigma(t.seed, t.id, g, n, sigma);
        } else if (p.gflags[g] & RANDES_SHIFT) {
            // rotate towards higher index by `shift`: slot k receives member k - shift
            const uint32_t shift = 1u + t.id % (n - 1u);
            sigma.resize(n);
            for (uint32_t k = 0; k < n; ++k) sigma[k] = (k + n - shift) % n;
        } else {
            continue;
        }
        for (size_t k = 0; k < mem.size(); ++k) {
            t.src_of_slot[mem[k]] = mem[sigma[k]];     // slot k receives member sigma(k)
            t.slot_of_pos[mem[sigma[k]]] = mem[k];
        }
    }
}

int find_task(const randes_plan_t& p, uint32_t id)
{
    for (size_t i = 0; i < p.tasks.size(); ++i)
        if (p.tasks[i].id == id) return static_cast<int>(i);
    return -1;
}

// the factor table of a plan with a general diagonal context, seen from task row `row`
ContextArgs context_args(const randes_plan_t& p, size_t row)
{
    ContextArgs x;
    x.table = p.dev<float>(p.lay.ctx_table) + row * p.ctx_stride;
    x.off = p.dev<uint32_t>(p.lay.ctx_off);
    x.stride = p.ctx_stride;
    return x;
}

// copy task rows [first, end) (descriptors + both tables) to the device
int upload_task_rows(randes_plan_t& p, size_t first, cudaStream_t s)
{
    const size_t L = p.n_layers;
    p.h_dev_tasks.resize(p.max_tasks);
    for (size_t i = first; i < p.tasks.size(); ++i) {
        const TaskEntry& t = p.tasks[i];
        DevTask d;
        d.id = t.id;
        d.key0 = static_cast<uint32_t>(t.seed);
        d.key1 = static_cast<uint32_t>(t.seed >> 32);
        d.pad = 0;
        p.h_dev_tasks[i] = d;
        cudaError_t e = cudaMemcpyAsync(p.dev<uint32_t>(p.lay.src_of_slot) + i * L, t.src_of_slot.data(),
                                        L * sizeof(uint32_t), cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(p.dev<uint32_t>(p.lay.slot_of_pos) + i * L, t.slot_of_pos.data(), L * sizeof(uint32_t),
                                cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return fail_cuda(e, "copy of task tables");
    }
    if (first < p.tasks.size()) {
        cudaError_t e = cudaMemcpyAsync(p.dev<DevTask>(p.lay.tasks) + first, p.h_dev_tasks.data() + first,
                                        (p.tasks.size() - first) * sizeof(DevTask), cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return fail_cuda(e, "copy of task descriptors");
        if (p.has_gauss) {   // the factors of these tasks, once, for every later call
            const int ce = launch_context_fill(context_args(p, 0), p.dev<DevLayer>(p.lay.layers), p.n_layers, p.max_cols, p.dev<DevTask>(p.lay.tasks),
                                               static_cast<uint32_t>(first), static_cast<uint32_t>(p.tasks.size() - first), s);
            if (ce) return fail_cuda(static_cast<cudaError_t>(ce), "launch of the context table kernel");
            ++g_launches;
        }
    }
    return RANDES_OK;
}

int check_ptrs(const randes_plan_t& p, const void* const* ptrs, const char* what, size_t elem, bool allow_null_array)
{
    if (!ptrs) return allow_null_array ? RANDES_OK : fail(RANDES_INVALID_ARGUMENT, "%s is NULL", what);
    for (uint32_t l = 0; l < p.n_layers; ++l) {
        const bool empty = p.layers[l].rows == 0 || p.layers[l].cols == 0;
        if (!ptrs[l] && !empty) return fail(RANDES_INVALID_ARGUMENT, "%s[%u] is NULL", what, l);
        if (reinterpret_cast<uintptr_t>(ptrs[l]) % elem)
            return fail(RANDES_MISALIGNED, "%s[%u] = %p is not aligned to %zu bytes", what, l, ptrs[l], elem);
    }
    return RANDES_OK;
}

// bring a device pointer table up to date; skips the copy when nothing changed
int stage_ptrs(randes_plan_t& p, std::vector<const void*>& mirror, bool& valid, size_t dev_off, const void* const* ptrs,
               cudaStream_t s)
{
    const size_t L = p.n_layers;
    if (valid && std::memcmp(mirror.data(), ptrs, L * sizeof(void*)) == 0) return RANDES_OK;
    mirror.assign(ptrs, ptrs + L);
    valid = true;
    cudaError_t e = cudaMemcpyAsync(p.ws + dev_off, mirror.data(), L * sizeof(void*), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) { valid = false; return fail_cuda(e, "copy of pointer table"); }
    return RANDES_OK;
}

int stage_task_ptrs(randes_plan_t& p, const void* const* ptrs, size_t n_tasks, cudaStream_t s)
{
    const size_t n = n_tasks * p.n_layers;
    if (p.tasks_valid == n && std::memcmp(p.h_tasks.data(), ptrs, n * sizeof(void*)) == 0) return RANDES_OK;
    if (p.h_tasks.size() < n) p.h_tasks.resize(static_cast<size_t>(p.max_tasks) * p.n_layers);
    std::memcpy(p.h_tasks.data(), ptrs, n * sizeof(void*));
    p.tasks_valid = n;
    cudaError_t e = cudaMemcpyAsync(p.ws + p.lay.task_ptrs, p.h_tasks.data(), n * sizeof(void*), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) { p.tasks_valid = 0; return fail_cuda(e, "copy of task pointer table"); }
    return RANDES_OK;
}

size_t elem_size(int dtype) { return dtype == RANDES_BF16 ? 2 : 4; }

int check_m(const void* M)
{
    if (!M) return fail(RANDES_INVALID_ARGUMENT, "M is NULL");
    if (reinterpret_cast<uintptr_t>(M) % 256) return fail(RANDES_MISALIGNED, "M = %p is not 256-byte aligned", M);
    return RANDES_OK;
}

int run_accumulate(randes_plan_t& p, size_t first_row, size_t n_rows, bool init_from_m, bool negate,
                   const void* const* base, const void* const* task_ptrs, void* M, cudaStream_t s)
{
    int rc;
    if (base && (rc = stage_ptrs(p, p.h_base, p.base_valid, p.lay.base_ptrs, base, s))) return rc;
    if ((rc = stage_task_ptrs(p, task_ptrs, n_rows, s))) return rc;
    AccumulateArgs a;
    a.layers = p.dev<DevLayer>(p.lay.layers);
    a.units = p.dev<DevUnit>(p.lay.units);
    a.n_units = static_cast<uint32_t>(p.units.size());
    // Compress from zero under a shuffle: the shuffled groups go to the group kernel, which needs W_0,
    // all tasks in one chunk, room for its tables, and 16-byte aligned tensors in those groups.
    bool staged = !init_from_m && n_rows >= 2 && n_rows <= static_cast<size_t>(kTaskChunk) && base != nullptr &&
                  !p.group_units.empty() && compress_group_fits(p.storage, p.max_staged_group, static_cast<uint32_t>(n_rows));
    for (uint32_t l = 0; staged && l < p.n_layers; ++l) {
        if (!p.group_staged[p.layers[l].group]) continue;
        staged = reinterpret_cast<uintptr_t>(base[l]) % 16 == 0;
        for (size_t i = 0; staged && i < n_rows; ++i) staged = reinterpret_cast<uintptr_t>(task_ptrs[i * p.n_layers + l]) % 16 == 0;
    }
    if (staged) {
        a.units = p.dev<DevUnit>(p.lay.staged_units);
        a.n_units = static_cast<uint32_t>(p.other_units.size());
    }
    a.n_layers = p.n_layers;
    a.src_of_slot = p.dev<uint32_t>(p.lay.src_of_slot) + first_row * p.n_layers;
    a.tasks = p.dev<DevTask>(p.lay.tasks) + first_row;
    a.n_tasks = static_cast<uint32_t>(n_rows);
    a.init_from_m = init_from_m;
    a.negate = negate;
    a.has_base = base != nullptr;
    a.base = p.dev<const void*>(p.lay.base_ptrs);
    a.task_ptrs = p.dev<const void*>(p.lay.task_ptrs);
    a.M = M;
    if (p.has_gauss) {
        if (a.n_units == 0) return RANDES_OK;
        const int e = launch_context_accumulate(p.storage, a, context_args(p, first_row), s);
        if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the general-context accumulate kernel");
        ++g_launches;
        return RANDES_OK;
    }
    if (staged) {
        CompressGroupArgs g;
        g.layers = a.layers;
        g.units = p.dev<DevUnit>(p.lay.staged_units) + p.other_units.size();
        g.n_units = static_cast<uint32_t>(p.group_units.size());
        g.n_layers = p.n_layers;
        g.src_of_slot = a.src_of_slot;
        g.tasks = a.tasks;
        g.n_tasks = a.n_tasks;
        g.base = a.base;
        g.task_ptrs = a.task_ptrs;
        g.M = M;
        g.members = p.dev<uint32_t>(p.lay.members);
        const int e = launch_compress_groups(p.storage, p.m_dtype, g, p.max_staged_group, p.sm_count, s);
        if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the group compress kernel");
        ++g_launches;
    }
    if (a.n_units == 0) return RANDES_OK;
    // one model, bf16 weights, fp32 superposition: the kernel whose requests are contiguous across a warp,
    // when every layer's width and every tensor's alignment allow it
    bool halves = n_rows == 1 && init_from_m && p.storage == RANDES_BF16 && p.m_dtype == RANDES_F32;
    for (uint32_t l = 0; halves && l < p.n_layers; ++l) {
        if (p.layers[l].rows == 0 || p.layers[l].cols == 0) continue;
        halves = p.layers[l].cols % 8 == 0 && reinterpret_cast<uintptr_t>(task_ptrs[l]) % 16 == 0 &&
                 (!base || reinterpret_cast<uintptr_t>(base[l]) % 16 == 0);
    }
    if (halves) {
        const int he = launch_add_halves(a, p.sm_count, s);
        if (he) return fail_cuda(static_cast<cudaError_t>(he), "launch of the add / remove kernel");
        ++g_launches;
        return RANDES_OK;
    }
    const int grid = std::min<int>(p.grid_acc[n_rows == 1], static_cast<int>(a.n_units));
    const int e = launch_accumulate(p.storage, p.m_dtype, a, grid, s);
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the accumulate kernel");
    ++g_launches;
    return RANDES_OK;
}

// The outputs of a retrieve may overlap neither the base tensors, nor M, nor each other (an output element is
// written by one thread while others still read their inputs).  Byte ranges, so that partial overlaps are caught
// too: the ranges of all tensors are sorted by their start and swept once.
int check_outputs_disjoint(const randes_plan_t& p, const void* const* base, const void* const* out, size_t n_out_models,
                           size_t out_elem, const void* M)
{
    struct Range { uintptr_t lo, hi; uint32_t layer; int kind; };   // kind: 0 base, 1 M, 2 + b output of model b
    std::vector<Range> r;
    r.reserve((n_out_models + 1) * p.n_layers + 1);
    for (uint32_t l = 0; l < p.n_layers; ++l) {
        const size_t elems = static_cast<size_t>(p.layers[l].rows) * p.layers[l].cols;
        if (!elems) continue;
        const uintptr_t b = reinterpret_cast<uintptr_t>(base[l]);
        r.push_back({b, b + elems * elem_size(p.storage), l, 0});
        for (size_t m = 0; m < n_out_models; ++m) {
            const uintptr_t o = reinterpret_cast<uintptr_t>(out[m * p.n_layers + l]);
            r.push_back({o, o + elems * out_elem, l, static_cast<int>(2 + m)});
        }
    }
    const uintptr_t m0 = reinterpret_cast<uintptr_t>(M);
    r.push_back({m0, m0 + p.m_bytes, 0, 1});
    std::sort(r.begin(), r.end(), [](const Range& a, const Range& b) { return a.lo < b.lo; });
    uintptr_t reach = 0;          // furthest end seen so far, and whose it is
    const Range* owner = nullptr;
    for (const Range& x : r) {
        if (owner && x.lo < reach && (x.kind >= 2 || owner->kind >= 2)) {
            const Range& o = x.kind >= 2 ? x : *owner;
            const Range& other = x.kind >= 2 ? *owner : x;
            return fail(RANDES_INVALID_ARGUMENT, "out[%d][%u] overlaps %s", o.kind - 2, o.layer,
                        other.kind == 0 ? "a base tensor" : (other.kind == 1 ? "M" : "another output tensor"));
        }
        if (x.hi > reach) { reach = x.hi; owner = &x; }
    }
    return RANDES_OK;
}

// Built with -DRANDES_NVTX every computing entry point is bracketed by an NVTX range named after it, so that
// a timeline shows which call enqueued which kernels.  Off by default: the header is not even included.
#ifdef RANDES_NVTX
struct CallRange {
    explicit CallRange(const char* name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
};
#else
struct CallRange {
    explicit CallRange(const char*) {}
};
#endif

// Runs the body of an entry point; nothing may cross the C ABI as an exception.
template <typename F> int guarded(const char* name, F&& body)
{
    const CallRange range(name);
    try {
        return body();
    } catch (const std::bad_alloc&) {
        return fail(RANDES_OUT_OF_MEMORY, "host allocation failed");
    } catch (...) {
        return fail(RANDES_INVALID_ARGUMENT, "unexpected internal error");
    }
}

}  // namespace

extern "C" {

const char* randes_last_error(void) { return g_error.c_str(); }

uint64_t randes_launch_count(void) { return g_launches.load(); }

size_t randes_plan_workspace_bytes(const randes_layer_t* layers, uint32_t n_layers, uint32_t max_tasks)
{
    if (check_layers(layers, n_layers) || max_tasks == 0) return 0;
    // the unit list depends on the storage type, which is not known here: take the larger
    std::vector<DevUnit> units;
    build_units(layers, n_layers, RANDES_F32, units);
    size_t n_units = units.size();
    build_units(layers, n_layers, RANDES_BF16, units);
    n_units = std::max(n_units, units.size());
    const size_t n_staged = std::max(max_mixed_units(layers, n_layers, RANDES_F32), max_mixed_units(layers, n_layers, RANDES_BF16));
    return layout_workspace(n_layers, n_units, n_staged, max_tasks).total;
}

size_t randes_plan_workspace_bytes_groups(const randes_layer_t* layers, uint32_t n_layers, const randes_group_t* groups, uint32_t n_groups,
                                          uint32_t max_tasks)
{
    const size_t plain = randes_plan_workspace_bytes(layers, n_layers, max_tasks);
    if (plain == 0 || !groups) return plain;
    bool gauss = false;
    for (uint32_t g = 0; g < n_groups; ++g) gauss = gauss || (groups[g].flags & RANDES_GAUSS);
    if (!gauss) return plain;
    if (context_stride(layers, n_layers) > 0xFFFFFFFFull) return 0;
    WorkspaceLayout w{};
    w.total = plain;
    layout_context(w, layers, n_layers, max_tasks);
    return w.total;
}

int randes_plan(const randes_layer_t* layers, uint32_t n_layers, const randes_group_t* groups, uint32_t n_groups,
                randes_dtype_t storage_dtype, randes_dtype_t m_dtype, const uint32_t* task_ids, const uint64_t* seeds, uint32_t n_tasks,
                uint32_t max_tasks, void* dev_workspace, size_t dev_workspace_bytes, void* stream,
                randes_plan_t** out_plan)
{
    if (!out_plan) return fail(RANDES_INVALID_ARGUMENT, "out_plan is NULL");
    *out_plan = nullptr;
    int rc = check_layers(layers, n_layers);
    if (rc) return rc;
    if (!groups || n_groups == 0) return fail(RANDES_INVALID_ARGUMENT, "groups is NULL or empty");
    if (storage_dtype != RANDES_F32 && storage_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "storage dtype %d is not supported", static_cast<int>(storage_dtype));
    if (m_dtype != RANDES_F32 && m_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "superposition dtype %d is not supported", static_cast<int>(m_dtype));
    if (max_tasks == 0 || n_tasks > max_tasks)
        return fail(RANDES_INVALID_ARGUMENT, "max_tasks = %u must be >= max(1, n_tasks = %u)", max_tasks, n_tasks);
    if (n_tasks && (!task_ids || !seeds)) return fail(RANDES_INVALID_ARGUMENT, "task_ids / seeds is NULL");
    for (uint32_t g = 0; g < n_groups; ++g)
    {
        if (groups[g].flags & ~static_cast<uint32_t>(RANDES_SHUFFLE | RANDES_FLIP | RANDES_SHIFT | RANDES_SKIP(0xFF) | RANDES_GAUSS))
            return fail(RANDES_INVALID_ARGUMENT, "group %u: unknown flag bits 0x%x", g, groups[g].flags);
        if ((groups[g].flags & RANDES_SHUFFLE) && (groups[g].flags & RANDES_SHIFT))
            return fail(RANDES_INVALID_ARGUMENT, "group %u: RANDES_SHUFFLE and RANDES_SHIFT exclude each other", g);
        if ((groups[g].flags & RANDES_FLIP) && (groups[g].flags & RANDES_GAUSS))
            return fail(RANDES_INVALID_ARGUMENT, "group %u: RANDES_FLIP and RANDES_GAUSS exclude each other", g);
        if ((groups[g].flags & RANDES_GAUSS) && m_dtype != RANDES_F32)
            return fail(RANDES_UNSUPPORTED_DTYPE, "group %u: RANDES_GAUSS needs an fp32 superposition", g);
    }
    for (uint32_t i = 0; i < n_tasks; ++i)
        for (uint32_t j = 0; j < i; ++j)
            if (task_ids[i] == task_ids[j]) return fail(RANDES_DUPLICATE_TASK, "task id %u appears twice", task_ids[i]);

    randes_plan_t* p = new (std::nothrow) randes_plan_t;
    if (!p) return fail(RANDES_OUT_OF_MEMORY, "host allocation failed");
    try {
        p->n_layers = n_layers;
        p->n_groups = n_groups;
        p->max_tasks = max_tasks;
        p->storage = storage_dtype;
        p->m_dtype = m_dtype;
        p->layers.assign(layers, layers + n_layers);
        p->gflags.resize(n_groups);
        for (uint32_t g = 0; g < n_groups; ++g) {
            p->gflags[g] = groups[g].flags;
            p->has_gauss = p->has_gauss || (groups[g].flags & RANDES_GAUSS);
        }
        p->members.assign(n_groups, {});
        for (uint32_t l = 0; l < n_layers; ++l) {
            if (layers[l].group >= n_groups) {
                delete p;
                return fail(RANDES_INVALID_ARGUMENT, "layer %u: group %u out of range (n_groups = %u)", l, layers[l].group,
                            n_groups);
            }
            const std::vector<uint32_t>& mem = p->members[layers[l].group];
            if (!mem.empty() && (layers[mem[0]].rows != layers[l].rows || layers[mem[0]].cols != layers[l].cols)) {
                const uint32_t first = mem[0];   // `mem` dies with the plan
                delete p;
                return fail(RANDES_SHAPE_MISMATCH, "group %u: layer %u is %ux%u but layer %u is %ux%u", layers[l].group, l,
                            layers[l].rows, layers[l].cols, first, layers[first].rows, layers[first].cols);
            }
            p->members[layers[l].group].push_back(l);
        }
        p->dev_layers.resize(n_layers);
        p->m_off_bytes.resize(n_layers);
        // The first slot starts 1 KiB into the arena.  Callers often keep a model's layers packed in one arena in layer
        // order with 256-byte alignment -- the very layout M has -- and allocators hand out large arenas on 2 MiB
        // boundaries: W_0[l] and M[l] would then sit at equal addresses modulo every power of two up to 2 MiB, and the
        // two read streams of retrieve collide in DRAM (measured: 1.6 % slower; any offset of 1 KiB or more cures it).
        size_t off = kSuperpositionLeadIn;
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint32_t g = layers[l].group;
            const std::vector<uint32_t>& mem = p->members[g];
            DevLayer d;
            d.m_off = off / elem_size(m_dtype);
            d.rows = layers[l].rows;
            d.cols = layers[l].cols;
            d.group = g;
            d.member = static_cast<uint32_t>(std::find(mem.begin(), mem.end(), l) - mem.begin());
            const uint32_t skip = std::max<uint32_t>(1, (p->gflags[g] >> 8) & 0xFFu);
            const bool takes_part = d.member % skip == 0;
            const size_t n_part = (mem.size() + skip - 1) / skip;
            d.flags = ((p->gflags[g] & RANDES_FLIP) && takes_part ? kFlagFlip : 0u) |
                      ((p->gflags[g] & RANDES_GAUSS) && takes_part ? kFlagGauss : 0u) |
                      ((p->gflags[g] & (RANDES_SHUFFLE | RANDES_SHIFT)) && takes_part && n_part >= 2 ? kFlagShuffle : 0u);
            d.group_size = static_cast<uint32_t>(mem.size());
            p->dev_layers[l] = d;
            p->m_off_bytes[l] = off;
            off = align_up(off + static_cast<size_t>(layers[l].rows) * layers[l].cols * elem_size(m_dtype), 256);
        }
        p->m_bytes = off;
        build_units(layers, n_layers, p->storage, p->units);
        {
            std::vector<uint32_t> member_base(n_groups, 0);
            p->group_staged.assign(n_groups, 0);
            bool any = false;
            for (uint32_t g = 0; g < n_groups; ++g) {
                const std::vector<uint32_t>& mem = p->members[g];
                member_base[g] = static_cast<uint32_t>(p->member_table.size());
                p->member_table.insert(p->member_table.end(), mem.begin(), mem.end());
                if (mem.empty() || !group_fits_stash(mem.size(), layers[mem[0]].cols, p->storage)) continue;
                bool shuffled = false;
                for (uint32_t l : mem) shuffled = shuffled || (p->dev_layers[l].flags & kFlagShuffle);
                // bf16 weights and many tasks: the group kernel decodes a task's signs once per three rows and is the faster
                // one even without a shuffle, so the large unrepeated matrices go through it too.  With few tasks a warp's
                // pipeline over one member's rows is too short to fill (measured: slower at 7 tasks, faster at 20), so
                // the choice follows the number of tasks registered when the plan is built.
                const bool large_single = p->storage == RANDES_BF16 && mem.size() == 1 && layers[mem[0]].rows >= 256 && n_tasks >= 16;
                const bool stage = shuffled || large_single;
                p->group_staged[g] = stage;
                any = any || stage;
                if (stage) p->max_staged_group = std::max<uint32_t>(p->max_staged_group, static_cast<uint32_t>(mem.size()));
            }
            if (any && !p->has_gauss) {
                build_units(layers, n_layers, p->storage, p->group_units, &p->group_staged, &member_base, kStagedGroups);
                build_units(layers, n_layers, p->storage, p->other_units, &p->group_staged, &member_base, kOtherGroups);
            }
        }
        p->tasks.resize(n_tasks);
        for (uint32_t i = 0; i < n_tasks; ++i) {
            p->tasks[i].id = task_ids[i];
            p->tasks[i].seed = seeds[i];
            make_task_tables(*p, p->tasks[i]);
        }
        p->lay = layout_workspace(n_layers, p->units.size(), p->group_units.size() + p->other_units.size(), max_tasks);
        if (p->has_gauss) {
            const size_t stride = context_stride(layers, n_layers);
            if (stride > 0xFFFFFFFFull) {
                delete p;
                return fail(RANDES_INVALID_ARGUMENT, "the layers have %zu columns in all: more than the factor table of a RANDES_GAUSS plan indexes", stride);
            }
            p->ctx_stride = static_cast<uint32_t>(stride);
            for (uint32_t l = 0; l < n_layers; ++l) p->max_cols = std::max(p->max_cols, layers[l].cols);
            layout_context(p->lay, layers, n_layers, max_tasks);
        }
    } catch (const std::bad_alloc&) {
        delete p;
        return fail(RANDES_OUT_OF_MEMORY, "host allocation failed");
    }

    if (dev_workspace) {
        // A plan without a workspace is host-only: tables and sizes can be
        // queried, the compute entry points refuse to run.
        if (reinterpret_cast<uintptr_t>(dev_workspace) % 256) {
            delete p;
            return fail(RANDES_MISALIGNED, "dev_workspace = %p is not 256-byte aligned", dev_workspace);
        }
        if (dev_workspace_bytes < p->lay.total) {
            const size_t need = p->lay.total;
            const bool gauss = p->has_gauss;
            delete p;
            return fail(RANDES_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, plan needs %zu%s", dev_workspace_bytes, need,
                        gauss ? " (a plan with a RANDES_GAUSS group holds a table of its factors: size it with randes_plan_workspace_bytes_groups)" : "");
        }
        p->ws = static_cast<char*>(dev_workspace);
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) { delete p; return fail_cuda(e, "device query"); }
        const int occ_acc = accumulate_ctas_per_sm(p->storage, p->m_dtype, false);
        const int occ_acc1 = accumulate_ctas_per_sm(p->storage, p->m_dtype, true);
        const int occ_r0 = retrieve_ctas_per_sm(p->storage, RANDES_F32, p->m_dtype);
        const int occ_r1 = retrieve_ctas_per_sm(p->storage, RANDES_BF16, p->m_dtype);
        if (occ_acc <= 0 || occ_acc1 <= 0 || occ_r0 <= 0 || occ_r1 <= 0) {
            delete p;
            return fail(RANDES_CUDA_ERROR, "kernels are not loadable on this device (built for sm_100a)");
        }
        p->grid_acc[0] = p->sm_count * occ_acc;
        p->grid_acc[1] = p->sm_count * occ_acc1;
        p->grid_ret[0] = p->sm_count * occ_r0;
        p->grid_ret[1] = p->sm_count * occ_r1;
        p->grid_gram = p->sm_count * std::max(1, gram_ctas_per_sm(p->storage));
        e = cudaMemcpyAsync(p->ws + p->lay.layers, p->dev_layers.data(), n_layers * sizeof(DevLayer),
                            cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && !p->units.empty())
            e = cudaMemcpyAsync(p->ws + p->lay.units, p->units.data(), p->units.size() * sizeof(DevUnit),
                                cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(p->ws + p->lay.members, p->member_table.data(), p->member_table.size() * sizeof(uint32_t),
                                cudaMemcpyHostToDevice, s);
        // [other units][group units]
        if (e == cudaSuccess && !p->other_units.empty())
            e = cudaMemcpyAsync(p->ws + p->lay.staged_units, p->other_units.data(), p->other_units.size() * sizeof(DevUnit),
                                cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && !p->group_units.empty())
            e = cudaMemcpyAsync(p->dev<DevUnit>(p->lay.staged_units) + p->other_units.size(), p->group_units.data(),
                                p->group_units.size() * sizeof(DevUnit), cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && !p->group_units.empty()) {
            const int ge = compress_group_prepare(p->storage, p->m_dtype);
            if (ge) { delete p; return fail_cuda(static_cast<cudaError_t>(ge), "set-up of the group compress kernel"); }
        }
        if (e == cudaSuccess && p->has_gauss) {
            std::vector<uint32_t> ctx_off(n_layers);
            size_t o = 0;
            for (uint32_t l = 0; l < n_layers; ++l) { ctx_off[l] = static_cast<uint32_t>(o); o += align_up(static_cast<size_t>(layers[l].cols), 4); }
            // pageable host memory: the copy has left the vector when the call returns
            e = cudaMemcpyAsync(p->ws + p->lay.ctx_off, ctx_off.data(), n_layers * sizeof(uint32_t), cudaMemcpyHostToDevice, s);
        }
        if (e != cudaSuccess) { delete p; return fail_cuda(e, "copy of plan tables"); }
        if ((rc = upload_task_rows(*p, 0, s))) { delete p; return rc; }
    }
    *out_plan = p;
    return RANDES_OK;
}

void randes_plan_destroy(randes_plan_t* plan) { delete plan; }

size_t randes_superposition_bytes(const randes_plan_t* plan) { return plan ? plan->m_bytes : 0; }

size_t randes_layer_offset(const randes_plan_t* plan, uint32_t layer)
{
    if (!plan || layer >= plan->n_layers) return static_cast<size_t>(-1);
    return plan->m_off_bytes[layer];
}

uint32_t randes_num_layers(const randes_plan_t* plan) { return plan ? plan->n_layers : 0; }
uint32_t randes_num_tasks(const randes_plan_t* plan) { return plan ? static_cast<uint32_t>(plan->tasks.size()) : 0; }

int randes_task_list(const randes_plan_t* plan, uint32_t* task_ids, uint64_t* seeds)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    for (size_t i = 0; i < plan->tasks.size(); ++i) {
        if (task_ids) task_ids[i] = plan->tasks[i].id;
        if (seeds) seeds[i] = plan->tasks[i].seed;
    }
    return RANDES_OK;
}

// ---- persistence: what the paper stores per model is a seed; a plan is its shapes, flags and seeds ----
namespace {
constexpr uint32_t kBlobMagic = 0x53444E52u;   // "RNDS"
constexpr uint32_t kBlobVersion = 1;
struct BlobHeader {
    uint32_t magic, version, n_layers, n_groups, storage, m_dtype, n_tasks, reserved;
};
size_t blob_bytes(uint32_t n_layers, uint32_t n_groups, uint32_t n_tasks)
{
    return sizeof(BlobHeader) + n_layers * sizeof(randes_layer_t) + n_groups * sizeof(uint32_t) + n_tasks * (sizeof(uint32_t) + sizeof(uint64_t));
}
}  // namespace

size_t randes_plan_serialize(const randes_plan_t* plan, void* buffer, size_t buffer_bytes)
{
    if (!plan) { fail(RANDES_INVALID_ARGUMENT, "plan is NULL"); return 0; }
    const uint32_t n_tasks = static_cast<uint32_t>(plan->tasks.size());
    const size_t need = blob_bytes(plan->n_layers, plan->n_groups, n_tasks);
    if (!buffer) return need;
    if (buffer_bytes < need) { fail(RANDES_WORKSPACE_TOO_SMALL, "buffer has %zu bytes, the plan needs %zu", buffer_bytes, need); return 0; }
    char* out = static_cast<char*>(buffer);
    const BlobHeader h = {kBlobMagic, kBlobVersion, plan->n_layers, plan->n_groups, static_cast<uint32_t>(plan->storage),
                          static_cast<uint32_t>(plan->m_dtype), n_tasks, 0};
    std::memcpy(out, &h, sizeof h); out += sizeof h;
    std::memcpy(out, plan->layers.data(), plan->n_layers * sizeof(randes_layer_t)); out += plan->n_layers * sizeof(randes_layer_t);
    std::memcpy(out, plan->gflags.data(), plan->n_groups * sizeof(uint32_t)); out += plan->n_groups * sizeof(uint32_t);
    for (const TaskEntry& t : plan->tasks) { std::memcpy(out, &t.id, sizeof t.id); out += sizeof t.id; }
    for (const TaskEntry& t : plan->tasks) { std::memcpy(out, &t.seed, sizeof t.seed); out += sizeof t.seed; }
    return need;
}

size_t randes_plan_workspace_needed(const randes_plan_t* plan) { return plan ? plan->lay.total : 0; }

int randes_plan_deserialize(const void* buffer, size_t buffer_bytes, uint32_t max_tasks, void* dev_workspace,
                            size_t dev_workspace_bytes, void* stream, randes_plan_t** out_plan)
{
    if (!out_plan) return fail(RANDES_INVALID_ARGUMENT, "out_plan is NULL");
    *out_plan = nullptr;
    if (!buffer || buffer_bytes < sizeof(BlobHeader)) return fail(RANDES_INVALID_ARGUMENT, "buffer is NULL or shorter than a header");
    BlobHeader h;
    std::memcpy(&h, buffer, sizeof h);
    if (h.magic != kBlobMagic || h.version != kBlobVersion)
        return fail(RANDES_INVALID_ARGUMENT, "not a serialized plan (magic 0x%x, version %u)", h.magic, h.version);
    if (h.n_layers > (1u << 24) || h.n_groups > (1u << 24) || h.n_tasks > (1u << 24) ||
        buffer_bytes < blob_bytes(h.n_layers, h.n_groups, h.n_tasks))
        return fail(RANDES_INVALID_ARGUMENT, "serialized plan is truncated or corrupt");
    return guarded("randes_plan_deserialize", [&] {
        const char* in = static_cast<const char*>(buffer) + sizeof h;
        std::vector<randes_layer_t> layers(h.n_layers);
        std::memcpy(layers.data(), in, h.n_layers * sizeof(randes_layer_t)); in += h.n_layers * sizeof(randes_layer_t);
        std::vector<randes_group_t> groups(h.n_groups);
        for (uint32_t g = 0; g < h.n_groups; ++g) { std::memcpy(&groups[g].flags, in, sizeof(uint32_t)); in += sizeof(uint32_t); }
        std::vector<uint32_t> ids(h.n_tasks);
        std::vector<uint64_t> seeds(h.n_tasks);
        std::memcpy(ids.data(), in, h.n_tasks * sizeof(uint32_t)); in += h.n_tasks * sizeof(uint32_t);
        std::memcpy(seeds.data(), in, h.n_tasks * sizeof(uint64_t));
        return randes_plan(layers.data(), h.n_layers, groups.data(), h.n_groups, static_cast<randes_dtype_t>(h.storage),
                           static_cast<randes_dtype_t>(h.m_dtype), ids.data(), seeds.data(), h.n_tasks,
                           std::max(max_tasks, std::max(1u, h.n_tasks)), dev_workspace, dev_workspace_bytes, stream, out_plan);
    });
}

int randes_task_tables(const randes_plan_t* plan, uint32_t task_id, uint32_t* src_of_slot, uint32_t* slot_of_pos)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    const int i = find_task(*plan, task_id);
    if (i < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_id);
    const TaskEntry& t = plan->tasks[i];
    if (src_of_slot) std::memcpy(src_of_slot, t.src_of_slot.data(), plan->n_layers * sizeof(uint32_t));
    if (slot_of_pos) std::memcpy(slot_of_pos, t.slot_of_pos.data(), plan->n_layers * sizeof(uint32_t));
    return RANDES_OK;
}

static int randes_compress_impl(randes_plan_t* plan, const void* const* base, const void* const* tasks, void* M, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    int rc;
    if ((rc = check_m(M))) return rc;
    if (plan->tasks.empty()) return fail(RANDES_INVALID_ARGUMENT, "no task is registered");
    if (!tasks) return fail(RANDES_INVALID_ARGUMENT, "tasks is NULL");
    // Beyond kTaskChunk tasks the kernel carries the partial sum through M between chunks; a bf16 M
    // would round it there, while compress promises one rounding at the end.
    if (plan->m_dtype == RANDES_BF16 && plan->tasks.size() > static_cast<size_t>(kTaskChunk))
        return fail(RANDES_CAPACITY, "with a bf16 superposition compress sums at most %d tasks per call (plan holds %zu); "
                    "use an fp32 superposition or add the remaining models with randes_add_model", kTaskChunk, plan->tasks.size());
    const size_t es = elem_size(plan->storage);
    if ((rc = check_ptrs(*plan, base, "base", es, true))) return rc;
    for (size_t i = 0; i < plan->tasks.size(); ++i)
        if ((rc = check_ptrs(*plan, tasks + i * plan->n_layers, "tasks", es, false))) return rc;
    return run_accumulate(*plan, 0, plan->tasks.size(), false, false, base, tasks, M, static_cast<cudaStream_t>(stream));
}

static int randes_add_model_impl(randes_plan_t* plan, uint32_t task_id, uint64_t seed, const void* const* base,
                     const void* const* task, void* M, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    int rc;
    if ((rc = check_m(M))) return rc;
    if (find_task(*plan, task_id) >= 0) return fail(RANDES_DUPLICATE_TASK, "task id %u is already registered", task_id);
    if (plan->tasks.size() >= plan->max_tasks)
        return fail(RANDES_CAPACITY, "plan already holds max_tasks = %u tasks", plan->max_tasks);
    const size_t es = elem_size(plan->storage);
    if ((rc = check_ptrs(*plan, base, "base", es, true))) return rc;
    if ((rc = check_ptrs(*plan, task, "task", es, false))) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TaskEntry t;
    t.id = task_id;
    t.seed = seed;
    try {
        make_task_tables(*plan, t);
        plan->tasks.push_back(std::move(t));
    } catch (const std::bad_alloc&) {
        return fail(RANDES_OUT_OF_MEMORY, "host allocation failed");
    }
    const size_t row = plan->tasks.size() - 1;
    if ((rc = upload_task_rows(*plan, row, s)) ||
        (rc = run_accumulate(*plan, row, 1, true, false, base, task, M, s))) {
        plan->tasks.pop_back();
        return rc;
    }
    return RANDES_OK;
}

static int randes_add_models_impl(randes_plan_t* plan, const uint32_t* task_ids, const uint64_t* seeds, uint32_t n_tasks,
                                  const void* const* base, const void* const* tasks, void* M, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    int rc;
    if ((rc = check_m(M))) return rc;
    if (n_tasks == 0) return RANDES_OK;
    if (!task_ids || !seeds || !tasks) return fail(RANDES_INVALID_ARGUMENT, "task_ids / seeds / tasks is NULL");
    for (uint32_t i = 0; i < n_tasks; ++i) {
        if (find_task(*plan, task_ids[i]) >= 0) return fail(RANDES_DUPLICATE_TASK, "task id %u is already registered", task_ids[i]);
        for (uint32_t j = 0; j < i; ++j)
            if (task_ids[i] == task_ids[j]) return fail(RANDES_DUPLICATE_TASK, "task id %u appears twice", task_ids[i]);
    }
    if (plan->tasks.size() + n_tasks > plan->max_tasks)
        return fail(RANDES_CAPACITY, "plan holds %zu tasks, %u more exceed max_tasks = %u", plan->tasks.size(), n_tasks, plan->max_tasks);
    // beyond kTaskChunk terms the kernel carries the partial sum through M, where a bf16 M would round it
    if (plan->m_dtype == RANDES_BF16 && n_tasks > static_cast<uint32_t>(kTaskChunk))
        return fail(RANDES_CAPACITY, "with a bf16 superposition at most %d models are added per call (got %u)", kTaskChunk, n_tasks);
    const size_t es = elem_size(plan->storage);
    if ((rc = check_ptrs(*plan, base, "base", es, true))) return rc;
    for (uint32_t i = 0; i < n_tasks; ++i)
        if ((rc = check_ptrs(*plan, tasks + static_cast<size_t>(i) * plan->n_layers, "tasks", es, false))) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t first = plan->tasks.size();
    try {
        for (uint32_t i = 0; i < n_tasks; ++i) {
            TaskEntry t;
            t.id = task_ids[i];
            t.seed = seeds[i];
            make_task_tables(*plan, t);
            plan->tasks.push_back(std::move(t));
        }
    } catch (const std::bad_alloc&) {
        plan->tasks.resize(first);
        return fail(RANDES_OUT_OF_MEMORY, "host allocation failed");
    }
    if ((rc = upload_task_rows(*plan, first, s)) || (rc = run_accumulate(*plan, first, n_tasks, true, false, base, tasks, M, s))) {
        plan->tasks.resize(first);
        return rc;
    }
    return RANDES_OK;
}

static int randes_remove_model_impl(randes_plan_t* plan, uint32_t task_id, const void* const* base, const void* const* task,
                        void* M, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    int rc;
    if ((rc = check_m(M))) return rc;
    const int row = find_task(*plan, task_id);
    if (row < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_id);
    const size_t es = elem_size(plan->storage);
    if ((rc = check_ptrs(*plan, base, "base", es, true))) return rc;
    if ((rc = check_ptrs(*plan, task, "task", es, false))) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((rc = run_accumulate(*plan, row, 1, true, true, base, task, M, s))) return rc;
    // close the gap in the registry; later rows move up one place on the device too
    plan->tasks.erase(plan->tasks.begin() + row);
    return upload_task_rows(*plan, row, s);
}

static int randes_retrieve_impl(randes_plan_t* plan, uint32_t task_id, float lambda, randes_dtype_t out_dtype,
                    const void* const* base, const void* M, void* const* out, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    if (out_dtype != RANDES_F32 && out_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "output dtype %d is not supported", static_cast<int>(out_dtype));
    int rc;
    if ((rc = check_m(M))) return rc;
    const int row = find_task(*plan, task_id);
    if (row < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_id);
    if ((rc = check_ptrs(*plan, base, "base", elem_size(plan->storage), false))) return rc;
    if ((rc = check_ptrs(*plan, const_cast<const void* const*>(out), "out", elem_size(out_dtype), false))) return rc;
    // (skipped when both pointer tables are the ones the last successful call checked)
    const size_t table_bytes = plan->n_layers * sizeof(void*);
    const bool seen = plan->base_valid && plan->out_valid && plan->checked_m == M && plan->checked_out_elem == elem_size(out_dtype) &&
                      std::memcmp(plan->h_base.data(), base, table_bytes) == 0 && std::memcmp(plan->h_out.data(), out, table_bytes) == 0;
    if (!seen && (rc = check_outputs_disjoint(*plan, base, const_cast<const void* const*>(out), 1, elem_size(out_dtype), M))) return rc;
    plan->checked_m = M;
    plan->checked_out_elem = elem_size(out_dtype);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((rc = stage_ptrs(*plan, plan->h_base, plan->base_valid, plan->lay.base_ptrs, base, s))) return rc;
    if ((rc = stage_ptrs(*plan, plan->h_out, plan->out_valid, plan->lay.out_ptrs, const_cast<const void* const*>(out), s)))
        return rc;
    RetrieveArgs a;
    a.layers = plan->dev<DevLayer>(plan->lay.layers);
    a.units = plan->dev<DevUnit>(plan->lay.units);
    a.n_units = static_cast<uint32_t>(plan->units.size());
    a.n_layers = plan->n_layers;
    a.slot_of_pos = plan->dev<uint32_t>(plan->lay.slot_of_pos) + static_cast<size_t>(row) * plan->n_layers;
    a.base = plan->dev<const void*>(plan->lay.base_ptrs);
    a.out = plan->dev<void*>(plan->lay.out_ptrs);
    a.M = M;
    a.task.id = plan->tasks[row].id;
    a.task.key0 = static_cast<uint32_t>(plan->tasks[row].seed);
    a.task.key1 = static_cast<uint32_t>(plan->tasks[row].seed >> 32);
    a.task.pad = 0;
    a.lambda = lambda;
    if (a.n_units == 0) return RANDES_OK;
    if (plan->has_gauss) {
        const int ce = launch_context_retrieve(plan->storage, out_dtype, a, context_args(*plan, static_cast<size_t>(row)), s);
        if (ce) return fail_cuda(static_cast<cudaError_t>(ce), "launch of the general-context retrieve kernel");
        ++g_launches;
        return RANDES_OK;
    }
    const int grid = std::min<int>(plan->grid_ret[out_dtype], static_cast<int>(a.n_units));
    const int e = launch_retrieve(plan->storage, out_dtype, plan->m_dtype, a, grid, s);
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the retrieve kernel");
    ++g_launches;
    return RANDES_OK;
}

size_t randes_delta_gram_scratch_bytes(const randes_plan_t* plan)
{
    if (!plan || !plan->ws) return 0;
    return static_cast<size_t>(plan->grid_gram) * kGramPartialDoubles * sizeof(double);
}

static int randes_delta_gram_impl(randes_plan_t* plan, const void* const* base, const void* const* tasks, double* gram, void* scratch,
                      size_t scratch_bytes, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (plan->has_gauss) return fail(RANDES_INVALID_ARGUMENT, "not offered for plans with a RANDES_GAUSS group");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    const size_t n = plan->tasks.size();
    if (n == 0) return fail(RANDES_INVALID_ARGUMENT, "no task is registered");
    if (n > static_cast<size_t>(kTaskChunk)) return fail(RANDES_CAPACITY, "the Gram matrix is limited to %d tasks; the plan holds %zu", kTaskChunk, n);
    if (!gram || reinterpret_cast<uintptr_t>(gram) % 8) return fail(RANDES_MISALIGNED, "gram = %p is NULL or not 8-byte aligned", (void*)gram);
    if (!scratch || reinterpret_cast<uintptr_t>(scratch) % 8) return fail(RANDES_MISALIGNED, "scratch = %p is NULL or not 8-byte aligned", scratch);
    if (scratch_bytes < randes_delta_gram_scratch_bytes(plan))
        return fail(RANDES_WORKSPACE_TOO_SMALL, "scratch has %zu bytes, the Gram matrix needs %zu", scratch_bytes,
                    randes_delta_gram_scratch_bytes(plan));
    if (!tasks) return fail(RANDES_INVALID_ARGUMENT, "tasks is NULL");
    int rc;
    const size_t es = elem_size(plan->storage);
    if ((rc = check_ptrs(*plan, base, "base", es, true))) return rc;
    for (size_t i = 0; i < n; ++i)
        if ((rc = check_ptrs(*plan, tasks + i * plan->n_layers, "tasks", es, false))) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (base && (rc = stage_ptrs(*plan, plan->h_base, plan->base_valid, plan->lay.base_ptrs, base, s))) return rc;
    if ((rc = stage_task_ptrs(*plan, tasks, n, s))) return rc;
    GramArgs a;
    a.layers = plan->dev<DevLayer>(plan->lay.layers);
    a.units = plan->dev<DevUnit>(plan->lay.units);
    a.n_units = static_cast<uint32_t>(plan->units.size());
    a.n_layers = plan->n_layers;
    a.src_of_slot = plan->dev<uint32_t>(plan->lay.src_of_slot);
    a.tasks = plan->dev<DevTask>(plan->lay.tasks);
    a.n_tasks = static_cast<uint32_t>(n);
    a.has_base = base != nullptr;
    a.base = plan->dev<const void*>(plan->lay.base_ptrs);
    a.task_ptrs = plan->dev<const void*>(plan->lay.task_ptrs);
    a.partial = static_cast<double*>(scratch);
    const int grid = std::max(1, std::min<int>(plan->grid_gram, static_cast<int>(a.n_units)));
    const int e = launch_gram(plan->storage, a, grid, gram, s);
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the Gram kernels");
    g_launches += 2;
    return RANDES_OK;
}

static int randes_retrieve_batch_impl(randes_plan_t* plan, const uint32_t* task_ids, uint32_t n_tasks, float lambda,
                          randes_dtype_t out_dtype, const void* const* base, const void* M, void* const* out, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (plan->has_gauss) return fail(RANDES_INVALID_ARGUMENT, "not offered for plans with a RANDES_GAUSS group");
    if (!plan->ws) return fail(RANDES_INVALID_ARGUMENT, "plan was built without a device workspace");
    if (out_dtype != RANDES_F32 && out_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "output dtype %d is not supported", static_cast<int>(out_dtype));
    if (!task_ids || n_tasks == 0) return fail(RANDES_INVALID_ARGUMENT, "task_ids is NULL or empty");
    if (n_tasks > static_cast<uint32_t>(kTaskChunk) || n_tasks > plan->max_tasks)
        return fail(RANDES_CAPACITY, "a batch holds at most %d tasks (and at most max_tasks = %u); got %u", kTaskChunk,
                    plan->max_tasks, n_tasks);
    int rc;
    if ((rc = check_m(M))) return rc;
    if ((rc = check_ptrs(*plan, base, "base", elem_size(plan->storage), false))) return rc;
    if (!out) return fail(RANDES_INVALID_ARGUMENT, "out is NULL");
    RetrieveBatchArgs a;
    for (uint32_t b = 0; b < n_tasks; ++b) {
        const int row = find_task(*plan, task_ids[b]);
        if (row < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_ids[b]);
        for (uint32_t c = 0; c < b; ++c)
            if (task_ids[c] == task_ids[b]) return fail(RANDES_DUPLICATE_TASK, "task id %u appears twice in the batch", task_ids[b]);
        a.task_rows[b] = static_cast<uint32_t>(row);
        void* const* ob = out + static_cast<size_t>(b) * plan->n_layers;
        if ((rc = check_ptrs(*plan, const_cast<const void* const*>(ob), "out", elem_size(out_dtype), false))) return rc;
    }
    if ((rc = check_outputs_disjoint(*plan, base, const_cast<const void* const*>(out), n_tasks, elem_size(out_dtype), M))) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((rc = stage_ptrs(*plan, plan->h_base, plan->base_valid, plan->lay.base_ptrs, base, s))) return rc;
    // the batch's output tables share the device area of the task pointer tables
    if ((rc = stage_task_ptrs(*plan, const_cast<const void* const*>(out), n_tasks, s))) return rc;
    a.layers = plan->dev<DevLayer>(plan->lay.layers);
    a.units = plan->dev<DevUnit>(plan->lay.units);
    a.n_units = static_cast<uint32_t>(plan->units.size());
    a.n_layers = plan->n_layers;
    a.slot_of_pos = plan->dev<uint32_t>(plan->lay.slot_of_pos);
    a.tasks = plan->dev<DevTask>(plan->lay.tasks);
    a.n_tasks = n_tasks;
    a.base = plan->dev<const void*>(plan->lay.base_ptrs);
    a.out = plan->dev<void*>(plan->lay.task_ptrs);
    a.M = M;
    a.lambda = lambda;
    a.members = plan->dev<uint32_t>(plan->lay.members);
    // fp32 weights and superposition: the shuffled groups go through the kernel that stages M and W_0 of a
    // whole group in shared memory (needs 16-byte aligned tensors there); the rest as before
    bool staged = plan->storage == RANDES_F32 && plan->m_dtype == RANDES_F32 && !plan->group_units.empty() &&
                  retrieve_batch_group_fits(plan->max_staged_group, n_tasks);
    for (uint32_t l = 0; staged && l < plan->n_layers; ++l) {
        if (!plan->group_staged[plan->layers[l].group]) continue;
        staged = reinterpret_cast<uintptr_t>(base[l]) % 16 == 0;
        for (uint32_t b = 0; staged && b < n_tasks; ++b) staged = reinterpret_cast<uintptr_t>(out[static_cast<size_t>(b) * plan->n_layers + l]) % 16 == 0;
    }
    if (staged) {
        int ge = retrieve_batch_group_prepare();
        if (ge) return fail_cuda(static_cast<cudaError_t>(ge), "set-up of the grouped batched retrieve kernel");
        RetrieveBatchArgs g = a;
        g.units = plan->dev<DevUnit>(plan->lay.staged_units) + plan->other_units.size();
        g.n_units = static_cast<uint32_t>(plan->group_units.size());
        ge = launch_retrieve_batch_groups(out_dtype, g, plan->max_staged_group, plan->sm_count, s);
        if (ge) return fail_cuda(static_cast<cudaError_t>(ge), "launch of the grouped batched retrieve kernel");
        ++g_launches;
        a.units = plan->dev<DevUnit>(plan->lay.staged_units);
        a.n_units = static_cast<uint32_t>(plan->other_units.size());
    }
    if (a.n_units == 0) return RANDES_OK;
    // one CTA per unit (the block scheduler balances the store-bound work over the SMs; a resident loop over units dealt
    // out in advance was 4 - 27 % slower)
    const int grid = static_cast<int>(std::min<uint64_t>(a.n_units, 0x7FFFFFFFull));
    const int e = launch_retrieve_batch(plan->storage, out_dtype, plan->m_dtype, a, grid, s);
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the batched retrieve kernel");
    ++g_launches;
    return RANDES_OK;
}

static int randes_retrieve_static_impl(const randes_plan_t* plan, uint32_t task_id, float lambda, randes_dtype_t out_dtype,
                           const void* const* base, const void* M, void* const* out, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (plan->has_gauss) return fail(RANDES_INVALID_ARGUMENT, "not offered for plans with a RANDES_GAUSS group");
    if (out_dtype != RANDES_F32 && out_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "output dtype %d is not supported", static_cast<int>(out_dtype));
    int rc;
    if ((rc = check_m(M))) return rc;
    const int row = find_task(*plan, task_id);
    if (row < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_id);
    if ((rc = check_ptrs(*plan, base, "base", elem_size(plan->storage), false))) return rc;
    if ((rc = check_ptrs(*plan, const_cast<const void* const*>(out), "out", elem_size(out_dtype), false))) return rc;
    if ((rc = check_outputs_disjoint(*plan, base, const_cast<const void* const*>(out), 1, elem_size(out_dtype), M))) return rc;
    const size_t need = retrieve_static_bytes(plan->n_layers, static_cast<uint32_t>(plan->units.size()));
    if (need > kStaticScratchBytes)
        return fail(RANDES_CAPACITY,
                    "this model needs %zu bytes of tables (%u layers, %zu tiles) but the built-in scratch holds %zu; "
                    "use randes_retrieve with a workspace instead",
                    need, plan->n_layers, plan->units.size(), static_cast<size_t>(kStaticScratchBytes));
    const TaskEntry& t = plan->tasks[row];
    DevTask dt;
    dt.id = t.id;
    dt.key0 = static_cast<uint32_t>(t.seed);
    dt.key1 = static_cast<uint32_t>(t.seed >> 32);
    dt.pad = 0;
    const int e = launch_retrieve_static(plan->storage, out_dtype, plan->m_dtype, plan->dev_layers.data(), plan->n_layers,
                                         plan->units.data(), static_cast<uint32_t>(plan->units.size()), t.slot_of_pos.data(), base,
                                         out, M, dt, lambda, stream);
    if (e == -1) return fail(RANDES_CAPACITY, "tables exceed the built-in scratch");
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "randes_retrieve_static");
    if (!plan->units.empty()) ++g_launches;
    return RANDES_OK;
}

int randes_compress(randes_plan_t* plan, const void* const* base, const void* const* tasks, void* M, void* stream)
{
    return guarded("randes_compress", [&] { return randes_compress_impl(plan, base, tasks, M, stream); });
}

int randes_add_model(randes_plan_t* plan, uint32_t task_id, uint64_t seed, const void* const* base,
                     const void* const* task, void* M, void* stream)
{
    return guarded("randes_add_model", [&] { return randes_add_model_impl(plan, task_id, seed, base, task, M, stream); });
}

int randes_add_models(randes_plan_t* plan, const uint32_t* task_ids, const uint64_t* seeds, uint32_t n_tasks,
                      const void* const* base, const void* const* tasks, void* M, void* stream)
{
    return guarded("randes_add_models", [&] { return randes_add_models_impl(plan, task_ids, seeds, n_tasks, base, tasks, M, stream); });
}

int randes_remove_model(randes_plan_t* plan, uint32_t task_id, const void* const* base, const void* const* task,
                        void* M, void* stream)
{
    return guarded("randes_remove_model", [&] { return randes_remove_model_impl(plan, task_id, base, task, M, stream); });
}

int randes_retrieve(randes_plan_t* plan, uint32_t task_id, float lambda, randes_dtype_t out_dtype,
                    const void* const* base, const void* M, void* const* out, void* stream)
{
    return guarded("randes_retrieve", [&] { return randes_retrieve_impl(plan, task_id, lambda, out_dtype, base, M, out, stream); });
}

static int randes_linear_impl(const randes_plan_t* plan, uint32_t task_id, float lambda, uint32_t layer, const void* x,
                              uint32_t n_tokens, const void* const* base, const void* M, void* y, randes_dtype_t y_dtype,
                              const uint32_t* gate, uint64_t wait_ns, void* stream)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    if (plan->has_gauss) return fail(RANDES_INVALID_ARGUMENT, "not offered for plans with a RANDES_GAUSS group");
    if (plan->storage != RANDES_BF16 || plan->m_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "randes_linear needs bf16 weights and a bf16 superposition (tensor-core operands)");
    if (y_dtype != RANDES_F32 && y_dtype != RANDES_BF16)
        return fail(RANDES_UNSUPPORTED_DTYPE, "output dtype %d is not supported", static_cast<int>(y_dtype));
    if (layer >= plan->n_layers) return fail(RANDES_INVALID_ARGUMENT, "layer %u out of range (n_layers = %u)", layer, plan->n_layers);
    const int row = find_task(*plan, task_id);
    if (row < 0) return fail(RANDES_UNKNOWN_TASK, "task id %u is not registered", task_id);
    int rc;
    if ((rc = check_m(M))) return rc;
    if (!base || !base[layer]) return fail(RANDES_INVALID_ARGUMENT, "base or base[%u] is NULL", layer);
    const uint32_t rows = plan->layers[layer].rows, cols = plan->layers[layer].cols;
    if (n_tokens == 0 || rows == 0 || cols == 0) return RANDES_OK;   // nothing to compute (x and y may be NULL then)
    if (!x || !y) return fail(RANDES_INVALID_ARGUMENT, "x or y is NULL");
    if (cols % 8) return fail(RANDES_INVALID_ARGUMENT, "layer %u: cols = %u is not a multiple of 8 (16-byte rows for the tensor maps)", layer, cols);
    if (reinterpret_cast<uintptr_t>(x) % 16 || reinterpret_cast<uintptr_t>(base[layer]) % 16)
        return fail(RANDES_MISALIGNED, "x and base[%u] must be 16-byte aligned", layer);
    if (reinterpret_cast<uintptr_t>(y) % elem_size(y_dtype)) return fail(RANDES_MISALIGNED, "y = %p is not aligned to its element size", y);
    if (reinterpret_cast<uintptr_t>(gate) % 4) return fail(RANDES_MISALIGNED, "gate = %p is not 4-byte aligned", (const void*)gate);
    if (n_tokens > 65535u * 128u) return fail(RANDES_INVALID_ARGUMENT, "n_tokens = %u exceeds the supported %u", n_tokens, 65535u * 128u);
    if (wait_ns > 60ull * 1000000000ull) return fail(RANDES_INVALID_ARGUMENT, "wait_ns = %llu exceeds the supported 60 s", (unsigned long long)wait_ns);
    const TaskEntry& t = plan->tasks[row];
    const uint32_t slot = t.slot_of_pos[layer];                    // sigma_t^-1(p)
    const bool flip = (plan->dev_layers[slot].flags & kFlagFlip) != 0;
    DevTask d;
    d.id = t.id;
    d.key0 = static_cast<uint32_t>(t.seed);
    d.key1 = static_cast<uint32_t>(t.seed >> 32);
    d.pad = 0;
    int e = linear_prepare(), launched = 0;
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "set-up of the linear kernel");
    e = launch_linear(x, n_tokens, base[layer], static_cast<const char*>(M) + plan->m_off_bytes[slot], rows, cols, flip, slot, d, lambda,
                      y, y_dtype == RANDES_BF16, gate, wait_ns, stream, &launched);
    g_launches += launched;
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "launch of the linear kernel");
    return RANDES_OK;
}

int randes_linear(const randes_plan_t* plan, uint32_t task_id, float lambda, uint32_t layer, const void* x, uint32_t n_tokens,
                  const void* const* base, const void* M, void* y, randes_dtype_t y_dtype, void* stream)
{
    return guarded("randes_linear", [&] { return randes_linear_impl(plan, task_id, lambda, layer, x, n_tokens, base, M, y, y_dtype, nullptr, 0, stream); });
}

int randes_linear_gated(const randes_plan_t* plan, uint32_t task_id, float lambda, uint32_t layer, const void* x, uint32_t n_tokens,
                        const void* const* base, const void* M, void* y, randes_dtype_t y_dtype, const uint32_t* gate,
                        uint64_t wait_ns, void* stream)
{
    if (!gate) return fail(RANDES_INVALID_ARGUMENT, "gate is NULL (use randes_linear for a call without a gate)");
    return guarded("randes_linear_gated", [&] { return randes_linear_impl(plan, task_id, lambda, layer, x, n_tokens, base, M, y, y_dtype, gate, wait_ns, stream); });
}

int randes_linear_giveups(unsigned int* count)
{
    if (!count) return fail(RANDES_INVALID_ARGUMENT, "count is NULL");
    const int e = linear_giveups(count);
    if (e) return fail_cuda(static_cast<cudaError_t>(e), "read of the give-up counter");
    return RANDES_OK;
}

int randes_retrieve_batch(randes_plan_t* plan, const uint32_t* task_ids, uint32_t n_tasks, float lambda,
                          randes_dtype_t out_dtype, const void* const* base, const void* M, void* const* out, void* stream)
{
    return guarded("randes_retrieve_batch", [&] { return randes_retrieve_batch_impl(plan, task_ids, n_tasks, lambda, out_dtype, base, M, out, stream); });
}

int randes_delta_gram(randes_plan_t* plan, const void* const* base, const void* const* tasks, double* gram, void* scratch,
                      size_t scratch_bytes, void* stream)
{
    return guarded("randes_delta_gram", [&] { return randes_delta_gram_impl(plan, base, tasks, gram, scratch, scratch_bytes, stream); });
}

// Self-check of a plan (a debugging aid; nothing in the compute calls depends on it having run).
static int randes_plan_validate_impl(const randes_plan_t* plan)
{
    if (!plan) return fail(RANDES_INVALID_ARGUMENT, "plan is NULL");
    const uint32_t L = plan->n_layers;
    // (1) slots of M: aligned, in order, not overlapping, inside the arena
    size_t end = 0;
    for (uint32_t l = 0; l < L; ++l) {
        const size_t off = plan->m_off_bytes[l];
        if (off % 256 || off < end) return fail(RANDES_INVALID_ARGUMENT, "slot %u of M starts at byte %zu (previous slot ends at %zu)", l, off, end);
        end = off + static_cast<size_t>(plan->layers[l].rows) * plan->layers[l].cols * elem_size(plan->m_dtype);
        if (plan->dev_layers[l].m_off * elem_size(plan->m_dtype) != off) return fail(RANDES_INVALID_ARGUMENT, "slot %u: element and byte offsets disagree", l);
    }
    if (end > plan->m_bytes) return fail(RANDES_INVALID_ARGUMENT, "M holds %zu bytes but the last slot ends at %zu", plan->m_bytes, end);
    // (2) every task's sigma is a bijection that stays inside groups (Section 4.3), and sigma^-1 inverts it
    for (const TaskEntry& t : plan->tasks) {
        std::vector<char> hit(L, 0);
        for (uint32_t l = 0; l < L; ++l) {
            const uint32_t src = t.src_of_slot[l];
            if (src >= L || hit[src]) return fail(RANDES_INVALID_ARGUMENT, "task %u: sigma is not a bijection at slot %u", t.id, l);
            hit[src] = 1;
            if (plan->layers[src].group != plan->layers[l].group) return fail(RANDES_INVALID_ARGUMENT, "task %u: slot %u receives layer %u of another group", t.id, l, src);
            if (t.slot_of_pos[src] != l) return fail(RANDES_INVALID_ARGUMENT, "task %u: sigma^-1(sigma(%u)) = %u", t.id, l, t.slot_of_pos[src]);
            if (src != l && !(plan->dev_layers[l].flags & kFlagShuffle)) return fail(RANDES_INVALID_ARGUMENT, "task %u: slot %u moved without the shuffle flag", t.id, l);
        }
    }
    // (3) each unit list tiles every layer exactly once: cells = (row, warp-wide column block)
    const uint32_t span = cols_per_warp(plan->storage);
    std::vector<size_t> first(L + 1, 0);
    for (uint32_t l = 0; l < L; ++l)
        first[l + 1] = first[l] + static_cast<size_t>(plan->layers[l].rows) * ((plan->layers[l].cols + span - 1) / span);
    auto check_list = [&](const std::vector<DevUnit>& per_layer, const std::vector<DevUnit>& per_group, const char* name) -> int {
        std::vector<unsigned char> seen(first[L], 0);
        auto mark = [&](uint32_t layer, uint32_t row0, uint32_t nrows, uint32_t cb0, uint32_t nbc, size_t index) -> int {
            if (layer >= L) return fail(RANDES_INVALID_ARGUMENT, "%s unit %zu: layer %u out of range", name, index, layer);
            const uint32_t rows = plan->layers[layer].rows, nb = (plan->layers[layer].cols + span - 1) / span;
            if (nrows == 0 || row0 + nrows > rows) return fail(RANDES_INVALID_ARGUMENT, "%s unit %zu: rows [%u, %u) leave layer %u (%u rows)", name, index, row0, row0 + nrows, layer, rows);
            for (uint32_t cb = cb0; cb < cb0 + nbc; ++cb) {
                if (cb >= nb) continue;   // a unit may be wider than a ragged layer: the kernels skip those column blocks
                for (uint32_t r = row0; r < row0 + nrows; ++r) {
                    unsigned char& cell = seen[first[layer] + static_cast<size_t>(r) * nb + cb];
                    if (cell) return fail(RANDES_INVALID_ARGUMENT, "%s unit %zu: layer %u row %u column block %u is covered twice", name, index, layer, r, cb);
                    cell = 1;
                }
            }
            return RANDES_OK;
        };
        int rc;
        for (size_t i = 0; i < per_layer.size(); ++i) {
            const DevUnit& u = per_layer[i];
            if (u.nbc == 0 || u.nbc > kWarpsPerCta || (u.nbc & (u.nbc - 1))) return fail(RANDES_INVALID_ARGUMENT, "%s unit %zu: %u column blocks", name, i, u.nbc);
            if ((rc = mark(u.layer, u.row0, u.nrows, u.cb0, u.nbc, i))) return rc;
        }
        for (size_t i = 0; i < per_group.size(); ++i) {
            const DevUnit& u = per_group[i];
            if (u.nbc != 0 || u.layer >= plan->member_table.size()) return fail(RANDES_INVALID_ARGUMENT, "%s group unit %zu is malformed", name, i);
            const uint32_t g = plan->layers[plan->member_table[u.layer]].group;
            const std::vector<uint32_t>& mem = plan->members[g];
            if (plan->member_table[u.layer] != mem[0]) return fail(RANDES_INVALID_ARGUMENT, "%s group unit %zu does not start at its group's first member", name, i);
            if (static_cast<size_t>(mem.size()) * u.nrows * kStashTileBytes > stash_bytes(plan->storage))
                return fail(RANDES_INVALID_ARGUMENT, "%s group unit %zu: %zu members x %u rows exceed the stash", name, i, mem.size(), u.nrows);
            for (uint32_t l : mem)
                if ((rc = mark(l, u.row0, u.nrows, u.cb0, 1, i))) return rc;
        }
        for (uint32_t l = 0; l < L; ++l)
            for (size_t c = first[l]; c < first[l + 1]; ++c)
                if (!seen[c]) {
                    const uint32_t nb = (plan->layers[l].cols + span - 1) / span;
                    return fail(RANDES_INVALID_ARGUMENT, "%s: layer %u row %zu column block %zu is covered by no unit", name, l, (c - first[l]) / nb, (c - first[l]) % nb);
                }
        return RANDES_OK;
    };
    int rc;
    if ((rc = check_list(plan->units, {}, "the unit list"))) return rc;
    if (!plan->group_units.empty() && (rc = check_list(plan->other_units, plan->group_units, "the grouped unit list"))) return rc;
    // a general diagonal context: the factor table holds every column of every layer for max_tasks rows, inside the workspace
    if (plan->has_gauss) {
        if (plan->ctx_stride != context_stride(plan->layers.data(), L))
            return fail(RANDES_INVALID_ARGUMENT, "the factor table has %u floats per task, the layers need %zu", plan->ctx_stride, context_stride(plan->layers.data(), L));
        if (plan->ws && (plan->lay.ctx_off + L * sizeof(uint32_t) > plan->lay.ctx_table ||
                         plan->lay.ctx_table + static_cast<size_t>(plan->max_tasks) * plan->ctx_stride * sizeof(float) > plan->lay.total))
            return fail(RANDES_INVALID_ARGUMENT, "the factor table does not fit the workspace layout");
    }
    return RANDES_OK;
}

int randes_plan_validate(const randes_plan_t* plan)
{
    return guarded("randes_plan_validate", [&] { return randes_plan_validate_impl(plan); });
}

int randes_debug_violation(uint64_t* word, int* checked_build)
{
    if (!word) return fail(RANDES_INVALID_ARGUMENT, "word is NULL");
#ifdef RANDES_CHECKED
    if (checked_build) *checked_build = 1;
#else
    if (checked_build) *checked_build = 0;
#endif
    const unsigned long long w[3] = {violation_in_streaming_kernels(), violation_in_group_kernel(), violation_in_batch_kernels()};
    *word = w[0] ? w[0] : (w[1] ? w[1] : w[2]);
    if (*word == ~0ull) return fail(RANDES_CUDA_ERROR, "the violation word could not be read");
    return RANDES_OK;
}

// Section 3, norm of the interference: || lambda sum_{j != t} T_t^-1 T_j d_j ||^2 = lambda^2 sum_{j,l != t} <T_j d_j, T_l d_l>,
// because T_t^-1 is orthogonal.
int randes_interference_norm(const double* gram, uint32_t n, uint32_t t, double lambda, double* norm)
{
    if (!gram || !norm) return fail(RANDES_INVALID_ARGUMENT, "gram or norm is NULL");
    if (n == 0 || t >= n) return fail(RANDES_INVALID_ARGUMENT, "task index %u out of range (n = %u)", t, n);
    double total = 0.0;
    for (uint32_t j = 0; j < n; ++j) {
        if (j == t) continue;
        double row = 0.0;
        for (uint32_t l = 0; l < n; ++l)
            if (l != t) row += gram[static_cast<size_t>(j) * n + l];
        total += row;
    }
    *norm = lambda * std::sqrt(total > 0.0 ? total : 0.0);
    return RANDES_OK;
}

int randes_pairwise_cosines(const double* gram, uint32_t n, int32_t exclude, double* cosines, double* mean)
{
    if (!gram) return fail(RANDES_INVALID_ARGUMENT, "gram is NULL");
    if (n == 0) return fail(RANDES_INVALID_ARGUMENT, "n is 0");
    if (exclude >= 0 && static_cast<uint32_t>(exclude) >= n)
        return fail(RANDES_INVALID_ARGUMENT, "exclude = %d out of range (n = %u)", exclude, n);
    auto cosine = [&](uint32_t j, uint32_t l) {
        if (j == l) return 1.0;
        const double d = std::sqrt(gram[static_cast<size_t>(j) * n + j] * gram[static_cast<size_t>(l) * n + l]);
        return d > 0.0 ? gram[static_cast<size_t>(j) * n + l] / d : 0.0;
    };
    double sum = 0.0;
    uint64_t pairs = 0;
    for (uint32_t j = 0; j < n; ++j)
        for (uint32_t l = 0; l < n; ++l) {
            const double c = cosine(j, l);
            if (cosines) cosines[static_cast<size_t>(j) * n + l] = c;
            if (j < l && static_cast<int64_t>(j) != exclude && static_cast<int64_t>(l) != exclude) { sum += c; ++pairs; }
        }
    if (mean) *mean = pairs ? sum / static_cast<double>(pairs) : 0.0;
    return RANDES_OK;
}

int randes_retrieve_static(const randes_plan_t* plan, uint32_t task_id, float lambda, randes_dtype_t out_dtype,
                           const void* const* base, const void* M, void* const* out, void* stream)
{
    return guarded("randes_retrieve_static", [&] { return randes_retrieve_static_impl(plan, task_id, lambda, out_dtype, base, M, out, stream); });
}

}  // extern "C"
