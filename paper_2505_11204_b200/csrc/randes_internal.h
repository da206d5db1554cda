// Structures shared by the host side (plan, C ABI) and the kernels of the
// RanDeS library.  Not part of the public interface.
#pragma once

#include <cstddef>
#include <cstdint>

namespace randes {

constexpr uint32_t kFlagShuffle = 1u;   // layer may move inside its group for some task
constexpr uint32_t kFlagFlip = 2u;      // per-column sign flip on this slot
constexpr uint32_t kFlagGauss = 4u;     // per-column Gaussian-like factor on this slot instead (general diagonal context)

constexpr size_t kSuperpositionLeadIn = 1024;   // bytes before the first slot of M (see randes_plan)
constexpr int kWarpsPerCta = 8;
constexpr int kThreadsPerCta = kWarpsPerCta * 32;
constexpr int kRowsPerWarp = 16;        // rows one warp walks per unit (8 to 16 measured best; 32 and 64 slower)
constexpr int kTaskChunk = 32;          // tasks whose pointers / sign blocks a warp holds at once
constexpr uint32_t kTagSign = 0x5349474Eu;  // counter word 2 of the sign stream ("SIGN")
constexpr uint32_t kTagPerm = 0x5045524Du;  // counter word 2 of the permutation stream ("PERM")
constexpr uint32_t kTagGauss = 0x47415553u; // counter word 2 of the Gaussian-like context stream ("GAUS")

// A lane always moves 16 bytes of a weight tensor: 4 fp32 or 8 bf16 columns.  A
// warp therefore spans 128 (fp32) or 256 (bf16) columns = 1 or 2 Philox blocks
// of sign bits.
constexpr int cols_per_lane(int storage_dtype) { return storage_dtype == 1 ? 8 : 4; }
constexpr int cols_per_warp(int storage_dtype) { return 32 * cols_per_lane(storage_dtype); }

// One layer of the model == one slot of M (same index space).
struct DevLayer {
    unsigned long long m_off;  // first element of this slot in the fp32 arena M
    uint32_t rows, cols;
    uint32_t flags;            // kFlagShuffle | kFlagFlip, already resolved (shuffle only if group size >= 2)
    uint32_t group;
    uint32_t member;           // index of this layer inside its group
    uint32_t group_size;
};
static_assert(sizeof(DevLayer) == 32, "DevLayer layout");

// One unit of work for a CTA: `nrows` rows x `nbc` warp-wide column blocks of
// one layer.  Warp w owns column block cb0 + (w % nbc) and the rows
// row0 + (w / nbc), stepping by kWarpsPerCta / nbc.
struct DevUnit {
    uint32_t layer;
    uint32_t row0;
    uint32_t nrows;
    uint16_t cb0;
    uint16_t nbc;              // 1, 2, 4 or 8
};
static_assert(sizeof(DevUnit) == 16, "DevUnit layout");

// A group unit (nbc == 0) covers `nrows` rows x one warp-wide column block of EVERY member of a
// shuffled group: the CTA first stashes the W_0 tiles of all members in shared memory, then its
// warps sum the tasks' deltas slot by slot, subtracting W_0[sigma_i(l)] from the stash.  `layer`
// is then the index of the group's first entry in the member table.
constexpr uint32_t kUnitChunk = 8;                    // group units of one (group, column block) kept adjacent in the unit list
constexpr uint32_t kStashTileBytes = 512;             // 32 lanes x 16 bytes
constexpr uint32_t kStashBytes = 48 * 1024;           // fp32 weights
constexpr uint32_t kItemRows = 4;                     // rows of one slot a warp sums in one go, fp32 weights
// With bf16 weights a lane's 16 bytes hold twice the columns, so the sign records are twice as large and the
// row loop is bound by instruction issue: items are 3 rows taken as one stage (more rows per sign decode), and
// the stash is 36 KiB so that records for 20 tasks x 24 members still fit beside two resident CTAs.
constexpr uint32_t stash_bytes(int storage_dtype) { return storage_dtype == 1 ? 36u * 1024u : kStashBytes; }
constexpr uint32_t item_rows(int storage_dtype) { return storage_dtype == 1 ? 3u : kItemRows; }
// rows per group unit for a group of G members (0: the group is too large for the stash)
constexpr uint32_t group_unit_rows(uint32_t G, int storage_dtype)
{
    const uint32_t ir = item_rows(storage_dtype);
    const uint32_t fit = G ? stash_bytes(storage_dtype) / kStashTileBytes / G : 0;
    // four items per member, and at least one item for each of the CTA's warps (a group of one member: eight items)
    const uint32_t items = G && (static_cast<uint32_t>(kWarpsPerCta) + G - 1) / G > 4u ? (static_cast<uint32_t>(kWarpsPerCta) + G - 1) / G : 4u;
    return fit >= items * ir ? items * ir : (fit >= ir ? fit / ir * ir : fit);
}

struct DevTask {
    uint32_t id;
    uint32_t key0, key1;       // low / high half of the 64-bit seed
    uint32_t pad;
};

struct RetrieveArgs {
    const DevLayer* layers;
    const DevUnit* units;
    uint32_t n_units;
    uint32_t n_layers;
    const uint32_t* slot_of_pos;   // this task's sigma^-1, n_layers entries
    const void* const* base;       // device array of n_layers device pointers
    void* const* out;
    const void* M;                 // fp32 or bf16 arena
    DevTask task;
    float lambda;
};

struct AccumulateArgs {
    const DevLayer* layers;
    const DevUnit* units;
    uint32_t n_units;
    uint32_t n_layers;
    const uint32_t* src_of_slot;   // rows of sigma, one per task to sum, n_layers entries each
    const DevTask* tasks;          // matching task descriptors
    uint32_t n_tasks;
    uint32_t init_from_m;          // 0: start from +0 (compress); 1: start from M (add / remove)
    uint32_t negate;               // 1: subtract (remove)
    uint32_t has_base;             // 0: task tensors already hold deltas
    const void* const* base;       // device array [n_layers]
    const void* const* task_ptrs;  // device array [n_tasks][n_layers]
    void* M;                       // fp32 or bf16 arena
};

// compress over group units (randes_group.cu)
struct CompressGroupArgs {
    const DevLayer* layers;
    const DevUnit* units;          // group units only (nbc == 0; `layer` indexes `members`)
    uint32_t n_units;
    uint32_t n_layers;
    const uint32_t* src_of_slot;   // rows of sigma, one per task to sum
    const DevTask* tasks;
    uint32_t n_tasks;              // 2 .. kTaskChunk
    const void* const* base;       // device array [n_layers]
    const void* const* task_ptrs;  // device array [n_tasks][n_layers]
    void* M;
    const uint32_t* members;       // layers of every group, group after group, in member order
};

struct RetrieveBatchArgs {
    const DevLayer* layers;
    const DevUnit* units;
    uint32_t n_units;
    uint32_t n_layers;
    const uint32_t* slot_of_pos;   // all registered tasks' sigma^-1 rows, n_layers entries each
    const DevTask* tasks;          // all registered tasks' descriptors
    uint32_t task_rows[kTaskChunk];   // which rows to rebuild, in output order
    uint32_t n_tasks;              // <= kTaskChunk
    const void* const* base;       // device array [n_layers]
    void* const* out;              // device array [n_tasks][n_layers]
    const void* M;
    float lambda;
    const uint32_t* members;       // layers of every group, group after group, in member order (group units only)
};

constexpr int kGramBlocks = 10;   // blocks of 8 x 8 in the upper triangle of a kTaskChunk x kTaskChunk Gram matrix
constexpr int kGramPartialDoubles = kGramBlocks * 64;   // what one CTA hands to the final reduction

struct GramArgs {
    const DevLayer* layers;
    const DevUnit* units;
    uint32_t n_units;
    uint32_t n_layers;
    const uint32_t* src_of_slot;   // sigma rows of all registered tasks
    const DevTask* tasks;
    uint32_t n_tasks;              // <= kTaskChunk
    uint32_t has_base;
    const void* const* base;
    const void* const* task_ptrs;  // [n_tasks][n_layers]
    double* partial;               // [grid][kGramPartialDoubles]
};

// Launchers (randes_kernels.cu).  Return a cudaError_t as int.
int launch_retrieve(int storage_dtype, int out_dtype, int m_dtype, const RetrieveArgs& a, int grid, void* stream);
int launch_accumulate(int storage_dtype, int m_dtype, const AccumulateArgs& a, int grid, void* stream);
// add / remove of one model, bf16 weights, fp32 superposition, every layer cols % 8 == 0 and 16-byte aligned tensors
int launch_add_halves(const AccumulateArgs& a, int sm_count, void* stream);
// randes_context.cu: all of a plan's layers under a general diagonal context (plans with a RANDES_GAUSS group).
// The diagonal factors live in a table in the plan's workspace: table[task row][off[slot] + column], `stride` floats per
// row (every slot's span padded to a multiple of four, so that four neighbouring factors are one aligned 16-byte load).
// launch_context_fill writes the rows of newly registered tasks; for accumulate `table` points at the first task row
// to sum, for retrieve at the row of the task to rebuild.
struct ContextArgs {
    const float* table;
    const uint32_t* off;           // device array [n_layers]
    uint32_t stride;
};
int launch_context_fill(const ContextArgs& x, const DevLayer* layers, uint32_t n_layers, uint32_t max_cols, const DevTask* tasks,
                        uint32_t first_row, uint32_t n_rows, void* stream);
int launch_context_accumulate(int storage_dtype, const AccumulateArgs& a, const ContextArgs& x, void* stream);
int launch_context_retrieve(int storage_dtype, int out_dtype, const RetrieveArgs& a, const ContextArgs& x, void* stream);
// randes_group.cu: compress over group units.  `max_group` = the largest staged group.
int compress_group_prepare(int storage_dtype, int m_dtype);   // once per device: opts into the shared memory the kernel needs
bool compress_group_fits(int storage_dtype, uint32_t max_group, uint32_t n_tasks);
int launch_compress_groups(int storage_dtype, int m_dtype, const CompressGroupArgs& a, uint32_t max_group, int sm_count, void* stream);
// Resident CTAs per SM of each kernel (for sizing persistent grids); 0 if the
// kernels cannot run on the current device.  Also opts the kernels into the
// dynamic shared memory they need: call once per device before launching.
int retrieve_ctas_per_sm(int storage_dtype, int out_dtype, int m_dtype);
int accumulate_ctas_per_sm(int storage_dtype, int m_dtype, bool single_task);
// randes_diag.cu: the Gram kernel (one pass over the weights) plus the fixed-order reduction into gram
int launch_gram(int storage_dtype, const GramArgs& a, int grid, double* gram, void* stream);
int gram_ctas_per_sm(int storage_dtype);
// randes_batch.cu
int launch_retrieve_batch(int storage_dtype, int out_dtype, int m_dtype, const RetrieveBatchArgs& a, int grid, void* stream);
// batched retrieve over group units (fp32 weights and superposition): M and W_0 tiles of a whole group staged in shared memory
int retrieve_batch_group_prepare();
bool retrieve_batch_group_fits(uint32_t max_group, uint32_t n_tasks);
int launch_retrieve_batch_groups(int out_dtype, const RetrieveBatchArgs& a, uint32_t max_group, int sm_count, void* stream);


// Checked build (-DRANDES_CHECKED): the first bounds violation recorded by the kernels of each file, 0 if none
// (always 0 in the ordinary build); all-ones if the word could not be read.
unsigned long long violation_in_streaming_kernels();
unsigned long long violation_in_group_kernel();
unsigned long long violation_in_batch_kernels();

// randes_linear.cu: y = x W_0^T + lambda (x D) M_slot^T on the tensor cores (bf16 operands, fp32 accumulators).
// All return a cudaError_t as int.
int linear_prepare();   // opts the kernel into its shared memory on the current device
int launch_linear(const void* x, uint32_t n_tokens, const void* w0, const void* m_slot, uint32_t rows, uint32_t cols, bool flip,
                  uint32_t slot, const DevTask& task, float lambda, void* y, bool y_bf16, const uint32_t* gate,
                  unsigned long long wait_ns, void* stream, int* n_launched);   // gate: NULL or a device word to wait on; wait_ns: 0 = one second
int linear_giveups(unsigned int* count);   // CTAs that gave up on a bounded wait since the library was loaded (synchronises)

// Retrieve with its tables in a fixed device array inside the library (no workspace).
// Returns a cudaError_t as int, or -1 when the tables exceed kStaticScratchBytes.
constexpr size_t kStaticScratchBytes = 1u << 20;
size_t retrieve_static_bytes(uint32_t n_layers, uint32_t n_units);
int launch_retrieve_static(int storage_dtype, int out_dtype, int m_dtype, const DevLayer* layers, uint32_t n_layers, const DevUnit* units,
                           uint32_t n_units, const uint32_t* slot_of_pos, const void* const* base, void* const* out,
                           const void* M, const DevTask& task, float lambda, void* stream);

}  // namespace randes
