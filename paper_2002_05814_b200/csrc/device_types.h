// Structures shared by the host planner and the kernels: the device-resident object directory
// and the wave descriptors that are passed to the kernels as launch parameters.
#pragma once
#include <cstdint>

namespace hpl {

// One row of the object directory in device memory (arXiv 2002.05814, Section 3.2: per object its
// size and, per location, the progress; here one row per copy, progress as a chunk prefix).
struct DirRow {
    unsigned long long ptr;     // device address of this copy (0 while unknown)
    unsigned long long bytes;   // object size
    unsigned int n_chunks;
    unsigned int ready_chunks;  // chunks published so far; written by the host (copy engine), polled by kernels
    unsigned int dtype;
    unsigned int owner;
};
static_assert(sizeof(DirRow) == 32, "directory row layout");

// Error record the kernels write when a bounded wait runs out.
struct DeviceStatus {
    unsigned int error;      // 0, 1 = a wait on a progress counter expired, 2 = (bounds-checking build) an access outside its object
    unsigned int row;        // directory row that was waited for
    unsigned int chunk;      // chunk index that was waited for
    unsigned int abort;      // set together with error: other CTAs stop waiting
    unsigned long long waits;  // polls that did not succeed at the first look
    unsigned long long pad;
};

constexpr int kTileElems = 4096;        // elements of the reduce output per tile (one CTA iteration)
constexpr int kReduceThreads = 256;
constexpr int kMaxAcc = 8;              // accumulators (tree depth that can be fused in registers)
constexpr int kFanoutTileBytes = 32768;
constexpr int kFanoutThreads = 256;

enum : uint8_t { OPC_LOAD = 0, OPC_ADD_LOAD = 1, OPC_ADD_ACC = 2 };
enum : uint8_t { SRC_F32 = 0, SRC_BF16 = 1 };

// One step of a fused subtree evaluation.  LOAD: acc[a] = operand; ADD_LOAD: acc[a] = acc[a] (+) operand;
// ADD_ACC: acc[a] = acc[a] (+) acc[b].  The result of a task is acc[0].
// A step travels to the kernel as one 64-bit record: the operand's device address in the low 56 bits (known to
// the planner when the task is planned, so a launch does not depend on a directory update that is still on its
// way) and, in the top byte, code (2 bits), accumulator (3 bits), operand kind (1 bit).  The directory row of
// the operand travels beside it: it is what a polling task waits on.
struct ReduceStep {
    uint8_t code;
    uint8_t a;
    uint8_t b;
    uint8_t kind;       // SRC_F32 / SRC_BF16 for loads
    uint32_t row;       // directory row of the operand
    unsigned long long ptr;   // device address of the operand (loads)
};

constexpr int kRecShift = 56;
inline unsigned long long pack_step(const ReduceStep& st) {
    const unsigned long long meta = (unsigned long long)st.code | ((unsigned long long)st.a << 2) | ((unsigned long long)st.kind << 5);
    return (st.ptr & ((1ull << kRecShift) - 1)) | (meta << kRecShift);
}

// Tile size of a fan-out wave.  A tile is one CTA's unit of work: read once, then one bulk copy per receiver, a chain of
// latencies.  When an object has far fewer full tiles than there are resident CTAs (`slots`) the tiles are made smaller
// so that more CTAs share the chain -- 256 KiB to 16 receivers is 8 full tiles, or 64 tiles of 4 KiB on 64 CTAs, a
// third faster.  From a quarter of the slots upwards the full tile stays (measured: nothing to gain there).
inline uint32_t spread_tile_bytes(unsigned long long full_tiles, unsigned long long slots, uint32_t full, uint32_t gran, uint32_t floor) {
    if (full_tiles == 0 || full_tiles * 4 >= slots) return full;
    unsigned long long size = ((unsigned long long)full * full_tiles + slots - 1) / slots;
    size = (size + gran - 1) / gran * gran;
    if (size < floor) size = floor;
    return size > full ? full : (uint32_t)size;
}

struct ReduceTask {
    unsigned long long out_ptr;   // fp32 result (partial or target)
    unsigned long long elems;     // elements in the whole object
    uint32_t chunk_elems;
    uint32_t c_begin, c_end;      // chunk range [c_begin, c_end)
    uint32_t tiles_per_chunk;
    uint32_t tile_begin;          // index of this task's first tile within the wave
    uint32_t step_begin, n_steps;
    uint32_t red_op;
    uint32_t poll;                // 1: operands' progress counters must be polled before each chunk
    uint32_t fan_begin, n_fan;    // receivers of a broadcast of this result that take each tile straight from the
                                  // reduce (indices into ReduceWave::fan_ptrs); 0 = the result goes to out_ptr only
    uint32_t out_row;             // directory row of the result buffer (read by the bounds-checking build only)
};

constexpr int kMaxTasksPerWave = 24;
constexpr int kMaxStepsPerWave = 640;
constexpr int kMaxFusedDst = 128;       // receivers served by the reduce tasks of one wave

struct ReduceWave {
    const DirRow* dir;
    DeviceStatus* status;
    unsigned long long budget_ns;
    uint32_t n_tasks;
    uint32_t total_tiles;
    ReduceTask tasks[kMaxTasksPerWave];
    unsigned long long recs[kMaxStepsPerWave];   // packed steps (pack_step)
    uint32_t rows[kMaxStepsPerWave];             // directory row of each load step's operand
    unsigned long long fan_ptrs[kMaxFusedDst];   // device addresses of receivers' buffers (fused reduce -> fan-out)
    uint32_t fan_rows[kMaxFusedDst];             // their directory rows (bounds-checking build)
};

struct FanoutTask {
    unsigned long long src_ptr;      // device address of the copy that is read
    uint32_t src_row;                // its directory row (polled when the task polls)
    uint32_t c_begin, c_end;
    uint32_t tiles_per_chunk;
    uint32_t tile_bytes;             // bytes per tile: kFanoutTileBytes, or fewer for small objects (a multiple of 512)
    uint32_t tile_begin;
    uint32_t dst_begin, n_dst;
    uint32_t poll;
    unsigned long long bytes;        // object size
    unsigned long long chunk_bytes;
};

constexpr int kMaxFanoutTasks = 24;
constexpr int kMaxFanoutDst = 1024;

struct FanoutWave {
    const DirRow* dir;
    DeviceStatus* status;
    unsigned long long budget_ns;
    uint32_t n_tasks;
    uint32_t total_tiles;
    FanoutTask tasks[kMaxFanoutTasks];
    unsigned long long dst_ptrs[kMaxFanoutDst];   // device addresses of the receivers' buffers
    uint32_t dst_rows[kMaxFanoutDst];             // their directory rows (bounds-checking build)
};

// Launchers (kernels.cu).  Return a cudaError_t as int.
int launch_reduce_wave(const ReduceWave& w, int n_acc, bool bf16, bool fan, int grid, void* stream);
int launch_fanout_wave(const FanoutWave& w, int grid, void* stream);
int reduce_ctas_per_sm(int n_acc, bool bf16, bool fan);
int fanout_ctas_per_sm();

}  // namespace hpl
