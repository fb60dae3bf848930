// hpl_reduce_noalloc: the fused tree reduce for callers that must not allocate.
//
// Who needs this: code that runs where a device allocation is forbidden or would stall -- inside a
// memory-pool or caching-allocator callback, in a latency-critical serving loop that has frozen
// its memory map, in a process whose device memory is entirely handed out to other owners.  Such
// callers cannot give the library an arena either, so the small amount of device memory the reduce
// kernel needs besides its inputs and output (the directory rows of the operands and the status
// record of the bounded waits) lives in the file-scope array below.  The array is part of the
// loaded library image: every GPU that loads the library holds these few KiB until the process
// exits.
//
// The array's name is only a handle in host code; its device address is looked up once per
// device with cudaGetSymbolAddress and that address is what the kernels receive.
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

#include "../../include/hpl.h"
#include "device_types.h"
#include "sched_reduce.h"

namespace hpl {

constexpr int kNoAllocMaxSources = HPL_NOALLOC_MAX_SOURCES;
constexpr size_t kNoAllocRowsBytes = sizeof(DirRow) * kNoAllocMaxSources;
constexpr size_t kNoAllocScratchBytes = kNoAllocRowsBytes + 256;   // rows, then the status record

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

struct NoAllocRows {
    unsigned long long ptr[kNoAllocMaxSources];
    unsigned long long bytes;
    unsigned int n, dtype;
};

// Writes the operands' directory rows into the scratch array and clears the status record, which must
// start at zero for every call (the array keeps whatever the previous call left).
__global__ void noalloc_fill_kernel(const __grid_constant__ NoAllocRows r) {
    DirRow* rows = reinterpret_cast<DirRow*>(g_noalloc_scratch);
    for (unsigned int i = threadIdx.x; i < r.n; i += blockDim.x) {
        DirRow d;
        d.ptr = r.ptr[i];
        d.bytes = r.bytes;
        d.n_chunks = 1;
        d.ready_chunks = 1;   // every operand is complete: nothing is polled
        d.dtype = r.dtype;
        d.owner = i;
        rows[i] = d;
    }
    if (threadIdx.x == 0) {
        DeviceStatus z = {};
        *reinterpret_cast<DeviceStatus*>(g_noalloc_scratch + kNoAllocRowsBytes) = z;
    }
}

namespace {

std::mutex g_mu;
std::vector<unsigned char*> g_scratch_of_device;   // device address of the array, per device ordinal
std::vector<int> g_sm_of_device;

// Steps of the whole tree with every member ready, in the association order of the tree: first child's
// subtree, the node's own object, then the other children (a fused child subtree takes one more accumulator).
void gen_all_ready(const ReduceTreeSchedule& s, int u, int acc, uint8_t kind, std::vector<ReduceStep>& out, int& n_acc) {
    if (acc + 1 > n_acc) n_acc = acc + 1;
    auto load = [&](int q, uint8_t code) {
        ReduceStep st{};
        st.code = code;
        st.a = (uint8_t)acc;
        st.kind = kind;
        st.row = (uint32_t)s.object_at(q);   // object i sits in row i
        out.push_back(st);
    };
    if (s.is_leaf(u)) {
        load(u, OPC_LOAD);
        return;
    }
    const int c0 = s.first_child(u), nc = s.n_children(u);
    for (int j = 0; j < nc; ++j) {
        const int cj = c0 + j;
        if (s.is_leaf(cj)) {
            load(cj, j == 0 ? OPC_LOAD : OPC_ADD_LOAD);
        } else if (j == 0) {
            gen_all_ready(s, cj, acc, kind, out, n_acc);
        } else {
            gen_all_ready(s, cj, acc + 1, kind, out, n_acc);
            ReduceStep st{};
            st.code = OPC_ADD_ACC;
            st.a = (uint8_t)acc;
            st.b = (uint8_t)(acc + 1);
            out.push_back(st);
        }
        if (j == 0) load(u, OPC_ADD_LOAD);
    }
}

}  // namespace
}  // namespace hpl

using namespace hpl;

extern "C" int hpl_reduce_noalloc(const void* const* src_bufs, int32_t n, int32_t degree, int32_t op, int32_t dtype,
                                  uint64_t elems, void* out, void* cuda_stream) {
    if (!src_bufs || !out || n < 1 || degree < 1 || elems == 0) return HPL_ERR_INVALID;
    if (n > kNoAllocMaxSources || elems > HPL_NOALLOC_MAX_ELEMS) return HPL_ERR_INVALID;   // beyond the fixed scratch / index range
    if (op < HPL_SUM || op > HPL_MAX || (dtype != HPL_F32 && dtype != HPL_BF16)) return HPL_ERR_INVALID;
    if ((uintptr_t)out % 16) return HPL_ERR_INVALID;
    for (int i = 0; i < n; ++i)
        if (!src_bufs[i] || (uintptr_t)src_bufs[i] % 16) return HPL_ERR_INVALID;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HPL_ERR_CUDA;
    unsigned char* scratch = nullptr;
    int n_sm = 0;
    {
        // first call on this device: look the array's device address up (not an allocation)
        std::lock_guard<std::mutex> lock(g_mu);
        if ((int)g_scratch_of_device.size() <= dev) {
            g_scratch_of_device.resize(dev + 1, nullptr);
            g_sm_of_device.resize(dev + 1, 0);
        }
        if (!g_scratch_of_device[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return HPL_ERR_CUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return HPL_ERR_CUDA;
            g_scratch_of_device[dev] = (unsigned char*)p;
            g_sm_of_device[dev] = sms;
        }
        scratch = g_scratch_of_device[dev];
        n_sm = g_sm_of_device[dev];
    }

    // the tree: objects arrive in index order, all complete
    std::vector<int64_t> ids(n);
    for (int i = 0; i < n; ++i) ids[i] = i;
    ReduceTreeSchedule sched(ids, n, degree);
    for (int i = 0; i < n; ++i) sched.arrive(i);
    std::vector<ReduceStep> steps;
    int n_acc = 1;
    gen_all_ready(sched, 0, 0, dtype == HPL_BF16 ? SRC_BF16 : SRC_F32, steps, n_acc);
    if (n_acc > kMaxAcc || steps.size() > (size_t)kMaxStepsPerWave) return HPL_ERR_INVALID;   // tree too deep to fuse

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    static thread_local NoAllocRows rows;
    for (int i = 0; i < n; ++i) rows.ptr[i] = (unsigned long long)(uintptr_t)src_bufs[i];
    rows.bytes = elems * (dtype == HPL_BF16 ? 2ull : 4ull);
    rows.n = (unsigned)n;
    rows.dtype = (unsigned)dtype;
    noalloc_fill_kernel<<<1, 256, 0, stream>>>(rows);
    if (cudaGetLastError() != cudaSuccess) return HPL_ERR_CUDA;

    static thread_local ReduceWave w;
    w.dir = reinterpret_cast<const DirRow*>(scratch);
    w.status = reinterpret_cast<DeviceStatus*>(scratch + kNoAllocRowsBytes);
    w.budget_ns = 1000000ull;
    w.n_tasks = 1;
    const uint32_t chunk_elems = 1u << 22;   // tiling unit only: there is one task over the whole object
    const uint32_t C = (uint32_t)((elems + chunk_elems - 1) / chunk_elems);
    const uint32_t ce = elems < chunk_elems ? (uint32_t)elems : chunk_elems;
    const uint32_t tpc = (ce + kTileElems - 1) / kTileElems;
    ReduceTask& t = w.tasks[0];
    t.out_ptr = (unsigned long long)(uintptr_t)out;
    t.elems = elems;
    t.chunk_elems = ce;
    t.c_begin = 0;
    t.c_end = C;
    t.tiles_per_chunk = tpc;
    t.tile_begin = 0;
    t.step_begin = 0;
    t.n_steps = (uint32_t)steps.size();
    t.red_op = (uint32_t)op;
    t.poll = 0;
    t.fan_begin = t.n_fan = 0;
    t.out_row = 0xFFFFFFFFu;   // the output has no directory row: the bounds-checking build leaves this task alone
    for (size_t i = 0; i < steps.size(); ++i) {
        w.recs[i] = pack_step(steps[i]);   // address 0: the kernel takes it from the row in the scratch array
        w.rows[i] = steps[i].row;
    }
    w.total_tiles = C * tpc;
    const bool bf16 = dtype == HPL_BF16;
    int occ = reduce_ctas_per_sm(n_acc, bf16, false);
    uint64_t grid = (uint64_t)n_sm * (occ < 1 ? 1 : occ);
    if (grid > w.total_tiles) grid = w.total_tiles;
    if (grid < 1) grid = 1;
    if (launch_reduce_wave(w, n_acc, bf16, false, (int)grid, stream) != 0) return HPL_ERR_CUDA;
    return HPL_OK;
}
