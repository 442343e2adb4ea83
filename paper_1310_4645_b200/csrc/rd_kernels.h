// Launch interface between the C ABI (host C++) and the CUDA kernels.
#ifndef RD_KERNELS_H_
#define RD_KERNELS_H_

#include <cstddef>
#include <cstdint>

namespace rd {

// One unit of work of the tree kernel: a run of elements inside one segment.
struct TileDesc {
    uint64_t elem_off;   // first element
    uint32_t len;        // elements in the tile (<= tile capacity)
    uint32_t prog;       // first word of the segment's program in the operation table
};

constexpr int kTreeThreads = 256;
constexpr int kPackedPtrs = 256;      // up to this many input pointers travel as kernel parameters

struct TreeLaunch {
    const void *const *host_ptrs;     // p device pointers (host array)
    const void *const *dev_ptr_table; // device copy of the same, used when p > kPackedPtrs
    void *out;
    const TileDesc *tiles;            // device
    const uint32_t *ops;              // device
    uint32_t n_tiles;
    int p;
    int stack_depth;
    int dtype, op;                    // rd_dtype_t, rd_op_t
    int vec;                          // 4: 128-bit path, 1: element path
    int sm_count;
    int device;
    void *stream;
    // streaming variant only
    const uint32_t *cta_first;        // device: n_ctas + 1 offsets into tiles
    uint32_t n_ctas;
    int stages;
    int stage_elems;
    int *status;                      // device word
};

// Elements one tile of the element-path kernel may hold for the given vector width.
uint32_t tree_tile_elems(int vec);
// Launches the tree kernel; returns a cudaError_t value (0 = success).
int launch_tree(const TreeLaunch &a);
// Streaming variant (128-bit path): stage size for a CTA's share of the message, ring shape for a
// stack depth and the SM's shared memory, launch.
int stream_stage_elems(uint64_t elems_per_cta);
void stream_shape(int stack_depth, int smem_per_sm, int stage_elems, int *ctas_per_sm, int *stages);
size_t stream_smem_bytes(int stages, int depth, int stage_elems);
int launch_tree_stream(const TreeLaunch &a);

}  // namespace rd
#endif
