// Output tiles leaving through shared memory and the TMA: the epilogue of the GEMM kernels.
// A thread that holds one accumulator row per lane would store 16 bytes to 32 different rows with every
// instruction - 32 memory wavefronts each, which measured 12-14 % of a whole 32768 x 6144 x 4096 GEMM.
// Instead a warp lays its 32 rows out in shared memory as boxes of 64 bf16 columns (128 bytes per row, the
// 16-byte chunks XOR-swizzled by row as a SWIZZLE_128B tensor map expects, which also makes the shared-memory
// stores conflict-free) and one lane hands each finished box to the TMA, which writes whole lines and clips
// rows and columns past the matrix.
#pragma once
#include <cstdint>

namespace pec {
namespace sm100 {

constexpr uint32_t kStoreBoxCols = 64, kStoreBoxRows = 32, kStoreBoxBytes = kStoreBoxCols * 2 * kStoreBoxRows;   // 4 KB

// 8 bf16 (16 bytes) of row `lane` of a box at `box` (shared-memory address, 1024-byte aligned), chunk 0..7.
__device__ __forceinline__ void box_put(uint32_t box, int lane, int chunk, uint32_t p0, uint32_t p1, uint32_t p2, uint32_t p3)
{
    const uint32_t addr = box + (uint32_t)lane * 128u + ((uint32_t)(chunk ^ (lane & 7)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(p0), "r"(p1), "r"(p2), "r"(p3) : "memory");
}
// Box -> global memory at (column x, row y) of the tensor map (x a multiple of 8 elements); joins the thread's bulk group.
__device__ __forceinline__ void box_store(const void *tmap, uint32_t box, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(tmap), "r"(box), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until the TMA has read every box this thread committed (the shared memory may then be given up).
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// Orders the warp's ordinary shared-memory stores before the TMA's reads of them.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

}  // namespace sm100
}  // namespace pec
