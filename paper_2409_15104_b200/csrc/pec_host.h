// Host-side helpers shared by the launchers of the tensor-core kernels: TMA tensor-map encoding
// with a small cache, and per-device one-time kernel set-up.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <cstring>
#include <mutex>

namespace pec {
namespace host {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point (the library does not link libcuda).
inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// What determines a bf16 tensor map of up to three dimensions with 128-byte swizzle.
struct MapKey {
    const void *base;
    uint64_t dims[3];
    uint64_t strides[2];       // bytes
    uint32_t box[3];
    uint32_t rank;
    bool operator==(const MapKey &o) const { return std::memcmp(this, &o, sizeof(MapKey)) == 0; }
};

// Encoded maps are pure functions of their key, so a launcher that is called with the same tensors
// again (every step of a prefill, every layer of a model) can reuse them.  Direct-mapped, per thread:
// no locking, and a stale entry is merely overwritten.
inline bool cached_map(CUtensorMap *out, const MapKey &key)
{
    constexpr int kSlots = 64;
    struct Entry { MapKey key; CUtensorMap map; bool valid; };
    static thread_local Entry cache[kSlots] = {};
    uint64_t h = reinterpret_cast<uintptr_t>(key.base) * 0x9E3779B97F4A7C15ull;
    h ^= (key.dims[2] + 0x7F4A7C15ull * key.dims[1]) * 0xC2B2AE3D27D4EB4Full;
    h ^= key.strides[1] * 0x165667B19E3779F9ull + key.box[2];
    Entry &e = cache[(h >> 40) % kSlots];
    if (e.valid && e.key == key) { *out = e.map; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {key.dims[0], key.dims[1], key.dims[2]};
    cuuint64_t strides[2] = {key.strides[0], key.strides[1]};
    cuuint32_t box[3] = {key.box[0], key.box[1], key.box[2]};
    cuuint32_t estr[3] = {1, 1, 1};
    if (fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, key.rank, const_cast<void *>(key.base), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.key = key; e.map = *out; e.valid = true;
    return true;
}

// [rows, heads, 128] bf16 tensor with element strides (stride_t, stride_h); box = 64 channels x 1 head x 128 rows.
inline bool make_qkv_map(CUtensorMap *map, const void *base, int64_t rows, int32_t heads, int64_t stride_t, int64_t stride_h)
{
    MapKey key;
    std::memset(&key, 0, sizeof(key));
    key.base = base;
    key.dims[0] = 128; key.dims[1] = (uint64_t)heads; key.dims[2] = (uint64_t)(rows > 0 ? rows : 1);
    key.strides[0] = (uint64_t)stride_h * 2; key.strides[1] = (uint64_t)stride_t * 2;
    key.box[0] = 64; key.box[1] = 1; key.box[2] = 128;
    key.rank = 3;
    return cached_map(map, key);
}

// [rows, cols] bf16 matrix, row stride in elements; box = 64 columns x box_rows rows.
inline bool make_matrix_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t stride, int box_rows)
{
    MapKey key;
    std::memset(&key, 0, sizeof(key));
    key.base = base;
    key.dims[0] = (uint64_t)cols; key.dims[1] = (uint64_t)rows;
    key.strides[0] = (uint64_t)stride * 2;
    key.box[0] = 64; key.box[1] = (uint32_t)box_rows;
    key.rank = 2;
    return cached_map(map, key);
}

// Runs `setup` (which returns true on success) once per device for one kernel; later calls on that
// device only read a flag (under the mutex).  `state` is a zero-initialised array of kMaxDevices flags owned by the caller.
constexpr int kMaxDevices = 64;
template <class Setup>
inline bool once_per_device(unsigned char (&state)[kMaxDevices], std::mutex &mu, Setup setup)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (state[dev]) return true;
    if (!setup()) return false;
    state[dev] = 1;
    return true;
}

}  // namespace host
}  // namespace pec
