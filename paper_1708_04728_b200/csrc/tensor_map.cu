// Tensor-map (TMA descriptor) encoding for all kernels of the library, with a process-wide memo.
//
// A tensor map depends only on the arguments it is encoded from (address, extents, strides, box, swizzle), so the
// 128-byte result is kept in a table keyed by exactly those arguments: a layer called again on the same buffers —
// every layer of a prepared network, every step of a training loop — costs one table lookup per map instead of a
// driver call.  The table is bounded (it is emptied when it reaches MAX_ENTRIES) and guarded by a mutex.
// Integer tunables from the environment are read once per name and kept the same way.
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_map>

#include "conv_common.cuh"

namespace dr {

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*PFN_encodeIm2col)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                     const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static PFN_encodeTiled g_encode_tiled = nullptr;
static PFN_encodeIm2col g_encode_im2col = nullptr;
static std::atomic<long long> g_driver_encodes{0};

static bool load_encoders() {
    if (g_encode_tiled && g_encode_im2col) return true;
    cudaDriverEntryPointQueryResult q;
    void* f = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !f) return false;
    g_encode_tiled = (PFN_encodeTiled)f;
    f = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !f) return false;
    g_encode_im2col = (PFN_encodeIm2col)f;
    return true;
}

namespace {
struct Key {
    uint64_t ptr;
    uint64_t dims[5], strides[4];
    uint32_t box[5], es[5];
    int32_t lower[2], upper[2];
    uint32_t rank, mode, channels, pixels, swizzle, l2;
    bool operator==(const Key& o) const { return std::memcmp(this, &o, sizeof(Key)) == 0; }
};
struct KeyHash {
    size_t operator()(const Key& k) const {
        const unsigned char* b = reinterpret_cast<const unsigned char*>(&k);
        uint64_t h = 1469598103934665603ull;
        for (size_t i = 0; i < sizeof(Key); ++i) { h ^= b[i]; h *= 1099511628211ull; }
        return (size_t)h;
    }
};
struct alignas(64) Map64 { CUtensorMap m; };
constexpr size_t MAX_ENTRIES = 8192;
std::mutex g_mu;
std::unordered_map<Key, Map64, KeyHash> g_memo;
std::unordered_map<std::string, int> g_tunables;

bool lookup(const Key& k, CUtensorMap* out) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_memo.find(k);
    if (it == g_memo.end()) return false;
    std::memcpy(out, &it->second.m, sizeof(CUtensorMap));
    return true;
}
void remember(const Key& k, const CUtensorMap* m) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_memo.size() >= MAX_ENTRIES) g_memo.clear();
    Map64 v;
    std::memcpy(&v.m, m, sizeof(CUtensorMap));
    g_memo.emplace(k, v);
}
}  // namespace

// Tiled map over a bf16 tensor of `rank` dimensions (innermost first); element strides 1, no interleave, zero fill.
int tmap_tiled(CUtensorMap* map, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
               CUtensorMapSwizzle swizzle, CUtensorMapL2promotion l2) {
    if (rank < 1 || rank > 5 || !load_encoders()) return DR_ERR_CUDA;
    Key k;
    std::memset(&k, 0, sizeof(k));
    k.ptr = (uint64_t)(uintptr_t)ptr; k.rank = (uint32_t)rank; k.mode = 0; k.swizzle = (uint32_t)swizzle; k.l2 = (uint32_t)l2;
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; k.es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
    if (lookup(k, map)) return DR_OK;
    g_driver_encodes.fetch_add(1, std::memory_order_relaxed);
    if (g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, l2, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DR_ERR_CUDA;
    remember(k, map);
    return DR_OK;
}

// im2col-mode map over an NHWC bf16 tensor (dims C, W, H, N): `channels` x `pixels` per load, the bounding box
// corners of the positions the filter's first tap visits, traversal stride `stride` in W and H.
int tmap_im2col(CUtensorMap* map, const void* ptr, const cuuint64_t dims[4], const cuuint64_t strides[3], const int lower[2], const int upper[2],
                unsigned channels, unsigned pixels, unsigned stride, CUtensorMapL2promotion l2) {
    if (!load_encoders()) return DR_ERR_CUDA;
    Key k;
    std::memset(&k, 0, sizeof(k));
    k.ptr = (uint64_t)(uintptr_t)ptr; k.rank = 4; k.mode = 1; k.swizzle = (uint32_t)CU_TENSOR_MAP_SWIZZLE_128B; k.l2 = (uint32_t)l2;
    k.channels = channels; k.pixels = pixels;
    const cuuint32_t es[4] = {1, stride, stride, 1};
    for (int i = 0; i < 4; ++i) { k.dims[i] = dims[i]; k.es[i] = es[i]; }
    for (int i = 0; i < 3; ++i) k.strides[i] = strides[i];
    for (int i = 0; i < 2; ++i) { k.lower[i] = lower[i]; k.upper[i] = upper[i]; }
    if (lookup(k, map)) return DR_OK;
    g_driver_encodes.fetch_add(1, std::memory_order_relaxed);
    if (g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, lower, upper, channels, pixels, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, l2, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DR_ERR_CUDA;
    remember(k, map);
    return DR_OK;
}

long long tmap_driver_encodes() { return g_driver_encodes.load(std::memory_order_relaxed); }

// Integer tunable from the environment (for A/B timing); the environment is read once per name.
int tunable(const char* name, int dflt) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_tunables.find(name);
    if (it != g_tunables.end()) return it->second == INT32_MIN ? dflt : it->second;
    const char* v = getenv(name);
    g_tunables.emplace(name, v ? atoi(v) : INT32_MIN);
    return v ? atoi(v) : dflt;
}

}  // namespace dr

extern "C" long long dr_tensor_map_encodes(void) { return dr::tmap_driver_encodes(); }
