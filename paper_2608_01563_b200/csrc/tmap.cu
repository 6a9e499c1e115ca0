// Host-side construction of TMA tensor maps.  The driver's encoder is reached through
// the runtime (cudaGetDriverEntryPoint), so the library does not link libcuda directly.
#include <mutex>

#include "kernels.h"

namespace mgn {
namespace {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode()
{
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    });
    return fn;
}

// Small cache of encoded maps.  A training or serving loop calls the library with the same
// buffers and shapes step after step; encoding a map takes about a microsecond of host time, and
// a call needs three to five of them, which shows in calls that last a few tens of microseconds.
// Key: everything the encoder is given.  Least-recently-used replacement, one mutex.
struct MapKey {
    const void* base;
    int elem_bytes, is_bf16, BH, S, D, box_d, box_rows;
    bool operator==(const MapKey& o) const {
        return base == o.base && elem_bytes == o.elem_bytes && is_bf16 == o.is_bf16 && BH == o.BH && S == o.S &&
               D == o.D && box_d == o.box_d && box_rows == o.box_rows;
    }
};
constexpr int kCacheSlots = 64;
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    unsigned long long last_use;   // 0: empty
};
MapSlot g_cache[kCacheSlots];
unsigned long long g_tick = 0;
std::mutex g_cache_mu;

}  // namespace

int make_tmap_3d(CUtensorMap* out, const void* base, int elem_bytes, int is_bf16, int BH, int S, int D, int box_d,
                 int box_rows)
{
    const MapKey key{base, elem_bytes, is_bf16, BH, S, D, box_d, box_rows};
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        for (MapSlot& sl : g_cache)
            if (sl.last_use != 0 && sl.key == key) {
                sl.last_use = ++g_tick;
                *out = sl.map;
                return 0;
            }
    }
    EncodeFn enc = get_encode();
    if (!enc) return 1;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S), static_cast<cuuint64_t>(BH)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * elem_bytes,
                                   static_cast<cuuint64_t>(S) * D * elem_bytes};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(box_d), static_cast<cuuint32_t>(box_rows), 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    auto encode = [&] {
        return enc(out, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                   const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    };
    CUresult r = encode();
    if (r != CUDA_SUCCESS) {
        // The encoder is a driver call and wants a current context: a host thread whose first CUDA work is
        // this library call has none bound yet (the runtime binds it lazily, and nothing before this point
        // needs it).  Bind it -- cudaFree(nullptr) allocates and frees nothing -- and try once more.
        cudaFree(nullptr);
        r = encode();
    }
    if (r != CUDA_SUCCESS) return 2;
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        MapSlot* victim = &g_cache[0];
        for (MapSlot& sl : g_cache)
            if (sl.last_use < victim->last_use) victim = &sl;
        victim->key = key;
        victim->map = *out;
        victim->last_use = ++g_tick;
    }
    return 0;
}

}  // namespace mgn
