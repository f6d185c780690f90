// Pieces the tensor-core translation units share: tile constants, the bounded mbarrier wait,
// packed-fp32 helpers, swizzled row stores, tensor-map builders and the per-device set-up table.
// Everything sits in an anonymous namespace: each translation unit gets its own copy.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include <mutex>

#include "arl2_internal.h"
#include "tc_ptx.cuh"

namespace arl2 {
namespace {

using namespace ptx;

constexpr int kTile = 128;               // query rows per tile = keys per tile = head dim
constexpr int kTileBytes = kTile * kTile * 2;
constexpr int kHalfBytes = kTileBytes / 2;  // one 64-column TMA box of a tile

constexpr uint32_t kSpinLimit = 1u << 24;

struct Abort {
    volatile int* flag;   // in shared memory
    uint32_t* status;     // device status block
    uint32_t limit;       // polls before a wait gives up
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Abort& ab, int site)
{
    for (uint32_t it = 0; it < ab.limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *ab.flag) return false;
    }
    *ab.flag = 1;
    if (atomicCAS(ab.status + kStatusError, 0u, (uint32_t)(-ARL2_ERR_TIMEOUT)) == 0u)
        ab.status[kStatusWhere] = (uint32_t)site;
    return false;
}

// Bounded wait that ignores the abort flag: used on the way out, for copies still in flight.
__device__ __forceinline__ void drain_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it)
        if (mbar_try_wait(bar, parity)) return;
}

__device__ __forceinline__ float sigmoid_fast(float x) { return 1.0f / (1.0f + __expf(-x)); }

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// packed pairs of fp32 (one 64-bit register pair per operand)
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}


// (cos, sin) of one rotation pair, stored as half2
__device__ __forceinline__ void unpack_cs(uint32_t h2, float& c, float& s)
{
    const __half2 v = *reinterpret_cast<const __half2*>(&h2);
    const float2 f = __half22float2(v);
    c = f.x;
    s = f.y;
}


__device__ __forceinline__ void store_row_bf16_swizzled(uint8_t* tile, int r, const uint32_t (&x)[128], float f)
{
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(x[c * 8 + 0]) * f, __uint_as_float(x[c * 8 + 1]) * f);
        v.y = pack_bf16(__uint_as_float(x[c * 8 + 2]) * f, __uint_as_float(x[c * 8 + 3]) * f);
        v.z = pack_bf16(__uint_as_float(x[c * 8 + 4]) * f, __uint_as_float(x[c * 8 + 5]) * f);
        v.w = pack_bf16(__uint_as_float(x[c * 8 + 6]) * f, __uint_as_float(x[c * 8 + 7]) * f);
        const int off = (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
        *reinterpret_cast<uint4*>(tile + off) = v;
    }
}
// half of row r (64 columns = one 64-column box of the tile)
__device__ __forceinline__ void store_half_row_bf16_swizzled(uint8_t* tile, int r, int half, const uint32_t (&x)[64], float f)
{
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(x[c * 8 + 0]) * f, __uint_as_float(x[c * 8 + 1]) * f);
        v.y = pack_bf16(__uint_as_float(x[c * 8 + 2]) * f, __uint_as_float(x[c * 8 + 3]) * f);
        v.z = pack_bf16(__uint_as_float(x[c * 8 + 4]) * f, __uint_as_float(x[c * 8 + 5]) * f);
        v.w = pack_bf16(__uint_as_float(x[c * 8 + 6]) * f, __uint_as_float(x[c * 8 + 7]) * f);
        *reinterpret_cast<uint4*>(tile + half * kHalfBytes + r * 128 + ((c ^ (r & 7)) << 4)) = v;
    }
}
__device__ __forceinline__ void store_row_bf16_global(__nv_bfloat16* dst, const uint32_t (&x)[128], float f)
{
#pragma unroll
    for (int c = 0; c < 16; ++c) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(x[c * 8 + 0]) * f, __uint_as_float(x[c * 8 + 1]) * f);
        v.y = pack_bf16(__uint_as_float(x[c * 8 + 2]) * f, __uint_as_float(x[c * 8 + 3]) * f);
        v.z = pack_bf16(__uint_as_float(x[c * 8 + 4]) * f, __uint_as_float(x[c * 8 + 5]) * f);
        v.w = pack_bf16(__uint_as_float(x[c * 8 + 6]) * f, __uint_as_float(x[c * 8 + 7]) * f);
        *reinterpret_cast<uint4*>(dst + c * 8) = v;
    }
}


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [B, L, H, 128] bf16 viewed as a 4-D tensor (d, h, l, b); box = 64 columns x 128 rows of one head.
int make_map_blhd(CUtensorMap* m, const void* base, const Shape& s)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return ARL2_ERR_CUDA; }
    cuuint64_t dims[4] = {(cuuint64_t)s.D, (cuuint64_t)s.H, (cuuint64_t)s.L, (cuuint64_t)s.B};
    cuuint64_t strides[3] = {(cuuint64_t)s.D * 2, (cuuint64_t)s.H * s.D * 2, (cuuint64_t)s.L * s.H * s.D * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled([B,L,H,D]) failed with %d", (int)r); return ARL2_ERR_CUDA; }
    return 0;
}

// [rows, 128] bf16 row-major; box = 64 columns x 128 rows.
int make_map_rows(CUtensorMap* m, const void* base, size_t rows, int box_rows = kTile)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return ARL2_ERR_CUDA; }
    cuuint64_t dims[2] = {(cuuint64_t)kTile, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kTile * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled([rows,128]) failed with %d", (int)r); return ARL2_ERR_CUDA; }
    return 0;
}


// Per-device, once, under a lock: the SM count and whatever the translation unit has to set for
// its kernels on that device (the opt-in to large dynamic shared memory belongs to the device
// that is current when it is set).
constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    int num_sms = 0;
};

template <typename K>
cudaError_t opt_in_smem(K kernel, int bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// `configure()` returns a cudaError_t and runs once per device with that device current.
template <typename F>
int device_setup_once(std::mutex& mutex, DeviceSetup (&table)[kMaxDevices], F configure, int* num_sms)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_error("cannot identify the current device (%s)", cudaGetErrorString(e));
        return ARL2_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mutex);
    DeviceSetup& d = table[dev];
    if (!d.ready) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
            set_error("cannot read the SM count of device %d", dev);
            return ARL2_ERR_CUDA;
        }
        e = configure();
        if (e != cudaSuccess) {
            set_error("cudaFuncSetAttribute(dynamic shared memory) on device %d: %s", dev, cudaGetErrorString(e));
            return ARL2_ERR_CUDA;
        }
        d.num_sms = sms;
        d.ready = true;
    }
    *num_sms = d.num_sms;
    return 0;
}

}  // namespace
}  // namespace arl2
