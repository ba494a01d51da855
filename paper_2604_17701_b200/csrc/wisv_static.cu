// wisv_lm_head_reduce_static: the LM-head reduction (logits -> argmax and
// log-sum-exp per row) for callers that must not allocate device memory.
//
// Some users of this library run inside a process where every byte of device
// memory is handed out up front - an inference server whose framework owns the
// whole GPU through its own pool, or a latency-critical loop that may not enter
// the driver's allocator because cudaMalloc / cudaFree stall the device.  Such
// callers cannot use wisv_create (it allocates a workspace).  For them this file
// keeps the scratch the LM-head pass needs - the bf16 copy of the rows and the
// per-tile (max, index, sum-exp) partials - in one fixed array that is part of the
// loaded library image.  Every GPU that loads the library holds the array
// (about 4 MiB) until the process exits.
//
// The array is shared by all calls on a device and keeps what the last call left
// in it: each call rewrites everything it later reads and clears its error word,
// and two calls that overlap on the GPU (different streams, no ordering) race on
// it - order them.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/wisv.h"
#include "wisv_gemm.cuh"

using namespace wisv;

namespace {

constexpr int kStaticMaxRows = WISV_STATIC_MAX_ROWS;      // one row tile
constexpr int kStaticMaxH = WISV_STATIC_MAX_H;
constexpr int kStaticMaxV = WISV_STATIC_MAX_V;
constexpr int kStaticTileN = 256;
constexpr int kStaticMaxTiles = kStaticMaxV / kStaticTileN;

constexpr size_t kOffX = 0;                                                        // bf16 [128][H]
constexpr size_t kBytesX = (size_t)kStaticMaxRows * kStaticMaxH * 2;
constexpr size_t kOffPart = kOffX + kBytesX;                                       // float4 [128][n_tiles]
constexpr size_t kBytesPart = (size_t)kStaticMaxRows * kStaticMaxTiles * 16;
constexpr size_t kOffTok = kOffPart + kBytesPart;                                  // int32 [128], all -1
constexpr size_t kOffTokLogit = kOffTok + kStaticMaxRows * 4;                      // float [128], unused sink
constexpr size_t kOffErr = kOffTokLogit + kStaticMaxRows * 4;                      // int32 error word
constexpr size_t kScratchBytes = kOffErr + 256;

// Device-resident scratch.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels receive the address obtained from it.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceSetup {
    bool ready = false;
    unsigned char* scratch = nullptr;
    int sm_count = 0;
    int max_smem = 0;
    EncodeTiledFn encode = nullptr;
};

constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// fp32 rows -> bf16 (nearest even) into the scratch copy; marks every row as carrying no draft token
__global__ void __launch_bounds__(256) static_cast_rows_kernel(const float* __restrict__ src,
                                                               __nv_bfloat16* __restrict__ dst,
                                                               int32_t* __restrict__ row_tok, int H)
{
    const int r = blockIdx.x;
    if (threadIdx.x == 0) row_tok[r] = -1;
    const float* s = src + (size_t)r * H;
    __nv_bfloat16* d = dst + (size_t)r * H;
    for (int i = threadIdx.x * 8; i < H; i += blockDim.x * 8) {
        const float4 a = *reinterpret_cast<const float4*>(s + i);
        const float4 b = *reinterpret_cast<const float4*>(s + i + 4);
        __nv_bfloat162 o[4];
        o[0] = __floats2bfloat162_rn(a.x, a.y);
        o[1] = __floats2bfloat162_rn(a.z, a.w);
        o[2] = __floats2bfloat162_rn(b.x, b.y);
        o[3] = __floats2bfloat162_rn(b.z, b.w);
        *reinterpret_cast<uint4*>(d + i) = *reinterpret_cast<const uint4*>(o);
    }
}

// one warp per row: merge the per-tile partials (lowest token id wins ties)
__global__ void __launch_bounds__(128) static_merge_rows_kernel(const float4* __restrict__ part, int n_tiles, int R,
                                                                const int32_t* __restrict__ err,
                                                                int32_t* __restrict__ argmax, float* __restrict__ lse)
{
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= R) return;
    float mx = -CUDART_INF_F, sum = 0.0f;
    int idx = 0x7fffffff;
    auto merge = [&](float omx, int oidx, float osum) {
        if (omx == -CUDART_INF_F && osum == 0.0f) return;
        if (omx > mx) { sum = sum * expf(mx - omx) + osum; mx = omx; idx = oidx; }
        else { sum += osum * expf(omx - mx); if (omx == mx && oidx < idx) idx = oidx; }
    };
    for (int n = lane; n < n_tiles; n += 32) {
        const float4 v = part[(size_t)r * n_tiles + n];
        merge(v.x, __float_as_int(v.y), v.z);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float omx = __shfl_xor_sync(0xffffffffu, mx, off);
        const int oidx = __shfl_xor_sync(0xffffffffu, idx, off);
        const float osum = __shfl_xor_sync(0xffffffffu, sum, off);
        merge(omx, oidx, osum);
    }
    if (lane == 0) {
        const bool failed = *err != 0;            // a bounded wait in the GEMM gave up
        argmax[r] = failed ? -1 : idx;
        lse[r] = failed ? CUDART_NAN_F : mx + logf(sum);
    }
}

int setup_device(int dev, DeviceSetup** out)
{
    if (dev < 0 || dev >= kMaxDevices) return WISV_ESHAPE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[dev];
    if (!s.ready) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
        if (prop.major != 10) return WISV_EARCH;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return WISV_ECUDA;
        }
        if (cudaFuncSetAttribute(gemm_rowreduce_kernel<EPI_LMHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)prop.sharedMemPerBlockOptin) != cudaSuccess) {
            (void)cudaGetLastError();
            return WISV_ECUDA;
        }
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return WISV_ECUDA;
        }
        s.scratch = static_cast<unsigned char*>(ptr);
        s.sm_count = prop.multiProcessorCount;
        s.max_smem = (int)prop.sharedMemPerBlockOptin;
        s.encode = reinterpret_cast<EncodeTiledFn>(fn);
        s.ready = true;
    }
    *out = &s;
    return WISV_OK;
}

int encode_bf16_2d(EncodeTiledFn fn, CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer,
                   uint32_t box_outer)
{
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_outer};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                          estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WISV_OK : WISV_ECUDA;
}

}  // namespace

extern "C" int wisv_lm_head_reduce_static(const void* lm_head, int32_t V, int32_t H, const float* target_hidden,
                                          int32_t R, int32_t* argmax, float* lse, void* cuda_stream)
{
    if (!lm_head || !target_hidden || !argmax || !lse) return WISV_EINVAL;
    if (R < 1 || R > kStaticMaxRows || V < 1 || V > kStaticMaxV || H < 64 || H > kStaticMaxH || H % 8)
        return WISV_ECAPACITY;
    if ((reinterpret_cast<uintptr_t>(lm_head) & 15u) || (reinterpret_cast<uintptr_t>(target_hidden) & 15u))
        return WISV_EALIGN;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
    DeviceSetup* s = nullptr;
    const int src = setup_device(dev, &s);
    if (src != WISV_OK) return src;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    __nv_bfloat16* X = reinterpret_cast<__nv_bfloat16*>(s->scratch + kOffX);
    float4* part = reinterpret_cast<float4*>(s->scratch + kOffPart);
    int32_t* row_tok = reinterpret_cast<int32_t*>(s->scratch + kOffTok);
    float* tok_logit = reinterpret_cast<float*>(s->scratch + kOffTokLogit);
    int32_t* err = reinterpret_cast<int32_t*>(s->scratch + kOffErr);

    const int tile_n = V >= kStaticTileN ? kStaticTileN : (V + 15) / 16 * 16;
    const int n_tiles = (V + tile_n - 1) / tile_n;

    // descriptors are plain host structs: encoding them touches no device memory
    CUtensorMap tmX, tmW;
    int rc = encode_bf16_2d(s->encode, &tmX, X, (uint64_t)H, (uint64_t)kStaticMaxRows, kTileM);
    if (rc == WISV_OK) rc = encode_bf16_2d(s->encode, &tmW, lm_head, (uint64_t)H, (uint64_t)V, (uint32_t)tile_n);
    if (rc != WISV_OK) return rc;

    // the error word must start at zero; rows beyond R in the bf16 copy are never reduced
    if (cudaMemsetAsync(err, 0, sizeof(int32_t), st) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
    static_cast_rows_kernel<<<R, 256, 0, st>>>(target_hidden, X, row_tok, H);

    GemmParams gp;
    memset(&gp, 0, sizeof gp);
    gp.rows = R; gp.n_total = V; gp.k_blocks = (H + kBlockK - 1) / kBlockK; gp.tile_n = tile_n;
    gp.m_tiles = 1; gp.n_tiles = n_tiles; gp.a_rows = kTileM; gp.mma_m = kTileM; gp.carry = 0; gp.part_stride = n_tiles;
    gp.k_splits = 1; gp.kb_per_split = gp.k_blocks;
    const size_t fixed = 1024 + gemm_tail_bytes(tile_n, 0);
    int stages = (int)(((size_t)s->max_smem - fixed) / gemm_stage_bytes(tile_n));
    if (stages > kMaxStages) stages = kMaxStages;
    gp.stages = stages;
    gp.err = err; gp.lm_part = part; gp.row_tok = row_tok; gp.tok_logit = tok_logit;
    const size_t smem = fixed + (size_t)stages * gemm_stage_bytes(tile_n);
    const int ctas = n_tiles < s->sm_count ? n_tiles : s->sm_count;
    gemm_rowreduce_kernel<EPI_LMHEAD><<<ctas, kGemmThreads, smem, st>>>(tmX, tmW, tmW, gp);

    static_merge_rows_kernel<<<(R + 3) / 4, 128, 0, st>>>(part, n_tiles, R, err, argmax, lse);
    if (cudaGetLastError() != cudaSuccess) return WISV_ECUDA;
    return WISV_OK;
}

extern "C" int wisv_debug_poison_static(void* cuda_stream)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return WISV_ECUDA; }
    DeviceSetup* s = nullptr;
    const int src = setup_device(dev, &s);
    if (src != WISV_OK) return src;
    if (cudaMemsetAsync(s->scratch, 0xFF, kScratchBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return WISV_ECUDA;
    }
    return WISV_OK;
}
