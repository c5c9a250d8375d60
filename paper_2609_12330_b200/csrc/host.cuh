// Host-side plumbing shared by the entry points: argument checks, the cached driver entry
// point for tensor-map encoding, device properties, error bookkeeping.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/equiforge.h"

namespace ef {

// Workspace header: [0,16) status word, [16,256) reserved, [256, kHeaderBytes) arrival counters.
constexpr size_t kHeaderBytes = 4096;
constexpr size_t kCounterOffset = 256;
constexpr size_t kMaxCounters = (kHeaderBytes - kCounterOffset) / sizeof(uint32_t);  // 960
// [kHeaderBytes, kDataOffset) holds only words that are zero between calls (per-tile / per-unit arrival counters) and is
// inside the window ef_workspace_init clears; whatever a call leaves behind non-zero (partial slots, T, Khat) starts at
// kDataOffset -- at a FIXED offset, so that calls of one entry point with different shapes can share a workspace.
constexpr size_t kDataOffset = 65536;

extern thread_local int g_last_cuda_error;

struct DeviceInfo {
    int device = -1;
    int cc_major = 0;
    int num_sms = 0;
    int max_smem_optin = 0;
};
// Properties of the CURRENT device (cached per device id).  Returns false on CUDA failure.
bool current_device_info(DeviceInfo* out);

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Encode a tiled tensor map over bf16 data.  dims/box are innermost-first; strides_bytes[i] is
// the byte stride of dimension i+1 (rank-1 entries).  swizzle: CU_TENSOR_MAP_SWIZZLE_*.
ef_status encode_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                           const uint64_t* strides_bytes, const uint32_t* box, CUtensorMapSwizzle swizzle);

// Launch with programmatic stream serialization (see pdl_wait() on the device side).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Skinny-M tail of the LoRA-fused linear (csrc/skinny.cu), used by ef_lora_linear for M <= 16.
namespace skinny {
constexpr int kLoraTailMaxM = 16;
size_t lora_tail_counters_bytes(int N);
size_t lora_tail_partials_bytes();
ef_status launch_lora_head(const void* X, const void* A, void* T, int M, int K, float alpha, uint32_t* status,
                           uint32_t* counters, float* partials, const DeviceInfo& di, cudaStream_t stream);
ef_status launch_lora_tail(const void* X, const void* W, const void* T, const void* Bm, void* Y, int M, int K, int N,
                           uint32_t* status, uint32_t* counters, float* partials, const DeviceInfo& di, cudaStream_t stream);
}  // namespace skinny

#define EF_CUDA_CHECK(expr)                                  \
    do {                                                     \
        cudaError_t _e = (expr);                             \
        if (_e != cudaSuccess) {                             \
            ::ef::g_last_cuda_error = static_cast<int>(_e);  \
            return EF_ERR_CUDA;                              \
        }                                                    \
    } while (0)

}  // namespace ef
