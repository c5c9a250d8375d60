// Host-side plumbing: device info cache, tensor-map encoding through the driver entry point,
// workspace init / status check, status strings.
#include "host.cuh"

#include <mutex>

namespace ef {

thread_local int g_last_cuda_error = 0;

namespace {
std::mutex g_mu;
constexpr int kMaxDevices = 64;
DeviceInfo g_info[kMaxDevices];
bool g_info_valid[kMaxDevices] = {};

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

EncodeTiledFn get_encode_fn() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_encode) return g_encode;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        g_last_cuda_error = static_cast<int>(e != cudaSuccess ? e : cudaErrorUnknown);
        return nullptr;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return g_encode;
}
}  // namespace

bool current_device_info(DeviceInfo* out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        g_last_cuda_error = static_cast<int>(e);
        return false;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_info_valid[dev]) {
        DeviceInfo di;
        di.device = dev;
        if ((e = cudaDeviceGetAttribute(&di.cc_major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&di.num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&di.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) !=
                cudaSuccess) {
            g_last_cuda_error = static_cast<int>(e);
            return false;
        }
        g_info[dev] = di;
        g_info_valid[dev] = true;
    }
    *out = g_info[dev];
    return true;
}

ef_status encode_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                           const uint64_t* strides_bytes, const uint32_t* box, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return EF_ERR_CUDA;
    cuuint64_t gdims[5];
    cuuint64_t gstrides[4];
    cuuint32_t gbox[5];
    cuuint32_t estr[5];
    for (int i = 0; i < rank; ++i) {
        gdims[i] = dims[i];
        gbox[i] = box[i];
        estr[i] = 1;
    }
    for (int i = 0; i + 1 < rank; ++i) gstrides[i] = strides_bytes[i];
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base),
                    gdims, gstrides, gbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = static_cast<int>(r);
        return EF_ERR_CUDA;
    }
    return EF_OK;
}

}  // namespace ef

extern "C" {

ef_status ef_workspace_init(void* ws, size_t ws_bytes, void* stream) {
    if (!ws) return EF_ERR_NULL;
    if (!ef::aligned(ws, 256)) return EF_ERR_ALIGN;
    if (ws_bytes < ef::kHeaderBytes) return EF_ERR_WORKSPACE;
    size_t n = ws_bytes < 65536 ? ws_bytes : 65536;
    EF_CUDA_CHECK(cudaMemsetAsync(ws, 0, n, static_cast<cudaStream_t>(stream)));
    return EF_OK;
}

ef_status ef_check_status(const void* ws, void* stream) {
    if (!ws) return EF_ERR_NULL;
    uint32_t word = 0;
    EF_CUDA_CHECK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    EF_CUDA_CHECK(cudaMemcpy(&word, ws, sizeof(word), cudaMemcpyDeviceToHost));
    return word == 0 ? EF_OK : EF_ERR_DEVICE_TIMEOUT;
}

const char* ef_status_string(ef_status s) {
    switch (s) {
        case EF_OK: return "ok";
        case EF_ERR_NULL: return "null pointer argument";
        case EF_ERR_SHAPE: return "non-positive or inconsistent dimensions";
        case EF_ERR_UNSUPPORTED: return "shape not covered by any kernel (no CPU fallback)";
        case EF_ERR_ALIGN: return "pointer not sufficiently aligned";
        case EF_ERR_WORKSPACE: return "workspace missing or too small";
        case EF_ERR_ARCH: return "device is not compute capability 10.x";
        case EF_ERR_CUDA: return "CUDA call failed (see ef_last_cuda_error)";
        case EF_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    }
    return "unknown status";
}

int ef_last_cuda_error(void) { return ef::g_last_cuda_error; }
int ef_version(void) { return 100; }

}  // extern "C"
