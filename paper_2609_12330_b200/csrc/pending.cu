// Entry points whose kernels are not built yet: they validate nothing and report
// EF_ERR_UNSUPPORTED (there is no fallback path).  Each moves to its own file when built.
#include "host.cuh"

extern "C" {
size_t ef_qknorm_attn_workspace_bytes(int, int, int, int) { return ef::kHeaderBytes; }
ef_status ef_qknorm_attn(const void*, const void*, const void*, const void*, const void*, void*, int, int, int, int,
                         float, float, int, void*, size_t, void*) {
    return EF_ERR_UNSUPPORTED;
}
}
