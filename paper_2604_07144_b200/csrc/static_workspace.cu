// ap_attention_iteration_static: attention with the split-K scratch held in a
// fixed device array that is part of the library image, for callers that must
// not allocate device memory (see the declaration in ap_serving.h).
#include "internal.h"

namespace {

constexpr size_t kStaticWorkspaceBytes = AP_STATIC_WORKSPACE_BYTES;

// The scratch itself.  It lives in every CUDA context that loads this library,
// from load until the process exits.  In host code this name is only a handle
// for the runtime's symbol table, never an address a kernel may be given: the
// device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

constexpr int kMaxDevices = 64;
void *g_workspace_addr[kMaxDevices] = {};

// Device address of the array on `device`, which must be the current device.
int static_workspace_address(int device, void **addr) {
    if (device < 0 || device >= kMaxDevices) return AP_ERR_UNSUPPORTED;
    if (!g_workspace_addr[device]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return AP_ERR_CUDA;
        }
        g_workspace_addr[device] = p;
    }
    *addr = g_workspace_addr[device];
    return AP_OK;
}

}  // namespace

namespace ap {

// Set-up step, run by ap_kv_pool_create with the pool's device current: looks the array's device
// address up once per device.  The first lookup may make the runtime load this file's module (which
// is when the array comes into being on that device), so it belongs where allocation is expected
// and no stream is being captured, not in the serving loop.
int prepare_static_workspace(int device) {
    void *unused = nullptr;
    return static_workspace_address(device, &unused);
}

}  // namespace ap

extern "C" {

size_t ap_static_workspace_bytes(void) { return kStaticWorkspaceBytes; }

int ap_attention_iteration_static(ap_kv_pool *pool, const ap_plan *plan, const void *q, void *out, float *lse,
                                  void *stream) {
    if (!pool || !plan || plan->pool != pool) return AP_ERR_INVALID_ARG;
    if (pool->desc.device < 0) return AP_ERR_CUDA;
    if (plan->info.n_new == 0) return AP_OK;
    if (!q || !out || (((uintptr_t)q | (uintptr_t)out) & 15u)) return AP_ERR_INVALID_ARG;
    if (plan->ws.bytes > kStaticWorkspaceBytes) return AP_ERR_WORKSPACE_TOO_SMALL;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { (void)cudaGetLastError(); prev = -1; }
    if (cudaSetDevice(pool->desc.device) != cudaSuccess) { (void)cudaGetLastError(); return AP_ERR_CUDA; }

    int rc = AP_OK;
    void *ws = nullptr;
    rc = static_workspace_address(pool->desc.device, &ws);
    if (rc == AP_OK) {
        cudaStream_t st = (cudaStream_t)stream;
        // Every partial slot is written in full by its decode item before the
        // last-arriving item of the stream merges them, so nothing left over
        // from an earlier call is ever read and nothing needs clearing.
        float *o_part = plan->ws.bytes ? (float *)((char *)ws + plan->ws.o_part_off) : nullptr;
        float *lse_part = plan->ws.bytes ? (float *)((char *)ws + plan->ws.lse_part_off) : nullptr;
        const cudaError_t e = ap::launch_attention_kernels(pool, plan, q, out, lse, o_part, lse_part, st);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            rc = e == cudaErrorNotSupported ? AP_ERR_UNSUPPORTED : AP_ERR_CUDA;
        }
    }
    if (prev >= 0) (void)cudaSetDevice(prev);
    return rc;
}

}  // extern "C"
