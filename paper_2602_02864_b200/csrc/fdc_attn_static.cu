// fdc_decode_attn_static: the masked attention of one layer with the split partials kept in a
// buffer that is part of the library image, so that the call needs no device memory from
// anybody.
//
// Who this is for.  fdc_decode_attn leaves its scratch (the split pass's partial results) to
// the caller, who normally gets it from cudaMalloc or from a framework's allocator.  Some hosts
// of a driving stack cannot do that once they are running: an in-vehicle runtime that fixes
// its device memory budget at start-up and forbids allocation inside the decode loop
// (cudaMalloc synchronises the whole device, takes an unbounded time and can fail when the KV
// pool already owns all of HBM), or a host that reaches this library through a plugin
// interface whose per-step call is not allowed to allocate.  For them the scratch lives in
// the file-scope array below: FDC_STATIC_WS_BYTES on every GPU that loads the library, held
// until the process exits, whether or not this entry point is ever called.
//
// The array's name is only usable as an address in device code.  On the host the same name is
// a stand-in object of the host image; handing it to a kernel would make the kernel read
// and write host addresses.  The device address is therefore looked up once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels get.
#include <mutex>

#include "fdc_internal.h"

namespace {

static __device__ __align__(256) unsigned char g_static_ws[FDC_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_ws_addr[kMaxDevices];          // device address of g_static_ws, per device ordinal (nullptr: not looked up yet)

// Device address of the array on the CURRENT device (looked up on first use).
int static_ws_address(int device, void** out)
{
    if (device < 0 || device >= kMaxDevices) return FDC_ERR_RANGE;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_ws_addr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_ws);
        if (e != cudaSuccess) return fdc::set_cuda_error(e);
        if (!p || ((uintptr_t)p & 255)) return FDC_ERR_WORKSPACE;
        g_ws_addr[device] = p;
    }
    *out = g_ws_addr[device];
    return FDC_OK;
}

}  // namespace

extern "C" int fdc_decode_attn_static(fdc_plan* p, const fdc_kv_desc* kv, int32_t layer,
                                      const int32_t* d_n_active, const uint64_t* d_mask, const int32_t* d_tiles,
                                      const int32_t* d_ntiles, const void* d_q, void* d_out, float scale,
                                      void* stream)
{
    size_t need = 0;
    int rc = fdc_attn_workspace_bytes(p, kv, &need);          // also validates plan and cache view
    if (rc) return rc;
    if (need > (size_t)FDC_STATIC_WS_BYTES) return FDC_ERR_STATIC_LIMIT;
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return fdc::set_cuda_error(e);
    if (device != p->device) return FDC_ERR_RANGE;            // the plan's tables live on another GPU
    void* ws = nullptr;
    rc = static_ws_address(device, &ws);
    if (rc) return rc;
    // Every partial the combine pass reads has been written by the split pass of the same call,
    // so nothing in the buffer has to start at zero and it is not cleared.
    return fdc_decode_attn(p, kv, layer, d_n_active, d_mask, d_tiles, d_ntiles, d_q, d_out, scale, ws,
                           (size_t)FDC_STATIC_WS_BYTES, stream);
}
