// tb_factor_static: the factorisation of tb_factor for callers that cannot
// provide a workspace, with the scratch held in a fixed array of device memory
// that belongs to the library.
#include "tb_common.cuh"

namespace tb {

// the factorisation itself (tb_factor.cu); lookahead = false keeps it on the caller's stream
tb_status factor_run(const float* H, int n_batch, int d, float* U, float* Hinv, int* info, void* ws, size_t ws_bytes,
                     void* stream, bool lookahead);

// 32 MiB: enough for 64 matrices of 128 x 128 (the per-head H_out of a
// 64-head attention layer) or one matrix of 1024 x 1024.  Each GPU on which
// the library is loaded keeps this array until the process exits.
static const size_t kStaticScratchBytes = (size_t)32 << 20;
static __device__ __align__(256) unsigned char g_factor_scratch[kStaticScratchBytes];

// Device address of the array, looked up once per device.  In host code the
// name g_factor_scratch is only a handle for the runtime; the pointer a kernel
// may use comes from cudaGetSymbolAddress on the device that is current.
static void* g_scratch_ptr[64] = {nullptr};

static tb_status scratch_address(void** out) {
  int dev = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    TB_CUDA_CHECK(cudaGetSymbolAddress(&p, g_factor_scratch));
    if (!p) return TB_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return TB_OK;
}

}  // namespace tb

extern "C" size_t tb_factor_static_capacity(void) { return tb::kStaticScratchBytes; }

extern "C" tb_status tb_factor_static(const float* H, int n_batch, int d, float* U, int* info,
                                      void* stream) {
  if (!H || !U || !info || n_batch <= 0 || n_batch > 65535 || d <= 0) return TB_ERR_INVALID_ARG;
  const size_t need = tb_factor_workspace(n_batch, d);
  if (need == 0 || need > tb::kStaticScratchBytes) return TB_ERR_UNSUPPORTED;  // beyond the fixed scratch
  void* scratch = nullptr;
  TB_TRY(tb::scratch_address(&scratch));
  // tb_factor clears the parts of its workspace that must start at zero (the
  // inverse factor and the info words) on the stream before it uses them, so
  // what an earlier call left in the array cannot leak into this one.
  // single stream: this entry point creates nothing, not even the helper stream of tb_factor's look-ahead
  return tb::factor_run(H, n_batch, d, U, nullptr, info, scratch, tb::kStaticScratchBytes, stream, false);
}
