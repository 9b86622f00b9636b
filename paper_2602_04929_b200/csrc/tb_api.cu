// Status strings and the host-buffer entry point that chains the whole path:
// Hessians -> factors -> quantizer (Algorithm 1 for one projection).
#include "tb_common.cuh"

using namespace tb;

namespace tb {
unsigned long long g_launch_count = 0;
}

extern "C" unsigned long long tb_launch_count(void) { return tb::g_launch_count; }

extern "C" const char* tb_status_string(tb_status st) {
  switch (st) {
    case TB_OK: return "ok";
    case TB_ERR_INVALID_ARG: return "invalid argument";
    case TB_ERR_UNSUPPORTED: return "unsupported configuration";
    case TB_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TB_ERR_NOT_SPD: return "matrix not positive definite";
    case TB_ERR_CUDA: return "CUDA runtime error";
    case TB_ERR_TIMEOUT: return "bounded device wait ran out";
  }
  return "unknown status";
}

namespace {

struct HostPlan {
  float *W, *G, *Hsum, *Hin, *Uin, *Hout, *Uout, *scales, *What;
  __nv_bfloat16* X;
  int *info, *zeros;
  unsigned char* codes;
  double* loss;
  void* sub;    // workspace of the calls on the caller's stream
  void* sub2;   // workspace of the H_out build and factor, which run beside the factor of H_in
  size_t sub_bytes, sub2_bytes, total;
};

// One helper stream per device for the part of the path that runs beside the factor of H_in,
// created on first use and kept for the life of the process.
enum { COPY_CHUNKS_MAX = 16 };
struct SideStream {
  cudaStream_t stream;
  cudaEvent_t fork, join;
  cudaEvent_t chunk[COPY_CHUNKS_MAX];  // one per piece of X in flight
  bool ready;
};

SideStream* side_stream() {
  static SideStream per_device[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SideStream* s = &per_device[dev];
  if (!s->ready) {
    if (cudaStreamCreateWithFlags(&s->stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < COPY_CHUNKS_MAX; ++i)
      if (cudaEventCreateWithFlags(&s->chunk[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    s->ready = true;
  }
  return s;
}

size_t max_sz(size_t a, size_t b) { return a > b ? a : b; }

HostPlan host_plan(const tb_layer_desc* D, long long n_tok, int g_heads, void* ws) {
  HostPlan h;
  Bump b(ws);
  const size_t d = (size_t)D->d_in, dout = (size_t)D->d_out;
  const size_t ng = D->quant_group > 0 ? d / (size_t)D->quant_group : 1;
  h.W = b.take<float>(dout * d);
  h.X = b.take<__nv_bfloat16>((size_t)n_tok * d);
  h.G = g_heads > 0 ? b.take<float>((size_t)g_heads * D->d_head * d) : nullptr;
  h.Hsum = b.take<float>(d * d);
  h.Hin = b.take<float>(d * d);
  h.Uin = b.take<float>(d * d);
  h.Hout = g_heads > 0 ? b.take<float>((size_t)D->n_heads * D->d_head * D->d_head) : nullptr;
  h.Uout = g_heads > 0 ? b.take<float>((size_t)D->n_heads * D->d_head * D->d_head) : nullptr;
  h.info = b.take<int>((size_t)D->n_heads + 1);
  h.codes = b.take<unsigned char>(dout * d);
  h.scales = b.take<float>(dout * ng);
  h.zeros = b.take<int>(dout * ng);
  h.What = b.take<float>(dout * d);
  h.loss = b.take<double>((size_t)D->n_heads);
  size_t sub = tb_factor_workspace(1, D->d_in);
  sub = max_sz(sub, tb_quantize_layer_workspace(D, 0, 1));
  h.sub = b.take<unsigned char>(sub);
  h.sub_bytes = sub;
  h.sub2 = nullptr;
  h.sub2_bytes = 0;
  if (g_heads > 0) {
    h.sub2_bytes = max_sz(tb_factor_workspace(D->n_heads, D->d_head),
                          tb_build_hout_workspace(g_heads, D->d_head, D->d_in));
    h.sub2 = b.take<unsigned char>(h.sub2_bytes);
  }
  h.total = b.total();
  return h;
}

bool desc_ok(const tb_layer_desc* D, long long n_tok, int g_heads) {
  if (!D || n_tok <= 0 || g_heads < 0) return false;
  if (D->d_out <= 0 || D->d_in <= 0 || D->n_heads <= 0 || D->d_head <= 0) return false;
  if ((long long)D->n_heads * D->d_head != D->d_out) return false;
  if (D->quant_group < 0 || (D->quant_group > 0 && D->d_in % D->quant_group)) return false;
  if (g_heads > 0 && (g_heads >= D->n_heads ? g_heads % D->n_heads : D->n_heads % g_heads)) return false;
  return true;
}

}  // namespace

extern "C" size_t tb_quantize_from_host_workspace(const tb_layer_desc* desc, long long n_tok,
                                                  int g_heads) {
  if (!desc_ok(desc, n_tok, g_heads)) return 0;
  return host_plan(desc, n_tok, g_heads, nullptr).total;
}

namespace {

// Everything tb_quantize_from_host enqueues; returns at the first failure.  The caller joins the
// helper stream and synchronises whatever the outcome, so no copy is in flight when it returns.
tb_status from_host_enqueue(const tb_layer_desc* desc, const HostPlan& h, SideStream* ss, const float* W_host,
                            const void* X_host, long long n_tok, const float* G_host, int g_heads, float damp_in,
                            float damp_out, unsigned char* codes_host, float* scales_host, int* zeros_host,
                            float* W_hat_host, double* loss_host, int* info_host, int n_info, void* stream) {
  cudaStream_t st = as_stream(stream);
  const size_t d = (size_t)desc->d_in, dout = (size_t)desc->d_out;
  const size_t ng = desc->quant_group > 0 ? d / (size_t)desc->quant_group : 1;
  const int H = desc->n_heads, dh = desc->d_head;
  // X is by far the largest transfer: it goes over in pieces on the helper stream while the Hessian
  // of the pieces that have arrived accumulates on the caller's stream.  Pieces are multiples of 2048
  // tokens, so the sums are those of a single accumulation over all tokens.
  long long piece = ((n_tok + COPY_CHUNKS_MAX / 2 - 1) / (COPY_CHUNKS_MAX / 2) + 2047) / 2048 * 2048;  // about 8 pieces
  TB_CUDA_CHECK(cudaMemsetAsync(h.Hin, 0, d * d * sizeof(float), st));
  int n_pieces = 0;
  for (long long t0 = 0; t0 < n_tok; t0 += piece, ++n_pieces) {
    const long long nt = (n_tok - t0 < piece) ? (n_tok - t0) : piece;
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(X_host) + (size_t)t0 * d;
    TB_CUDA_CHECK(cudaMemcpyAsync(h.X + (size_t)t0 * d, src, (size_t)nt * d * sizeof(__nv_bfloat16),
                                  cudaMemcpyHostToDevice, ss->stream));
    TB_CUDA_CHECK(cudaEventRecord(ss->chunk[n_pieces], ss->stream));
    if (n_pieces == 0) {  // the small inputs ride on the caller's stream beside the first piece
      TB_CUDA_CHECK(cudaMemcpyAsync(h.W, W_host, dout * d * sizeof(float), cudaMemcpyHostToDevice, st));
      if (g_heads > 0)
        TB_CUDA_CHECK(cudaMemcpyAsync(h.G, G_host, (size_t)g_heads * dh * d * sizeof(float),
                                      cudaMemcpyHostToDevice, st));
    }
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, ss->chunk[n_pieces], 0));
    TB_TRY(tb_accumulate_hessian(h.Hin, h.X + (size_t)t0 * d, TB_BF16, nt, (int)d, stream));
  }
  TB_TRY(tb_finalize_hessian(h.Hin, nullptr, h.Hsum, (int)d, n_tok, damp_in, stream));
  if (g_heads > 0) {
    // H_out and its factor need the Hessian only: they run on the helper stream beside the factor of
    // H_in (a chain of small launches that leaves SMs idle), with their own part of the workspace
    TB_CUDA_CHECK(cudaEventRecord(ss->fork, st));
    TB_CUDA_CHECK(cudaStreamWaitEvent(ss->stream, ss->fork, 0));
    TB_TRY(tb_build_hout(h.Hout, h.G, h.Hsum, H, g_heads, dh, (int)d, damp_out, h.sub2, h.sub2_bytes, ss->stream));
    TB_TRY(tb_factor(h.Hout, H, dh, h.Uout, nullptr, h.info + 1, h.sub2, h.sub2_bytes, ss->stream));
    TB_CUDA_CHECK(cudaEventRecord(ss->join, ss->stream));
  } else {
    TB_CUDA_CHECK(cudaMemsetAsync(h.info + 1, 0, sizeof(int) * (size_t)H, st));
  }
  TB_TRY(tb_factor(h.Hin, 1, (int)d, h.Uin, nullptr, h.info, h.sub, h.sub_bytes, stream));
  if (g_heads > 0) TB_CUDA_CHECK(cudaStreamWaitEvent(st, ss->join, 0));
  TB_TRY(tb_quantize_layer(desc, h.W, h.Hin, h.Uin, h.Hout, h.Uout, nullptr, nullptr, nullptr,
                           h.codes, h.scales, h.zeros, nullptr, W_hat_host ? h.What : nullptr,
                           nullptr, loss_host ? h.loss : nullptr, nullptr, h.sub, h.sub_bytes, stream));
  TB_CUDA_CHECK(cudaMemcpyAsync(codes_host, h.codes, dout * d, cudaMemcpyDeviceToHost, st));
  TB_CUDA_CHECK(cudaMemcpyAsync(scales_host, h.scales, dout * ng * sizeof(float), cudaMemcpyDeviceToHost, st));
  TB_CUDA_CHECK(cudaMemcpyAsync(zeros_host, h.zeros, dout * ng * sizeof(int), cudaMemcpyDeviceToHost, st));
  if (W_hat_host)
    TB_CUDA_CHECK(cudaMemcpyAsync(W_hat_host, h.What, dout * d * sizeof(float), cudaMemcpyDeviceToHost, st));
  if (loss_host)
    TB_CUDA_CHECK(cudaMemcpyAsync(loss_host, h.loss, sizeof(double) * (size_t)H, cudaMemcpyDeviceToHost, st));
  TB_CUDA_CHECK(cudaMemcpyAsync(info_host, h.info, sizeof(int) * (size_t)n_info, cudaMemcpyDeviceToHost, st));
  return TB_OK;
}

}  // namespace

extern "C" tb_status tb_quantize_from_host(const tb_layer_desc* desc, const float* W_host,
                                           const void* X_host, long long n_tok,
                                           const float* G_host, int g_heads, float damp_in,
                                           float damp_out, unsigned char* codes_host,
                                           float* scales_host, int* zeros_host, float* W_hat_host,
                                           double* loss_host, void* dev_ws, size_t ws_bytes,
                                           void* stream) {
  // The whole description is checked before anything is enqueued: the quantizer's own workspace
  // query rejects every description tb_quantize_layer would reject (it returns 0), and the
  // tensor-core Hessian needs a width that is a multiple of 8.
  if (!desc_ok(desc, n_tok, G_host ? g_heads : 0)) return TB_ERR_INVALID_ARG;
  if (!W_host || !X_host || !codes_host || !scales_host || !zeros_host) return TB_ERR_INVALID_ARG;
  if (desc->n_hin != 1) return TB_ERR_UNSUPPORTED;  // one shared H_in on this entry point
  if (desc->d_in % 8) return TB_ERR_INVALID_ARG;
  if (tb_quantize_layer_workspace(desc, 0, 1) == 0) {
    // tell an unsupported shape from an invalid one the way tb_quantize_layer does
    return (desc->d_in % 128 || (desc->quant_group > 0 && desc->quant_group % 32)) ? TB_ERR_UNSUPPORTED
                                                                                  : TB_ERR_INVALID_ARG;
  }
  if (!G_host) g_heads = 0;
  const HostPlan hs = host_plan(desc, n_tok, g_heads, nullptr);
  if (!dev_ws || !aligned(dev_ws, 256) || ws_bytes < hs.total) return TB_ERR_WORKSPACE;
  const HostPlan h = host_plan(desc, n_tok, g_heads, dev_ws);
  cudaStream_t st = as_stream(stream);
  const int H = desc->n_heads;
  SideStream* ss = side_stream();
  if (!ss) return TB_ERR_CUDA;
  // earlier work on the caller's stream may still use the buffers: the helper stream starts after it
  TB_CUDA_CHECK(cudaEventRecord(ss->fork, st));
  TB_CUDA_CHECK(cudaStreamWaitEvent(ss->stream, ss->fork, 0));
  int info_host[1 + 4096];
  const int n_info = 1 + (H < 4096 ? H : 4096);
  tb_status status = from_host_enqueue(desc, h, ss, W_host, X_host, n_tok, G_host, g_heads, damp_in, damp_out,
                                       codes_host, scales_host, zeros_host, W_hat_host, loss_host, info_host,
                                       n_info, stream);
  // One way out, success or not: the helper stream joins the caller's, and the call waits until
  // nothing it enqueued (copies from and to the caller's host buffers included) is still in flight.
  bool sync_ok = cudaEventRecord(ss->join, ss->stream) == cudaSuccess &&
                 cudaStreamWaitEvent(st, ss->join, 0) == cudaSuccess;
  sync_ok = (cudaStreamSynchronize(st) == cudaSuccess) && sync_ok;
  if (!sync_ok) {
    (void)cudaGetLastError();
    return status != TB_OK ? status : TB_ERR_CUDA;
  }
  if (status != TB_OK) return status;
  // a bounded wait inside one of the tensor-core kernels ran out: the results are incomplete
  const int flag = tb_device_error_flag();
  if (flag != 0) return flag > 0 ? TB_ERR_TIMEOUT : TB_ERR_CUDA;
  for (int i = 0; i < n_info; ++i)
    if (info_host[i] != 0) return TB_ERR_NOT_SPD;
  return TB_OK;
}
