// Block level of Algorithm 1: its outer loop over the projections of one attention layer
// (W_Q, W_K, W_V, and the output projection in the H_out = I mode of Table 1), with the
// statistics each projection needs.
//
//   tb_quantize_block    several prepared projections, side by side on helper streams
//   tb_attention_layer   activations -> Hessians (Table 1), deviation correlations (Algorithm 1,
//                        deviation step), factors (Eq. 2), propagated-error operands
//                        (Algorithm 2 / Proposition 3.2), H_out of every projection (Table 1),
//                        then the four quantizer calls; activations, weights and results either
//                        device-resident or in host memory (then the activations cross in
//                        pieces while the Hessian of the pieces that have arrived accumulates)
#include "tb_common.cuh"
#include "tb_profile.cuh"

using namespace tb;

namespace {

enum { N_HELPERS = 4, STAGE_SLOTS = 8 };

// Helper streams and events of the block level, one set per device, created on first use and
// kept for the life of the process.
struct BlockSide {
  cudaStream_t helper[N_HELPERS];
  cudaStream_t copy;
  cudaEvent_t fork, join[N_HELPERS], dep[8];
  cudaEvent_t staged[STAGE_SLOTS], consumed[STAGE_SLOTS];
  bool ready;
};

BlockSide* block_side() {
  static BlockSide per_device[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  BlockSide* s = &per_device[dev];
  if (!s->ready) {
    int prio_low = 0, prio_high = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high) != cudaSuccess) return nullptr;
    for (int i = 0; i < N_HELPERS; ++i) {
      // the last helper is the ingest stream of the host mode: its short Hessian launches go first when SMs
      // fall free, so that the staging slots drain while long quantizer launches hold the GPU
      const int prio = (i == N_HELPERS - 1) ? prio_high : prio_low;
      if (cudaStreamCreateWithPriority(&s->helper[i], cudaStreamNonBlocking, prio) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s->join[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    if (cudaStreamCreateWithFlags(&s->copy, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < 8; ++i)
      if (cudaEventCreateWithFlags(&s->dep[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < STAGE_SLOTS; ++i) {
      if (cudaEventCreateWithFlags(&s->staged[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s->consumed[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    s->ready = true;
  }
  return s;
}

tb_status run_job(const tb_projection_job& j, cudaStream_t st) {
  return tb_quantize_layer(&j.desc, j.W, j.H_in, j.U_in, j.H_out, j.U_out, j.R, j.P, j.C, j.codes, j.scales, j.zeros,
                           j.cand, j.W_hat, j.W_comp, j.loss, j.stats, j.ws, j.ws_bytes, st);
}

// dst[c][r] = src[r][c]
__global__ void k_transpose_f32(const float* __restrict__ src, float* __restrict__ dst, int rows, int cols) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    tile[i][threadIdx.x] = (r < rows && c < cols) ? src[(long long)r * cols + c] : 0.0f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) dst[(long long)c * rows + r] = tile[threadIdx.x][i];
  }
}

size_t max_sz(size_t a, size_t b) { return a > b ? a : b; }

}  // namespace

extern "C" tb_status tb_quantize_block(const tb_projection_job* jobs, int n_jobs, int concurrent, void* stream) {
  if (!jobs || n_jobs <= 0 || n_jobs > 1 + N_HELPERS) return TB_ERR_INVALID_ARG;
  // Every description, pointer and workspace is checked before the first launch of any job: the
  // quantizer's own checks run again inside, but by then earlier jobs would be in flight.
  for (int i = 0; i < n_jobs; ++i) {
    const tb_projection_job& j = jobs[i];
    if (!j.W || !j.H_in || !j.U_in || !j.codes || !j.scales || !j.zeros) return TB_ERR_INVALID_ARG;
    if ((j.H_out == nullptr) != (j.U_out == nullptr)) return TB_ERR_INVALID_ARG;
    if ((j.R != nullptr) != (j.P != nullptr) || (j.R != nullptr) != (j.C != nullptr)) return TB_ERR_INVALID_ARG;
    const size_t need = tb_quantize_layer_workspace(&j.desc, j.R != nullptr, j.loss != nullptr);
    if (need == 0) return TB_ERR_INVALID_ARG;
    if (!j.ws || !aligned(j.ws, 256) || j.ws_bytes < need) return TB_ERR_WORKSPACE;
    for (int k = 0; k < i; ++k)
      if (concurrent && jobs[k].ws == j.ws) return TB_ERR_INVALID_ARG;  // side-by-side jobs need their own scratch
  }
  cudaStream_t st = as_stream(stream);
  if (!concurrent || n_jobs == 1) {
    for (int i = 0; i < n_jobs; ++i) TB_TRY(run_job(jobs[i], st));
    return TB_OK;
  }
  BlockSide* bs = block_side();
  if (!bs) return TB_ERR_CUDA;
  TB_CUDA_CHECK(cudaEventRecord(bs->fork, st));
  tb_status status = TB_OK;
  int forked = 0;
  for (int i = 1; i < n_jobs && status == TB_OK; ++i) {
    cudaStream_t hs = bs->helper[i - 1];
    if (cudaStreamWaitEvent(hs, bs->fork, 0) != cudaSuccess) {
      status = TB_ERR_CUDA;
      break;
    }
    forked = i;
    status = run_job(jobs[i], hs);
  }
  if (status == TB_OK) status = run_job(jobs[0], st);
  // the helper streams always join the caller's, whatever happened above
  for (int i = 1; i <= forked; ++i) {
    if (cudaEventRecord(bs->join[i - 1], bs->helper[i - 1]) != cudaSuccess ||
        cudaStreamWaitEvent(st, bs->join[i - 1], 0) != cudaSuccess) {
      (void)cudaGetLastError();
      if (status == TB_OK) status = TB_ERR_CUDA;
    }
  }
  return status;
}

// ---------------------------------------------------------------------------
// tb_attention_layer
// ---------------------------------------------------------------------------
namespace {

struct InputSide {  // one input Hessian with what derives from it
  float *H, *Hsum, *U, *R, *P, *C;
};

struct LayerPlan {
  int d, dq, hq, hkv, dh;
  bool with_r, with_ro, per_head_v, on_host, concurrent;
  long long n_tok, piece;
  tb_layer_desc desc[4];   // q, k, v, o
  InputSide attn, vhead, oin;  // vhead.* hold hkv matrices when per_head_v
  float *Hout[3], *Uout[3];    // q, k, v
  float* WoT;
  int* info;                   // [info_count]
  int info_count;
  // device copies in host mode
  float* Wdev[4];
  unsigned char* codes[4];
  float* scales[4];
  int* zeros[4];
  float* What[4];
  double* loss[4];
  __nv_bfloat16* stage[STAGE_SLOTS][2];  // pieces of an activation tensor and of its full-precision twin
  // scratch
  void *ws_factor, *ws_factor_small[2], *ws_hout[2], *ws_cross, *ws_prep, *ws_quant[4];
  size_t factor_bytes, factor_small_bytes, hout_bytes, cross_bytes, prep_bytes, quant_bytes[4];
  size_t total;
};

bool layer_desc_ok(const tb_attention_desc* D) {
  if (!D) return false;
  if (D->d_model <= 0 || D->n_q_heads <= 0 || D->n_kv_heads <= 0 || D->d_head <= 0 || D->n_tok <= 0) return false;
  if (D->n_q_heads % D->n_kv_heads) return false;
  if (!(D->damp >= 0.0f)) return false;
  return true;
}

tb_status make_layer_plan(const tb_attention_desc* D, const tb_attention_io* io, void* ws, LayerPlan* out) {
  if (!layer_desc_ok(D) || !io) return TB_ERR_INVALID_ARG;
  LayerPlan& p = *out;
  p.d = D->d_model;
  p.hq = D->n_q_heads;
  p.hkv = D->n_kv_heads;
  p.dh = D->d_head;
  p.dq = p.hq * p.dh;
  p.n_tok = D->n_tok;
  p.with_r = io->X_fp != nullptr;
  p.with_ro = io->X_o_fp != nullptr;
  p.per_head_v = io->X_v != nullptr;
  p.on_host = D->on_host != 0;
  p.concurrent = D->concurrent != 0;
  if (p.d % 8 || p.dq % 8) return TB_ERR_INVALID_ARG;
  const int rows[4] = {p.dq, p.hkv * p.dh, p.hkv * p.dh, p.d};
  const int cols[4] = {p.d, p.d, p.d, p.dq};
  const int heads[4] = {p.hq, p.hkv, p.hkv, 1};
  const int dheads[4] = {p.dh, p.dh, p.dh, p.d};
  for (int i = 0; i < 4; ++i) {
    tb_layer_desc& L = p.desc[i];
    L.d_out = rows[i];
    L.d_in = cols[i];
    L.n_heads = heads[i];
    L.d_head = dheads[i];
    L.n_hin = (i == 2 && p.per_head_v) ? p.hkv : 1;
    L.bits = D->bits;
    L.quant_group = D->quant_group;
    L.out_block = (i == 3) ? dheads[i] : D->out_block;
    L.n_cand = D->n_cand;
    L.cd_iters = D->cd_iters;
    L.flags = D->flags;
  }
  const bool r_of[4] = {p.with_r, p.with_r, p.with_r && !p.per_head_v, p.with_ro};
  for (int i = 0; i < 4; ++i)
    if (tb_quantize_layer_workspace(&p.desc[i], r_of[i], 1) == 0)
      return (cols[i] % 128 || (D->quant_group > 0 && D->quant_group % 32)) ? TB_ERR_UNSUPPORTED : TB_ERR_INVALID_ARG;

  Bump b(ws);
  const size_t dd = (size_t)p.d * p.d, qq = (size_t)p.dq * p.dq;
  auto side = [&](InputSide& s, size_t n, size_t count, bool with_r, bool with_sum) {
    s.H = b.take<float>(n * count);
    s.Hsum = with_sum ? b.take<float>(n) : nullptr;
    s.U = b.take<float>(n * count);
    s.R = with_r ? b.take<float>(n) : nullptr;
    s.P = with_r ? b.take<float>(n) : nullptr;
    s.C = with_r ? b.take<float>(n) : nullptr;
  };
  side(p.attn, dd, 1, p.with_r, true);
  if (p.per_head_v)
    side(p.vhead, dd, (size_t)p.hkv, false, false);
  else
    p.vhead = p.attn;
  side(p.oin, qq, 1, p.with_ro, false);
  const size_t hh = (size_t)p.dh * p.dh;
  const int oh[3] = {p.hq, p.hkv, p.hkv};
  for (int i = 0; i < 3; ++i) {
    p.Hout[i] = b.take<float>(hh * oh[i]);
    p.Uout[i] = b.take<float>(hh * oh[i]);
  }
  p.WoT = b.take<float>((size_t)p.dq * p.d);
  p.info_count = 2 + (p.per_head_v ? p.hkv : 0) + p.hq + 2 * p.hkv;
  p.info = b.take<int>((size_t)p.info_count);
  for (int i = 0; i < 4; ++i) {
    const size_t n = (size_t)rows[i] * cols[i];
    const size_t ng = D->quant_group > 0 ? (size_t)cols[i] / D->quant_group : 1;
    p.Wdev[i] = p.on_host ? b.take<float>(n) : nullptr;
    p.codes[i] = p.on_host ? b.take<unsigned char>(n) : nullptr;
    p.scales[i] = p.on_host ? b.take<float>((size_t)rows[i] * ng) : nullptr;
    p.zeros[i] = p.on_host ? b.take<int>((size_t)rows[i] * ng) : nullptr;
    p.What[i] = (p.on_host && io->W_hat[i]) ? b.take<float>(n) : nullptr;
    p.loss[i] = (p.on_host && io->loss[i]) ? b.take<double>((size_t)heads[i]) : nullptr;
  }
  // pieces of an activation tensor: multiples of 2048 tokens (the Hessian's accumulation runs), so
  // that the sums equal those of one call over all tokens
  p.piece = 16384;
  if (p.piece > ((p.n_tok + 2047) / 2048) * 2048) p.piece = ((p.n_tok + 2047) / 2048) * 2048;
  const size_t wide = (size_t)(p.d > p.dq ? p.d : p.dq);
  for (int s = 0; s < STAGE_SLOTS; ++s)
    for (int t = 0; t < 2; ++t)
      p.stage[s][t] = p.on_host ? b.take<__nv_bfloat16>((size_t)p.piece * wide) : nullptr;

  p.factor_bytes = max_sz(tb_factor_workspace(1, p.d), tb_factor_workspace(1, p.dq));
  if (p.per_head_v) p.factor_bytes = max_sz(p.factor_bytes, tb_factor_workspace(p.hkv, p.d));
  p.ws_factor = b.take<unsigned char>(p.factor_bytes);
  p.factor_small_bytes = tb_factor_workspace(p.hq, p.dh);
  p.hout_bytes = max_sz(tb_build_hout_workspace(p.hq, p.dh, p.d), tb_build_hout_workspace(p.hkv, p.dh, p.d));
  for (int i = 0; i < 2; ++i) {
    p.ws_factor_small[i] = b.take<unsigned char>(p.factor_small_bytes);
    p.ws_hout[i] = b.take<unsigned char>(p.hout_bytes);
  }
  const long long cross_tok = p.on_host ? p.piece : p.n_tok;
  p.cross_bytes = (p.with_r || p.with_ro) ? tb_accumulate_cross_workspace(TB_BF16, cross_tok, (int)wide) : 0;
  p.ws_cross = p.cross_bytes ? b.take<unsigned char>(p.cross_bytes) : nullptr;
  p.prep_bytes = (p.with_r || p.with_ro) ? tb_prepare_correction_workspace(1, (int)wide) : 0;
  p.ws_prep = p.prep_bytes ? b.take<unsigned char>(p.prep_bytes) : nullptr;
  size_t qmax = 0;
  for (int i = 0; i < 4; ++i) {
    p.quant_bytes[i] = tb_quantize_layer_workspace(&p.desc[i], r_of[i], 1);
    qmax = max_sz(qmax, p.quant_bytes[i]);
  }
  if (p.concurrent) {
    for (int i = 0; i < 4; ++i) p.ws_quant[i] = b.take<unsigned char>(p.quant_bytes[i]);
  } else {
    void* shared = b.take<unsigned char>(qmax);
    for (int i = 0; i < 4; ++i) {
      p.ws_quant[i] = shared;
      p.quant_bytes[i] = qmax;
    }
  }
  p.total = b.total();
  return TB_OK;
}

// H (+ R) of one activation tensor [n_tok][width], un-normalised sums then finalised.
// Device-resident tensors go through in one call; host tensors in pieces through the staging
// slots on the copy stream, each piece accumulated as soon as it has arrived.
tb_status accumulate_input(const LayerPlan& p, BlockSide* bs, const void* X, const void* Xfp, int width, float* H,
                           float* R, float* Hsum, float damp, float alpha, cudaStream_t st) {
  const size_t n = (size_t)width * width;
  TB_CUDA_CHECK(cudaMemsetAsync(H, 0, n * sizeof(float), st));
  if (R) TB_CUDA_CHECK(cudaMemsetAsync(R, 0, n * sizeof(float), st));
  if (!p.on_host) {
    {
      PhaseScope ph(PH_HESSIAN, st);
      TB_TRY(tb_accumulate_hessian(H, X, TB_BF16, p.n_tok, width, st));
    }
    if (R) {
      PhaseScope ph(PH_CROSS, st);
      TB_TRY(tb_accumulate_cross(R, X, Xfp, TB_BF16, p.n_tok, width, alpha, p.ws_cross, p.cross_bytes, st));
    }
  } else {
    int it = 0;
    for (long long t0 = 0; t0 < p.n_tok; t0 += p.piece, ++it) {
      const long long nt = (p.n_tok - t0 < p.piece) ? (p.n_tok - t0) : p.piece;
      const int slot = it % STAGE_SLOTS;
      const size_t bytes = (size_t)nt * width * sizeof(__nv_bfloat16);
      // the slot is free once the accumulation of the piece that used it last has run
      TB_CUDA_CHECK(cudaStreamWaitEvent(bs->copy, bs->consumed[slot], 0));
      TB_CUDA_CHECK(cudaMemcpyAsync(p.stage[slot][0], static_cast<const __nv_bfloat16*>(X) + (size_t)t0 * width, bytes,
                                    cudaMemcpyHostToDevice, bs->copy));
      if (R)
        TB_CUDA_CHECK(cudaMemcpyAsync(p.stage[slot][1], static_cast<const __nv_bfloat16*>(Xfp) + (size_t)t0 * width,
                                      bytes, cudaMemcpyHostToDevice, bs->copy));
      TB_CUDA_CHECK(cudaEventRecord(bs->staged[slot], bs->copy));
      TB_CUDA_CHECK(cudaStreamWaitEvent(st, bs->staged[slot], 0));
      {
        PhaseScope ph(PH_HESSIAN, st);
        TB_TRY(tb_accumulate_hessian(H, p.stage[slot][0], TB_BF16, nt, width, st));
      }
      if (R) {
        PhaseScope ph(PH_CROSS, st);
        TB_TRY(tb_accumulate_cross(R, p.stage[slot][0], p.stage[slot][1], TB_BF16, nt, width, alpha, p.ws_cross,
                                   p.cross_bytes, st));
      }
      TB_CUDA_CHECK(cudaEventRecord(bs->consumed[slot], st));
    }
  }
  PhaseScope ph(PH_HESSIAN, st);
  return tb_finalize_hessian(H, R, Hsum, width, p.n_tok, damp, st);
}

tb_status layer_enqueue(const tb_attention_desc* D, const tb_attention_io* io, LayerPlan& p, BlockSide* bs,
                        cudaStream_t st) {
  const size_t dd = (size_t)p.d * p.d;
  const float* W[4];
  // ---- weights ----
  for (int i = 0; i < 4; ++i) {
    if (p.on_host) {
      const size_t n = (size_t)p.desc[i].d_out * p.desc[i].d_in;
      TB_CUDA_CHECK(cudaMemcpyAsync(p.Wdev[i], io->W[i], n * sizeof(float), cudaMemcpyHostToDevice, st));
      W[i] = p.Wdev[i];
    } else {
      W[i] = io->W[i];
    }
  }
  int* info_attn = p.info;
  int* info_o = p.info + 1;
  int* info_v = p.info + 2;
  int* info_out[3];
  info_out[0] = p.info + 2 + (p.per_head_v ? p.hkv : 0);
  info_out[1] = info_out[0] + p.hq;
  info_out[2] = info_out[1] + p.hkv;
  TB_CUDA_CHECK(cudaMemsetAsync(p.info, 0, sizeof(int) * (size_t)p.info_count, st));

  // With host buffers the Hessians accumulate on a stream of their own ("ingest"), piece by piece as the
  // copies land, and everything that is not a Hessian (factors, correction operands, the quantizer) runs on
  // the caller's stream behind an event per finished Hessian: the copy engine then never waits for a factor
  // or for the quantizer, and the order of the inputs is chosen so that as much as possible of that work
  // has run by the time the last activation has crossed: attention input, output projection's input, then
  // the value heads (each factored alone as soon as its Hessian is complete, which gives the batched
  // factor's numbers bit for bit), the value projection last.
  cudaStream_t in = p.on_host ? bs->helper[N_HELPERS - 1] : st;
  auto hessian_ready = [&]() -> tb_status {   // work enqueued on st from here on sees what `in` has done so far
    if (in == st) return TB_OK;
    TB_CUDA_CHECK(cudaEventRecord(bs->dep[N_HELPERS + 1], in));
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, bs->dep[N_HELPERS + 1], 0));
    return TB_OK;
  };
  if (in != st) TB_CUDA_CHECK(cudaStreamWaitEvent(in, bs->fork, 0));  // after the caller's earlier work

  // ---- the attention input: H_in of W_Q, W_K (and of W_V without per-head inputs), and R ----
  TB_TRY(accumulate_input(p, bs, io->X, io->X_fp, p.d, p.attn.H, p.attn.R, p.attn.Hsum, D->damp, D->alpha, in));
  TB_TRY(hessian_ready());

  // ---- out-channel Hessians of Table 1 and their factors: they need Hsum and the partner weights
  // only, so with `concurrent` they run on helper streams beside the factor of H_in ----
  cudaStream_t hs0 = p.concurrent ? bs->helper[0] : st;
  cudaStream_t hs1 = p.concurrent ? bs->helper[1] : st;
  if (p.concurrent) {
    TB_CUDA_CHECK(cudaEventRecord(bs->fork, st));
    TB_CUDA_CHECK(cudaStreamWaitEvent(hs0, bs->fork, 0));
    TB_CUDA_CHECK(cudaStreamWaitEvent(hs1, bs->fork, 0));
  }
  {
    // W_Q: K_h^T K_h from G = W_K (a query head takes the block of its key/value head);
    // W_K: Q_h^T Q_h from G = W_Q (a key/value head sums the blocks of its query heads)
    PhaseScope ph(PH_HOUT, hs0);
    TB_TRY(tb_build_hout(p.Hout[0], W[1], p.attn.Hsum, p.hq, p.hkv, p.dh, p.d, D->damp, p.ws_hout[0], p.hout_bytes, hs0));
    TB_TRY(tb_build_hout(p.Hout[1], W[0], p.attn.Hsum, p.hkv, p.hq, p.dh, p.d, D->damp, p.ws_hout[0], p.hout_bytes, hs0));
  }
  {
    PhaseScope ph(PH_FACTOR, hs0);
    TB_TRY(tb_factor(p.Hout[0], p.hq, p.dh, p.Uout[0], nullptr, info_out[0], p.ws_factor_small[0], p.factor_small_bytes, hs0));
    TB_TRY(tb_factor(p.Hout[1], p.hkv, p.dh, p.Uout[1], nullptr, info_out[1], p.ws_factor_small[0], p.factor_small_bytes, hs0));
  }
  {
    // W_V: W_out,h^T W_out,h, the Gram of the head's block of columns of the output projection,
    // i.e. of the rows of W_O^T
    PhaseScope ph(PH_HOUT, hs1);
    k_transpose_f32<<<dim3((p.dq + 31) / 32, (p.d + 31) / 32), dim3(32, 8), 0, hs1>>>(W[3], p.WoT, p.d, p.dq);
    TB_LAUNCH_CHECK();
    TB_TRY(tb_build_hout(p.Hout[2], p.WoT, nullptr, p.hkv, p.hq, p.dh, p.d, D->damp, p.ws_hout[1], p.hout_bytes, hs1));
  }
  {
    PhaseScope ph(PH_FACTOR, hs1);
    TB_TRY(tb_factor(p.Hout[2], p.hkv, p.dh, p.Uout[2], nullptr, info_out[2], p.ws_factor_small[1], p.factor_small_bytes, hs1));
  }
  if (p.concurrent) {
    TB_CUDA_CHECK(cudaEventRecord(bs->join[0], hs0));
    TB_CUDA_CHECK(cudaEventRecord(bs->join[1], hs1));
  }
  // Side by side, device-resident, with per-head value inputs: the factor of the attention input's Hessian
  // (one matrix: much of it waits on its own panel chain) runs on a helper stream beside the value heads'
  // Hessians and is joined before the next factor, which shares its scratch.
  cudaStream_t fs = (p.concurrent && !p.on_host && p.per_head_v) ? bs->helper[2] : st;
  if (fs != st) {
    TB_CUDA_CHECK(cudaEventRecord(bs->dep[N_HELPERS + 2], st));
    TB_CUDA_CHECK(cudaStreamWaitEvent(fs, bs->dep[N_HELPERS + 2], 0));
  }
  {
    PhaseScope ph(PH_FACTOR, fs);
    TB_TRY(tb_factor(p.attn.H, 1, p.d, p.attn.U, nullptr, info_attn, p.ws_factor, p.factor_bytes, fs));
  }
  if (p.with_r) {
    PhaseScope ph(PH_PREP, fs);
    TB_TRY(tb_prepare_correction(p.attn.R, p.attn.U, 1, p.d, p.attn.P, p.attn.C, p.ws_prep, p.prep_bytes, fs));
  }
  if (fs != st) TB_CUDA_CHECK(cudaEventRecord(bs->dep[N_HELPERS + 3], fs));

  // ---- the value projection's own input Hessians, one per key/value head (Table 1, W_V row) ----
  auto value_side = [&]() -> tb_status {
    if (!p.per_head_v) return TB_OK;
    for (int h = 0; h < p.hkv; ++h) {
      const __nv_bfloat16* Xh = static_cast<const __nv_bfloat16*>(io->X_v) + (size_t)h * p.n_tok * p.d;
      TB_TRY(accumulate_input(p, bs, Xh, nullptr, p.d, p.vhead.H + (size_t)h * dd, nullptr, nullptr, D->damp, 0.0f, in));
      if (in != st) {
        // host buffers: this head's factor runs while the next head's activations cross
        TB_TRY(hessian_ready());
        PhaseScope ph(PH_FACTOR, st);
        TB_TRY(tb_factor(p.vhead.H + (size_t)h * dd, 1, p.d, p.vhead.U + (size_t)h * dd, nullptr, info_v + h, p.ws_factor,
                         p.factor_bytes, st));
      }
    }
    if (in != st) return TB_OK;
    if (fs != st) TB_CUDA_CHECK(cudaStreamWaitEvent(st, bs->dep[N_HELPERS + 3], 0));  // the attention input's factor is done
    PhaseScope ph(PH_FACTOR, st);
    return tb_factor(p.vhead.H, p.hkv, p.d, p.vhead.U, nullptr, info_v, p.ws_factor, p.factor_bytes, st);
  };

  // ---- the output projection's input ----
  auto output_side = [&]() -> tb_status {
    TB_TRY(accumulate_input(p, bs, io->X_o, io->X_o_fp, p.dq, p.oin.H, p.oin.R, nullptr, D->damp, D->alpha, in));
    TB_TRY(hessian_ready());
    {
      PhaseScope ph(PH_FACTOR, st);
      TB_TRY(tb_factor(p.oin.H, 1, p.dq, p.oin.U, nullptr, info_o, p.ws_factor, p.factor_bytes, st));
    }
    if (p.with_ro) {
      PhaseScope ph(PH_PREP, st);
      TB_TRY(tb_prepare_correction(p.oin.R, p.oin.U, 1, p.dq, p.oin.P, p.oin.C, p.ws_prep, p.prep_bytes, st));
    }
    return TB_OK;
  };
  const bool value_last = p.on_host && p.per_head_v;   // host buffers: the value heads cross last
  if (!value_last) TB_TRY(value_side());
  TB_TRY(output_side());
  if (p.concurrent) {
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, bs->join[0], 0));
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, bs->join[1], 0));
  }

  // ---- Algorithm 1's loop over the projections ----
  tb_projection_job jobs[4];
  const InputSide* in_of[4] = {&p.attn, &p.attn, &p.vhead, &p.oin};
  for (int i = 0; i < 4; ++i) {
    tb_projection_job& j = jobs[i];
    j.desc = p.desc[i];
    j.W = W[i];
    j.H_in = in_of[i]->H;
    j.U_in = in_of[i]->U;
    j.H_out = (i < 3) ? p.Hout[i] : nullptr;
    j.U_out = (i < 3) ? p.Uout[i] : nullptr;
    const bool r = (i == 2 && p.per_head_v) ? false : (in_of[i]->R != nullptr);
    j.R = r ? in_of[i]->R : nullptr;
    j.P = r ? in_of[i]->P : nullptr;
    j.C = r ? in_of[i]->C : nullptr;
    j.codes = p.on_host ? p.codes[i] : io->codes[i];
    j.scales = p.on_host ? p.scales[i] : io->scales[i];
    j.zeros = p.on_host ? p.zeros[i] : io->zeros[i];
    j.cand = nullptr;
    j.W_hat = p.on_host ? p.What[i] : io->W_hat[i];
    j.W_comp = nullptr;
    j.loss = p.on_host ? p.loss[i] : io->loss[i];
    j.stats = nullptr;
    j.ws = p.ws_quant[i];
    j.ws_bytes = p.quant_bytes[i];
  }
  // results of projection i back to the host (host buffers only)
  auto results_home = [&](int i) -> tb_status {
    if (!p.on_host) return TB_OK;
    PhaseScope ph(PH_COPY, st);
    const size_t n = (size_t)p.desc[i].d_out * p.desc[i].d_in;
    const size_t ng = D->quant_group > 0 ? (size_t)p.desc[i].d_in / D->quant_group : 1;
    const size_t ns = (size_t)p.desc[i].d_out * ng;
    TB_CUDA_CHECK(cudaMemcpyAsync(io->codes[i], p.codes[i], n, cudaMemcpyDeviceToHost, st));
    TB_CUDA_CHECK(cudaMemcpyAsync(io->scales[i], p.scales[i], ns * sizeof(float), cudaMemcpyDeviceToHost, st));
    TB_CUDA_CHECK(cudaMemcpyAsync(io->zeros[i], p.zeros[i], ns * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (io->W_hat[i])
      TB_CUDA_CHECK(cudaMemcpyAsync(io->W_hat[i], p.What[i], n * sizeof(float), cudaMemcpyDeviceToHost, st));
    if (io->loss[i])
      TB_CUDA_CHECK(cudaMemcpyAsync(io->loss[i], p.loss[i], sizeof(double) * (size_t)p.desc[i].n_heads,
                                    cudaMemcpyDeviceToHost, st));
    return TB_OK;
  };
  if (!value_last) {
    // the two large projections first: their launches then fill the GPU while the small ones run beside them
    const tb_projection_job order[4] = {jobs[0], jobs[3], jobs[1], jobs[2]};
    TB_TRY(tb_quantize_block(order, 4, p.concurrent ? 1 : 0, st));
    for (int i = 0; i < 4; ++i) TB_TRY(results_home(i));
  } else {
    // q, o and k while the value heads' activations are still crossing; then the value projection
    const tb_projection_job first[3] = {jobs[0], jobs[3], jobs[1]};
    TB_TRY(tb_quantize_block(first, 3, p.concurrent ? 1 : 0, st));
    TB_TRY(results_home(0));
    TB_TRY(results_home(3));
    TB_TRY(results_home(1));
    TB_TRY(value_side());
    TB_TRY(tb_quantize_block(&jobs[2], 1, 0, st));
    TB_TRY(results_home(2));
  }

  if (io->info) {
    TB_CUDA_CHECK(cudaMemcpyAsync(io->info, p.info, sizeof(int) * (size_t)p.info_count,
                                  p.on_host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice, st));
  }
  return TB_OK;
}

}  // namespace

extern "C" int tb_attention_layer_info_count(const tb_attention_desc* desc, int per_head_v) {
  if (!layer_desc_ok(desc)) return 0;
  return 2 + (per_head_v ? desc->n_kv_heads : 0) + desc->n_q_heads + 2 * desc->n_kv_heads;
}

extern "C" size_t tb_attention_layer_workspace(const tb_attention_desc* desc, const tb_attention_io* io) {
  LayerPlan p;
  if (make_layer_plan(desc, io, nullptr, &p) != TB_OK) return 0;
  return p.total;
}

extern "C" tb_status tb_attention_layer(const tb_attention_desc* desc, const tb_attention_io* io, void* ws,
                                        size_t ws_bytes, void* stream) {
  if (!desc || !io) return TB_ERR_INVALID_ARG;
  if (!io->X || !io->X_o) return TB_ERR_INVALID_ARG;
  for (int i = 0; i < 4; ++i)
    if (!io->W[i] || !io->codes[i] || !io->scales[i] || !io->zeros[i]) return TB_ERR_INVALID_ARG;
  LayerPlan p;
  TB_TRY(make_layer_plan(desc, io, nullptr, &p));
  if (!ws || !aligned(ws, 256) || ws_bytes < p.total) return TB_ERR_WORKSPACE;
  TB_TRY(make_layer_plan(desc, io, ws, &p));
  BlockSide* bs = block_side();
  if (!bs) return TB_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  // The copy stream starts after the caller's earlier work (the buffers may still be in use), and
  // both staging slots start out free.
  TB_CUDA_CHECK(cudaEventRecord(bs->fork, st));
  TB_CUDA_CHECK(cudaStreamWaitEvent(bs->copy, bs->fork, 0));
  for (int s = 0; s < STAGE_SLOTS; ++s) TB_CUDA_CHECK(cudaEventRecord(bs->consumed[s], st));
  tb_status status = layer_enqueue(desc, io, p, bs, st);
  // One way out: every helper stream joins the caller's.  With host buffers the call also waits
  // until nothing it enqueued is in flight, then reads the info words.
  bool ok = true;
  cudaStream_t others[N_HELPERS + 1] = {bs->helper[0], bs->helper[1], bs->helper[2], bs->helper[3], bs->copy};
  for (int i = 0; i < N_HELPERS + 1; ++i) {
    ok = cudaEventRecord(bs->dep[i], others[i]) == cudaSuccess && ok;
    ok = cudaStreamWaitEvent(st, bs->dep[i], 0) == cudaSuccess && ok;
  }
  if (p.on_host) ok = cudaStreamSynchronize(st) == cudaSuccess && ok;
  if (!ok) {
    (void)cudaGetLastError();
    return status != TB_OK ? status : TB_ERR_CUDA;
  }
  if (status != TB_OK || !p.on_host) return status;
  const int flag = tb_device_error_flag();
  if (flag != 0) return flag > 0 ? TB_ERR_TIMEOUT : TB_ERR_CUDA;
  int info_host[2 + 3 * 4096];
  const int n_info = p.info_count < 2 + 3 * 4096 ? p.info_count : 2 + 3 * 4096;
  TB_CUDA_CHECK(cudaMemcpy(info_host, p.info, sizeof(int) * (size_t)n_info, cudaMemcpyDeviceToHost));
  for (int i = 0; i < n_info; ++i)
    if (info_host[i] != 0) return TB_ERR_NOT_SPD;
  return TB_OK;
}
