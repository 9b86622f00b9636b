// Calibration Hessians (Table 1; Algorithm 1, statistics steps):
//   tb_accumulate_hessian  H += X^T X          (X token-major, so this is the paper's X X^T)
//   tb_accumulate_cross    R += alpha (X - Xfp)^T X
//   tb_finalize_hessian    normalisation by the token count and diagonal damping
//   tb_build_hout          H_out,h = G_h Hsum G_h^T  or  G_h G_h^T, per head
#include "tb_common.cuh"
#include "tb_gemm.cuh"

namespace tb {

tb_status syrk_bf16_tensor(float* H, const __nv_bfloat16* X, long long n_tok, int d, cudaStream_t st);
size_t cross_bf16_workspace(long long n_tok, int d);
tb_status cross_bf16_tensor(float* R, const __nv_bfloat16* X, const __nv_bfloat16* Xfp, long long n_tok, int d,
                            float alpha, void* ws, cudaStream_t st);
tb_status gemm_split_tensor(double* C, long long ldc, const float* A, const float* B, __nv_bfloat16* AT,
                            __nv_bfloat16* Bp, long long M, int N, int K, cudaStream_t st);

// G Hsum runs on the tensor cores when the shapes fit the TMA boxes of that kernel
static bool hout_on_tensor(int rows, int d) { return (rows % 8 == 0) && (d % 32 == 0); }

// Tokens per launch: partial sums of one launch stay in float registers, the
// running sum in H absorbs one rounding per launch.
static const long long kTokChunk = 4096;

// upper triangle <- lower triangle (the accumulation only forms tiles on or below the diagonal)
__global__ void k_mirror_lower(float* __restrict__ H, int d) {
  const long long n = (long long)d * d;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    // only entries outside the 128-wide diagonal tiles were skipped
    if (j / GEMM_BN > i / GEMM_BM) H[idx] = H[(long long)j * d + i];
  }
}

// R += alpha (X - Xfp)^T X over one token chunk.
template <typename TX>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
    k_cross(float* __restrict__ R, const TX* __restrict__ X, const TX* __restrict__ Xfp,
            long long n_tok, int d, float alpha) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int m0 = blockIdx.y * GEMM_BM, n0 = blockIdx.x * GEMM_BN;
  GemmAcc<float> acc;
  acc.clear();
  const int K = (int)n_tok;
  struct Pair {
    TX x, xfp;
  };
  auto la = [&](int mm, int k) -> Pair {
    const int m = m0 + mm;
    Pair p{zero_of<TX>(), zero_of<TX>()};
    if (m < d && k < K) {
      const long long o = (long long)k * d + m;
      p.x = X[o];
      p.xfp = Xfp[o];
    }
    return p;
  };
  auto ca = [](Pair p, int, int) -> float { return cvt<float, TX>(p.x) - cvt<float, TX>(p.xfp); };
  auto lb = [&](int nn, int k) -> TX {
    const int n = n0 + nn;
    return (n < d && k < K) ? X[(long long)k * d + n] : zero_of<TX>();
  };
  auto cb = [](TX v, int, int) -> float { return cvt<float, TX>(v); };
  gemm_mainloop<float, true, true>(acc, la, ca, lb, cb, 0, K, smem_raw);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + GemmAcc<float>::row(i);
    if (m >= d) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int n = n0 + GemmAcc<float>::col(j);
      if (n < d) R[(long long)m * d + n] = fmaf(alpha, acc.at(i, j), R[(long long)m * d + n]);
    }
  }
}

// Off-diagonal entries: H <- H / n (and the optional copy); R <- R / n.
__global__ void k_normalise(float* __restrict__ H, float* __restrict__ R, float* __restrict__ Hsum,
                            int d, double inv_n) {
  const long long n = (long long)d * d;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    if (R) R[idx] = (float)((double)R[idx] * inv_n);
    if (i == j) continue;  // the diagonal waits for the damping kernel
    const float v = (float)((double)H[idx] * inv_n);
    H[idx] = v;
    if (Hsum) Hsum[idx] = v;
  }
}

// Diagonal: mean of diag(H / n) in a fixed order, then H_ii <- H_ii / n + damp * mean.
__global__ void __launch_bounds__(256) k_damp_diagonal(float* __restrict__ H,
                                                       float* __restrict__ Hsum, int d,
                                                       double inv_n, double damp) {
  __shared__ double part[256];
  double acc = 0.0;
  for (int i = threadIdx.x; i < d; i += 256) acc += (double)H[(long long)i * d + i] * inv_n;
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
    __syncthreads();
  }
  const double mean = part[0] / (double)d;
  for (int i = threadIdx.x; i < d; i += 256) {
    const double v = (double)H[(long long)i * d + i] * inv_n;
    if (Hsum) Hsum[(long long)i * d + i] = (float)v;
    H[(long long)i * d + i] = (float)(v + damp * mean);
  }
}

// H_out[h] = combination of the per-block Grams, plus damp * mean(diag) on the diagonal.
__global__ void __launch_bounds__(256) k_combine_hout(float* __restrict__ Hout,
                                                      const double* __restrict__ blocks,
                                                      int n_heads, int g_heads, int dh, double damp) {
  __shared__ double part[256];
  const int h = blockIdx.x;
  const long long bb = (long long)dh * dh;
  int b_first, b_count;
  if (g_heads >= n_heads) {
    b_count = g_heads / n_heads;
    b_first = h * b_count;
  } else {
    b_count = 1;
    b_first = h / (n_heads / g_heads);
  }
  double acc = 0.0;
  for (int i = threadIdx.x; i < dh; i += 256) {
    double v = 0.0;
    for (int b = 0; b < b_count; ++b) v += blocks[(b_first + b) * bb + (long long)i * dh + i];
    acc += v;
  }
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
    __syncthreads();
  }
  const double mean = part[0] / (double)dh;
  for (long long idx = threadIdx.x; idx < bb; idx += 256) {
    double v = 0.0;
    for (int b = 0; b < b_count; ++b) v += blocks[(b_first + b) * bb + idx];
    if (idx / dh == idx % dh) v += damp * mean;
    Hout[h * bb + idx] = (float)v;
  }
}

template <typename TX>
static tb_status accumulate_typed(float* H, const TX* X, long long n_tok, int d, cudaStream_t st) {
  for (long long t0 = 0; t0 < n_tok; t0 += kTokChunk) {
    const long long nt = (n_tok - t0 < kTokChunk) ? (n_tok - t0) : kTokChunk;
    GemmP g = gemm_params();
    g.A = X + t0 * d;  // A(m, k) = X[k][m]
    g.a_m = 1;
    g.a_k = d;
    g.B = X + t0 * d;  // B(k, n) = X[k][n]
    g.b_k = d;
    g.b_n = 1;
    g.C = H;
    g.ldc = d;
    g.M = d;
    g.N = d;
    g.K = (int)nt;
    g.alpha = 1.0;
    g.beta = 1.0;
    g.flags = GEMM_LOWER_TILES;
    TB_TRY((gemm_launch<TX, TX, float, float, true, true>(g, st)));
  }
  k_mirror_lower<<<148 * 8, 256, 0, st>>>(H, d);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

template <typename TX>
static tb_status cross_typed(float* R, const TX* X, const TX* Xfp, long long n_tok, int d,
                             float alpha, cudaStream_t st) {
  auto kern = k_cross<TX>;
  static bool configured[64] = {false};
  TB_TRY(allow_smem(kern, GemmSmem<float>::bytes, configured));
  dim3 grid((d + GEMM_BN - 1) / GEMM_BN, (d + GEMM_BM - 1) / GEMM_BM);
  for (long long t0 = 0; t0 < n_tok; t0 += kTokChunk) {
    const long long nt = (n_tok - t0 < kTokChunk) ? (n_tok - t0) : kTokChunk;
    kern<<<grid, GEMM_THREADS, GemmSmem<float>::bytes, st>>>(R, X + t0 * d, Xfp + t0 * d, nt, d, alpha);
    TB_LAUNCH_CHECK();
  }
  return TB_OK;
}

}  // namespace tb

using namespace tb;

extern "C" tb_status tb_accumulate_hessian(float* H, const void* X, tb_dtype x_type,
                                           long long n_tok, int d, void* stream) {
  if (!H || n_tok < 0 || d <= 0 || (d % 8)) return TB_ERR_INVALID_ARG;
  if (x_type != TB_F32 && x_type != TB_BF16) return TB_ERR_INVALID_ARG;
  if (n_tok == 0) return TB_OK;  // nothing to add; X may be NULL
  if (!X) return TB_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (x_type == TB_BF16) {
    // bf16 activations: tensor cores (products exact in float, short float accumulations)
    if (!aligned(X, 16) || !aligned(H, 16)) return TB_ERR_INVALID_ARG;
    TB_TRY(syrk_bf16_tensor(H, static_cast<const __nv_bfloat16*>(X), n_tok, d, st));
    k_mirror_lower<<<148 * 8, 256, 0, st>>>(H, d);
    TB_LAUNCH_CHECK();
    return TB_OK;
  }
  // float activations keep every product exact only on the FP32 pipe
  return accumulate_typed<float>(H, static_cast<const float*>(X), n_tok, d, st);
}

extern "C" size_t tb_accumulate_cross_workspace(tb_dtype x_type, long long n_tok, int d) {
  if (x_type != TB_BF16 || n_tok <= 0 || d <= 0) return 0;
  return cross_bf16_workspace(n_tok, d);
}

extern "C" tb_status tb_accumulate_cross(float* R, const void* X, const void* Xfp, tb_dtype x_type,
                                         long long n_tok, int d, float alpha, void* ws, size_t ws_bytes,
                                         void* stream) {
  if (!R || n_tok < 0 || d <= 0 || (d % 8)) return TB_ERR_INVALID_ARG;
  if (x_type != TB_F32 && x_type != TB_BF16) return TB_ERR_INVALID_ARG;
  if (n_tok == 0) return TB_OK;
  if (!X || !Xfp) return TB_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (x_type == TB_BF16) {
    // bf16 activations: tensor cores, the deviation in two exact bf16 pieces
    if (!aligned(X, 16) || !aligned(Xfp, 16) || !aligned(R, 16)) return TB_ERR_INVALID_ARG;
    if (!ws || !aligned(ws, 256) || ws_bytes < cross_bf16_workspace(n_tok, d)) return TB_ERR_WORKSPACE;
    return cross_bf16_tensor(R, static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(Xfp),
                             n_tok, d, alpha, ws, st);
  }
  return cross_typed<float>(R, static_cast<const float*>(X), static_cast<const float*>(Xfp), n_tok, d,
                            alpha, st);
}

extern "C" tb_status tb_finalize_hessian(float* H, float* R, float* Hsum_out, int d,
                                         long long n_total, float damp, void* stream) {
  if (!H || d <= 0 || n_total <= 0 || !(damp >= 0.0f)) return TB_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  const double inv_n = 1.0 / (double)n_total;
  k_normalise<<<148 * 8, 256, 0, st>>>(H, R, Hsum_out, d, inv_n);
  TB_LAUNCH_CHECK();
  k_damp_diagonal<<<1, 256, 0, st>>>(H, Hsum_out, d, inv_n, (double)damp);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

extern "C" size_t tb_build_hout_workspace(int g_heads, int d_head, int d) {
  if (g_heads <= 0 || d_head <= 0 || d <= 0) return 0;
  Bump b(nullptr);
  b.take<double>((size_t)g_heads * d_head * d);       // G Hsum
  b.take<double>((size_t)g_heads * d_head * d_head);  // per-block Grams
  if (hout_on_tensor(g_heads * d_head, d)) {
    b.take<__nv_bfloat16>((size_t)3 * g_heads * d_head * d);  // G^T in three bf16 pieces
    b.take<__nv_bfloat16>((size_t)3 * d * d);                 // Hsum in three bf16 pieces
  }
  return b.total();
}

extern "C" tb_status tb_build_hout(float* H_out, const float* G, const float* Hsum, int n_heads,
                                   int g_heads, int d_head, int d, float damp, void* ws,
                                   size_t ws_bytes, void* stream) {
  if (!H_out || !G || n_heads <= 0 || g_heads <= 0 || d_head <= 0 || d <= 0 || !(damp >= 0.0f))
    return TB_ERR_INVALID_ARG;
  if (g_heads >= n_heads ? (g_heads % n_heads) : (n_heads % g_heads)) return TB_ERR_INVALID_ARG;
  if (!ws || !aligned(ws, 256) || ws_bytes < tb_build_hout_workspace(g_heads, d_head, d))
    return TB_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  Bump b(ws);
  double* T = b.take<double>((size_t)g_heads * d_head * d);
  double* blocks = b.take<double>((size_t)g_heads * d_head * d_head);
  const int rows = g_heads * d_head;
  GemmP q = gemm_params();
  if (Hsum && hout_on_tensor(rows, d)) {
    // T = G Hsum from exact bf16 splits of both operands (float-accurate products, double chunk sums)
    __nv_bfloat16* GT = b.take<__nv_bfloat16>((size_t)3 * rows * d);
    __nv_bfloat16* Hp = b.take<__nv_bfloat16>((size_t)3 * d * d);
    TB_TRY(gemm_split_tensor(T, d, G, Hsum, GT, Hp, rows, d, d, st));
    q.A = T;
  } else if (Hsum) {
    GemmP g = gemm_params();  // T = G Hsum
    g.A = G;
    g.a_m = d;
    g.a_k = 1;
    g.B = Hsum;
    g.b_k = d;
    g.b_n = 1;
    g.C = T;
    g.ldc = d;
    g.M = rows;
    g.N = d;
    g.K = d;
    TB_TRY((gemm_launch<float, float, double, double, false, true>(g, st)));
    q.A = T;  // blocks_b = T_b G_b^T
  }
  q.a_m = d;
  q.a_k = 1;
  q.a_batch = (long long)d_head * d;
  q.B = G;  // B(k, n) = G_b[n][k]
  q.b_k = 1;
  q.b_n = d;
  q.b_batch = (long long)d_head * d;
  q.C = blocks;
  q.ldc = d_head;
  q.c_batch = (long long)d_head * d_head;
  q.M = d_head;
  q.N = d_head;
  q.K = d;
  q.n_batch = g_heads;
  if (Hsum) {
    TB_TRY((gemm_launch<double, float, double, double, false, false>(q, st)));
  } else {
    q.A = G;
    TB_TRY((gemm_launch<float, float, double, double, false, false>(q, st)));
  }
  k_combine_hout<<<n_heads, 256, 0, st>>>(H_out, blocks, n_heads, g_heads, d_head, (double)damp);
  TB_LAUNCH_CHECK();
  return TB_OK;
}
