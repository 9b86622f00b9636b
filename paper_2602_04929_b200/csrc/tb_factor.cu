// tb_factor: U upper triangular with H^{-1} = U^T U (Eq. 2), batched, and
// tb_prepare_correction: P and C of Algorithm 2 line 2 / Proposition 3.2.
//
// Route taken for U (the positive-diagonal factor is unique, so any route to it
// is the factor of Eq. 2): with J the index reversal, J H J = L L^T is an
// ordinary lower Cholesky factorisation; then H = (J L J)(J L J)^T with
// M = J L J upper triangular, H^{-1} = M^{-T} M^{-1}, hence U = M^{-1} = J L^{-1} J.
// No inverse of H is formed.  Everything runs in double: with cond(H_in) ~ 1e5
// a float factorisation would lose most of U's digits.
//
//   1. A = J H J                                        (k_reverse_in)
//   2. right-looking blocked Cholesky, 64-column panels:
//        k_potrf64   factor the 64 x 64 diagonal block in shared memory and
//                    invert it (forward substitution, one thread per column)
//        GEMM        panel below the block  <- panel * inv(L_kk)^T
//        GEMM        trailing matrix -= panel panel^T   (tiles on/below the diagonal)
//   3. L^{-1} by block rows: X[i, 0:i] = -inv(L_ii) (L[i, 0:i] X[0:i, 0:i])
//   4. U = J L^{-1} J, written as float with an explicit zero lower triangle.
#include "tb_common.cuh"
#include "tb_gemm.cuh"

namespace tb {

enum { FNB = 64 };

__global__ void k_reverse_in(const float* __restrict__ H, double* __restrict__ A, int d) {
  const long long n = (long long)d * d;
  const float* Hb = H + (long long)blockIdx.y * n;
  double* Ab = A + (long long)blockIdx.y * n;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    Ab[idx] = (double)Hb[(long long)(d - 1 - i) * d + (d - 1 - j)];
  }
}

__global__ void k_reverse_out(const double* __restrict__ Li, float* __restrict__ U, int d) {
  const long long n = (long long)d * d;
  const double* Lb = Li + (long long)blockIdx.y * n;
  float* Ub = U + (long long)blockIdx.y * n;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    Ub[idx] = (j >= i) ? (float)Lb[(long long)(d - 1 - i) * d + (d - 1 - j)] : 0.0f;
  }
}

// Factor the diagonal block [k0, k0 + nb) of A in place (lower Cholesky) and
// write its inverse to Dinv (64 x 64, zero above the diagonal) and to the
// diagonal block of Li.  A non-positive pivot is recorded in info (first one
// wins) and replaced by 1 so that no NaN or Inf is produced by this kernel.
__global__ void __launch_bounds__(256) k_potrf64(double* __restrict__ A, double* __restrict__ Li,
                                                 double* __restrict__ Dinv, int* __restrict__ info,
                                                 int d, int k0, int nb, int n_blk) {
  __shared__ double Ls[FNB][FNB + 1];
  __shared__ double rdiag[FNB];
  const int b = blockIdx.x, tid = threadIdx.x;
  double* Ab = A + (long long)b * d * d;
  for (int idx = tid; idx < FNB * FNB; idx += 256) {
    const int r = idx / FNB, c = idx % FNB;
    double v = (r == c) ? 1.0 : 0.0;
    if (r < nb && c < nb) v = Ab[(long long)(k0 + r) * d + k0 + c];
    Ls[r][c] = v;
  }
  __syncthreads();
  for (int j = 0; j < FNB; ++j) {
    const double pv = Ls[j][j];
    const bool bad = !(pv > 0.0);
    const double dj = bad ? 1.0 : sqrt(pv);
    if (bad && tid == 0 && j < nb) atomicCAS(&info[b], 0, k0 + j + 1);
    __syncthreads();
    if (tid == 0) Ls[j][j] = dj;
    if (tid > j && tid < FNB) Ls[tid][j] = Ls[tid][j] / dj;
    __syncthreads();
    for (int idx = tid; idx < FNB * FNB; idx += 256) {
      const int r = idx / FNB, c = idx % FNB;
      if (c > j && c <= r) Ls[r][c] = fma(-Ls[r][j], Ls[c][j], Ls[r][c]);
    }
    __syncthreads();
  }
  for (int idx = tid; idx < FNB * FNB; idx += 256) {
    const int r = idx / FNB, c = idx % FNB;
    if (r < nb && c < nb && c <= r) Ab[(long long)(k0 + r) * d + k0 + c] = Ls[r][c];
  }
  if (tid < FNB) rdiag[tid] = 1.0 / Ls[tid][tid];
  __syncthreads();
  if (tid < FNB) {
    // column `tid` of inv(L): L x = e_tid by forward substitution, x in registers
    const int c = tid;
    double x[FNB];
#pragma unroll
    for (int r = 0; r < FNB; ++r) {
      double s = (r == c) ? 1.0 : 0.0;
#pragma unroll
      for (int k = 0; k < r; ++k) s = fma(-Ls[r][k], x[k], s);
      x[r] = (r < c) ? 0.0 : s * rdiag[r];
    }
    double* Db = Dinv + ((long long)b * n_blk + k0 / FNB) * FNB * FNB;
    double* Lb = Li + (long long)b * d * d;
#pragma unroll
    for (int r = 0; r < FNB; ++r) {
      Db[r * FNB + c] = x[r];
      if (r < nb && c < nb) Lb[(long long)(k0 + r) * d + k0 + c] = x[r];
    }
  }
}

__global__ void k_copy_panel(const double* __restrict__ A, double* __restrict__ Pn, int d, int r0,
                             int k0, int nb) {
  const long long rows = d - r0;
  const double* Ab = A + (long long)blockIdx.y * d * d;
  double* Pb = Pn + (long long)blockIdx.y * d * FNB;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < rows * nb;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long r = idx / nb;
    const int c = (int)(idx % nb);
    Pb[r * FNB + c] = Ab[(r0 + r) * d + k0 + c];
  }
}

// strictly-upper mask of a square matrix (Algorithm 2 line 2: (R U^T) .* M_U)
__global__ void k_mask_strict_upper(const double* __restrict__ src, double* __restrict__ dst, int d) {
  const long long n = (long long)d * d;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    dst[idx] = (j > i) ? src[idx] : 0.0;
  }
}

struct FactorWs {
  double *A, *Li, *Dinv, *Pn, *tmp;
  int n_blk;
  size_t total;
};

static FactorWs factor_ws(int n_batch, int d, void* ws) {
  FactorWs f;
  Bump b(ws);
  f.n_blk = (d + FNB - 1) / FNB;
  f.A = b.take<double>((size_t)n_batch * d * d);
  f.Li = b.take<double>((size_t)n_batch * d * d);
  f.Dinv = b.take<double>((size_t)n_batch * f.n_blk * FNB * FNB);
  f.Pn = b.take<double>((size_t)n_batch * d * FNB);
  f.tmp = b.take<double>((size_t)n_batch * FNB * d);
  f.total = b.total();
  return f;
}

}  // namespace tb

using namespace tb;

extern "C" size_t tb_factor_workspace(int n_batch, int d) {
  if (n_batch <= 0 || d <= 0) return 0;
  return factor_ws(n_batch, d, nullptr).total;
}

extern "C" tb_status tb_factor(const float* H, int n_batch, int d, float* U, float* Hinv, int* info,
                               void* ws, size_t ws_bytes, void* stream) {
  if (!H || !U || !info || n_batch <= 0 || n_batch > 65535 || d <= 0) return TB_ERR_INVALID_ARG;
  if (!ws || !aligned(ws, 256) || ws_bytes < tb_factor_workspace(n_batch, d)) return TB_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  FactorWs f = factor_ws(n_batch, d, ws);
  const long long dd = (long long)d * d;
  TB_CUDA_CHECK(cudaMemsetAsync(info, 0, sizeof(int) * (size_t)n_batch, st));
  TB_CUDA_CHECK(cudaMemsetAsync(f.Li, 0, sizeof(double) * (size_t)n_batch * dd, st));
  int eb = (int)((dd + 255) / 256);
  if (eb > 148 * 8) eb = 148 * 8;
  k_reverse_in<<<dim3(eb, n_batch), 256, 0, st>>>(H, f.A, d);
  TB_LAUNCH_CHECK();

  for (int k0 = 0; k0 < d; k0 += FNB) {
    const int nb = (d - k0 < FNB) ? (d - k0) : FNB;
    k_potrf64<<<n_batch, 256, 0, st>>>(f.A, f.Li, f.Dinv, info, d, k0, nb, f.n_blk);
    TB_LAUNCH_CHECK();
    const int r0 = k0 + nb, m = d - r0;
    if (m <= 0) break;
    k_copy_panel<<<dim3(64, n_batch), 256, 0, st>>>(f.A, f.Pn, d, r0, k0, nb);
    TB_LAUNCH_CHECK();
    GemmP g = gemm_params();  // panel <- panel inv(L_kk)^T
    g.A = f.Pn;
    g.a_m = FNB;
    g.a_k = 1;
    g.a_batch = (long long)d * FNB;
    g.B = f.Dinv + (long long)(k0 / FNB) * FNB * FNB;  // B(k, n) = Dinv[n][k]
    g.b_k = 1;
    g.b_n = FNB;
    g.b_batch = (long long)f.n_blk * FNB * FNB;
    g.C = f.A + (long long)r0 * d + k0;
    g.ldc = d;
    g.c_batch = dd;
    g.M = m;
    g.N = nb;
    g.K = nb;
    g.n_batch = n_batch;
    TB_TRY((gemm_launch<double, double, double, double, false, false>(g, st)));
    GemmP s = gemm_params();  // trailing -= panel panel^T, tiles on or below the diagonal
    s.A = f.A + (long long)r0 * d + k0;
    s.a_m = d;
    s.a_k = 1;
    s.a_batch = dd;
    s.B = f.A + (long long)r0 * d + k0;  // B(k, n) = panel[n][k]
    s.b_k = 1;
    s.b_n = d;
    s.b_batch = dd;
    s.C = f.A + (long long)r0 * d + r0;
    s.ldc = d;
    s.c_batch = dd;
    s.M = m;
    s.N = m;
    s.K = nb;
    s.n_batch = n_batch;
    s.alpha = -1.0;
    s.beta = 1.0;
    s.flags = GEMM_LOWER_TILES;
    TB_TRY((gemm_launch<double, double, double, double, false, false>(s, st)));
  }

  // L^{-1}, block row by block row (diagonal blocks are already in place)
  for (int r0 = FNB; r0 < d; r0 += FNB) {
    const int nb = (d - r0 < FNB) ? (d - r0) : FNB;
    GemmP g = gemm_params();  // tmp = L[r0:r0+nb, 0:r0] * Li[0:r0, 0:r0]
    g.A = f.A + (long long)r0 * d;
    g.a_m = d;
    g.a_k = 1;
    g.a_batch = dd;
    g.B = f.Li;
    g.b_k = d;
    g.b_n = 1;
    g.b_batch = dd;
    g.C = f.tmp;
    g.ldc = d;
    g.c_batch = (long long)FNB * d;
    g.M = nb;
    g.N = r0;
    g.K = r0;
    g.n_batch = n_batch;
    g.btrim = 2;  // Li is lower triangular: Li(k, n) = 0 for k < n
    g.boff = 0;
    TB_TRY((gemm_launch<double, double, double, double, false, true>(g, st)));
    GemmP h = gemm_params();  // Li[r0:r0+nb, 0:r0] = -inv(L_ii) tmp
    h.A = f.Dinv + (long long)(r0 / FNB) * FNB * FNB;
    h.a_m = FNB;
    h.a_k = 1;
    h.a_batch = (long long)f.n_blk * FNB * FNB;
    h.B = f.tmp;
    h.b_k = d;
    h.b_n = 1;
    h.b_batch = (long long)FNB * d;
    h.C = f.Li + (long long)r0 * d;
    h.ldc = d;
    h.c_batch = dd;
    h.M = nb;
    h.N = r0;
    h.K = nb;
    h.n_batch = n_batch;
    h.alpha = -1.0;
    TB_TRY((gemm_launch<double, double, double, double, false, true>(h, st)));
  }
  k_reverse_out<<<dim3(eb, n_batch), 256, 0, st>>>(f.Li, U, d);
  TB_LAUNCH_CHECK();

  if (Hinv) {
    // Hinv = U^T U with U(k, m) = Li[d-1-k][d-1-m]: negative strides from the last element
    GemmP g = gemm_params();
    const double* last = f.Li + dd - 1;
    g.A = last;  // A(m, k) = U[k][m]
    g.a_m = -1;
    g.a_k = -(long long)d;
    g.a_batch = dd;
    g.B = last;  // B(k, n) = U[k][n]
    g.b_k = -(long long)d;
    g.b_n = -1;
    g.b_batch = dd;
    g.C = Hinv;
    g.ldc = d;
    g.c_batch = dd;
    g.M = d;
    g.N = d;
    g.K = d;
    g.n_batch = n_batch;
    g.btrim = 1;  // U(k, n) = 0 for k > n
    g.atrim = 1;  // U(k, m) = 0 for k > m
    TB_TRY((gemm_launch<double, double, float, double, true, true>(g, st)));
  }
  return TB_OK;
}

extern "C" size_t tb_prepare_correction_workspace(int n_batch, int d) {
  if (n_batch <= 0 || d <= 0) return 0;
  Bump b(nullptr);
  b.take<double>((size_t)d * d);
  b.take<double>((size_t)d * d);
  return b.total();
}

extern "C" tb_status tb_prepare_correction(const float* R, const float* U_in, int n_batch, int d,
                                           float* P, float* C, void* ws, size_t ws_bytes,
                                           void* stream) {
  if (!R || !U_in || !P || !C || n_batch <= 0 || d <= 0) return TB_ERR_INVALID_ARG;
  if (!ws || !aligned(ws, 256) || ws_bytes < tb_prepare_correction_workspace(n_batch, d))
    return TB_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  Bump b(ws);
  double* T1 = b.take<double>((size_t)d * d);
  double* T2 = b.take<double>((size_t)d * d);
  const long long dd = (long long)d * d;
  int eb = (int)((dd + 255) / 256);
  if (eb > 148 * 8) eb = 148 * 8;
  for (int i = 0; i < n_batch; ++i) {
    const float* Rb = R + i * dd;
    const float* Ub = U_in + i * dd;
    GemmP g = gemm_params();  // T1 = R U^T
    g.A = Rb;
    g.a_m = d;
    g.a_k = 1;
    g.B = Ub;  // B(k, n) = U[n][k], zero for k < n
    g.b_k = 1;
    g.b_n = d;
    g.C = T1;
    g.ldc = d;
    g.M = d;
    g.N = d;
    g.K = d;
    g.btrim = 2;
    TB_TRY((gemm_launch<float, float, double, double, false, false>(g, st)));
    GemmP c = gemm_params();  // C = T1 U
    c.A = T1;
    c.a_m = d;
    c.a_k = 1;
    c.B = Ub;  // B(k, n) = U[k][n], zero for k > n
    c.b_k = d;
    c.b_n = 1;
    c.C = C + i * dd;
    c.ldc = d;
    c.M = d;
    c.N = d;
    c.K = d;
    c.btrim = 1;
    TB_TRY((gemm_launch<double, float, float, double, false, true>(c, st)));
    k_mask_strict_upper<<<eb, 256, 0, st>>>(T1, T2, d);
    TB_LAUNCH_CHECK();
    GemmP p = c;  // P = (strictly upper part of T1) U
    p.A = T2;
    p.C = P + i * dd;
    p.atrim = 2;  // T2(m, k) = 0 for k < m + 1
    p.aoff = 1;
    TB_TRY((gemm_launch<double, float, float, double, false, true>(p, st)));
  }
  return TB_OK;
}
