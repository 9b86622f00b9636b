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
// The matrix is embedded in a dp x dp one (dp = 64 * 2^k >= d, identity in the
// padding) so that every block step below is uniform.
//   1. A = J H J                                        (k_reverse_in)
//   2. right-looking blocked Cholesky, 64-column panels, two launches per panel:
//        k_chol_panel  every CTA factors the 64 x 64 diagonal block (one thread
//                      per row, the row in registers, left-looking) and then
//                      solves its 128 rows of the panel against it
//        GEMM          trailing matrix -= panel panel^T  (tiles on/below the diagonal)
//   3. inverses of the 64 x 64 diagonal blocks, all at once (k_inv_diag64)
//   4. L^{-1} by recursive doubling: for block size s = 64, 128, ... every pair of
//      neighbouring inverted blocks A, B with coupling C = L[B rows, A cols] gets
//      its off-diagonal block -B^{-1} C A^{-1} from two batched GEMMs
//   5. U = J L^{-1} J, written as float with an explicit zero lower triangle.
#include "tb_common.cuh"
#include "tb_gemm.cuh"

namespace tb {

enum { FNB = 64 };

// A (dp x dp) <- J H J in the leading d x d block, identity elsewhere
__global__ void k_reverse_in(const float* __restrict__ H, double* __restrict__ A, int d, int dp) {
  const long long n = (long long)dp * dp;
  const float* Hb = H + (long long)blockIdx.y * d * d;
  double* Ab = A + (long long)blockIdx.y * n;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / dp), j = (int)(idx % dp);
    double v = (i == j) ? 1.0 : 0.0;
    if (i < d && j < d) v = (double)Hb[(long long)(d - 1 - i) * d + (d - 1 - j)];
    Ab[idx] = v;
  }
}

__global__ void k_reverse_out(const double* __restrict__ Li, float* __restrict__ U, int d, int dp) {
  const long long n = (long long)d * d;
  const double* Lb = Li + (long long)blockIdx.y * dp * dp;
  float* Ub = U + (long long)blockIdx.y * n;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    Ub[idx] = (j >= i) ? (float)Lb[(long long)(d - 1 - i) * dp + (d - 1 - j)] : 0.0f;
  }
}

// One panel step of the Cholesky factorisation, columns k0 .. k0+63 of the dp x dp matrix.
// Every CTA factors the diagonal block itself (same arithmetic everywhere, so the same
// result); CTA x then solves rows k0+64+128x .. +127 of the panel, X L_kk^T = A_panel.
// A non-positive pivot is recorded in info (first one wins) and replaced by 1.
__global__ void __launch_bounds__(128) k_chol_panel(double* __restrict__ A, int* __restrict__ info,
                                                    int dp, int k0) {
  __shared__ double sL[FNB][FNB + 1];
  __shared__ double rdiag[FNB];
  const int tid = threadIdx.x, b = blockIdx.y;
  double* Ab = A + (long long)b * dp * dp;
  if (tid < FNB) {
    // left-looking factorisation, thread r owns row r of the block
    const int r = tid;
    double a[FNB];
    const double* src = Ab + (long long)(k0 + r) * dp + k0;
#pragma unroll
    for (int c = 0; c < FNB; ++c) a[c] = src[c];
#pragma unroll
    for (int j = 0; j < FNB; ++j) {
      // t = a[r][j] - sum_{k<j} L[r][k] L[j][k]
      double t0 = a[j], t1 = 0.0;
#pragma unroll
      for (int k = 0; k + 1 < j; k += 2) {
        t0 = fma(-a[k], sL[j][k], t0);
        t1 = fma(-a[k + 1], sL[j][k + 1], t1);
      }
      if (j & 1) t0 = fma(-a[j - 1], sL[j][j - 1], t0);
      const double t = t0 + t1;
      if (r == j) {
        const bool bad = !(t > 0.0);
        if (bad && blockIdx.x == 0) atomicCAS(&info[b], 0, k0 + j + 1);
        const double dj = bad ? 1.0 : sqrt(t);
        sL[j][j] = dj;
        rdiag[j] = 1.0 / dj;
        a[j] = dj;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");  // all 128 threads (the other 64 pass the same barriers below)
      if (r > j) {
        a[j] = t * rdiag[j];
        sL[r][j] = a[j];
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    if (blockIdx.x == 0) {
      double* dst = Ab + (long long)(k0 + r) * dp + k0;
#pragma unroll
      for (int c = 0; c < FNB; ++c)
        if (c <= r) dst[c] = a[c];
    }
  } else {
#pragma unroll 1
    for (int j = 0; j < 2 * FNB; ++j) asm volatile("bar.sync 1, 128;" ::: "memory");
  }
  // rows of the panel below the block
  const long long row = (long long)k0 + FNB + (long long)blockIdx.x * 128 + tid;
  if (row < dp) {
    double x[FNB];
    double* src = Ab + row * dp + k0;
#pragma unroll
    for (int c = 0; c < FNB; ++c) x[c] = src[c];
#pragma unroll
    for (int j = 0; j < FNB; ++j) {
      double t0 = x[j], t1 = 0.0;
#pragma unroll
      for (int k = 0; k + 1 < j; k += 2) {
        t0 = fma(-x[k], sL[j][k], t0);
        t1 = fma(-x[k + 1], sL[j][k + 1], t1);
      }
      if (j & 1) t0 = fma(-x[j - 1], sL[j][j - 1], t0);
      x[j] = (t0 + t1) * rdiag[j];
    }
#pragma unroll
    for (int c = 0; c < FNB; ++c) src[c] = x[c];
  }
}

// Inverse of every 64 x 64 diagonal block of L into the same block of Li (lower triangular):
// forward substitution, one thread per column, the column in registers.
__global__ void __launch_bounds__(64) k_inv_diag64(const double* __restrict__ A, double* __restrict__ Li, int dp) {
  __shared__ double Ls[FNB][FNB + 1];
  __shared__ double rdiag[FNB];
  const int blk = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const long long off = (long long)b * dp * dp + (long long)blk * FNB * (dp + 1);
  for (int r = 0; r < FNB; ++r) Ls[r][c] = A[off + (long long)r * dp + c];
  __syncthreads();
  rdiag[c] = 1.0 / Ls[c][c];
  __syncthreads();
  double x[FNB];
#pragma unroll
  for (int r = 0; r < FNB; ++r) {
    double s0 = (r == c) ? 1.0 : 0.0;
#pragma unroll
    for (int k = 0; k < r; ++k) s0 = fma(-Ls[r][k], x[k], s0);
    x[r] = (r < c) ? 0.0 : s0 * rdiag[r];
  }
#pragma unroll
  for (int r = 0; r < FNB; ++r) Li[off + (long long)r * dp + c] = x[r];
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
  double *A, *Li, *tmp;
  int dp;
  size_t total;
};

static int padded_dim(int d) {
  int dp = FNB;
  while (dp < d) dp <<= 1;
  return dp;
}

static FactorWs factor_ws(int n_batch, int d, void* ws) {
  FactorWs f;
  Bump b(ws);
  f.dp = padded_dim(d);
  const size_t n = (size_t)f.dp * f.dp;
  f.A = b.take<double>((size_t)n_batch * n);
  f.Li = b.take<double>((size_t)n_batch * n);
  f.tmp = b.take<double>((size_t)n_batch * n / 4 + 64);
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
  const int dp = f.dp;
  const long long pp = (long long)dp * dp;
  TB_CUDA_CHECK(cudaMemsetAsync(info, 0, sizeof(int) * (size_t)n_batch, st));
  TB_CUDA_CHECK(cudaMemsetAsync(f.Li, 0, sizeof(double) * (size_t)n_batch * pp, st));
  int eb = (int)((pp + 255) / 256);
  if (eb > 148 * 8) eb = 148 * 8;
  k_reverse_in<<<dim3(eb, n_batch), 256, 0, st>>>(H, f.A, d, dp);
  TB_LAUNCH_CHECK();

  // the padding is an identity block decoupled from the rest: factor the leading part only
  const int d_fact = ((d + FNB - 1) / FNB) * FNB;
  for (int k0 = 0; k0 < d_fact; k0 += FNB) {
    const int r0 = k0 + FNB, m = d_fact - r0;
    const int xt = (m > 0) ? (m + 127) / 128 : 1;
    k_chol_panel<<<dim3(xt, n_batch), 128, 0, st>>>(f.A, info, dp, k0);
    TB_LAUNCH_CHECK();
    if (m <= 0) break;
    GemmP s = gemm_params();  // trailing -= panel panel^T, tiles on or below the diagonal
    s.A = f.A + (long long)r0 * dp + k0;
    s.a_m = dp;
    s.a_k = 1;
    s.a_batch = pp;
    s.B = f.A + (long long)r0 * dp + k0;  // B(k, n) = panel[n][k]
    s.b_k = 1;
    s.b_n = dp;
    s.b_batch = pp;
    s.C = f.A + (long long)r0 * dp + r0;
    s.ldc = dp;
    s.c_batch = pp;
    s.M = m;
    s.N = m;
    s.K = FNB;
    s.n_batch = n_batch;
    s.alpha = -1.0;
    s.beta = 1.0;
    s.flags = GEMM_LOWER_TILES;
    TB_TRY((gemm_launch<double, double, double, double, false, false>(s, st)));
  }

  // L^{-1}: diagonal blocks, then recursive doubling
  k_inv_diag64<<<dim3(dp / FNB, n_batch), 64, 0, st>>>(f.A, f.Li, dp);
  TB_LAUNCH_CHECK();
  for (int sblk = FNB; sblk < dp; sblk <<= 1) {
    const int pairs = dp / (2 * sblk);
    // one batched launch covers all pairs of one matrix, or (a single pair per matrix) all matrices
    const int outer = (pairs == 1) ? 1 : n_batch;
    for (int mb = 0; mb < outer; ++mb) {
      const long long moff = (long long)mb * pp;
      const long long pair_stride = (pairs == 1) ? pp : (long long)2 * sblk * (dp + 1);
      const int batch = (pairs == 1) ? n_batch : pairs;
      double* tmp = f.tmp + (long long)mb * (pp / 4);
      const long long tmp_stride = (pairs == 1) ? (pp / 4) : (long long)sblk * sblk;
      GemmP g = gemm_params();  // T = C A^{-1}: C = L[s:2s, 0:s], A^{-1} = Li[0:s, 0:s] (lower triangular)
      g.A = f.A + moff + (long long)sblk * dp;
      g.a_m = dp;
      g.a_k = 1;
      g.a_batch = pair_stride;
      g.B = f.Li + moff;
      g.b_k = dp;
      g.b_n = 1;
      g.b_batch = pair_stride;
      g.C = tmp;
      g.ldc = sblk;
      g.c_batch = tmp_stride;
      g.M = sblk;
      g.N = sblk;
      g.K = sblk;
      g.n_batch = batch;
      g.btrim = 2;
      TB_TRY((gemm_launch<double, double, double, double, false, true>(g, st)));
      GemmP h = gemm_params();  // Li[s:2s, 0:s] = -B^{-1} T, B^{-1} = Li[s:2s, s:2s] (lower triangular)
      h.A = f.Li + moff + (long long)sblk * (dp + 1);
      h.a_m = dp;
      h.a_k = 1;
      h.a_batch = pair_stride;
      h.B = tmp;
      h.b_k = sblk;
      h.b_n = 1;
      h.b_batch = tmp_stride;
      h.C = f.Li + moff + (long long)sblk * dp;
      h.ldc = dp;
      h.c_batch = pair_stride;
      h.M = sblk;
      h.N = sblk;
      h.K = sblk;
      h.n_batch = batch;
      h.alpha = -1.0;
      h.atrim = 1;
      TB_TRY((gemm_launch<double, double, double, double, false, true>(h, st)));
    }
  }
  int eo = (int)(((long long)d * d + 255) / 256);
  if (eo > 148 * 8) eo = 148 * 8;
  k_reverse_out<<<dim3(eo, n_batch), 256, 0, st>>>(f.Li, U, d, dp);
  TB_LAUNCH_CHECK();

  if (Hinv) {
    // Hinv = U^T U with U(k, m) = Li[d-1-k][d-1-m]: negative strides from element (d-1, d-1)
    GemmP g = gemm_params();
    const double* last = f.Li + (long long)(d - 1) * dp + (d - 1);
    g.A = last;  // A(m, k) = U[k][m]
    g.a_m = -1;
    g.a_k = -(long long)dp;
    g.a_batch = pp;
    g.B = last;  // B(k, n) = U[k][n]
    g.b_k = -(long long)dp;
    g.b_n = -1;
    g.b_batch = pp;
    g.C = Hinv;
    g.ldc = d;
    g.c_batch = (long long)d * d;
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
