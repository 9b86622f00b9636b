// tb_factor: U upper triangular with H^{-1} = U^T U (Eq. 2), batched, and
// tb_prepare_correction: P and C of Algorithm 2 (masked operand) / Proposition 3.2.
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
//                      per row, the row in registers, right-looking) and then
//                      solves its 64 rows of the panel against it
//                      (after applying the previous panel's update to its own columns)
//        GEMM          trailing matrix -= panel panel^T from the panel after the next on
//                      (tiles on/below the diagonal)
//   3. inverses of the 64 x 64 diagonal blocks (k_inv_diag64)
//   4. L^{-1} by recursive doubling: for block size s = 64, 128, ... every pair of
//      neighbouring inverted blocks A, B with coupling C = L[B rows, A cols] gets
//      its off-diagonal block -B^{-1} C A^{-1} from two batched GEMMs.  Steps 3 and 4
//      follow the factorisation block by block of 512 columns, so that with the
//      look-ahead they run beside the later panels.
//   5. U = J L^{-1} J, written as float with an explicit zero lower triangle.
#include "tb_common.cuh"
#include "tb_gemm.cuh"
#include "tb_gemm64.cuh"

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
// result); CTA x then solves rows k0+64+64x .. +63 of the panel, X L_kk^T = A_panel.
// L_kk itself is stored in Ldiag[k0 / 64] (64 x 64, row-major), not in A.
// A non-positive pivot is recorded in info (first one wins) and replaced by 1.
//
// 256 threads; thread (r, q) keeps columns 16q .. 16q+15 of row r in registers, a warp
// shares q.  The loops over 16-column blocks are rolled (straight-line code executed once
// is bound by instruction fetch), the 16 steps inside a block are unrolled.
//
// Factorisation, right-looking.  Step j: the owners publish their (final) entries of
// column j, one barrier, then every thread forms the reciprocal pivot itself and applies
// a[c] -= a[j] / piv * col_j[c] to its part of the row.  The published raw columns stay in
// shared memory: the panel solve runs the same elimination on its rows (x_j = a_j / L_jj,
// then a_c -= x_j / L_jj * col_j[c]), so neither L nor an inverse is stored in between.
// Entries right of the diagonal go through the same updates and are never used.
//
// update_first: the previous panel's rank-64 update of these 64 columns has not been applied yet (the
// trailing update after a panel leaves out the next panel's columns); the kernel applies it to the
// diagonal block and to its own rows before it starts, from the previous panel's rows staged
// k-major.  That keeps a GEMM launch per panel off the chain of dependent launches.
enum { PLD = 66, PQ = 16, PANEL_THREADS = 256 };  // PLD: row pitch of the staged 64 x 64 tiles (doubles)
static constexpr size_t PANEL_SMEM = (4 * 64 * PLD + 64 + 2 * PQ * 64) * sizeof(double);

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}

__global__ void __launch_bounds__(PANEL_THREADS) k_chol_panel(double* __restrict__ A, double* __restrict__ Ldiag,
                                                              long long ldiag_batch, int* __restrict__ info, int dp,
                                                              int k0, int d_fact, int update_first) {
  extern __shared__ __align__(16) unsigned char panel_raw[];
  double* sA = reinterpret_cast<double*>(panel_raw);  // this CTA's 64 panel rows
  double* sC = sA + 64 * PLD;                         // the diagonal block, then its raw columns: sC[j * PLD + r]
  double* rsv = sC + 64 * PLD;                        // 1 / L_jj
  double* sY = rsv + 64;                              // multipliers of the panel solve, [2][16][64]
  double* sPd = sY + 2 * PQ * 64;                     // previous panel, rows of the diagonal block: sPd[k * PLD + row]
  double* sPr = sPd + 64 * PLD;                       // previous panel, this CTA's rows, same layout
  const int tid = threadIdx.x, r = tid & 63, q = tid >> 6, b = blockIdx.y;
  double* Ab = A + (long long)b * dp * dp;
  double* diag = Ab + (long long)k0 * dp + k0;
  const long long row0 = (long long)k0 + FNB + (long long)FNB * blockIdx.x;
  const bool has_rows = row0 < d_fact;
  double* pan = Ab + row0 * dp + k0;
  {
    const int ch = tid & 31, rr0 = tid >> 5;  // 16-byte piece ch of rows rr0, rr0 + 8, ...
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int rr = 8 * i + rr0;
      cp_async_16(sC + rr * PLD + 2 * ch, diag + (long long)rr * dp + 2 * ch);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (has_rows) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = 8 * i + rr0;
        cp_async_16(sA + rr * PLD + 2 * ch, pan + (long long)rr * dp + 2 * ch);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (update_first) {
      const double* dprev = diag - FNB;
      const double* pprev = pan - FNB;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = 8 * i + rr0;
        const double2 v = *reinterpret_cast<const double2*>(dprev + (long long)rr * dp + 2 * ch);
        sPd[(2 * ch) * PLD + rr] = v.x;
        sPd[(2 * ch + 1) * PLD + rr] = v.y;
        if (has_rows) {
          const double2 w = *reinterpret_cast<const double2*>(pprev + (long long)rr * dp + 2 * ch);
          sPr[(2 * ch) * PLD + rr] = w.x;
          sPr[(2 * ch + 1) * PLD + rr] = w.y;
        }
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    }
  }
  __syncthreads();
  double a[PQ];
#pragma unroll
  for (int i = 0; i < PQ; i += 2) {
    const double2 v = *reinterpret_cast<const double2*>(sC + r * PLD + q * PQ + i);
    a[i] = v.x;
    a[i + 1] = v.y;
  }
  if (update_first) {
    // a[c] -= sum_k Pd[r][k] Pd[c][k], and the same for this CTA's rows against Pr[r][k]
    double xr[PQ];
#pragma unroll
    for (int i = 0; i < PQ; i += 2) {
      const double2 v = has_rows ? *reinterpret_cast<const double2*>(sA + r * PLD + q * PQ + i) : make_double2(0.0, 0.0);
      xr[i] = v.x;
      xr[i + 1] = v.y;
    }
#pragma unroll 2
    for (int k = 0; k < FNB; ++k) {
      const double pd = sPd[k * PLD + r];
      const double pr = has_rows ? sPr[k * PLD + r] : 0.0;
#pragma unroll
      for (int i = 0; i < PQ; i += 2) {
        const double2 c = *reinterpret_cast<const double2*>(sPd + k * PLD + q * PQ + i);
        a[i] = fma(-pd, c.x, a[i]);
        a[i + 1] = fma(-pd, c.y, a[i + 1]);
        xr[i] = fma(-pr, c.x, xr[i]);
        xr[i + 1] = fma(-pr, c.y, xr[i + 1]);
      }
    }
    if (has_rows) {
#pragma unroll
      for (int i = 0; i < PQ; i += 2)
        *reinterpret_cast<double2*>(sA + r * PLD + q * PQ + i) = make_double2(xr[i], xr[i + 1]);
    }
  }
  __syncthreads();  // the block has been read: its storage now takes the columns
#pragma unroll 1
  for (int jb = 0; jb < FNB / PQ; ++jb) {
#pragma unroll
    for (int jl = 0; jl < PQ; ++jl) {
      const int j = jb * PQ + jl;
      if (q == jb) sC[j * PLD + r] = a[jl];
      __syncthreads();
      if (q < jb || (r | 31) < j) continue;  // warps wholly left of or above the pivot only keep the barriers
      const double* col = sC + j * PLD;
      double piv = col[j];
      if (!(piv > 0.0)) {
        if (tid == j + 64 * jb && blockIdx.x == 0) atomicCAS(&info[b], 0, k0 + j + 1);
        piv = 1.0;
      }
      const double mult = col[r] * __drcp_rn(piv);
      if (q == jb) {
#pragma unroll
        for (int i = jl + 1; i < PQ; ++i) a[i] = fma(-mult, col[jb * PQ + i], a[i]);
        const double rs = rsqrt(piv);
        a[jl] = (r == j) ? piv * rs : a[jl] * rs;
        if (r == j) rsv[j] = rs;
      } else {
#pragma unroll
        for (int i = 0; i < PQ; ++i) a[i] = fma(-mult, col[q * PQ + i], a[i]);
      }
    }
  }
  if (blockIdx.x == 0) {
    // The factored block goes to its own array, never over the input: the CTAs of this launch need
    // not run at the same time, and one that starts late must still find the unfactored block.
    double* dst = Ldiag + (long long)b * ldiag_batch + (long long)(k0 / FNB) * FNB * FNB + r * FNB + q * PQ;
#pragma unroll
    for (int i = 0; i < PQ; ++i) dst[i] = (q * PQ + i <= r) ? a[i] : 0.0;
  }
  if (!has_rows) return;
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();  // panel rows staged by every thread; rsv complete
  double x[PQ];
#pragma unroll
  for (int i = 0; i < PQ; i += 2) {
    const double2 v = *reinterpret_cast<const double2*>(sA + r * PLD + q * PQ + i);
    x[i] = v.x;
    x[i + 1] = v.y;
  }
#pragma unroll 1
  for (int jb = 0; jb < FNB / PQ; ++jb) {
    double* yb = sY + (jb & 1) * PQ * 64;
    if (q == jb) {
#pragma unroll
      for (int jl = 0; jl < PQ; ++jl) {
        const int j = jb * PQ + jl;
        const double rs = rsv[j];
        const double xj = x[jl] * rs;
        x[jl] = xj;
        const double y = xj * rs;
        yb[jl * 64 + r] = y;
#pragma unroll
        for (int i = jl + 1; i < PQ; ++i) x[i] = fma(-y, sC[j * PLD + jb * PQ + i], x[i]);
      }
    }
    __syncthreads();
    if (q > jb) {
#pragma unroll
      for (int jl = 0; jl < PQ; ++jl) {
        const double y = yb[jl * 64 + r];
        const double* col = sC + (jb * PQ + jl) * PLD + q * PQ;
#pragma unroll
        for (int i = 0; i < PQ; ++i) x[i] = fma(-y, col[i], x[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < PQ; i += 2)
    *reinterpret_cast<double2*>(sA + r * PLD + q * PQ + i) = make_double2(x[i], x[i + 1]);
  __syncthreads();
  {
    const int ch = tid & 31, rr0 = tid >> 5;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int rr = 8 * i + rr0;
      *reinterpret_cast<double2*>(pan + (long long)rr * dp + 2 * ch) =
          *reinterpret_cast<const double2*>(sA + rr * PLD + 2 * ch);
    }
  }
}

// Inverse of every 64 x 64 diagonal block of L into the same block of Li (lower triangular):
// forward substitution, one thread per column, the column in registers.
__global__ void __launch_bounds__(64) k_inv_diag64(const double* __restrict__ Ldiag, long long ldiag_batch,
                                                   int n_factored, double* __restrict__ Li, int dp, int blk0) {
  __shared__ double Ls[FNB][FNB + 1];
  __shared__ double rdiag[FNB];
  const int blk = blk0 + blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const long long off = (long long)b * dp * dp + (long long)blk * FNB * (dp + 1);
  // blocks of the identity padding were never factored: their factor is the identity
  const double* src = Ldiag + (long long)b * ldiag_batch + (long long)blk * FNB * FNB;
  for (int r = 0; r < FNB; ++r) Ls[r][c] = (blk < n_factored) ? src[r * FNB + c] : (r == c ? 1.0 : 0.0);
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

// strictly-upper mask of a square matrix (Algorithm 2: (R U^T) .* M_U)
__global__ void k_mask_strict_upper(const double* __restrict__ src, double* __restrict__ dst, int d) {
  const long long n = (long long)d * d;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d), j = (int)(idx % d);
    dst[idx] = (j > i) ? src[idx] : 0.0;
  }
}

enum { INV_BLOCK = 512 };  // the inverse is completed block by block of this many columns (see factor_run)

struct FactorWs {
  double *A, *Li, *tmp;
  int dp;
  size_t tmp_per;   // doubles of tmp per matrix
  size_t low_off;   // products of the doubling levels inside one block of INV_BLOCK columns (two regions in turn)
  size_t high_off;  // products of the levels above, one region per level (level s at high_off + sum of the lower s^2)
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
  // tmp per matrix: the factored diagonal blocks (dp x 64), then the intermediate products of the
  // doubling steps.  The inverse proceeds while later panels are still being factored, and a product
  // of a high level stays alive while lower levels run, so each gets a region of its own.
  const size_t gdim = (f.dp < INV_BLOCK) ? (size_t)f.dp : (size_t)INV_BLOCK;
  f.low_off = (size_t)f.dp * FNB;
  f.high_off = f.low_off + 2 * (gdim * gdim / 4);  // two regions: neighbouring blocks are inverted side by side
  f.tmp_per = f.high_off;
  for (size_t sb = gdim; sb < (size_t)f.dp; sb <<= 1) f.tmp_per += sb * sb;
  f.tmp = b.take<double>((size_t)n_batch * f.tmp_per + 64);
  f.total = b.total();
  return f;
}

// Helper stream of the look-ahead (one per device, created on first use, kept until exit).
// The panels with the update of their own 64 columns are the critical path: they get a stream of the
// highest priority, so that their few CTAs are placed before the many tiles of a trailing update that
// is still being dispatched.  The first products of the upper doubling levels are large, and nothing
// needs them before the pair's second half has been factored and inverted: they get a stream of the
// lowest priority of their own (one per level: a small product must not queue behind a large one of the
// level above), so that the block-by-block part of the inverse does not wait for them needlessly.
struct FactorSide {
  cudaStream_t crit;    // panels (each applies the previous panel's update to its own columns first)
  cudaStream_t stream;  // trailing updates
  cudaStream_t inv;     // the inverse above the blocks: second products of the upper levels
  cudaStream_t low[2];  // the inverse inside a block of 512 columns, blocks in turn
  cudaStream_t inv2[8];  // first products of the doubling levels above one block, a stream per level
  cudaStream_t rest;    // the wide rank-256 updates beyond the next outer block's columns
  cudaEvent_t fork, panel, trail[2], block_done, inv_done, crit_done, half_done, first_done[8], low_done[2];
  cudaEvent_t outer_panels, strip_done, rest_done;
  bool ready;
};

static FactorSide* factor_side() {
  static FactorSide per_device[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  FactorSide* s = &per_device[dev];
  if (!s->ready) {
    int least = 0, greatest = 0;
    if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) return nullptr;
    const int middle = (greatest < least) ? greatest + 1 : least;  // numerically lower = more urgent
    if (cudaStreamCreateWithPriority(&s->crit, cudaStreamNonBlocking, greatest) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&s->stream, cudaStreamNonBlocking, middle) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->crit_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->panel, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->trail[0], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->trail[1], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&s->inv, cudaStreamNonBlocking, middle) != cudaSuccess) return nullptr;
    for (int i = 0; i < 8; ++i)
      if (cudaStreamCreateWithPriority(&s->inv2[i], cudaStreamNonBlocking, least) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->half_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < 2; ++i) {
      if (cudaStreamCreateWithPriority(&s->low[i], cudaStreamNonBlocking, middle) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&s->low_done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    for (int i = 0; i < 8; ++i)
      if (cudaEventCreateWithFlags(&s->first_done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->block_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->inv_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithPriority(&s->rest, cudaStreamNonBlocking, least) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->outer_panels, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->strip_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&s->rest_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    s->ready = true;
  }
  return s;
}

tb_status factor_run(const float* H, int n_batch, int d, float* U, float* Hinv, int* info, void* ws, size_t ws_bytes,
                     void* stream, bool lookahead);

}  // namespace tb

using namespace tb;

extern "C" size_t tb_factor_workspace(int n_batch, int d) {
  if (n_batch <= 0 || d <= 0) return 0;
  return factor_ws(n_batch, d, nullptr).total;
}

extern "C" tb_status tb_factor(const float* H, int n_batch, int d, float* U, float* Hinv, int* info,
                               void* ws, size_t ws_bytes, void* stream) {
  return factor_run(H, n_batch, d, U, Hinv, info, ws, ws_bytes, stream, true);
}

// lookahead: the panels run on a stream of high priority, the trailing updates (which leave out the
// next panel's columns: that panel applies its share itself) on a second stream beside the next panel,
// the inverse of the blocks already factored on a third.  Every entry still receives its updates in
// the same order and every product is the same launch, so the result is the same bit for bit.  Without
// it (callers that must not create a stream) everything runs on the caller's stream.
tb_status tb::factor_run(const float* H, int n_batch, int d, float* U, float* Hinv, int* info, void* ws,
                         size_t ws_bytes, void* stream, bool lookahead) {
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

  static bool panel_configured[64] = {false};
  TB_TRY(allow_smem(k_chol_panel, PANEL_SMEM, panel_configured));
  // the padding is an identity block decoupled from the rest: factor the leading part only
  const int d_fact = ((d + FNB - 1) / FNB) * FNB;
  FactorSide* side = nullptr;
  if (lookahead && d_fact >= 16 * FNB) {
    side = factor_side();
    if (!side) return TB_ERR_CUDA;
    TB_CUDA_CHECK(cudaEventRecord(side->fork, st));
    TB_CUDA_CHECK(cudaStreamWaitEvent(side->stream, side->fork, 0));
    TB_CUDA_CHECK(cudaStreamWaitEvent(side->crit, side->fork, 0));
    TB_CUDA_CHECK(cudaStreamWaitEvent(side->rest, side->fork, 0));
  }
  // L^{-1} block by block of G columns.  Block j can be inverted as soon as its last panel is factored:
  // its 64 x 64 diagonal inverses, the doubling levels inside the block, then every level above whose
  // pair this block completes (second product), and the first product of the one pair whose first half
  // it completes (that product needs only columns already final).  With the look-ahead all of this runs
  // on a stream of its own beside the later panels, and little of the inverse is left after the last
  // panel; without it the same launches follow the panels on the caller's stream.  Every product is
  // the same launch either way, so the result is the same bit for bit.
  const int G = (dp < INV_BLOCK) ? dp : INV_BLOCK;
  const int n_inv_blocks = dp / G, n_panels = d_fact / FNB;
  cudaStream_t inv_st = side ? side->inv : st;
  cudaStream_t cs = side ? side->crit : st;  // stream of the panels
  // first product of a pair at level sblk: T = C A^{-1}, C = L[s:2s, 0:s], A^{-1} = Li[0:s, 0:s] (lower triangular)
  // Launched in pieces of at most 768 columns (96 tiles at 2048 rows): the tiles of the upper levels
  // run for hundreds of microseconds, and a launch that fills every SM with them would keep the panels
  // waiting.  The first columns meet the longest part of the triangle, so the pieces get shorter.  A
  // piece is the same set of tiles, so nothing changes in the result.
  auto pair_first = [&](int sblk, long long off, long long pair_stride, int batch, double* tmp, long long tmp_stride,
                        cudaStream_t stream_first) -> tb_status {
    GemmP g = gemm_params();
    g.A = f.A + off + (long long)sblk * dp;
    g.a_m = dp;
    g.a_k = 1;
    g.a_batch = pair_stride;
    g.B = f.Li + off;
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
    g.flags = GEMM_HEAVY_N_FIRST;
    const int piece = (sblk > 1024) ? 768 : sblk;
    for (int n0 = 0; n0 < sblk; n0 += piece) {
      GemmP gp = g;
      gp.B = f.Li + off + n0;  // B(k, n0 + n), zero for k < n0 + n
      gp.boff = n0;
      gp.C = tmp + n0;
      gp.N = (sblk - n0 < piece) ? sblk - n0 : piece;
      TB_TRY((gemm64_launch<true>(gp, stream_first)));
    }
    return TB_OK;
  };
  // second product: Li[s:2s, 0:s] = -B^{-1} T, B^{-1} = Li[s:2s, s:2s] (lower triangular)
  auto pair_second = [&](int sblk, long long off, long long pair_stride, int batch, double* tmp, long long tmp_stride,
                         cudaStream_t stream_second) -> tb_status {
    GemmP h = gemm_params();
    h.A = f.Li + off + (long long)sblk * (dp + 1);
    h.a_m = dp;
    h.a_k = 1;
    h.a_batch = pair_stride;
    h.B = tmp;
    h.b_k = sblk;
    h.b_n = 1;
    h.b_batch = tmp_stride;
    h.C = f.Li + off + (long long)sblk * dp;
    h.ldc = dp;
    h.c_batch = pair_stride;
    h.M = sblk;
    h.N = sblk;
    h.K = sblk;
    h.n_batch = batch;
    h.alpha = -1.0;
    h.atrim = 1;
    h.flags = GEMM_HEAVY_M_LAST;
    return gemm64_launch<true>(h, stream_second);
  };
  auto high_tmp = [&](int sblk) {  // region of the level-sblk product (first matrix of the batch)
    size_t o = f.high_off;
    for (size_t sb = (size_t)G; sb < (size_t)sblk; sb <<= 1) o += sb * sb;
    return f.tmp + o;
  };
  auto invert_block = [&](int j) -> tb_status {
    const long long boff = (long long)j * G * (dp + 1);
    // inside the block: a stream per block parity, so that a block does not wait for its neighbour's
    // upper levels; the caller has just recorded block_done
    cudaStream_t low_st = side ? side->low[j & 1] : inv_st;
    const size_t low_region = f.low_off + (size_t)(j & 1) * ((size_t)G * G / 4);
    if (side) TB_CUDA_CHECK(cudaStreamWaitEvent(low_st, side->block_done, 0));
    k_inv_diag64<<<dim3(G / FNB, n_batch), 64, 0, low_st>>>(f.tmp, (long long)f.tmp_per, n_panels, f.Li, dp,
                                                             j * (G / FNB));
    TB_LAUNCH_CHECK();
    for (int sblk = FNB; sblk < G; sblk <<= 1) {
      const int pairs = G / (2 * sblk);
      // one batched launch covers all pairs of one matrix's block, or (a single pair) all matrices
      const int outer = (pairs == 1) ? 1 : n_batch;
      for (int mb = 0; mb < outer; ++mb) {
        const long long off = (long long)mb * pp + boff;
        const long long pair_stride = (pairs == 1) ? pp : (long long)2 * sblk * (dp + 1);
        const int batch = (pairs == 1) ? n_batch : pairs;
        double* tmp = f.tmp + (size_t)mb * f.tmp_per + low_region;
        const long long tmp_stride = (pairs == 1) ? (long long)f.tmp_per : (long long)sblk * sblk;
        TB_TRY(pair_first(sblk, off, pair_stride, batch, tmp, tmp_stride, low_st));
        TB_TRY(pair_second(sblk, off, pair_stride, batch, tmp, tmp_stride, low_st));
      }
    }
    if (side) {
      TB_CUDA_CHECK(cudaEventRecord(side->low_done[j & 1], low_st));
      TB_CUDA_CHECK(cudaStreamWaitEvent(side->inv, side->low_done[j & 1], 0));
    }
    int level = 0;
    for (int sblk = G; sblk < dp; sblk <<= 1, ++level) {
      const int mblk = sblk / G;  // blocks per half of a pair at this level
      if ((j + 1) % mblk) break;
      const int halves = (j + 1) / mblk;
      if (halves & 1) {  // block j completes the first half of its pair
        if (side) {
          TB_CUDA_CHECK(cudaEventRecord(side->half_done, side->inv));
          TB_CUDA_CHECK(cudaStreamWaitEvent(side->inv2[level & 7], side->half_done, 0));
        }
        TB_TRY(pair_first(sblk, (long long)(j + 1 - mblk) * G * (dp + 1), pp, n_batch, high_tmp(sblk),
                          (long long)f.tmp_per, side ? side->inv2[level & 7] : inv_st));
        if (side) TB_CUDA_CHECK(cudaEventRecord(side->first_done[level & 7], side->inv2[level & 7]));
        break;
      }
      if (side) TB_CUDA_CHECK(cudaStreamWaitEvent(side->inv, side->first_done[level & 7], 0));
      TB_TRY(pair_second(sblk, (long long)(j + 1 - 2 * mblk) * G * (dp + 1), pp, n_batch, high_tmp(sblk),
                         (long long)f.tmp_per, inv_st));
    }
    return TB_OK;
  };
  int next_inv_block = 0;

  // Two levels of blocking.  Outer blocks of OB = 256 columns (four panels).  Panel k applies the
  // update of panel k-1 to its own 64 columns itself; the rank-64 update after panel k covers the
  // columns from panel k+2 on up to ZL = 128 columns past the end of its outer block (a strip at most
  // 256 columns wide), so that the first two panels of the next block never wait for anything wide.
  // After a block's last panel its 256 columns update everything further right in one rank-256
  // product, in two launches: the columns up to ZL past the next block's end ("near": the next block's
  // third panel is the first to need it), then the rest ("far").  A rank-64 update of the whole
  // trailing matrix moves the matrix through memory once per panel and is bound by that traffic;
  // rank-256 updates move it a quarter as often and run at the GEMM engine's large-K efficiency.
  // With the look-ahead: panels on the high-priority stream, the rank-64 strips and the near updates
  // in order on the trailing stream, the far updates on a low-priority stream beside the next block's
  // panels.  The far update of block J and the near update of block J+1 overlap in their columns, so
  // the latter waits for the former: every entry receives its updates in the same order as in the
  // single-stream schedule, and the results agree bit for bit.
  enum { OB = 4 * FNB, ZL = 2 * FNB };
  bool trail_set[2] = {false, false};
  bool strip_set = false, rest_set = false;
  auto rank_update = [&](int k_lo, int k_cnt, int c_lo, int c_hi, cudaStream_t stream_u) -> tb_status {
    // A[r][c] -= sum_k L[r][k_lo + k] L[c][k_lo + k] for c in [c_lo, c_hi), r >= c (tiles on or below the diagonal)
    if (c_hi <= c_lo) return TB_OK;
    GemmP t = gemm_params();
    t.A = f.A + (long long)c_lo * dp + k_lo;
    t.a_m = dp;
    t.a_k = 1;
    t.a_batch = pp;
    t.B = t.A;  // B(k, n) = L[c_lo + n][k_lo + k]
    t.b_k = 1;
    t.b_n = dp;
    t.b_batch = pp;
    t.C = f.A + (long long)c_lo * dp + c_lo;
    t.ldc = dp;
    t.c_batch = pp;
    t.M = d_fact - c_lo;
    t.N = c_hi - c_lo;
    t.K = k_cnt;
    t.n_batch = n_batch;
    t.alpha = -1.0;
    t.beta = 1.0;
    t.flags = GEMM_LOWER_TILES;
    return gemm64_launch<false>(t, stream_u);
  };
  for (int k0 = 0; k0 < d_fact; k0 += FNB) {
    const int r0 = k0 + FNB, m = d_fact - r0;
    const int xt = (m > 0) ? m / FNB : 1;
    const int pi = k0 / FNB;
    const int j0 = (k0 / OB) * OB;                               // first column of this outer block
    const int j1 = (j0 + OB < d_fact) ? j0 + OB : d_fact;        // one past its last column
    const bool last_in_block = (r0 >= j1);
    auto clip = [&](int c) { return c < d_fact ? c : d_fact; };
    if (side && trail_set[pi & 1]) TB_CUDA_CHECK(cudaStreamWaitEvent(cs, side->trail[pi & 1], 0));
    k_chol_panel<<<dim3(xt, n_batch), PANEL_THREADS, PANEL_SMEM, cs>>>(f.A, f.tmp, (long long)f.tmp_per, info, dp, k0,
                                                                       d_fact, k0 > 0 ? 1 : 0);
    TB_LAUNCH_CHECK();
    if (side) {
      // blocks whose last factored panel this was (the identity padding needs no panel)
      bool waited = false;
      while (next_inv_block < n_inv_blocks) {
        int last = (next_inv_block + 1) * (G / FNB) - 1;
        if (last > n_panels - 1) last = n_panels - 1;
        if (last != pi) break;
        if (!waited) {
          TB_CUDA_CHECK(cudaEventRecord(side->block_done, cs));
          TB_CUDA_CHECK(cudaStreamWaitEvent(side->inv, side->block_done, 0));
          waited = true;
        }
        TB_TRY(invert_block(next_inv_block));
        ++next_inv_block;
      }
    }
    if (m <= 0) break;
    trail_set[pi & 1] = false;
    // rank-64 strip: the columns from panel k+2 on, up to ZL past the end of the outer block
    const int t_lo = clip(r0 + FNB), t_hi = clip(j1 + ZL);
    if (side && (t_hi > t_lo || last_in_block)) {
      TB_CUDA_CHECK(cudaEventRecord(side->panel, cs));
      TB_CUDA_CHECK(cudaStreamWaitEvent(side->stream, side->panel, 0));
    }
    if (t_hi > t_lo) {
      TB_TRY(rank_update(k0, FNB, t_lo, t_hi, side ? side->stream : st));
      if (side) {
        TB_CUDA_CHECK(cudaEventRecord(side->trail[pi & 1], side->stream));
        trail_set[pi & 1] = true;
      }
    }
    if (!last_in_block) continue;
    // the block is factored: rank-(j1 - j0) update of everything further right
    const int n_lo = clip(j1 + ZL), n_hi = clip(j1 + OB + ZL);
    if (!side) {
      TB_TRY(rank_update(j0, j1 - j0, n_lo, n_hi, st));
      TB_TRY(rank_update(j0, j1 - j0, n_hi, d_fact, st));
      continue;
    }
    if (n_hi > n_lo) {
      // near: overlaps the previous block's far update in these columns, so after it
      if (rest_set) TB_CUDA_CHECK(cudaStreamWaitEvent(side->stream, side->rest_done, 0));
      TB_TRY(rank_update(j0, j1 - j0, n_lo, n_hi, side->stream));
      // later strips of this stream follow it in order; the panels that need it wait for those strips
      TB_CUDA_CHECK(cudaEventRecord(side->strip_done, side->stream));
      strip_set = true;
    }
    if (n_hi < d_fact) {
      TB_CUDA_CHECK(cudaStreamWaitEvent(side->rest, side->panel, 0));
      TB_TRY(rank_update(j0, j1 - j0, n_hi, d_fact, side->rest));
      TB_CUDA_CHECK(cudaEventRecord(side->rest_done, side->rest));
      rest_set = true;
    }
  }
  if (side) {
    for (int i = 0; i < 2; ++i)
      if (trail_set[i]) TB_CUDA_CHECK(cudaStreamWaitEvent(st, side->trail[i], 0));
    if (strip_set) TB_CUDA_CHECK(cudaStreamWaitEvent(st, side->strip_done, 0));
    if (rest_set) TB_CUDA_CHECK(cudaStreamWaitEvent(st, side->rest_done, 0));
    TB_CUDA_CHECK(cudaEventRecord(side->crit_done, side->crit));
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, side->crit_done, 0));
  }

  // what is left of the inverse (all of it without the look-ahead)
  while (next_inv_block < n_inv_blocks) {
    TB_TRY(invert_block(next_inv_block));
    ++next_inv_block;
  }
  if (side) {
    TB_CUDA_CHECK(cudaEventRecord(side->inv_done, side->inv));
    TB_CUDA_CHECK(cudaStreamWaitEvent(st, side->inv_done, 0));
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

// P and C: three products on the FP64 engine.  (Products from bf16 splits on the tensor cores were 3x
// faster, but R U^T U cancels heavily at large widths: their error, a few 1e-7 of sum |a||b|, came to
// 1.5e-5 of the result at 4096 columns.)
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
