// Double-precision GEMM with 128 x 64 tiles, two CTAs per SM.
//
// Same interface (GemmP) and the same arithmetic per entry as the 128 x 128 engine of tb_gemm.cuh
// for double operands: C = alpha A B + beta C on the FP64 tensor pipe (mma.sync m8n8k4), K walked
// in chunks of 16 through a three-stage ring of shared-memory tiles that asynchronous copies fill
// straight from global memory (no staging through registers), one barrier per chunk.  The smaller tile
// keeps 32 x 32 accumulators per warp (64 registers instead of 128), so two CTAs share an SM: while
// one of them sits at its barrier, stages operands or reads and writes its C tile, the other keeps
// the tensor pipe busy.  That matters where K is short (the rank-64 / rank-256 updates of the
// factorisation), where the C traffic of a tile is comparable to its arithmetic.
#pragma once

#include "tb_gemm.cuh"

namespace tb {

enum { G64_BM = 128, G64_BN = 64, G64_BK = 16, G64_THREADS = 256, G64_STAGES = 3 };
// Shared-memory tiles keep the global layout (rows of 16 contraction steps for a k-contiguous operand,
// rows of 64 columns for an n-contiguous B), filled by 16-byte asynchronous copies.  Row pitches of
// 20 and 68 doubles put the 8 x 4 (or 4 x 8) elements of an m8n8k4 fragment in distinct banks.
enum { G64_LDK = G64_BK + 4, G64_LDN = G64_BN + 4 };
enum { G64_A_STAGE = G64_BM * G64_LDK, G64_B_STAGE = G64_BN * G64_LDK };  // doubles; 16 x G64_LDN is smaller
static constexpr size_t G64_SMEM = (size_t)G64_STAGES * (G64_A_STAGE + G64_B_STAGE) * sizeof(double);

__device__ __forceinline__ void g64_cp16(double* smem_dst, const double* gsrc, bool valid) {
  // 16 bytes global -> shared; with valid == false nothing is read and the destination is zero-filled
  const unsigned n = valid ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)),
               "l"(gsrc), "r"(n)
               : "memory");
}

// A(m, k) has k contiguous (a_k == 1); B(k, n) has n contiguous (B_NCONTIG, b_n == 1) or k contiguous
// (b_k == 1).  The K range of every tile is a multiple of 16, every operand row starts on a 16-byte
// boundary (the launcher checks both and the callers' strides).
template <bool B_NCONTIG>
__global__ void __launch_bounds__(G64_THREADS, 2) gemm64_kernel(GemmP p) {
  extern __shared__ __align__(16) unsigned char g64_smem[];
  int tm = blockIdx.y, tn = blockIdx.x;
  if (p.flags & (GEMM_HEAVY_N_FIRST | GEMM_HEAVY_M_LAST)) {
    const int lin = blockIdx.y * gridDim.x + blockIdx.x, tiles_m = gridDim.y, tiles_n = gridDim.x;
    if (p.flags & GEMM_HEAVY_N_FIRST) {
      tn = lin / tiles_m;
      tm = lin % tiles_m;
    } else {
      tm = tiles_m - 1 - lin / tiles_n;
      tn = lin % tiles_n;
    }
  }
  const int m0 = tm * G64_BM, n0 = tn * G64_BN;
  if ((p.flags & GEMM_LOWER_TILES) && n0 >= m0 + G64_BM) return;
  const int batch = blockIdx.z;
  const double* A = static_cast<const double*>(p.A) + (long long)batch * p.a_batch;
  const double* B = static_cast<const double*>(p.B) + (long long)batch * p.b_batch;
  double* C = static_cast<double*>(p.C) + (long long)batch * p.c_batch;

  int k_begin = 0, k_end = p.K;
  if (p.btrim == 1) k_end = min(k_end, n0 + G64_BN + p.boff);
  if (p.btrim == 2) k_begin = max(k_begin, n0 + p.boff);
  if (p.atrim == 1) k_end = min(k_end, m0 + G64_BM + p.aoff);
  if (p.atrim == 2) k_begin = max(k_begin, m0 + p.aoff);
  k_begin = (k_begin / G64_BK) * G64_BK;
  k_end = ((k_end + G64_BK - 1) / G64_BK) * G64_BK;   // K is a multiple of 16: never beyond it
  if (k_end > p.K) k_end = p.K;

  double* As = reinterpret_cast<double*>(g64_smem);       // [stages][128][LDK]
  double* Bs = As + G64_STAGES * G64_A_STAGE;             // [stages][64][LDK] or [stages][16][LDN]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = p.M, N = p.N;
  const long long a_m = p.a_m, b_k = p.b_k, b_n = p.b_n;

  auto issue = [&](int stage, int k0) {
    double* as = As + stage * G64_A_STAGE;
    double* bs = Bs + stage * G64_B_STAGE;
    // A: 128 rows x 8 pieces of 2 doubles
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + 256 * i, mm = idx >> 3, pc = idx & 7;
      const bool ok = (m0 + mm) < M;
      const double* src = A + (long long)(ok ? m0 + mm : m0) * a_m + k0 + 2 * pc;
      g64_cp16(as + mm * G64_LDK + 2 * pc, src, ok);
    }
    if (B_NCONTIG) {
      // B: 16 rows (k) x 32 pieces along n
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int idx = tid + 256 * i, kk = idx >> 5, pc = idx & 31;
        const bool ok = (n0 + 2 * pc) < N;   // N is even: a piece is wholly inside or outside
        const double* src = B + (long long)(k0 + kk) * b_k + (ok ? n0 + 2 * pc : n0);
        g64_cp16(bs + kk * G64_LDN + 2 * pc, src, ok);
      }
    } else {
      // B: 64 rows (n) x 8 pieces along k
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int idx = tid + 256 * i, nn = idx >> 3, pc = idx & 7;
        const bool ok = (n0 + nn) < N;
        const double* src = B + (long long)(ok ? n0 + nn : n0) * b_n + k0 + 2 * pc;
        g64_cp16(bs + nn * G64_LDK + 2 * pc, src, ok);
      }
    }
  };

  // warp w: rows 32 (w / 2) .. +31, columns 32 (w % 2) .. +31 as 4 x 4 fragments of 8 x 8; a fragment
  // gives this thread row lane / 4 and columns 2 (lane % 4), 2 (lane % 4) + 1
  double acc[4][4][2];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
  const int kq = lane & 3, rq = lane >> 2;
  const int wr = (warp >> 1) * 32, wc = (warp & 1) * 32;

  const int n_chunks = (k_end > k_begin) ? (k_end - k_begin) / G64_BK : 0;
  // prologue: stages 0 .. STAGES-2 in flight (empty groups keep the group count uniform)
#pragma unroll
  for (int s = 0; s < G64_STAGES - 1; ++s) {
    if (s < n_chunks) issue(s, k_begin + s * G64_BK);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  for (int c = 0; c < n_chunks; ++c) {
    asm volatile("cp.async.wait_group %0;" ::"n"(G64_STAGES - 2) : "memory");
    __syncthreads();   // chunk c has landed for every thread; everyone is done with chunk c - 1's stage
    {
      const int nc = c + G64_STAGES - 1;
      if (nc < n_chunks) issue(nc % G64_STAGES, k_begin + nc * G64_BK);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const int st = c % G64_STAGES;
    const double* ap = As + st * G64_A_STAGE + (wr + rq) * G64_LDK + kq;
    const double* bp = B_NCONTIG ? (Bs + st * G64_B_STAGE + kq * G64_LDN + wc + rq)
                                 : (Bs + st * G64_B_STAGE + (wc + rq) * G64_LDK + kq);
#pragma unroll
    for (int k4 = 0; k4 < G64_BK / 4; ++k4) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = ap[i * 8 * G64_LDK + k4 * 4];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = B_NCONTIG ? bp[k4 * 4 * G64_LDN + j * 8] : bp[j * 8 * G64_LDK + k4 * 4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                       : "+d"(acc[i][j][0]), "+d"(acc[i][j][1])
                       : "d"(a[i]), "d"(b[j]));
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");

  const double alpha = p.alpha, beta = p.beta;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + wr + i * 8 + rq;
    if (m >= M) continue;
    double* crow = C + (long long)m * p.ldc;
    double2 cold[4];
    if (beta != 0.0) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + wc + j * 8 + 2 * kq;
        cold[j].x = (n < N) ? crow[n] : 0.0;
        cold[j].y = (n + 1 < N) ? crow[n + 1] : 0.0;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + wc + j * 8 + 2 * kq;
      const double v0 = (beta != 0.0) ? fma(beta, cold[j].x, alpha * acc[i][j][0]) : alpha * acc[i][j][0];
      const double v1 = (beta != 0.0) ? fma(beta, cold[j].y, alpha * acc[i][j][1]) : alpha * acc[i][j][1];
      if (n < N) crow[n] = v0;
      if (n + 1 < N) crow[n + 1] = v1;
    }
  }
}

// Host launcher, double operands only.  Problems outside what the asynchronous copies need (a
// contraction length that is not a multiple of 16, operand rows off a 16-byte boundary, an odd N with
// an n-contiguous B) go to the 128 x 128 engine, which has no such conditions.
template <bool B_NCONTIG>
tb_status gemm64_launch(const GemmP& p, cudaStream_t stream) {
  if (p.M <= 0 || p.N <= 0 || p.n_batch <= 0) return TB_OK;
  const bool strides_ok = p.a_k == 1 && (B_NCONTIG ? p.b_n == 1 : p.b_k == 1);
  const long long brow = B_NCONTIG ? p.b_k : p.b_n;
  const bool aligned_ok = aligned(p.A, 16) && aligned(p.B, 16) && (p.a_m % 2 == 0) && (brow % 2 == 0) &&
                          (p.a_batch % 2 == 0) && (p.b_batch % 2 == 0) && (!B_NCONTIG || p.N % 2 == 0);
  const bool trim_ok = (p.boff % 2 == 0) && (p.aoff % 2 == 0);
  if (!strides_ok || !aligned_ok || !trim_ok || (p.K % G64_BK))
    return gemm_launch<double, double, double, double, false, B_NCONTIG>(p, stream);
  auto kern = gemm64_kernel<B_NCONTIG>;
  static bool configured[64] = {false};
  TB_TRY(allow_smem(kern, G64_SMEM, configured));
  const int zmax = 65535;
  for (int b0 = 0; b0 < p.n_batch; b0 += zmax) {
    GemmP q = p;
    const int nb = (p.n_batch - b0 < zmax) ? (p.n_batch - b0) : zmax;
    q.A = static_cast<const double*>(p.A) + (long long)b0 * p.a_batch;
    q.B = static_cast<const double*>(p.B) + (long long)b0 * p.b_batch;
    q.C = static_cast<double*>(p.C) + (long long)b0 * p.c_batch;
    q.n_batch = nb;
    dim3 grid((p.N + G64_BN - 1) / G64_BN, (p.M + G64_BM - 1) / G64_BM, nb);
    kern<<<grid, G64_THREADS, G64_SMEM, stream>>>(q);
    TB_LAUNCH_CHECK();
  }
  return TB_OK;
}

}  // namespace tb
