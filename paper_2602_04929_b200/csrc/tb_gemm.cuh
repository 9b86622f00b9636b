// Batched strided GEMM on the CUDA cores, C = alpha * A * B + beta * C, with
// the accumulator type chosen by the caller (double for everything that feeds
// an integer decision or a small difference of large terms).
//
// One CTA of 256 threads owns a 128 x 128 tile of C and walks K in chunks of
// 16 through double-buffered shared memory; every thread keeps an 8 x 8 block
// of accumulators.  Operands may be float, double or bf16 and are converted
// once, when they are staged.  A(m,k) and B(k,n) are addressed with element
// strides, so transposed operands need no copy; the template flags only say
// which index is contiguous so that the staging loads coalesce.
//
// The main loop takes its operands through two functors, so other kernels can
// run the same tile engine on operands they produce on the fly (the grid
// search stages quantization errors it computes from the weights; the fused
// column-sweep kernel runs trailing-update tiles next to its panel work).
#pragma once

#include "tb_common.cuh"

namespace tb {

enum { GEMM_BM = 128, GEMM_BN = 128, GEMM_BK = 16, GEMM_THREADS = 256 };
enum {
  GEMM_LOWER_TILES = 1,  // skip tiles that lie strictly above the diagonal
  // Launch order of the tiles when the K range depends on the tile (btrim / atrim): blocks start in
  // linear order as SMs free up, so the tiles with the longest K range are given the lowest indices.
  GEMM_HEAVY_N_FIRST = 2,  // K range grows as n0 falls (btrim 2): column tiles ascending, slowest index
  GEMM_HEAVY_M_LAST = 4    // K range grows with m0 (atrim 1): row tiles descending, slowest index
};

struct GemmP {
  const void* A;
  const void* B;
  void* C;
  long long a_m, a_k;  // element strides of A(m, k)
  long long b_k, b_n;  // element strides of B(k, n)
  long long ldc;       // row stride of C (columns contiguous)
  long long a_batch, b_batch, c_batch;
  int M, N, K;
  int n_batch;
  double alpha, beta;
  int flags;
  // Known-zero structure, used only to shorten the K range of a tile:
  // btrim 1: B(k,n) = 0 for k > n + boff;  2: B(k,n) = 0 for k < n + boff
  // atrim 1: A(m,k) = 0 for k > m + aoff;  2: A(m,k) = 0 for k < m + aoff
  int btrim, boff, atrim, aoff;
};

inline GemmP gemm_params() {
  GemmP p;
  p.A = p.B = nullptr;
  p.C = nullptr;
  p.a_m = p.a_k = p.b_k = p.b_n = p.ldc = 0;
  p.a_batch = p.b_batch = p.c_batch = 0;
  p.M = p.N = p.K = 0;
  p.n_batch = 1;
  p.alpha = 1.0;
  p.beta = 0.0;
  p.flags = 0;
  p.btrim = p.boff = p.atrim = p.aoff = 0;
  return p;
}

template <typename TAcc>
struct GemmSmem {
  static constexpr int LD = 132;
  static constexpr size_t bytes = 2ull * 2ull * GEMM_BK * LD * sizeof(TAcc);
};

// Per-thread accumulators of a 128 x 128 tile: an 8 x 8 block per thread in
// both engines, addressed as at(i, j) with tile-local row(i) and col(j).
//   float : SIMT FFMA engine, rows ty*4+i / 64+ty*4+i-4, columns likewise in tx.
//   double: FP64 tensor-core engine (mma.sync m8n8k4).  Warp w owns rows
//           64 (w / 4) .. +63 and columns 32 (w % 4) .. +31 as 8 x 4 fragments of
//           8 x 8; a fragment gives this thread row lane / 4 and columns
//           2 (lane % 4), 2 (lane % 4) + 1.
template <typename TAcc>
struct GemmAcc;

template <>
struct GemmAcc<float> {
  float v[8][8];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) v[i][j] = 0.0f;
  }
  __device__ __forceinline__ float at(int i, int j) const { return v[i][j]; }
  static __device__ __forceinline__ int row(int i) {
    const int ty = threadIdx.x >> 4;
    return (i < 4) ? (ty * 4 + i) : (64 + ty * 4 + i - 4);
  }
  static __device__ __forceinline__ int col(int j) {
    const int tx = threadIdx.x & 15;
    return (j < 4) ? (tx * 4 + j) : (64 + tx * 4 + j - 4);
  }
};

template <>
struct GemmAcc<double> {
  double v[8][4][2];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) v[i][j][0] = v[i][j][1] = 0.0;
  }
  __device__ __forceinline__ double at(int i, int j) const { return v[i][j >> 1][j & 1]; }
  static __device__ __forceinline__ int row(int i) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    return (warp >> 2) * 64 + i * 8 + (lane >> 2);
  }
  static __device__ __forceinline__ int col(int j) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    return (warp & 3) * 32 + (j >> 1) * 8 + (lane & 3) * 2 + (j & 1);
  }
};

// One K chunk (16) of the tile product from shared memory.
__device__ __forceinline__ void gemm_chunk(GemmAcc<float>& acc, const float* as, const float* bs) {
  constexpr int LD = GemmSmem<float>::LD;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int kk = 0; kk < GEMM_BK; ++kk) {
    float a[8], b[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      a[i] = as[kk * LD + ty * 4 + i];
      a[4 + i] = as[kk * LD + 64 + ty * 4 + i];
      b[i] = bs[kk * LD + tx * 4 + i];
      b[4 + i] = bs[kk * LD + 64 + tx * 4 + i];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc.v[i][j] = fmaf(a[i], b[j], acc.v[i][j]);
  }
}

__device__ __forceinline__ void gemm_chunk(GemmAcc<double>& acc, const double* as, const double* bs) {
  constexpr int LD = GemmSmem<double>::LD;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kq = lane & 3, rq = lane >> 2;
  const double* ap = as + kq * LD + (warp >> 2) * 64 + rq;
  const double* bp = bs + kq * LD + (warp & 3) * 32 + rq;
#pragma unroll
  for (int k4 = 0; k4 < GEMM_BK / 4; ++k4) {
    double a[8], b[4];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = ap[k4 * 4 * LD + i * 8];
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = bp[k4 * 4 * LD + j * 8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                     : "+d"(acc.v[i][j][0]), "+d"(acc.v[i][j][1])
                     : "d"(a[i]), "d"(b[j]));
  }
}

// acc += A_tile * B_tile over k in [k_begin, k_end), k_begin a multiple of 16.
// load_a(mm, k) / load_b(nn, k) fetch the raw operand for tile-local row /
// column 0..127 and absolute k (a value that converts to 0 outside the
// problem); conv_a(raw, mm, k) / conv_b(raw, nn, k) turn it into TAcc.  The
// fetch of the next chunk is issued before the current chunk's arithmetic and
// its conversion after it, so that the latency of global memory hides behind
// the arithmetic.  Every thread of the CTA must call this; `smem` must hold
// GemmSmem<TAcc>::bytes.  On return all threads have passed a barrier, so the
// shared buffer may be reused at once.
template <typename TAcc, bool A_MCONTIG, bool B_NCONTIG, typename FA, typename CA, typename FB, typename CB>
__device__ __forceinline__ void gemm_mainloop(GemmAcc<TAcc>& acc, FA load_a, CA conv_a, FB load_b, CB conv_b,
                                              int k_begin, int k_end, unsigned char* smem) {
  constexpr int LD = GemmSmem<TAcc>::LD;
  TAcc* As = reinterpret_cast<TAcc*>(smem);  // [2][BK][LD]
  TAcc* Bs = As + 2 * GEMM_BK * LD;          // [2][BK][LD]
  const int tid = threadIdx.x;

  decltype(load_a(0, 0)) ra[8];
  decltype(load_b(0, 0)) rb[8];
  auto load_regs = [&](int k0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int mm, kk;
      if (A_MCONTIG) {
        mm = tid & 127;
        kk = (tid >> 7) + 2 * i;
      } else {
        kk = tid & 15;
        mm = (tid >> 4) + 16 * i;
      }
      ra[i] = load_a(mm, k0 + kk);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int nn, kk;
      if (B_NCONTIG) {
        nn = tid & 127;
        kk = (tid >> 7) + 2 * i;
      } else {
        kk = tid & 15;
        nn = (tid >> 4) + 16 * i;
      }
      rb[i] = load_b(nn, k0 + kk);
    }
  };
  auto store_smem = [&](int buf, int k0) {
    TAcc* as = As + buf * GEMM_BK * LD;
    TAcc* bs = Bs + buf * GEMM_BK * LD;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int mm, kk;
      if (A_MCONTIG) {
        mm = tid & 127;
        kk = (tid >> 7) + 2 * i;
      } else {
        kk = tid & 15;
        mm = (tid >> 4) + 16 * i;
      }
      as[kk * LD + mm] = conv_a(ra[i], mm, k0 + kk);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int nn, kk;
      if (B_NCONTIG) {
        nn = tid & 127;
        kk = (tid >> 7) + 2 * i;
      } else {
        kk = tid & 15;
        nn = (tid >> 4) + 16 * i;
      }
      bs[kk * LD + nn] = conv_b(rb[i], nn, k0 + kk);
    }
  };

  if (k_begin < k_end) {
    load_regs(k_begin);
    store_smem(0, k_begin);
  }
  __syncthreads();
  int buf = 0;
  for (int k0 = k_begin; k0 < k_end; k0 += GEMM_BK) {
    const bool more = (k0 + GEMM_BK) < k_end;
    if (more) load_regs(k0 + GEMM_BK);
    gemm_chunk(acc, As + buf * GEMM_BK * LD, Bs + buf * GEMM_BK * LD);
    if (more) store_smem(buf ^ 1, k0 + GEMM_BK);
    __syncthreads();
    buf ^= 1;
  }
}

// One 128 x 128 tile of the strided GEMM described by p.
template <typename TA, typename TB, typename TC, typename TAcc, bool A_MCONTIG, bool B_NCONTIG>
__device__ __forceinline__ void gemm_tile(const GemmP& p, int m0, int n0, int batch,
                                          unsigned char* smem) {
  const TA* A = static_cast<const TA*>(p.A) + (long long)batch * p.a_batch;
  const TB* B = static_cast<const TB*>(p.B) + (long long)batch * p.b_batch;
  TC* C = static_cast<TC*>(p.C) + (long long)batch * p.c_batch;

  int k_begin = 0, k_end = p.K;
  if (p.btrim == 1) k_end = min(k_end, n0 + GEMM_BN + p.boff);
  if (p.btrim == 2) k_begin = max(k_begin, n0 + p.boff);
  if (p.atrim == 1) k_end = min(k_end, m0 + GEMM_BM + p.aoff);
  if (p.atrim == 2) k_begin = max(k_begin, m0 + p.aoff);
  k_begin = (k_begin / GEMM_BK) * GEMM_BK;

  GemmAcc<TAcc> acc;
  acc.clear();

  const int M = p.M, N = p.N;
  const long long a_m = p.a_m, a_k = p.a_k, b_k = p.b_k, b_n = p.b_n;
  auto la = [&](int mm, int k) -> TA {
    const int m = m0 + mm;
    return (m < M && k < k_end) ? A[(long long)m * a_m + (long long)k * a_k] : zero_of<TA>();
  };
  auto lb = [&](int nn, int k) -> TB {
    const int n = n0 + nn;
    return (n < N && k < k_end) ? B[(long long)k * b_k + (long long)n * b_n] : zero_of<TB>();
  };
  auto ca = [](TA v, int, int) -> TAcc { return cvt<TAcc, TA>(v); };
  auto cb = [](TB v, int, int) -> TAcc { return cvt<TAcc, TB>(v); };
  gemm_mainloop<TAcc, A_MCONTIG, B_NCONTIG>(acc, la, ca, lb, cb, k_begin, k_end, smem);

  const TAcc alpha = static_cast<TAcc>(p.alpha), beta = static_cast<TAcc>(p.beta);
  if (p.beta == 0.0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int m = m0 + GemmAcc<TAcc>::row(i);
      if (m >= M) continue;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int n = n0 + GemmAcc<TAcc>::col(j);
        if (n < N) C[(long long)m * p.ldc + n] = static_cast<TC>(alpha * acc.at(i, j));
      }
    }
    return;
  }
  // C is read and written: the old values of row i + 1 are fetched before row i is stored,
  // so that the loads of a row go out together and their latency overlaps the stores
  // (a load placed after a store through the same pointer type cannot be moved above it).
  TAcc cold[2][8];
  auto fetch_row = [&](int i, TAcc* dst) {
    const int m = m0 + GemmAcc<TAcc>::row(i);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int n = n0 + GemmAcc<TAcc>::col(j);
      dst[j] = (m < M && n < N) ? static_cast<TAcc>(C[(long long)m * p.ldc + n]) : TAcc(0);
    }
  };
  fetch_row(0, cold[0]);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (i + 1 < 8) fetch_row(i + 1, cold[(i + 1) & 1]);
    const int m = m0 + GemmAcc<TAcc>::row(i);
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int n = n0 + GemmAcc<TAcc>::col(j);
      if (n < N) C[(long long)m * p.ldc + n] = static_cast<TC>(fma(beta, cold[i & 1][j], alpha * acc.at(i, j)));
    }
  }
}

template <typename TA, typename TB, typename TC, typename TAcc, bool A_MCONTIG, bool B_NCONTIG>
__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(GemmP p) {
  extern __shared__ __align__(16) unsigned char gemm_smem[];
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
  const int m0 = tm * GEMM_BM, n0 = tn * GEMM_BN;
  if ((p.flags & GEMM_LOWER_TILES) && n0 >= m0 + GEMM_BM) return;
  gemm_tile<TA, TB, TC, TAcc, A_MCONTIG, B_NCONTIG>(p, m0, n0, blockIdx.z, gemm_smem);
}

// Raise the dynamic shared-memory limit of a kernel once per device.
template <typename K>
tb_status allow_smem(K kern, size_t bytes, bool* done_per_device) {
  int dev = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!done_per_device[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    done_per_device[dev] = true;
  }
  return TB_OK;
}

// Host launcher.  Empty problems are a no-op.
template <typename TA, typename TB, typename TC, typename TAcc, bool A_MCONTIG, bool B_NCONTIG>
tb_status gemm_launch(const GemmP& p, cudaStream_t stream) {
  if (p.M <= 0 || p.N <= 0 || p.n_batch <= 0) return TB_OK;
  auto kern = gemm_kernel<TA, TB, TC, TAcc, A_MCONTIG, B_NCONTIG>;
  static bool configured[64] = {false};
  TB_TRY(allow_smem(kern, GemmSmem<TAcc>::bytes, configured));
  const int zmax = 65535;
  for (int b0 = 0; b0 < p.n_batch; b0 += zmax) {
    GemmP q = p;
    const int nb = (p.n_batch - b0 < zmax) ? (p.n_batch - b0) : zmax;
    q.A = static_cast<const TA*>(p.A) + (long long)b0 * p.a_batch;
    q.B = static_cast<const TB*>(p.B) + (long long)b0 * p.b_batch;
    q.C = static_cast<TC*>(p.C) + (long long)b0 * p.c_batch;
    q.n_batch = nb;
    dim3 grid((p.N + GEMM_BN - 1) / GEMM_BN, (p.M + GEMM_BM - 1) / GEMM_BM, nb);
    kern<<<grid, GEMM_THREADS, GemmSmem<TAcc>::bytes, stream>>>(q);
    TB_LAUNCH_CHECK();
  }
  return TB_OK;
}

}  // namespace tb
