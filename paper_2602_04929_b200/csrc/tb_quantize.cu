// tb_quantize_layer: the out-channel-group loop of Algorithm 1 and its closing steps.
//
// Per step i (a group of g = out_block rows of every head, M = n_heads * g
// rows in all, heads being independent):
//   grid     k_grid           Algorithm 1, grid     candidate search per (row, column group)
//   sweep    k_sweep_rows     Algorithm 2 / Eq. 2   one launch, 8 rows per CTA for the whole sweep
//   residual k_residual       E = W0 - Q_B          (Proposition 3.1)
//            GEMM             E -= W0 C             (Proposition 3.2, only with R)
//   update   GEMM             W~[rem] -= T_i E      (Algorithm 1, update)
// then, once: coordinate descent on the scales (Algorithm 3), Q = s (W_int - z),
// and the loss of the proofs of Propositions 3.1 / 3.2.
//
// All of this runs in IEEE double on the CUDA cores.  The codes are integer
// decisions inside an error-feedback chain d_in steps long; in float the
// accumulated rounding error of the chain (a few 1e-6 code units) exceeds the
// 1e-6 band inside which a rounding decision may legitimately differ, and one
// different decision changes every later code of its row.
#include <cooperative_groups.h>

#include "tb_common.cuh"
#include "tb_gemm.cuh"
#include "tb_profile.cuh"
#include "tb_tma.cuh"

namespace cg = cooperative_groups;

namespace tb {
// tensor-core blockwise product of the scale refinement (tb_gemm_tc.cu)
tb_status yw_tensor(float* Yw, const unsigned char* codes, const int* zeros, const float* H_in, __nv_bfloat16* WbT,
                    __nv_bfloat16* Hp, bool split_h, long long rows, int d, int seg, int ng, int hunits,
                    cudaStream_t st);
// C (+)= A B in double from operands split into three bf16 pieces each (tb_gemm_tc.cu)
tb_status gemm_split_presplit(double* C, long long ldc, const __nv_bfloat16* AT, const __nv_bfloat16* Bp, long long M,
                              int N, int K, bool accumulate, cudaStream_t st, int hunits = 1);
tb_status split3_transpose(const double* A, __nv_bfloat16* AT, long long M, int K, cudaStream_t st);
tb_status split3_transpose(const float* A, __nv_bfloat16* AT, long long M, int K, cudaStream_t st);
tb_status split3(const float* B, __nv_bfloat16* Bp, long long n, cudaStream_t st);
}

namespace tb {

// ---------------------------------------------------------------------------
// Row bookkeeping.  Active row m of a step maps to head m / g, row i0 + m % g
// of that head.  "Units" are sets of rows that share one H_in / U_in: the
// whole step when H_in is shared, one head otherwise.
// ---------------------------------------------------------------------------
struct RowMap {
  int g, d_head, i0;
  __host__ __device__ long long row(int m) const {
    return (long long)(m / g) * d_head + i0 + (m % g);
  }
};

__global__ void k_widen(const float* __restrict__ W, double* __restrict__ Wt, long long n) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x)
    Wt[i] = (double)W[i];
}

// Wk[m][:] = W~[row(m)][:]  (and a second untouched copy W0c when the
// propagated-error term needs the snapshot as a contiguous GEMM operand)
__global__ void k_gather(const double* __restrict__ Wt, double* __restrict__ Wk,
                         double* __restrict__ W0c, RowMap rm, int M, int d) {
  const long long n = (long long)M * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / d), k = (int)(i % d);
    const double v = Wt[rm.row(m) * d + k];
    Wk[i] = v;
    if (W0c) W0c[i] = v;
  }
}

// ---------------------------------------------------------------------------
// Compensation matrices of Propositions 3.1 / 3.2 for every head and step:
//   T = [U_out^T]_{rem,B} ([U_out^T]_{B,B})^{-1},  B = {i0..i0+g-1}, rem = rows after B.
// With A = U_out^T lower triangular, T A_BB = A_remB is solved row by row,
// last column first.  T is stored [head][step][d_head][g] (first rem rows used).
// ---------------------------------------------------------------------------
__global__ void k_comp_matrices(const float* __restrict__ Uout, double* __restrict__ T, int dh,
                                int g, int n_steps) {
  const int step = blockIdx.x, head = blockIdx.y;
  const int i0 = step * g, r0 = i0 + g, nrem = dh - r0;
  const float* Uo = Uout + (long long)head * dh * dh;
  double* Th = T + ((long long)head * n_steps + step) * dh * g;
  for (int r = threadIdx.x; r < nrem; r += blockDim.x) {
    double* Tr = Th + (long long)r * g;
    for (int c = g - 1; c >= 0; --c) {
      const float* urow = Uo + (long long)(i0 + c) * dh;
      double v = (double)urow[r0 + r];
      for (int c2 = c + 1; c2 < g; ++c2) v -= Tr[c2] * (double)urow[i0 + c2];
      Tr[c] = v / (double)urow[i0 + c];
    }
  }
}

// ---------------------------------------------------------------------------
// Grid search (Algorithm 1, grid step).  For every (row, column group): n_cand
// clipped min-max grids, p_k = 1 - k/32; score e H_in[G,G] e^T with e the
// round-to-nearest error on that grid; the lowest score wins, lowest k on ties.
//
// One CTA takes RT = 128 / NCP rows (NCP = n_cand rounded up to a power of
// two) of one column group: RT * NCP = 128 "candidate rows".  The scores are
// the row-wise dots of (E H) with E, where E [128 x seg] holds the candidate
// errors; E H runs on the GEMM tile engine with E produced on the fly.
// ---------------------------------------------------------------------------
struct GridP {
  const double* Wt;   // [d_out][d]
  const float* Hin;   // [n_hin][d][d]
  double* sD;         // [d_out][ng]
  float* s_out;       // [d_out][ng]
  int* z_out;         // [d_out][ng]
  unsigned char* cand_out;  // or nullptr
  RowMap rm;
  int M, d, seg, ng, maxq, n_cand, ncp, rt;
  int units, rows_per_unit, tiles_per_unit;
  const double* Wloc;  // or nullptr: the step's rows as a contiguous [M][d] working copy, read instead of Wt
  int grp0;            // column group of blockIdx.x = 0
};

__global__ void __launch_bounds__(GEMM_THREADS, 1) k_grid(GridP p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ double c_s[128], c_rs[128], c_z[128], c_J[128];
  __shared__ long long c_row[128];  // global row of a candidate row, or -1

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = p.grp0 + blockIdx.x;
  const int unit = blockIdx.y / p.tiles_per_unit;
  const int tile = blockIdx.y % p.tiles_per_unit;
  const int seg0 = grp * p.seg;
  const double maxq = (double)p.maxq;

  // Phase 1: min / max of every row segment, then the candidates' (s, z).
  for (int r = warp; r < p.rt; r += GEMM_THREADS / 32) {
    const int rloc = tile * p.rt + r;
    const bool valid = rloc < p.rows_per_unit;
    long long grow = -1;
    double mn = 0.0, mx = 0.0;
    if (valid) {
      grow = p.rm.row(unit * p.rows_per_unit + rloc);
      const double* w = p.Wt + grow * p.d + seg0;
      for (int a = lane; a < p.seg; a += 32) {
        const double v = w[a];
        mn = fmin(mn, v);
        mx = fmax(mx, v);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
    }
    if (lane < p.ncp) {
      const int k = lane, cr = r * p.ncp + k;
      double s = 1.0, z = 0.0;
      if (valid && k < p.n_cand) {
        const double pk = 1.0 - (double)k / 32.0;
        const double lo = pk * mn, hi = pk * mx;
        if (hi != lo) {
          s = (hi - lo) / maxq;
          z = fmin(fmax(rne(-lo / s), 0.0), maxq);
        }
      }
      c_s[cr] = s;
      c_rs[cr] = 1.0 / s;
      c_z[cr] = z;
      c_row[cr] = (valid && k < p.n_cand) ? grow : -1;
    }
  }
  // candidate rows beyond rt * ncp do not exist when ncp divides 128 (it does)
  __syncthreads();

  const float* H = p.Hin + (long long)unit * p.d * p.d * (p.units > 1 ? 1 : 0);
  const double* Wt = p.Wt;
  const int d = p.d, seg = p.seg;

  // round-to-nearest error of weight w on the grid of candidate row cr (0 for w = 0,
  // which is what rows and columns outside the problem are given)
  auto err_of = [&](int cr, double w) -> double {
    const double s = c_s[cr], z = c_z[cr];
    double q = rne(fma(w, c_rs[cr], z));
    q = fmin(fmax(q, 0.0), maxq);
    return w - s * (q - z);
  };
  // quantization error of candidate row cr at segment column a
  auto err_at = [&](int cr, int a) -> double {
    const long long grow = c_row[cr];
    if (grow < 0 || a >= seg) return 0.0;
    return err_of(cr, Wt[grow * d + seg0 + a]);
  };

  double jpart[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) jpart[i] = 0.0;

  for (int a0 = 0; a0 < seg; a0 += GEMM_BN) {
    GemmAcc<double> acc;
    acc.clear();
    // fetch the weight; the candidate's error is formed when the chunk is staged
    auto la = [&](int mm, int k) -> double {
      const long long grow = c_row[mm];
      return (grow >= 0 && k < seg) ? Wt[grow * d + seg0 + k] : 0.0;
    };
    auto ca = [&](double w, int mm, int) -> double { return err_of(mm, w); };
    auto lb = [&](int nn, int k) -> float {
      const int a = a0 + nn;
      return (a < seg && k < seg) ? H[(long long)(seg0 + k) * d + seg0 + a] : 0.0f;
    };
    auto cb = [](float v, int, int) -> double { return (double)v; };
    gemm_mainloop<double, true, true>(acc, la, ca, lb, cb, 0, seg, smem_raw);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int cr = GemmAcc<double>::row(i);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        jpart[i] = fma(acc.at(i, j), err_at(cr, a0 + GemmAcc<double>::col(j)), jpart[i]);
    }
  }
  // A candidate row's score is spread over the 4 lanes of a quad and the 4 warps that
  // share its rows; quads reduce by shuffle, warps through shared memory in a fixed order.
  double* c_Jw = reinterpret_cast<double*>(smem_raw);  // [4][128], the tile buffers are free now
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    double v = jpart[i];
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    if ((lane & 3) == 0) c_Jw[(warp & 3) * 128 + GemmAcc<double>::row(i)] = v;
  }
  __syncthreads();
  if (tid < 128) c_J[tid] = ((c_Jw[tid] + c_Jw[128 + tid]) + c_Jw[256 + tid]) + c_Jw[384 + tid];
  __syncthreads();

  // Phase 3: argmin per row, strict '<' so that the lowest k wins ties.
  if (tid < p.rt) {
    const int r = tid;
    const long long grow = c_row[r * p.ncp];
    if (grow >= 0) {
      int best = 0;
      double bj = c_J[r * p.ncp];
      for (int k = 1; k < p.n_cand; ++k) {
        const double j = c_J[r * p.ncp + k];
        if (j < bj) {
          bj = j;
          best = k;
        }
      }
      const int cr = r * p.ncp + best;
      const long long o = grow * p.ng + grp;
      p.sD[o] = c_s[cr];
      p.s_out[o] = (float)c_s[cr];
      p.z_out[o] = (int)c_z[cr];
      if (p.cand_out) p.cand_out[o] = (unsigned char)best;
    }
  }
}

// ---------------------------------------------------------------------------
// The same search for groups of at most 128 columns, where the whole problem of a
// CTA (128 candidate rows x one group) fits shared memory.  H_in[G,G] is symmetric,
// so e H e^T = 2 e T e^T with T the upper triangle of H (diagonal halved): only the
// part k <= n of the product is formed, about half of the tensor-pipe work.  The
// scores are compared, never output, so the factor 2 is dropped.  The candidate
// errors are staged once (and read again for the row dots), T as float; after one
// barrier the product runs without further synchronisation.  Column fragments
// (8 columns) are dealt to the warps so that every warp has the same share of the
// triangle: warp column c owns fragments c, 7-c, 8+c, 15-c.  Reads the upper
// triangle of H_in only.
// ---------------------------------------------------------------------------
enum { GT_LDE = 132, GT_LDB = 136 };
static constexpr size_t GRID_TRI_SMEM = (size_t)128 * GT_LDE * sizeof(double) + (size_t)128 * GT_LDB * sizeof(float);

__global__ void __launch_bounds__(GEMM_THREADS, 1) k_grid_tri(GridP p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* Es = reinterpret_cast<double*>(smem_raw);                                    // [k][candidate row]
  float* Bs = reinterpret_cast<float*>(smem_raw + (size_t)128 * GT_LDE * sizeof(double));  // [k][n]
  __shared__ double c_s[128], c_rs[128], c_z[128], c_J[128];
  __shared__ long long c_row[128];  // global row of a candidate row, or -1
  __shared__ long long c_src[128];  // element offset of that row's first column in the source matrix

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = p.grp0 + blockIdx.x;
  const int unit = blockIdx.y / p.tiles_per_unit;
  const double* Wsrc = p.Wloc ? p.Wloc : p.Wt;
  const int tile = blockIdx.y % p.tiles_per_unit;
  const int seg0 = grp * p.seg;
  const int d = p.d, seg = p.seg;
  const double maxq = (double)p.maxq;
  const float* H = p.Hin + (long long)unit * p.d * p.d * (p.units > 1 ? 1 : 0);

  // T = upper triangle of H_in[G,G], diagonal halved; issued first, it lands while phase 1 runs
  {
    const int n = tid & 127;
    float hv[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) {
      const int k = (tid >> 7) + 2 * i;
      hv[i] = (k <= n && n < seg) ? H[(long long)(seg0 + k) * d + seg0 + n] : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 64; ++i) {
      const int k = (tid >> 7) + 2 * i;
      Bs[k * GT_LDB + n] = (k == n) ? 0.5f * hv[i] : hv[i];
    }
  }

  // Phase 1: min / max of every row segment, then the candidates' (s, z).
  for (int r = warp; r < p.rt; r += GEMM_THREADS / 32) {
    const int rloc = tile * p.rt + r;
    const bool valid = rloc < p.rows_per_unit;
    long long grow = -1, src = 0;
    double mn = 0.0, mx = 0.0;
    if (valid) {
      grow = p.rm.row(unit * p.rows_per_unit + rloc);
      src = (p.Wloc ? (long long)(unit * p.rows_per_unit + rloc) : grow) * p.d;
      const double* w = Wsrc + src + seg0;
      for (int a = lane; a < p.seg; a += 32) {
        const double v = w[a];
        mn = fmin(mn, v);
        mx = fmax(mx, v);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
    }
    if (lane < p.ncp) {
      const int k = lane, cr = r * p.ncp + k;
      double s = 1.0, z = 0.0;
      if (valid && k < p.n_cand) {
        const double pk = 1.0 - (double)k / 32.0;
        const double lo = pk * mn, hi = pk * mx;
        if (hi != lo) {
          s = (hi - lo) / maxq;
          z = fmin(fmax(rne(-lo / s), 0.0), maxq);
        }
      }
      c_s[cr] = s;
      c_rs[cr] = 1.0 / s;
      c_z[cr] = z;
      c_row[cr] = (valid && k < p.n_cand) ? grow : -1;
      c_src[cr] = src;
    }
  }
  __syncthreads();

  // Phase 2: the candidates' round-to-nearest errors, Es[k][cr] (0 outside the problem)
  {
    const int cr = tid & 127;
    const long long grow = c_row[cr];
    const double s = c_s[cr], rs = c_rs[cr], z = c_z[cr];
    const double magic = 6755399441055744.0;  // 1.5 * 2^52
    const double zm = z + magic;
    const double* w = Wsrc + (grow < 0 ? 0 : c_src[cr]) + seg0;
#pragma unroll 8
    for (int i = 0; i < 64; ++i) {
      const int k = (tid >> 7) + 2 * i;
      double e = 0.0;
      if (grow >= 0 && k < seg) {
        // the fused multiply-add into z + 1.5 * 2^52 rounds to nearest-even and leaves the integer in the
        // low word (|v / s + z| < 2^31), where the clamp is two integer instructions
        const double v = w[k];
        int n = __double2loint(fma(v, rs, zm));
        n = min(max(n, 0), p.maxq);
        const double q = __hiloint2double(0x43380000, n) - magic;
        e = v - s * (q - z);
      }
      Es[k * GT_LDE + cr] = e;
    }
  }
  __syncthreads();

  // Phase 3: acc = E T on the FP64 tensor pipe, fragments with k <= n only
  const int wc = warp & 3, kq = lane & 3, rq = lane >> 2;
  int fr[4];
  fr[0] = wc;
  fr[1] = 7 - wc;
  fr[2] = 8 + wc;
  fr[3] = 15 - wc;
  double acc[8][4][2];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
  const double* ap = Es + kq * GT_LDE + (warp >> 2) * 64 + rq;
  const float* bp = Bs + kq * GT_LDB + rq;
  const int k4_end = (seg + 3) / 4;
#pragma unroll 1
  for (int k4 = 0; k4 < k4_end; ++k4) {
    double a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = ap[k4 * 4 * GT_LDE + i * 8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (8 * fr[j] + 7 < 4 * k4 || 8 * fr[j] >= seg) continue;  // wholly below the diagonal, or outside the group
      const double b = (double)bp[k4 * 4 * GT_LDB + 8 * fr[j]];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                     : "+d"(acc[i][j][0]), "+d"(acc[i][j][1])
                     : "d"(a[i]), "d"(b));
    }
  }

  // Phase 4: row dots of (E T) with E.  A candidate row's score is spread over the 4 lanes of a
  // quad and the 4 warps that share its rows; quads reduce by shuffle, warps through shared
  // memory in a fixed order.
  double jpart[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int cr = (warp >> 2) * 64 + i * 8 + rq;
    double v = 0.0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = 8 * fr[j] + 2 * kq;
      v = fma(acc[i][j][0], Es[n * GT_LDE + cr], v);
      v = fma(acc[i][j][1], Es[(n + 1) * GT_LDE + cr], v);
    }
    jpart[i] = v;
  }
  __syncthreads();  // every warp is done with Bs: its storage takes the partial scores
  double* c_Jw = reinterpret_cast<double*>(Bs);  // [4][128]
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    double v = jpart[i];
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    if (kq == 0) c_Jw[wc * 128 + (warp >> 2) * 64 + i * 8 + rq] = v;
  }
  __syncthreads();
  if (tid < 128) c_J[tid] = ((c_Jw[tid] + c_Jw[128 + tid]) + c_Jw[256 + tid]) + c_Jw[384 + tid];
  __syncthreads();

  // Phase 5: argmin per row, strict '<' so that the lowest k wins ties.
  if (tid < p.rt) {
    const int r = tid;
    const long long grow = c_row[r * p.ncp];
    if (grow >= 0) {
      int best = 0;
      double bj = c_J[r * p.ncp];
      for (int k = 1; k < p.n_cand; ++k) {
        const double j = c_J[r * p.ncp + k];
        if (j < bj) {
          bj = j;
          best = k;
        }
      }
      const int cr = r * p.ncp + best;
      const long long o = grow * p.ng + grp;
      p.sD[o] = c_s[cr];
      p.s_out[o] = (float)c_s[cr];
      p.z_out[o] = (int)c_z[cr];
      if (p.cand_out) p.cand_out[o] = (unsigned char)best;
    }
  }
}

// ---------------------------------------------------------------------------
// Column sweep (Algorithm 2; Eq. 2), one launch per step.  Rows never interact
// inside the sweep, so a CTA keeps 8 active rows for the whole sweep and no CTA
// ever waits for another.
//
// Left-looking form: the values of block b on arrival are
//   w[:, b] = W0[:, b] - Err[:, 0 : 128 b] U[0 : 128 b, b]  (- Arr[:, 0 : 128 b] P[0 : 128 b, b]),
// where Err holds the normalised errors and Arr the arrival values of the
// columns already quantized (the second product only with the propagated-error
// term, WITH_P).  16 warps: warps 0-7 are the panel warps (one row each, one
// lane per column, the 128 columns of a block strictly in order); warps 8-15
// are the update warps (two 8-column fragments each, on the FP64 tensor pipe,
// four accumulators per fragment in turn so that enough independent tensor
// instructions are in flight).
// While the panel warps walk block b, the update warps form the part of block
// b+1's sum that needs only blocks < b: 64-row chunks of U (and P) and of the
// histories arrive by TMA (one box each, 8 spare columns per row so that
// fragment loads are free of bank conflicts) in a ring guarded by full / empty
// mbarriers; when the panel is done they add the last 128 terms (block b's
// errors and arrival values straight from shared memory) and hand block b+1
// over.  The two warp groups meet at hardware barriers with fixed participant
// counts; every trip count depends on the block index alone.  mbarrier waits
// are bounded: when a bound runs out the kernel raises a device error word and
// stops computing, but still passes every barrier, so it always terminates.
// ---------------------------------------------------------------------------
enum { RS_CCHUNK = 128, RS_CLDE = 132 };  // cluster form: contraction rows per chunk, row pitch of its history box
enum { RS_THREADS = 512, RS_LDB = 136, RS_LDE = 68, RS_CHUNK = 64, RS_LDW = 132, RS_TRI = 10240 };
struct RowSweepP {
  const double* Wt;      // [d_out][d] current W~ (rows of the step are read, never written)
  const float* U;        // [n_hin][d][d]
  const float* P;        // [n_hin][d][d] (WITH_P)
  double* ErrG;          // [M][d] normalised errors of the step's rows
  double* ArrG;          // [M][d] arrival values of the step's rows (WITH_P)
  unsigned char* codes;  // [d_out][d]
  const double* sD;      // [d_out][ng]
  const int* z;          // [d_out][ng]
  tb_stats* stats;       // or nullptr
  RowMap rm;
  int M, d, seg, ng, maxq, nblk;
  int units, rows_per_unit, ctas_per_unit;
  int cs;                // CTAs that share a group of 8 rows (1, or a cluster of 2 or 4 when rows are few)
};
struct RowSweepStage {
  float Ub[RS_CHUNK][RS_LDB];   // 64 rows of U or P: 128 columns of the target block + 8 spare
  double Eb[8][RS_LDE];         // the same 64 columns of a history (+ 4 spare), 8 rows
};
// The panel only touches the upper triangle of a diagonal block: rows of sub-block sb
// (32 rows) are stored from column 32 sb on, 128 - 32 sb wide.
__host__ __device__ constexpr int tri_base(int sb) { return sb * 4096 - 512 * sb * (sb - 1); }
template <bool WITH_P>
struct RowSweepSmem {
  static constexpr int STAGES = WITH_P ? 3 : 4;
  float sU[RS_TRI];             // diagonal block of U, upper part
  float sP[WITH_P ? RS_TRI : 4];
  alignas(128) RowSweepStage ring[STAGES];  // TMA destinations
  double wblk[8][128];          // arrival values of the current block before its own feedback
  double Es[8][RS_LDW];         // normalised errors of the current block
  double As[WITH_P ? 8 : 1][RS_LDW];  // arrival values of the current block
  unsigned long long full_bar[STAGES], empty_bar[STAGES];
  unsigned long long cfull_bar[8], cempty_bar[8];  // ring of the cluster form (more, smaller stages)
  int abort_flag;
};
__device__ int g_sweep_error = 0;

__device__ __forceinline__ void mma_f64(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}
__device__ __forceinline__ void bar_all() { asm volatile("bar.sync 3, 512;" ::: "memory"); }


template <bool WITH_P>
__global__ void __launch_bounds__(RS_THREADS, 1)
    k_sweep_rows(RowSweepP p, const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_e,
                 const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_a) {
  extern __shared__ __align__(128) unsigned char rs_raw[];
  using Smem = RowSweepSmem<WITH_P>;
  constexpr int STAGES = Smem::STAGES;
  constexpr int NOP = WITH_P ? 2 : 1;  // operand pairs per 64-row chunk: (Err, U) and (Arr, P)
  Smem& sm = *reinterpret_cast<Smem*>(rs_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // With few rows per launch a cluster of cs CTAs shares a group of 8 rows: each prepares 128 / cs
  // columns of the next block (its share of the contraction work) and writes them into the shared
  // memory of all; the panel runs in every CTA on the same values, so all of them hold the block's
  // errors and write identical results.
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = p.cs;
  const int crank = (cs > 1) ? (int)cluster.block_rank() : 0;
  const int grp = blockIdx.x / cs;
  const int unit = grp / p.ctas_per_unit;
  const int r_first = (grp % p.ctas_per_unit) * 8;  // first row of this group inside its unit
  // arrival values of the blocks: with a cluster the buffers alternate (a fast CTA may write block b + 1
  // while a slow one still reads block b); the second one sits in the part of ring stage 0 that the
  // narrower boxes of a cluster leave free
  // The cluster form cuts the ring's memory into more, smaller stages (its boxes of U are 128 / cs + 8
  // floats wide), as many as fit beside the second arrival buffer, at most 8: with short chunks only
  // the number of loads in flight hides their latency.
  const int c_ldb = 128 / cs + 8;
  const int c_stage_bytes = RS_CCHUNK * c_ldb * (int)sizeof(float) + 8 * RS_CLDE * (int)sizeof(double);
  const int c_nst = min(8, (int)((sizeof(sm.ring) - sizeof(sm.wblk)) / c_stage_bytes));
  unsigned char* ring_base = reinterpret_cast<unsigned char*>(&sm.ring[0]);
  double* wbuf0 = &sm.wblk[0][0];
  double* wbuf1 = (cs > 1) ? reinterpret_cast<double*>(ring_base + (size_t)c_nst * c_stage_bytes) : wbuf0;
  const int d = p.d;
  const long long uoff = (long long)unit * d * d * (p.units > 1 ? 1 : 0);
  const float* U = p.U + uoff;
  const float* Pm = WITH_P ? p.P + uoff : nullptr;
  const double maxq = (double)p.maxq;
  const int m_base = unit * p.rows_per_unit + r_first;
  const int rows_here = min(8, p.rows_per_unit - r_first);

  // block 0 arrives unchanged
  for (int idx = tid; idx < 8 * 128; idx += RS_THREADS) {
    const int r = idx >> 7, c = idx & 127;
    sm.wblk[r][c] = (r < rows_here) ? p.Wt[p.rm.row(m_base + r) * d + c] : 0.0;
  }
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&sm.full_bar[s]), 1);
      mbar_init(smem_u32(&sm.empty_bar[s]), 8);  // one arrival per update warp
    }
    for (int s = 0; s < 8; ++s) {
      mbar_init(smem_u32(&sm.cfull_bar[s]), 1);
      mbar_init(smem_u32(&sm.cempty_bar[s]), (cs > 1) ? 16 / cs : 8);  // one arrival per working update warp
    }
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  bar_all();

  if (warp < 8) {
    // =========================== panel warps: row `warp` ===========================
    const bool valid = warp < rows_here;
    const long long grow = valid ? p.rm.row(m_base + warp) : 0;
    const double magic = 6755399441055744.0;  // 1.5 * 2^52: adding it rounds to an integer, ties to even
    unsigned int n_near = 0, n_clamp = 0;
    for (int b = 0; b < p.nblk; ++b) {
      const int c0 = b * 128;
      // grids of this lane's four columns (fetched while the diagonal block is staged)
      double s4[4], z4[4];
#pragma unroll
      for (int sb = 0; sb < 4; ++sb) {
        const long long so = grow * p.ng + (c0 + sb * 32 + lane) / p.seg;
        s4[sb] = valid ? p.sD[so] : 1.0;
        z4[sb] = valid ? (double)p.z[so] : 0.0;
      }
      // upper part of the diagonal block(s): row r of sub-block sb from column 32 sb on
      for (int idx = tid; idx < 128 * 32; idx += 256) {
        const int r = idx >> 5, c4 = (idx & 31) * 4, sb = r >> 5;
        if (c4 >= 32 * sb) {
          const int o = tri_base(sb) + (r - 32 * sb) * (128 - 32 * sb) + (c4 - 32 * sb);
          *reinterpret_cast<float4*>(sm.sU + o) =
              *reinterpret_cast<const float4*>(U + (long long)(c0 + r) * d + c0 + c4);
          if (WITH_P)
            *reinterpret_cast<float4*>(sm.sP + o) =
                *reinterpret_cast<const float4*>(Pm + (long long)(c0 + r) * d + c0 + c4);
        }
      }
      asm volatile("bar.sync 2, 256;" ::: "memory");
      double w[4], rs4[4], rd4[4];
#pragma unroll
      for (int sb = 0; sb < 4; ++sb) {
        w[sb] = ((b & 1) ? wbuf1 : wbuf0)[warp * 128 + sb * 32 + lane];
        rs4[sb] = 1.0 / s4[sb];
        rd4[sb] = 1.0 / (double)sm.sU[tri_base(sb) + lane * (128 - 32 * sb) + lane];
      }
#pragma unroll 1
      for (int sb = 0; sb < 4; ++sb) {
        const int cl = sb * 32 + lane, col = c0 + cl;
        const int wd = 128 - 32 * sb;                 // width of this sub-block's stored rows
        const float* ub = sm.sU + tri_base(sb) + lane;  // element (32 sb + j, 32 sb + lane + 32 t) at ub[j * wd + 32 t]
        const float* pb = sm.sP + (WITH_P ? tri_base(sb) + lane : 0);
        const double s_l = (sb == 0) ? s4[0] : (sb == 1) ? s4[1] : (sb == 2) ? s4[2] : s4[3];
        const double z_l = (sb == 0) ? z4[0] : (sb == 1) ? z4[1] : (sb == 2) ? z4[2] : z4[3];
        const double rs_l = (sb == 0) ? rs4[0] : (sb == 1) ? rs4[1] : (sb == 2) ? rs4[2] : rs4[3];
        const double rd_l = (sb == 0) ? rd4[0] : (sb == 1) ? rd4[1] : (sb == 2) ? rd4[2] : rd4[3];
        const double srd_l = s_l * rd_l;
        const double szrd_l = s_l * z_l * rd_l;
        const double zm_l = z_l + magic;
        float u[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) u[j] = ub[j * wd];
        double v = (sb == 0) ? w[0] : (sb == 1) ? w[1] : (sb == 2) ? w[2] : w[3];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          // e = (v - s (q - z)) / U_jj = (v / U_jj + s z / U_jj) - (s / U_jj) q, with q = clamp(rne(v / s + z)).
          // The fused multiply-add into z + 1.5 * 2^52 performs the rounding itself and leaves the
          // integer in the low word of the result, where the clamp is two integer instructions
          // instead of two slow double-precision min / max.  The low word alone is the integer only
          // for |v / s + z| < 2^31; the high word tells (it is the constant's, or one less for a
          // negative integer, exactly when the low word's sign says the same), and beyond that
          // range, infinities included, the code saturates like the clamp of the full value.
          const double ard = fma(v, rd_l, szrd_l);
          const double xm = fma(v, rs_l, zm_l);
          const int lo = __double2loint(xm), hw = __double2hiint(xm) - 0x43380000;
          int n = min(max(lo, 0), p.maxq);
          n = (hw == (lo >> 31)) ? n : ((hw >= 0) ? p.maxq : 0);
          const double q = __hiloint2double(0x43380000, n) - magic;
          const double e = fma(-srd_l, q, ard);
          const double ej = shfl_d(e, j);
          if (WITH_P) {
            const double vj = shfl_d(v, j);  // value of column j on arrival
            if (lane > j) v = fma(-vj, (double)pb[j * wd], fma(-ej, (double)u[j], v));
          } else {
            if (lane > j) v = fma(-ej, (double)u[j], v);
          }
        }
        const double x = fma(v, rs_l, z_l);
        const double xr = fma(v, rs_l, zm_l) - magic;
        const double q = fmin(fmax(xr, 0.0), maxq);
        const double e_mine = fma(-srd_l, q, fma(v, rd_l, szrd_l));  // the value broadcast at step `lane`
        sm.Es[warp][cl] = valid ? e_mine : 0.0;
        if (WITH_P) sm.As[warp][cl] = valid ? v : 0.0;
        if (valid) {
          p.codes[grow * d + col] = (unsigned char)(int)q;
          p.ErrG[(long long)(m_base + warp) * d + col] = e_mine;
          if (WITH_P) p.ArrG[(long long)(m_base + warp) * d + col] = v;
          const double fl = floor(x);
          const double a0 = fmin(fmax(fl, 0.0), maxq), a1 = fmin(fmax(fl + 1.0, 0.0), maxq);
          if (fabs(x - (fl + 0.5)) < 1e-6 && a0 != a1) ++n_near;
          if (xr != q) ++n_clamp;
        }
        // the sub-block's errors (and arrival values) update the later sub-blocks of this block:
        // one branch-free loop per case, so that shuffles, loads and multiply-adds of different j overlap
        if (sb == 0) {
#pragma unroll 8
          for (int j = 0; j < 32; ++j) {
            const double ej = shfl_d(e_mine, j);
            w[1] = fma(-ej, (double)ub[j * 128 + 32], w[1]);
            w[2] = fma(-ej, (double)ub[j * 128 + 64], w[2]);
            w[3] = fma(-ej, (double)ub[j * 128 + 96], w[3]);
            if (WITH_P) {
              const double vj = shfl_d(v, j);
              w[1] = fma(-vj, (double)pb[j * 128 + 32], w[1]);
              w[2] = fma(-vj, (double)pb[j * 128 + 64], w[2]);
              w[3] = fma(-vj, (double)pb[j * 128 + 96], w[3]);
            }
          }
        } else if (sb == 1) {
#pragma unroll 8
          for (int j = 0; j < 32; ++j) {
            const double ej = shfl_d(e_mine, j);
            w[2] = fma(-ej, (double)ub[j * 96 + 32], w[2]);
            w[3] = fma(-ej, (double)ub[j * 96 + 64], w[3]);
            if (WITH_P) {
              const double vj = shfl_d(v, j);
              w[2] = fma(-vj, (double)pb[j * 96 + 32], w[2]);
              w[3] = fma(-vj, (double)pb[j * 96 + 64], w[3]);
            }
          }
        } else if (sb == 2) {
#pragma unroll 8
          for (int j = 0; j < 32; ++j) {
            const double ej = shfl_d(e_mine, j);
            w[3] = fma(-ej, (double)ub[j * 64 + 32], w[3]);
            if (WITH_P) {
              const double vj = shfl_d(v, j);
              w[3] = fma(-vj, (double)pb[j * 64 + 32], w[3]);
            }
          }
        }
      }
      // the histories are read back by TMA (async proxy): order these stores before it
      asm volatile("fence.proxy.async;" ::: "memory");
      bar_all();  // block b is quantized: its errors are in Es and in the history
      if (cs > 1)
        cluster.sync();  // block b+1 has been handed over by all CTAs of the cluster
      else
        bar_all();       // block b+1 has been handed over in wblk
    }
    if (p.stats && crank == 0) {
      n_near = __reduce_add_sync(0xffffffffu, n_near);
      n_clamp = __reduce_add_sync(0xffffffffu, n_clamp);
      if (lane == 0) {
        if (n_near) atomicAdd(&p.stats->near_tie_codes, (unsigned long long)n_near);
        if (n_clamp) atomicAdd(&p.stats->clamped_codes, (unsigned long long)n_clamp);
        if (grp == 0 && warp == 0) atomicAdd(&p.stats->column_steps, (unsigned long long)d);
      }
    }
    return;
  }

  // =========================== update warps ===========================
  const int uw = warp - 8;
  const int fr = lane >> 2, fk = lane & 3;   // fragment row / k (and column) index of this lane
  const bool fr_valid = fr < rows_here;
  const long long fr_grow = fr_valid ? p.rm.row(m_base + fr) : 0;
  // This warp owns columns n_lo .. n_lo+15 of the target block: fragment 0 the even ones,
  // fragment 1 the odd ones, so that one 8-byte load feeds both.
  const int n_lo = uw * 16;
  volatile int* abort_flag = &sm.abort_flag;
  // Loading a chunk costs its issuer a few hundred cycles, and a ring slot is only free once all eight
  // warps have released it, so a fixed issuer would hold everybody back: the duty rotates, chunk c of a
  // block is loaded by lane 0 of update warp c mod 8.  Every warp keeps the ring position of the
  // producer side itself (it is a function of the chunk count alone).
  const bool lane0 = (lane == 0);
  const int u_row0 = unit * d * (p.units > 1 ? 1 : 0);
  // ring positions: `c_*` of the consumers (all update warps), `p_*` of the producer thread
  int c_slot = 0, p_slot = 0;
  uint32_t c_phase = 0, p_phase = 0;
  if (cs > 1) {
    // ---- cluster form: this CTA prepares columns crank * wc .. + wc - 1 of the next block, one 8-column
    // fragment per working warp; the boxes of U are wc + 8 floats wide ----
    const int wc = 128 / cs, ldb = c_ldb, frags = 16 / cs;
    const int ub_bytes = RS_CCHUNK * ldb * (int)sizeof(float);
    const int eb_bytes = 8 * RS_CLDE * (int)sizeof(double);
    // chunks of 128 contraction rows (a whole block): with one fragment per warp a 64-row chunk is too
    // little work beside the fixed cost of a ring step
    const bool working = uw < frags;
    const int n_blk = crank * wc + uw * 8;   // first column of this warp's fragment inside the block
    for (int b = 0; b < p.nblk; ++b) {
      if (b + 1 >= p.nblk) {
        bar_all();
        cluster.sync();
        break;
      }
      const int cn = (b + 1) * 128;
      const int n_hist = b * NOP, n_all = n_hist + NOP;
      double* wnext = ((b + 1) & 1) ? wbuf1 : wbuf0;
      if (working) {
        double acc[8][2];  // eight accumulators in turn: one fragment per warp has to cover the latency alone
#pragma unroll
        for (int i = 0; i < 16; ++i) (&acc[0][0])[i] = 0.0;
        double w0[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) w0[e] = fr_valid ? p.Wt[fr_grow * d + cn + n_blk + 2 * fk + e] : 0.0;
        auto produce = [&](int c) {
          if (c < n_all) {
            if ((c % frags) == uw) {
              unsigned char* stg = ring_base + (size_t)p_slot * c_stage_bytes;
              const uint32_t fb = smem_u32(&sm.cfull_bar[p_slot]);
              if (mbar_wait(smem_u32(&sm.cempty_bar[p_slot]), p_phase ^ 1u, abort_flag, &g_sweep_error)) {
                const bool hist = c < n_hist;
                const bool second = WITH_P && (c & 1);
                const int kc = c / NOP;
                mbar_expect_tx(fb, (uint32_t)(ub_bytes + (hist ? eb_bytes : 0)));
                tma_load_2d(smem_u32(stg), second ? &map_p : &map_u, cn + crank * wc, u_row0 + kc * RS_CCHUNK, fb);
                if (hist) tma_load_2d(smem_u32(stg + ub_bytes), second ? &map_a : &map_e, kc * RS_CCHUNK, m_base, fb);
              }
            }
            if (++p_slot == c_nst) {
              p_slot = 0;
              p_phase ^= 1u;
            }
          }
        };
        if (lane0)
          for (int c = 0; c < c_nst - 1; ++c) produce(c);
        for (int c = 0; c < n_all; ++c) {
          if (c == n_hist) bar_all();
          const unsigned char* stg = ring_base + (size_t)c_slot * c_stage_bytes;
          const double* eb = reinterpret_cast<const double*>(stg + ub_bytes);  // [8][RS_CLDE]
          const bool ok = mbar_wait(smem_u32(&sm.cfull_bar[c_slot]), c_phase, abort_flag, &g_sweep_error);
          if (ok) {
            const double* ap;
            if (c < n_hist)
              ap = eb + fr * RS_CLDE + fk;
            else if (WITH_P && (c & 1))
              ap = &sm.As[fr][fk];
            else
              ap = &sm.Es[fr][fk];
            const float* bp = reinterpret_cast<const float*>(stg) + fk * ldb + uw * 8 + fr;
#pragma unroll
            for (int q = 0; q < RS_CCHUNK / 4; ++q) mma_f64(acc[q & 7], ap[4 * q], (double)bp[4 * q * ldb]);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&sm.cempty_bar[c_slot]));
          if (++c_slot == c_nst) {
            c_slot = 0;
            c_phase ^= 1u;
          }
          if (lane0) produce(c + c_nst - 1);
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const double v = w0[e] - (((acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e])) +
                                    ((acc[4][e] + acc[5][e]) + (acc[6][e] + acc[7][e])));
          for (int r = 0; r < cs; ++r) cluster.map_shared_rank(wnext, r)[fr * 128 + n_blk + 2 * fk + e] = v;
        }
      } else {
        bar_all();  // the barrier the working warps pass once the panel has finished block b
      }
      cluster.sync();  // block b+1 handed over
    }
    return;
  }
  for (int b = 0; b < p.nblk; ++b) {
    if (b + 1 >= p.nblk) {  // nothing left to prepare
      bar_all();
      bar_all();
      break;
    }
    const int cn = (b + 1) * 128;            // first column of the target block
    const int n_hist = 2 * b * NOP;          // steps whose left operand comes from a history (blocks < b)
    const int n_all = n_hist + 2 * NOP;      // plus the two chunks of block b itself
    // four accumulators per fragment, used in turn: with two there are not enough independent
    // tensor instructions in flight to cover their latency
    double acc[2][4][2];
#pragma unroll
    for (int i = 0; i < 16; ++i) (&acc[0][0][0])[i] = 0.0;
    // the block's own weights, needed at the end: tile-column ci = 2 fk + e is column n_lo + 2 ci + t
    double w0[2][2];
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int e = 0; e < 2; ++e)
        w0[t][e] = fr_valid ? p.Wt[fr_grow * d + cn + n_lo + 2 * (2 * fk + e) + t] : 0.0;

    // step c: 64-row chunk c / NOP of the contraction, operand pair c % NOP
    auto produce = [&](int c) {   // every lane 0 keeps count; the warp whose turn it is loads
      if (c < n_all) {
        if ((c & 7) == uw) {
        RowSweepStage& st = sm.ring[p_slot];
        const uint32_t fb = smem_u32(&sm.full_bar[p_slot]);
        if (mbar_wait(smem_u32(&sm.empty_bar[p_slot]), p_phase ^ 1u, abort_flag, &g_sweep_error)) {
          const bool hist = c < n_hist;
          const bool second = WITH_P && (c & 1);
          const int kc = c / NOP;
          mbar_expect_tx(fb, (uint32_t)(sizeof(st.Ub) + (hist ? sizeof(st.Eb) : 0)));
          tma_load_2d(smem_u32(&st.Ub[0][0]), second ? &map_p : &map_u, cn, u_row0 + kc * RS_CHUNK, fb);
          if (hist) tma_load_2d(smem_u32(&st.Eb[0][0]), second ? &map_a : &map_e, kc * RS_CHUNK, m_base, fb);
        }
        }
        if (++p_slot == STAGES) {
          p_slot = 0;
          p_phase ^= 1u;
        }
      }
    };
    if (lane0)
      for (int c = 0; c < STAGES - 1; ++c) produce(c);
    for (int c = 0; c < n_all; ++c) {
      if (c == n_hist) bar_all();  // the panel warps have finished block b: Es (and As) are complete
      const RowSweepStage& st = sm.ring[c_slot];
      const bool ok = mbar_wait(smem_u32(&sm.full_bar[c_slot]), c_phase, abort_flag, &g_sweep_error);
      if (ok) {
        const int own = (c - n_hist) / NOP;  // which of block b's two chunks (when c >= n_hist)
        const double* ap;
        if (c < n_hist)
          ap = &st.Eb[fr][fk];
        else if (WITH_P && (c & 1))
          ap = &sm.As[fr][own * RS_CHUNK + fk];
        else
          ap = &sm.Es[fr][own * RS_CHUNK + fk];
        const float* bp = &st.Ub[fk][n_lo + 2 * fr];
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const double a = ap[4 * q];
          const float2 bb = *reinterpret_cast<const float2*>(bp + 4 * q * RS_LDB);
          mma_f64(acc[0][q & 3], a, (double)bb.x);
          mma_f64(acc[1][q & 3], a, (double)bb.y);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[c_slot]));  // this warp is done with the stage
      if (++c_slot == STAGES) {
        c_slot = 0;
        c_phase ^= 1u;
      }
      if (lane0) produce(c + STAGES - 1);
    }
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int e = 0; e < 2; ++e)
        sm.wblk[fr][n_lo + 2 * (2 * fk + e) + t] =
            w0[t][e] - ((acc[t][0][e] + acc[t][1][e]) + (acc[t][2][e] + acc[t][3][e]));
    bar_all();  // block b+1 handed over
  }
}

int sweep_error_read_clear() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_sweep_error, sizeof(int)) != cudaSuccess) return -1;
  if (v) {
    int z = 0;
    cudaMemcpyToSymbol(g_sweep_error, &z, sizeof(int));
  }
  return v;
}

// ---------------------------------------------------------------------------
// Dynamic-grid variant of the sweep (the grid of a column group is searched when
// the sweep arrives at the group, from the group's current values).  Right-looking,
// one column group at a time on a contiguous working copy Wk [M][d] of the step's
// rows: k_grid_tri on the group's current values, this kernel for the group's
// columns (Algorithm 2's column loop restricted to the group: one warp per row, a
// lane per column of each 32-column sub-block, values in registers), then one GEMM
// that applies the group's errors (and, with R, its arrival values) to all later
// columns.  The group's errors only live until that GEMM has run.
// ---------------------------------------------------------------------------
struct GroupPanelP {
  double* Wk;            // [M][d] working values of the step's rows
  const float* U;        // [n_hin][d][d]
  const float* P;        // or nullptr
  double* Err;           // [M][seg] normalised errors of this group
  double* Arr;           // [M][seg] arrival values of this group (with P)
  unsigned char* codes;  // [d_out][d]
  const double* sD;      // [d_out][ng]
  const int* z;          // [d_out][ng]
  tb_stats* stats;
  RowMap rm;
  int M, d, seg, ng, maxq, grp;
  int units, rows_per_unit, ctas_per_unit;
};

__global__ void __launch_bounds__(256) k_group_panel(GroupPanelP p) {
  extern __shared__ float gp_sm[];   // U[c0 + j][c0 + c] at gp_sm[j * seg + c], then P likewise
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = p.seg, d = p.d, c0 = p.grp * seg, nsb = seg / 32;
  // a CTA takes 8 rows of one unit (rows that share an H_in / U_in); the last CTA of a unit may hold fewer
  const int unit = blockIdx.x / p.ctas_per_unit;
  const int m0 = unit * p.rows_per_unit + (blockIdx.x % p.ctas_per_unit) * 8;
  const long long uoff = (p.units > 1) ? (long long)unit * d * d : 0;
  const float* U = p.U + uoff;
  const float* Pm = p.P ? p.P + uoff : nullptr;
  float* sU = gp_sm;
  float* sP = gp_sm + seg * seg;
  for (int i = tid; i < seg * seg; i += blockDim.x) {
    const int j = i / seg, c = i % seg;
    sU[i] = (c >= j) ? U[(long long)(c0 + j) * d + c0 + c] : 0.0f;
    if (Pm) sP[i] = (c > j) ? Pm[(long long)(c0 + j) * d + c0 + c] : 0.0f;
  }
  __syncthreads();
  const int m = m0 + warp;
  if (m >= (unit + 1) * p.rows_per_unit) return;
  const long long grow = p.rm.row(m);
  const double s = p.sD[grow * p.ng + p.grp];
  const double zz = (double)p.z[grow * p.ng + p.grp];
  const double maxq = (double)p.maxq;
  double* wrow = p.Wk + (long long)m * d + c0;
  double v[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
  for (int t = 0; t < 4; ++t)
    if (t < nsb) v[t] = wrow[t * 32 + lane];
  unsigned int n_near = 0, n_clamp = 0;
  for (int j = 0; j < seg; ++j) {
    const int tj = j >> 5, lj = j & 31;
    const double mine = (tj == 0) ? v[0] : (tj == 1) ? v[1] : (tj == 2) ? v[2] : v[3];
    const double wj = shfl_d(mine, lj);   // value of column j on arrival
    const double x = wj / s + zz;
    const double q = fmin(fmax(rne(x), 0.0), maxq);
    const double ej = (wj - s * (q - zz)) / (double)sU[j * seg + j];
    if (lane == lj) {
      p.codes[grow * d + c0 + j] = (unsigned char)(int)q;
      p.Err[(long long)m * seg + j] = ej;
      if (Pm) p.Arr[(long long)m * seg + j] = wj;
      const double fl = floor(x);
      const double a0 = fmin(fmax(fl, 0.0), maxq), a1 = fmin(fmax(fl + 1.0, 0.0), maxq);
      if (fabs(x - (fl + 0.5)) < 1e-6 && a0 != a1) ++n_near;
      if (rne(x) != q) ++n_clamp;
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int c = t * 32 + lane;
      if (t < nsb && c > j) {
        double nv = fma(-ej, (double)sU[j * seg + c], v[t]);
        if (Pm) nv = fma(-wj, (double)sP[j * seg + c], nv);
        v[t] = nv;
      }
    }
  }
  if (p.stats) {
    n_near = __reduce_add_sync(0xffffffffu, n_near);
    n_clamp = __reduce_add_sync(0xffffffffu, n_clamp);
    if (lane == 0) {
      if (n_near) atomicAdd(&p.stats->near_tie_codes, (unsigned long long)n_near);
      if (n_clamp) atomicAdd(&p.stats->clamped_codes, (unsigned long long)n_clamp);
      if (m == 0) atomicAdd(&p.stats->column_steps, (unsigned long long)seg);
    }
  }
}

// E[m][k] = W~[row(m)][k] - s (code - z): the quantization error of the group on
// the weights it saw (Proposition 3.1's W_B - Q_B).
__global__ void k_residual(const double* __restrict__ Wt, const unsigned char* __restrict__ codes,
                           const double* __restrict__ sD, const int* __restrict__ z,
                           double* __restrict__ E, RowMap rm, int M, int d, int seg, int ng) {
  const long long n = (long long)M * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / d), k = (int)(i % d);
    const long long r = rm.row(m);
    const long long so = r * ng + k / seg;
    const double q = (double)codes[r * d + k] - (double)z[so];
    E[i] = Wt[r * d + k] - sD[so] * q;
  }
}

// ---------------------------------------------------------------------------
// Coordinate descent on the scales (Proposition 3.3 / Algorithm 3), with the
// codes frozen.  Wbar = W_int - z.  State kept current through the pass:
//   Dm = (Q - W) H_in + W R      [rows][d]
// and, so that a scale step costs no product with H_in,
//   Yw[r][g2][:] = Wbar[r, G_g2] H_in[G_g2, :]      (one row of products per scale)
// A step on scale (j, g2) by delta adds delta * Yw[j][g2][:] to row j of Dm.
// Rows of a head are visited in order (Gauss-Seidel); per row:
//   k_cd_row_stats : n0[g]  = <Wbar[j,G_g], (H_out Dm)[j,G_g]>
//                    A[g2][g] = <Yw[j][g2][G_g], Wbar[j,G_g]>   (A[g][g] is the denominator's
//                                                                Wbar H_in[G,G] Wbar^T)
//   k_cd_row_update: the scalar chain over the row's groups,
//                    delta_g2 = -num_g2 / (A[g2][g2] H_out[j][j]),  num_g += H_out[j][j] delta_g2 A[g2][g],
//                    then Dm[j,:] += sum_g2 delta_g2 Yw[j][g2][:] and s += delta.
// ---------------------------------------------------------------------------
__global__ void k_cd_prep(const float* __restrict__ W, const unsigned char* __restrict__ codes,
                          const double* __restrict__ sD, const int* __restrict__ z,
                          double* __restrict__ Dq, float* __restrict__ Wb, long long rows, int d,
                          int seg, int ng) {
  const long long n = rows * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / d;
    const int k = (int)(i % d);
    const long long so = r * ng + k / seg;
    const double wb = (double)codes[i] - (double)z[so];
    if (Wb) Wb[i] = (float)wb;
    Dq[i] = sD[so] * wb - (double)W[i];
  }
}

struct CdP {
  double* Dm;           // [rows][d]            (rows of this batch)
  const void* Yw;       // [rows][ng][d], element type TY of the kernel
  const float* Wb;      // [rows][d]
  const float* Hout;    // [heads][dh][dh] of this batch, or nullptr
  double* sD;           // [rows][ng]
  double* n0;           // [lines][ng]
  double* Amat;         // [lines][ng][ng]
  int d, seg, ng, dh, j0, lines_per_head;  // lines_per_head = 1 (row j0 of each head) or dh
  int groups_per_cta;
  int a_in_smem;
};

// line = head * lines_per_head + l; its row inside the head is j0 + l.
// Partial sums are kept per 32-column chunk and added in chunk order, so the
// result does not depend on warp scheduling.
template <typename TY>
__global__ void __launch_bounds__(256) k_cd_row_stats(CdP p) {
  extern __shared__ double cd_sm[];  // part[chunks][ng + 1], then hrow[dh]
  const int tid = threadIdx.x, lane = tid & 31;
  const int line = blockIdx.y, head = line / p.lines_per_head, j = p.j0 + line % p.lines_per_head;
  const int d = p.d, seg = p.seg, ng = p.ng, dh = p.dh;
  const int g_first = blockIdx.x * p.groups_per_cta;
  const int g_count = min(p.groups_per_cta, ng - g_first);
  const int c_first = g_first * seg, c_count = g_count * seg;
  const int chunks_per_group = seg / 32;
  const int max_chunks = p.groups_per_cta * chunks_per_group;
  const long long row = (long long)head * dh + j;
  double* part = cd_sm;                           // [max_chunks][ng + 1]
  double* hrow = cd_sm + (size_t)max_chunks * (ng + 1);  // [dh]
  if (p.Hout)
    for (int i = tid; i < dh; i += blockDim.x) hrow[i] = (double)p.Hout[((long long)head * dh + j) * dh + i];
  __syncthreads();
  const double* Dh = p.Dm + (long long)head * dh * d;
  const TY* Yr = static_cast<const TY*>(p.Yw) + row * ng * d;
  const float* wbr = p.Wb + row * d;
  // every warp walks 32 consecutive columns at a time; they lie in one group
  for (int cb = (tid >> 5) * 32; cb < c_count; cb += (blockDim.x >> 5) * 32) {
    const int col = c_first + cb + lane;
    const int chunk = cb / 32;
    const int g = g_first + cb / seg;
    const double wb = (double)wbr[col];
    double gj;
    if (p.Hout) {
      gj = 0.0;
      for (int i = 0; i < dh; ++i) gj = fma(hrow[i], Dh[(long long)i * d + col], gj);
    } else {
      gj = Dh[(long long)j * d + col];
    }
    const double v = warp_sum(wb * gj);
    if (lane == 0) part[chunk * (ng + 1) + ng] = v;
    for (int g2 = 0; g2 <= g; ++g2) {
      const double a = warp_sum((double)Yr[(long long)g2 * d + col] * wb);
      if (lane == 0) part[chunk * (ng + 1) + g2] = a;
    }
  }
  __syncthreads();
  for (int i = tid; i < g_count * (ng + 1); i += blockDim.x) {
    const int gl = i / (ng + 1), g2 = i % (ng + 1), g = g_first + gl;
    if (g2 != ng && g2 > g) continue;
    double t = 0.0;
    for (int c = 0; c < chunks_per_group; ++c) t += part[(gl * chunks_per_group + c) * (ng + 1) + g2];
    if (g2 == ng)
      p.n0[(long long)line * ng + g] = t;
    else
      p.Amat[((long long)line * ng + g2) * ng + g] = t;
  }
}

template <typename TY>
__global__ void __launch_bounds__(256) k_cd_row_update(CdP p) {
  extern __shared__ double cd_sm[];  // num[ng], delta[ng], then A[ng][ng] if it fits
  const int tid = threadIdx.x, lane = tid & 31;
  const int line = blockIdx.y, head = line / p.lines_per_head, j = p.j0 + line % p.lines_per_head;
  const int d = p.d, seg = p.seg, ng = p.ng, dh = p.dh;
  const long long row = (long long)head * dh + j;
  double* num = cd_sm;
  double* delta = cd_sm + ng;
  const double hjj = p.Hout ? (double)p.Hout[((long long)head * dh + j) * dh + j] : 1.0;
  const double* A = p.Amat + (long long)line * ng * ng;
  for (int g = tid; g < ng; g += blockDim.x) num[g] = p.n0[(long long)line * ng + g];
  if (p.a_in_smem) {
    double* As = cd_sm + 2 * ng;
    for (int i = tid; i < ng * ng; i += blockDim.x) {
      const int g2 = i / ng, g = i % ng;
      As[i] = (g >= g2) ? A[i] : 0.0;
    }
    A = As;
  }
  __syncthreads();
  if (tid < 32) {
    for (int g2 = 0; g2 < ng; ++g2) {
      const double den = A[(long long)g2 * ng + g2] * hjj;
      const double dl = (den == 0.0) ? 0.0 : -num[g2] / den;
      if (lane == 0) delta[g2] = dl;
      for (int g = g2 + 1 + lane; g < ng; g += 32) num[g] = fma(hjj * dl, A[(long long)g2 * ng + g], num[g]);
      __syncwarp();
    }
  }
  __syncthreads();
  const int g_first = blockIdx.x * p.groups_per_cta;
  const int g_count = min(p.groups_per_cta, ng - g_first);
  const int c_first = g_first * seg, c_count = g_count * seg;
  const TY* Yr = static_cast<const TY*>(p.Yw) + row * ng * d;
  double* dm = p.Dm + row * d;
  for (int c = tid; c < c_count; c += blockDim.x) {
    const int col = c_first + c;
    double acc = dm[col];
    for (int g2 = 0; g2 < ng; ++g2) acc = fma(delta[g2], (double)Yr[(long long)g2 * d + col], acc);
    dm[col] = acc;
  }
  if (blockIdx.x == 0)
    for (int g = tid; g < ng; g += blockDim.x) p.sD[row * ng + g] += delta[g];
}

// ---------------------------------------------------------------------------
// One Gauss-Seidel pass of Algorithm 3 over ALL rows of one head in a single
// launch.  A thread-block cluster of C CTAs owns a head; CTA r owns the column
// groups r ng/C .. (r+1) ng/C - 1 (whole groups, so every sum over a group is
// local to one CTA).  The cluster walks the head's rows in order and works on
//   G = H_out Dm    (rows of the head, formed once by a batched GEMM),
// whose row j is what the numerator of Proposition 3.3 needs.  A step on the
// scales of row i adds u_i = sum_g2 delta_g2 Yw[i][g2][:] to row i of Dm, hence
// H_out[j][i] u_i to every row j of G.  Those rank-1 terms are applied lazily:
// rows of the current block of 16 read the u_i of their block on the fly, and
// when a block is finished its 16 vectors are folded into the rows of G that
// are still to come.  Per row, each CTA forms n0[g] and A[.][g] for its groups,
// stores them into the shared memory of every CTA of the cluster (distributed
// shared memory, two buffers by row parity), and after one cluster barrier every
// CTA runs the short scalar chain itself.  The u_i are kept (Uacc) so that Dm
// can be refreshed after the pass.  All sums have a fixed order.
// ---------------------------------------------------------------------------
enum { CDH_THREADS = 512, CDH_BLOCK = 16 };
struct CdHeadP {
  double* G;           // [heads*dh][d]   H_out Dm, updated in place
  double* Uacc;        // [heads*dh][d]   out: the rank-1 vectors u_i
  const void* Yw;      // [heads*dh][ng][d], element type TY of the kernel
  const float* Wb;     // [heads*dh][d]
  const float* Hout;   // [heads][dh][dh]
  double* sD;          // [heads*dh][ng]
  int d, seg, ng, dh;
  int csize;           // CTAs per cluster (divides ng)
  int uw;              // columns per work unit (a divisor of seg, multiple of 32, at most 128)
};

template <typename TY>
__global__ void __launch_bounds__(CDH_THREADS, 1) k_cd_head(CdHeadP p) {
  extern __shared__ double cdh_sm[];
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / p.csize;
  const int d = p.d, seg = p.seg, ng = p.ng, dh = p.dh, uw = p.uw;
  const int gpc = ng / p.csize;                 // groups of this CTA
  const int g_lo = rank * gpc;
  const int upg = seg / uw;                     // units per group
  const int n_units = gpc * upg;                // units of this CTA
  const int c_lo = g_lo * seg, c_cnt = gpc * seg;  // its columns
  double* part = cdh_sm;                                   // [n_units][ng + 1]
  double* Am = part + (size_t)n_units * (ng + 1);          // [2][ng][ng]  (entries g2 <= g)
  double* num = Am + (size_t)2 * ng * ng;                  // [2][ng]
  double* delta = num + 2 * ng;                            // [ng]
  const long long row0 = (long long)head * dh;
  const float* Ho = p.Hout + (long long)head * dh * dh;

  for (int j = 0; j < dh; ++j) {
    const long long row = row0 + j;
    const int buf = j & 1;
    const int blk0 = (j / CDH_BLOCK) * CDH_BLOCK;
    const double hjj = (double)Ho[(long long)j * dh + j];
    const TY* Yr = static_cast<const TY*>(p.Yw) + row * ng * d;
    const float* wbr = p.Wb + row * d;
    const double* Gr = p.G + row * d;
    const float* hrow = Ho + (long long)j * dh;
    // ---- statistics of the row for this CTA's groups: n0[g] and A[g2][g], g2 <= g ----
    for (int u = warp; u < n_units; u += CDH_THREADS / 32) {
      const int g = g_lo + u / upg;
      const int cbase = g * seg + (u % upg) * uw;
      double wb[4], gv[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = cbase + lane + 32 * c;
        const bool on = lane + 32 * c < uw;
        wb[c] = on ? (double)wbr[col] : 0.0;
        gv[c] = on ? Gr[col] : 0.0;
      }
      for (int i = blk0; i < j; ++i) {
        const double h = (double)hrow[i];
        const double* ui = p.Uacc + (row0 + i) * d + cbase + lane;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (lane + 32 * c < uw) gv[c] = fma(h, ui[32 * c], gv[c]);
      }
      double v = 0.0;
#pragma unroll
      for (int c = 0; c < 4; ++c) v = fma(wb[c], gv[c], v);
      v = warp_sum(v);
      if (lane == 0) part[(size_t)u * (ng + 1) + ng] = v;
      const TY* yb = Yr + cbase + lane;
      int g2 = 0;
      for (; g2 + 4 <= g + 1; g2 += 4) {
        double a4[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (lane + 32 * c < uw) a4[t] = fma((double)yb[(long long)(g2 + t) * d + 32 * c], wb[c], a4[t]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int t = 0; t < 4; ++t) a4[t] += __shfl_xor_sync(0xffffffffu, a4[t], o);
        if (lane < 4) part[(size_t)u * (ng + 1) + g2 + lane] = (lane == 0) ? a4[0] : (lane == 1) ? a4[1] : (lane == 2) ? a4[2] : a4[3];
      }
      for (; g2 <= g; ++g2) {
        double a = 0.0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (lane + 32 * c < uw) a = fma((double)yb[(long long)g2 * d + 32 * c], wb[c], a);
        a = warp_sum(a);
        if (lane == 0) part[(size_t)u * (ng + 1) + g2] = a;
      }
    }
    __syncthreads();
    // ---- reduce the units of each group in order and publish to every CTA of the cluster ----
    for (int idx = tid; idx < gpc * (ng + 1); idx += CDH_THREADS) {
      const int gl = idx / (ng + 1), g2 = idx % (ng + 1), g = g_lo + gl;
      if (g2 != ng && g2 > g) continue;
      double t = 0.0;
      for (int c = 0; c < upg; ++c) t += part[(size_t)(gl * upg + c) * (ng + 1) + g2];
      for (int r = 0; r < p.csize; ++r) {
        if (g2 == ng)
          cluster.map_shared_rank(num, r)[buf * ng + g] = t;
        else
          cluster.map_shared_rank(Am, r)[((size_t)buf * ng + g2) * ng + g] = t;
      }
    }
    cluster.sync();
    // ---- the scalar chain over the row's groups (every CTA runs it) ----
    if (warp == 0) {
      double* nm = num + buf * ng;
      const double* A = Am + (size_t)buf * ng * ng;
      for (int g2 = 0; g2 < ng; ++g2) {
        const double den = A[(size_t)g2 * ng + g2] * hjj;
        const double dl = (den == 0.0) ? 0.0 : -nm[g2] / den;
        if (lane == 0) delta[g2] = dl;
        for (int g = g2 + 1 + lane; g < ng; g += 32) nm[g] = fma(hjj * dl, A[(size_t)g2 * ng + g], nm[g]);
        __syncwarp();
      }
    }
    __syncthreads();
    // ---- u_j on this CTA's columns, and the scales ----
    double* ur = p.Uacc + row * d;
    for (int c0 = tid; c0 < c_cnt; c0 += 4 * CDH_THREADS) {
      double acc[4] = {0.0, 0.0, 0.0, 0.0};
      for (int g2 = 0; g2 < ng; ++g2) {
        const double dl = delta[g2];
        const TY* y = Yr + (long long)g2 * d + c_lo + c0;
#pragma unroll
        for (int t = 0; t < 4; ++t)
          if (c0 + t * CDH_THREADS < c_cnt) acc[t] = fma(dl, (double)y[t * CDH_THREADS], acc[t]);
      }
#pragma unroll
      for (int t = 0; t < 4; ++t)
        if (c0 + t * CDH_THREADS < c_cnt) ur[c_lo + c0 + t * CDH_THREADS] = acc[t];
    }
    if (rank == 0)
      for (int g = tid; g < ng; g += CDH_THREADS) p.sD[row * ng + g] += delta[g];
    __syncthreads();
    // ---- end of a block: fold its vectors into the rows of G still to come ----
    if ((j + 1) % CDH_BLOCK == 0 && j + 1 < dh) {
      for (int c = tid; c < c_cnt; c += CDH_THREADS) {
        const int col = c_lo + c;
        double u16[CDH_BLOCK];
#pragma unroll
        for (int i = 0; i < CDH_BLOCK; ++i) u16[i] = p.Uacc[(row0 + blk0 + i) * d + col];
        for (int jj = j + 1; jj < dh; ++jj) {
          const float* hr = Ho + (long long)jj * dh + blk0;
          double gvv = p.G[(row0 + jj) * d + col];
#pragma unroll
          for (int i = 0; i < CDH_BLOCK; ++i) gvv = fma((double)hr[i], u16[i], gvv);
          p.G[(row0 + jj) * d + col] = gvv;
        }
      }
      __syncthreads();
    }
  }
  cluster.sync();  // no CTA may exit while another can still store into its shared memory
}

// ---------------------------------------------------------------------------
// Column-parallel form of the same pass, for up to 32 groups and at most 1024
// columns per CTA.  The quadratic forms A[g2][g] = Wbar_g2^T H_in[g2, g] Wbar_g
// of a row depend on the integers only, so k_cd_amat forms them for every row
// up front, in parallel.  In the walk, thread t owns columns 2t, 2t+1 of its
// CTA for the whole pass: the u_i of the current block of 16 rows stay in its
// registers, the lazily corrected row of G is formed there, and one row costs
// two block barriers, one cluster barrier and a 32-step chain run in registers
// by warp 0 of every CTA.  What the next row needs (its row of G, Wbar, A and
// H_out) is fetched while the current row is processed, and the next row's
// slice of Yw is pulled into L2.
// ---------------------------------------------------------------------------
template <typename TY>
__global__ void __launch_bounds__(256) k_cd_amat(const void* __restrict__ Yw_, const float* __restrict__ Wb,
                                                 double* __restrict__ Amat, int d, int seg, int ng) {
  extern __shared__ float amat_wb[];
  const long long row = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int c = tid; c < d; c += 256) amat_wb[c] = Wb[row * d + c];
  __syncthreads();
  const TY* Yr = static_cast<const TY*>(Yw_) + row * ng * d;
  double* A = Amat + row * ng * ng;
  for (int g2 = 0; g2 < ng; ++g2)
    for (int g = g2 + warp; g < ng; g += 8) {
      const TY* y = Yr + (long long)g2 * d + g * seg;
      const float* w = amat_wb + g * seg;
      double v = 0.0;
      for (int c = lane; c < seg; c += 32) v = fma((double)y[c], (double)w[c], v);
      v = warp_sum(v);
      if (lane == 0) A[g2 * ng + g] = v;
    }
}

enum { CDC_THREADS = 512, CDC_MAXG = 32 };
__device__ __forceinline__ double2 load_pair(const float* q) {
  const float2 v = *reinterpret_cast<const float2*>(q);
  return make_double2((double)v.x, (double)v.y);
}
__device__ __forceinline__ double2 load_pair(const double* q) { return *reinterpret_cast<const double2*>(q); }
struct CdColP {
  double* G;           // [heads*dh][d]   H_out Dm, rows still to come updated in place at block ends
  double* Uacc;        // [heads*dh][d]   out: the rank-1 vectors u_i
  const void* Yw;      // [heads*dh][ng][d], element type TY of the kernel
  const float* Wb;     // [heads*dh][d]
  const float* Hout;   // [heads][dh][dh]
  const double* Amat;  // [heads*dh][ng][ng], entries g2 <= g
  double* sD;          // [heads*dh][ng]
  int d, seg, ng, dh;
  int csize;           // CTAs per cluster (divides ng)
};

template <typename TY>
__global__ void __launch_bounds__(CDC_THREADS, 1) k_cd_head_cols(CdColP p) {
  __shared__ double part[CDC_THREADS];
  __shared__ double Am[2][CDC_MAXG * CDC_MAXG];
  __shared__ double num[2][CDC_MAXG];
  __shared__ double delta[CDC_MAXG];
  __shared__ float hs[2][CDH_BLOCK];
  __shared__ float hd[2];
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / p.csize;
  const int d = p.d, seg = p.seg, ng = p.ng, dh = p.dh;
  const int gpc = ng / p.csize, g_lo = rank * gpc;
  const int c_lo = g_lo * seg, c_cnt = gpc * seg;
  const int c0 = 2 * tid;
  const bool on = c0 < c_cnt;
  const int col = c_lo + c0;
  const long long row0 = (long long)head * dh;
  const float* Ho = p.Hout + (long long)head * dh * dh;
  const TY* Yw = static_cast<const TY*>(p.Yw);
  const int a_cnt = ng * ng;
  const int half = seg / 2;  // partial sums per group
  const size_t slab_lines = ((size_t)c_cnt * sizeof(TY) + 127) / 128;

  // what row 0 needs
  double2 gn = make_double2(0.0, 0.0);
  float2 wn = make_float2(0.0f, 0.0f);
  double an0 = 0.0, an1 = 0.0;
  if (on) {
    gn = *reinterpret_cast<const double2*>(p.G + row0 * d + col);
    wn = *reinterpret_cast<const float2*>(p.Wb + row0 * d + col);
  }
  if (tid < a_cnt) an0 = p.Amat[row0 * a_cnt + tid];
  if (tid + CDC_THREADS < a_cnt) an1 = p.Amat[row0 * a_cnt + tid + CDC_THREADS];
  double sdn = (rank == 0 && tid < ng) ? p.sD[row0 * ng + tid] : 0.0;  // the row's scales, fetched one row ahead
  // hs[.][k] multiplies ureg[k]; the vectors move down one slot per row, so slot k of row j
  // holds u of row j - 16 + k (zero while that row lies before the block)
  if (tid < CDH_BLOCK) hs[0][tid] = 0.0f;
  if (tid == CDH_BLOCK) hd[0] = Ho[0];
  __syncthreads();

  double2 ureg[CDH_BLOCK];
#pragma unroll
  for (int i = 0; i < CDH_BLOCK; ++i) ureg[i] = make_double2(0.0, 0.0);
#pragma unroll 1
  for (int j = 0; j < dh; ++j) {
    const long long row = row0 + j;
    const int buf = j & 1;
    double2 gv = gn;
    const float2 w = wn;
    const double sd_cur = sdn;
    if (tid < a_cnt) Am[buf][tid] = an0;
    if (tid + CDC_THREADS < a_cnt) Am[buf][tid + CDC_THREADS] = an1;
    // ---- fetch for row j + 1 ----
    if (j + 1 < dh) {
      const long long rn = row + 1;
      if (on) {
        gn = *reinterpret_cast<const double2*>(p.G + rn * d + col);
        wn = *reinterpret_cast<const float2*>(p.Wb + rn * d + col);
      }
      if (tid < a_cnt) an0 = p.Amat[rn * a_cnt + tid];
      if (tid + CDC_THREADS < a_cnt) an1 = p.Amat[rn * a_cnt + tid + CDC_THREADS];
      if (rank == 0 && tid < ng) sdn = p.sD[rn * ng + tid];
      const int blkn = ((j + 1) / CDH_BLOCK) * CDH_BLOCK;
      if (tid < CDH_BLOCK) {
        const int ci = j + 1 - CDH_BLOCK + tid;
        hs[buf ^ 1][tid] = (ci >= blkn && ci <= j) ? Ho[(long long)(j + 1) * dh + ci] : 0.0f;
      }
      if (tid == CDH_BLOCK) hd[buf ^ 1] = Ho[(long long)(j + 1) * dh + j + 1];
      for (size_t idx = tid; idx < slab_lines * ng; idx += CDC_THREADS) {
        const size_t g2 = idx / slab_lines, l = idx % slab_lines;
        const char* ptr = reinterpret_cast<const char*>(Yw + (rn * ng + (long long)g2) * d + c_lo) + l * 128;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
      }
    }
    // ---- numerators of this CTA's groups: Wbar . (G + pending rank-1 terms of the block) ----
#pragma unroll
    for (int i = 0; i < CDH_BLOCK; ++i) {
      const double h = (double)hs[buf][i];
      gv.x = fma(h, ureg[i].x, gv.x);
      gv.y = fma(h, ureg[i].y, gv.y);
    }
    part[tid] = on ? fma((double)w.y, gv.y, (double)w.x * gv.x) : 0.0;
    const double hjj = (double)hd[buf];
    __syncthreads();
    for (int gl = warp; gl < gpc; gl += CDC_THREADS / 32) {
      double v = 0.0;
      for (int k = lane; k < half; k += 32) v += part[gl * half + k];
      v = warp_sum(v);
      if (lane == 0)
        for (int r = 0; r < p.csize; ++r) cluster.map_shared_rank(&num[0][0], r)[buf * CDC_MAXG + g_lo + gl] = v;
    }
    cluster.sync();
    // ---- the scalar chain over the row's groups, lane g holding num[g] (every CTA runs it) ----
    if (warp == 0) {
      // delta_g2 = -num[g2] / (A[g2][g2] hjj); num[g] += hjj delta_g2 A[g2][g] for g > g2.  Only num is
      // carried from step to step: the factor -A[g2][g] / A[g2][g2] of lane g is formed beside the
      // chain, which is then one shuffle and one multiply-add per step.
      const bool in = lane < ng;
      double nm = in ? num[buf][lane] : 0.0;
      const double den = in ? Am[buf][lane * ng + lane] * hjj : 0.0;
      const double rinv = (den == 0.0) ? 0.0 : 1.0 / den;   // 1 / (A[g][g] hjj)
      const double ratio = -hjj * rinv;                     // -1 / A[g][g], or 0 for a skipped coordinate
      double mine = 0.0;
#pragma unroll 4
      for (int g2 = 0; g2 < ng; ++g2) {
        const double k = __shfl_sync(0xffffffffu, ratio, g2) * ((in && lane > g2) ? Am[buf][g2 * ng + lane] : 0.0);
        const double n2 = __shfl_sync(0xffffffffu, nm, g2);
        if (lane == g2) mine = -n2 * rinv;
        nm = fma(n2, k, nm);
      }
      if (in) {
        delta[lane] = mine;
        if (rank == 0) p.sD[row * ng + lane] = sd_cur + mine;
      }
    }
    __syncthreads();
    // ---- u_j on this thread's columns ----
    double2 u = make_double2(0.0, 0.0);
    if (on) {
      const TY* y = Yw + row * ng * d + col;
#pragma unroll 8
      for (int g2 = 0; g2 < ng; ++g2) {
        const double dl = delta[g2];
        const double2 yv = load_pair(y + (long long)g2 * d);
        u.x = fma(dl, yv.x, u.x);
        u.y = fma(dl, yv.y, u.y);
      }
      *reinterpret_cast<double2*>(p.Uacc + row * d + col) = u;
    }
#pragma unroll
    for (int i = 0; i + 1 < CDH_BLOCK; ++i) ureg[i] = ureg[i + 1];
    ureg[CDH_BLOCK - 1] = u;
    // ---- end of a block: fold its vectors into the rows of G still to come ----
    if ((j + 1) % CDH_BLOCK == 0 && j + 1 < dh) {
      const int blk0 = j + 1 - CDH_BLOCK;
      if (on) {
#pragma unroll 2
        for (int jj = j + 1; jj < dh; ++jj) {
          const float* hr = Ho + (long long)jj * dh + blk0;
          double2 g = *reinterpret_cast<const double2*>(p.G + (row0 + jj) * d + col);
#pragma unroll
          for (int i = 0; i < CDH_BLOCK; ++i) {
            const double h = (double)__ldg(hr + i);
            g.x = fma(h, ureg[i].x, g.x);
            g.y = fma(h, ureg[i].y, g.y);
          }
          *reinterpret_cast<double2*>(p.G + (row0 + jj) * d + col) = g;
          if (jj == j + 1) gn = g;
        }
      }
#pragma unroll
      for (int i = 0; i < CDH_BLOCK; ++i) ureg[i] = make_double2(0.0, 0.0);
    }
  }
  cluster.sync();  // no CTA may exit while another can still store into its shared memory
}

// Dm += Uacc (the effect of one pass on (Q - W) H_in + W R)
__global__ void k_axpy(double* __restrict__ y, const double* __restrict__ x, long long n) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x)
    y[i] += x[i];
}

// Q = s (W_int - z) in float, and the scales in float (Algorithm 1, final step).
__global__ void k_dequant(const unsigned char* __restrict__ codes, const double* __restrict__ sD,
                          const int* __restrict__ z, float* __restrict__ What,
                          float* __restrict__ s_out, long long rows, int d, int seg, int ng) {
  const long long n = rows * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / d;
    const int k = (int)(i % d);
    const long long so = r * ng + k / seg;
    if (What) What[i] = (float)(sD[so] * ((double)codes[i] - (double)z[so]));
    if (k % seg == 0) s_out[so] = (float)sD[so];
  }
}

// loss[h] = sum over the head's rows of <Z[r,:], dW[r,:]> (Z already multiplied by H_out when there
// is one: tr(H_out Z dW^T) = sum of (H_out Z) .* dW), in two steps with a fixed order: one partial
// sum per block of 32 rows, then the partial sums of a head.
__global__ void __launch_bounds__(256) k_loss_identity_partial(const double* __restrict__ Z,
                                                               const double* __restrict__ Dq,
                                                               double* __restrict__ partial,
                                                               long long rows_per_head, int d, int chunks) {
  __shared__ double part[8];
  const int h = blockIdx.y, c = blockIdx.x;
  const long long r0 = (long long)c * 32, r1 = (r0 + 32 < rows_per_head) ? r0 + 32 : rows_per_head;
  const long long base = ((long long)h * rows_per_head + r0) * d, n = (r1 - r0) * d;
  double acc = 0.0;
  for (long long i = threadIdx.x; i < n; i += blockDim.x) acc = fma(Z[base + i], Dq[base + i], acc);
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < 8; ++i) t += part[i];
    partial[(long long)h * chunks + c] = t;
  }
}
__global__ void k_loss_identity_final(const double* __restrict__ partial, double* __restrict__ loss, int chunks) {
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int c = 0; c < chunks; ++c) t += partial[(long long)blockIdx.x * chunks + c];
    loss[blockIdx.x] = t;
  }
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
struct Plan {
  int d_out, d, H, dh, n_hin, bits, seg, ng, g, S, maxq, n_cand, ncp, rt, cd_iters;
  bool adaptive, dynamic, cd, with_r, with_loss, has_hout;
  double *dynErr, *dynArr;  // [Mmax][seg] errors / arrival values of the current column group (dynamic grid)
  int Mmax;
  long long cd_rows;  // rows per coordinate-descent batch
  // workspace
  double *Wt, *Wk, *W0c, *E, *sD, *T, *Dq, *Dm, *Yw, *n0, *Amat, *G2;
  float* Wb;
  __nv_bfloat16 *WbT, *Hp;  // tensor-core path of the blockwise product
  bool yw_tensor;
  bool dm_tensor;  // (Q - W) H_in through the split-bf16 tensor-core product as well
  bool loss_tensor;  // the loss's own dW H_in (no scale refinement) through it too
  int loss_heads;    // with one H_in per head: heads per launch of that product (their pieces of H_in fit 2 GiB)
  size_t ws_total;
};

static int pow2_ceil(int v) {
  int p = 1;
  while (p < v) p <<= 1;
  return p;
}

static tb_status make_plan(const tb_layer_desc* D, bool has_hout, bool with_r, bool with_loss,
                           void* ws, Plan* pl) {
  if (!D) return TB_ERR_INVALID_ARG;
  if (D->d_out <= 0 || D->d_in <= 0 || D->n_heads <= 0 || D->d_head <= 0) return TB_ERR_INVALID_ARG;
  if ((long long)D->n_heads * D->d_head != D->d_out) return TB_ERR_INVALID_ARG;
  if (D->d_in % 128) return TB_ERR_UNSUPPORTED;
  if (D->n_hin != 1 && D->n_hin != D->n_heads) return TB_ERR_INVALID_ARG;
  if (D->bits < 2 || D->bits > 8) return TB_ERR_INVALID_ARG;
  if (D->quant_group < 0) return TB_ERR_INVALID_ARG;
  if (D->quant_group > 0 && (D->d_in % D->quant_group)) return TB_ERR_INVALID_ARG;
  if (D->quant_group > 0 && (D->quant_group % 32)) return TB_ERR_UNSUPPORTED;
  if (D->out_block < 1 || D->out_block > D->d_head || (D->d_head % D->out_block)) return TB_ERR_INVALID_ARG;
  if (D->n_cand < 1 || D->n_cand > 32) return TB_ERR_INVALID_ARG;
  if (D->cd_iters < 0) return TB_ERR_INVALID_ARG;
  Plan& p = *pl;
  p.d_out = D->d_out;
  p.d = D->d_in;
  p.H = D->n_heads;
  p.dh = D->d_head;
  p.n_hin = D->n_hin;
  p.bits = D->bits;
  p.seg = D->quant_group > 0 ? D->quant_group : D->d_in;
  p.ng = p.d / p.seg;
  p.has_hout = has_hout;
  p.g = has_hout ? D->out_block : D->d_head;  // H_out = I: all rows of a head at once
  p.S = p.dh / p.g;
  p.maxq = (1 << D->bits) - 1;
  p.n_cand = D->n_cand;
  p.ncp = pow2_ceil(D->n_cand);
  p.rt = 128 / p.ncp;
  p.cd_iters = D->cd_iters;
  // dynamic grid: with one group per row it IS the adaptive grid (the group arrives unchanged)
  p.dynamic = (D->flags & TB_F_DYNAMIC_GRID) != 0 && p.ng > 1;
  p.adaptive = (D->flags & TB_F_ADAPTIVE_GRID) != 0 || ((D->flags & TB_F_DYNAMIC_GRID) != 0 && !p.dynamic);
  if (p.dynamic && p.seg > 128) return TB_ERR_UNSUPPORTED;
  p.cd = (D->flags & TB_F_CD_REFINE) != 0 && D->cd_iters > 0;
  p.with_r = with_r;
  p.with_loss = with_loss;
  p.Mmax = p.H * p.g;
  if (p.ng > 1024) return TB_ERR_UNSUPPORTED;

  Bump b(ws);
  const size_t dd = (size_t)p.d;
  p.Wt = b.take<double>((size_t)p.d_out * dd);
  p.Wk = b.take<double>((size_t)p.Mmax * dd);
  p.E = b.take<double>((size_t)p.Mmax * dd);
  p.W0c = with_r ? b.take<double>((size_t)p.Mmax * dd) : nullptr;
  p.sD = b.take<double>((size_t)p.d_out * p.ng);
  p.T = (has_hout && p.S > 1) ? b.take<double>((size_t)p.H * p.S * p.dh * p.g) : nullptr;
  p.dynErr = p.dynamic ? b.take<double>((size_t)p.Mmax * p.seg) : nullptr;
  p.dynArr = (p.dynamic && with_r) ? b.take<double>((size_t)p.Mmax * p.seg) : nullptr;
  p.Dq = p.Dm = p.Yw = p.n0 = p.Amat = p.G2 = nullptr;
  p.Wb = nullptr;
  p.WbT = p.Hp = nullptr;
  p.yw_tensor = p.dm_tensor = false;
  p.cd_rows = 0;
  if (p.cd || with_loss) {
    p.Dq = b.take<double>((size_t)p.d_out * dd);
    p.Dm = b.take<double>((size_t)p.d_out * dd);
  }
  if (p.cd) {
    p.Wb = b.take<float>((size_t)p.d_out * dd);
    // batch of rows whose Yw fits 4 GiB: whole heads when rows of a head are coupled
    const size_t per_row = (size_t)p.ng * dd * sizeof(double);
    const size_t budget = (size_t)4 << 30;
    long long unit_rows = (has_hout || p.n_hin > 1) ? p.dh : 1;
    long long units = (long long)(budget / (per_row * unit_rows));
    if (units < 1) units = 1;
    long long rows = units * unit_rows;
    if (rows > p.d_out) rows = p.d_out;
    if (!(has_hout || p.n_hin > 1) && rows > 128) rows = (rows / 128) * 128;
    p.cd_rows = rows;
    p.Yw = b.take<double>((size_t)rows * p.ng * dd);
    // blockwise product on the tensor cores (float result): one shared H_in, groups that are whole TMA boxes
    // With one H_in per head the heads of a batch go through the same launches, each against its own
    // pieces of H_in; that needs heads of whole 128-row tiles and groups of at most 128 columns.
    const bool per_head_ok = (p.n_hin > 1) && (p.dh % 128 == 0) && (p.seg <= 128) && (rows % p.dh == 0);
    p.yw_tensor = (p.n_hin == 1 || per_head_ok) && (p.seg % 64 == 0) && (rows % 8 == 0) && (p.d_out % 8 == 0) &&
                  (p.dh % 8 == 0 || rows == p.d_out);
    if (p.yw_tensor) {
      p.WbT = b.take<__nv_bfloat16>((size_t)rows * dd);
      p.Hp = b.take<__nv_bfloat16>((size_t)3 * dd * dd * (p.n_hin > 1 ? (size_t)(rows / p.dh) : 1));
      p.dm_tensor = (p.d % 32 == 0);
    }
    const long long lines = rows;  // one set of statistics per row (the column-parallel pass keeps them all)
    p.n0 = b.take<double>((size_t)lines * p.ng);
    p.Amat = b.take<double>((size_t)lines * p.ng * p.ng);
  }
  // without the scale refinement the loss forms dW H_in itself: the same split-bf16 product
  // (with one H_in per head the heads of a batch share the launch, each against its own pieces: that
  // needs heads of whole 128-row tiles)
  p.loss_tensor = with_loss && !p.cd && (p.n_hin == 1 || p.dh % 128 == 0) && (p.d % 32 == 0) && (p.d_out % 8 == 0);
  p.loss_heads = 1;
  if (p.loss_tensor && p.n_hin > 1) {
    const size_t per_head = (size_t)3 * dd * dd * sizeof(__nv_bfloat16);
    size_t fit = ((size_t)2 << 30) / per_head;
    if (fit < 1) fit = 1;
    p.loss_heads = (fit < (size_t)p.H) ? (int)fit : p.H;
  }
  if (p.loss_tensor) p.Hp = b.take<__nv_bfloat16>((size_t)3 * dd * dd * (size_t)p.loss_heads);
  if (with_loss) p.G2 = b.take<double>((size_t)p.H * p.dh * (has_hout ? p.dh : 1));  // Z dW^T, or partial sums
  p.ws_total = b.total();
  return TB_OK;
}

static int ew_blocks(long long n) {
  long long b = (n + 255) / 256;
  if (b > 148 * 16) b = 148 * 16;
  if (b < 1) b = 1;
  return (int)b;
}

static tb_status run_grid(const Plan& p, const float* H_in, float* scales, int* zeros,
                          unsigned char* cand, RowMap rm, int M, cudaStream_t st) {
  GridP gp;
  gp.Wt = p.Wt;
  gp.Hin = H_in;
  gp.sD = p.sD;
  gp.s_out = scales;
  gp.z_out = zeros;
  gp.cand_out = cand;
  gp.rm = rm;
  gp.M = M;
  gp.d = p.d;
  gp.seg = p.seg;
  gp.ng = p.ng;
  gp.maxq = p.maxq;
  gp.n_cand = p.n_cand;
  gp.ncp = p.ncp;
  gp.rt = p.rt;
  gp.units = (p.n_hin == 1) ? 1 : p.H;
  gp.rows_per_unit = M / gp.units;
  gp.tiles_per_unit = (gp.rows_per_unit + p.rt - 1) / p.rt;
  gp.Wloc = nullptr;
  gp.grp0 = 0;
  static bool configured[64] = {false}, configured_tri[64] = {false};
  TB_TRY(allow_smem(k_grid, GemmSmem<double>::bytes, configured));
  TB_TRY(allow_smem(k_grid_tri, GRID_TRI_SMEM, configured_tri));
  const long long ytiles = (long long)gp.units * gp.tiles_per_unit;
  if (ytiles > 65535) return TB_ERR_UNSUPPORTED;
  dim3 grid(p.ng, (unsigned)ytiles);
  if (p.seg <= 128)
    k_grid_tri<<<grid, GEMM_THREADS, GRID_TRI_SMEM, st>>>(gp);
  else
    k_grid<<<grid, GEMM_THREADS, GemmSmem<double>::bytes, st>>>(gp);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

template <bool WITH_P>
static tb_status launch_sweep_rows(const RowSweepP& sp, const CUtensorMap& mu, const CUtensorMap& me,
                                   const CUtensorMap& mp, const CUtensorMap& ma, cudaStream_t st) {
  auto kern = k_sweep_rows<WITH_P>;
  static bool configured[64] = {false};
  TB_TRY(allow_smem(kern, sizeof(RowSweepSmem<WITH_P>), configured));
  const long long ctas = (long long)sp.ctas_per_unit * sp.units * sp.cs;
  if (sp.cs == 1) {
    kern<<<(unsigned)ctas, RS_THREADS, sizeof(RowSweepSmem<WITH_P>), st>>>(sp, mu, me, mp, ma);
    TB_LAUNCH_CHECK();
    return TB_OK;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas);
  cfg.blockDim = dim3(RS_THREADS);
  cfg.dynamicSmemBytes = sizeof(RowSweepSmem<WITH_P>);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)sp.cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  TB_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kern, sp, mu, me, mp, ma));
  TB_LAUNCH_CHECK();
  return TB_OK;
}

static tb_status run_sweep_rows(const Plan& p, const float* U_in, const float* P, unsigned char* codes,
                                const int* zeros, tb_stats* stats, RowMap rm, int M, cudaStream_t st) {
  RowSweepP sp;
  sp.Wt = p.Wt;
  sp.U = U_in;
  sp.P = P;
  sp.ErrG = p.Wk;  // error history of the step's rows
  sp.ArrG = p.E;   // arrival values; E itself is formed after the sweep
  sp.codes = codes;
  sp.sD = p.sD;
  sp.z = zeros;
  sp.stats = stats;
  sp.rm = rm;
  sp.M = M;
  sp.d = p.d;
  sp.seg = p.seg;
  sp.ng = p.ng;
  sp.maxq = p.maxq;
  sp.nblk = p.d / 128;
  sp.units = (p.n_hin == 1) ? 1 : p.H;
  sp.rows_per_unit = M / sp.units;
  sp.ctas_per_unit = (sp.rows_per_unit + 7) / 8;
  // few rows: a cluster of 2 or 4 CTAs per group of 8 rows shares the contraction work of the updates
  const long long groups = (long long)sp.ctas_per_unit * sp.units;
  sp.cs = (p.d >= 256 && groups * 4 <= 148) ? 4 : (p.d >= 256 && groups * 2 <= 148) ? 2 : 1;
  CUtensorMap map_u, map_e, map_p, map_a;
  const unsigned box_full = (unsigned)((p.d >= RS_LDB) ? RS_LDB : p.d);
  const unsigned box_u = (sp.cs > 1) ? (unsigned)(128 / sp.cs + 8) : box_full;
  const unsigned box_e = (sp.cs > 1) ? (unsigned)RS_CLDE : (unsigned)((p.d >= RS_LDE) ? RS_LDE : p.d);
  const unsigned box_k = (sp.cs > 1) ? (unsigned)RS_CCHUNK : (unsigned)RS_CHUNK;
  const unsigned long long mat_rows = (unsigned long long)p.d * sp.units;
  TB_TRY(make_map_2d(&map_u, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sizeof(float), U_in, (unsigned long long)p.d, mat_rows,
                     box_u, box_k, CU_TENSOR_MAP_SWIZZLE_NONE));
  TB_TRY(make_map_2d(&map_e, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, sizeof(double), sp.ErrG, (unsigned long long)p.d,
                     (unsigned long long)M, box_e, 8, CU_TENSOR_MAP_SWIZZLE_NONE));
  if (!P) return launch_sweep_rows<false>(sp, map_u, map_e, map_u, map_e, st);
  TB_TRY(make_map_2d(&map_p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sizeof(float), P, (unsigned long long)p.d, mat_rows,
                     box_u, box_k, CU_TENSOR_MAP_SWIZZLE_NONE));
  TB_TRY(make_map_2d(&map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, sizeof(double), sp.ArrG, (unsigned long long)p.d,
                     (unsigned long long)M, box_e, 8, CU_TENSOR_MAP_SWIZZLE_NONE));
  return launch_sweep_rows<true>(sp, map_u, map_e, map_p, map_a, st);
}

// Dynamic-grid variant: group by group on the working copy Wk of the step's rows.
static tb_status run_sweep_dynamic(const Plan& p, const float* H_in, const float* U_in, const float* P,
                                   unsigned char* codes, float* scales, int* zeros, unsigned char* cand,
                                   tb_stats* stats, RowMap rm, int M, cudaStream_t st) {
  const int d = p.d, seg = p.seg;
  const int units = (p.n_hin == 1) ? 1 : p.H;
  const long long dd = (long long)d * d;
  k_gather<<<ew_blocks((long long)M * d), 256, 0, st>>>(p.Wt, p.Wk, nullptr, rm, M, d);
  TB_LAUNCH_CHECK();
  GridP gp;
  gp.Wt = p.Wt;
  gp.Hin = H_in;
  gp.sD = p.sD;
  gp.s_out = scales;
  gp.z_out = zeros;
  gp.cand_out = cand;
  gp.rm = rm;
  gp.M = M;
  gp.d = d;
  gp.seg = seg;
  gp.ng = p.ng;
  gp.maxq = p.maxq;
  gp.n_cand = p.n_cand;
  gp.ncp = p.ncp;
  gp.rt = p.rt;
  gp.units = units;
  gp.rows_per_unit = M / units;
  gp.tiles_per_unit = (gp.rows_per_unit + p.rt - 1) / p.rt;
  gp.Wloc = p.Wk;
  const long long ytiles = (long long)gp.units * gp.tiles_per_unit;
  if (ytiles > 65535) return TB_ERR_UNSUPPORTED;
  static bool configured_tri[64] = {false}, configured_panel[64] = {false};
  TB_TRY(allow_smem(k_grid_tri, GRID_TRI_SMEM, configured_tri));
  const size_t panel_smem = (size_t)seg * seg * sizeof(float) * (P ? 2 : 1);
  TB_TRY(allow_smem(k_group_panel, 2 * 128 * 128 * sizeof(float), configured_panel));
  GroupPanelP pp;
  pp.Wk = p.Wk;
  pp.U = U_in;
  pp.P = P;
  pp.Err = p.dynErr;
  pp.Arr = p.dynArr;
  pp.codes = codes;
  pp.sD = p.sD;
  pp.z = zeros;
  pp.stats = stats;
  pp.rm = rm;
  pp.M = M;
  pp.d = d;
  pp.seg = seg;
  pp.ng = p.ng;
  pp.maxq = p.maxq;
  pp.units = units;
  pp.rows_per_unit = M / units;
  pp.ctas_per_unit = (pp.rows_per_unit + 7) / 8;
  for (int grp = 0; grp < p.ng; ++grp) {
    const int c0 = grp * seg, c1 = c0 + seg;
    gp.grp0 = grp;
    k_grid_tri<<<dim3(1, (unsigned)ytiles), GEMM_THREADS, GRID_TRI_SMEM, st>>>(gp);
    TB_LAUNCH_CHECK();
    pp.grp = grp;
    k_group_panel<<<(unsigned)(pp.ctas_per_unit * units), 256, panel_smem, st>>>(pp);
    TB_LAUNCH_CHECK();
    if (c1 >= d) break;
    // Wk[:, c1:] -= Err U[c0:c1, c1:]  (- Arr P[c0:c1, c1:])
    GemmP g = gemm_params();
    g.A = p.dynErr;
    g.a_m = seg;
    g.a_k = 1;
    g.a_batch = (long long)pp.rows_per_unit * seg;
    g.B = U_in + (long long)c0 * d + c1;
    g.b_k = d;
    g.b_n = 1;
    g.b_batch = (units > 1) ? dd : 0;
    g.C = p.Wk + c1;
    g.ldc = d;
    g.c_batch = (long long)pp.rows_per_unit * d;
    g.M = pp.rows_per_unit;
    g.N = d - c1;
    g.K = seg;
    g.n_batch = units;
    g.alpha = -1.0;
    g.beta = 1.0;
    TB_TRY((gemm_launch<double, float, double, double, false, true>(g, st)));
    if (P) {
      g.A = p.dynArr;
      g.B = P + (long long)c0 * d + c1;
      TB_TRY((gemm_launch<double, float, double, double, false, true>(g, st)));
    }
  }
  return TB_OK;
}

}  // namespace tb

using namespace tb;

namespace tb {
bool g_profile_on = false;
PhaseSpan g_spans[TB_MAX_SPANS];
int g_n_spans = 0;
}  // namespace tb

extern "C" void tb_profile_enable(int on) {
  for (int i = 0; i < g_n_spans; ++i) {
    cudaEventDestroy(g_spans[i].a);
    cudaEventDestroy(g_spans[i].b);
  }
  g_n_spans = 0;
  g_profile_on = (on != 0);
}

extern "C" int tb_profile_read(double* ms_by_phase, int n) {
  for (int i = 0; i < n; ++i) ms_by_phase[i] = 0.0;
  for (int i = 0; i < g_n_spans; ++i) {
    float ms = 0.0f;
    if (cudaEventSynchronize(g_spans[i].b) == cudaSuccess &&
        cudaEventElapsedTime(&ms, g_spans[i].a, g_spans[i].b) == cudaSuccess && g_spans[i].phase < n)
      ms_by_phase[g_spans[i].phase] += (double)ms;
    cudaEventDestroy(g_spans[i].a);
    cudaEventDestroy(g_spans[i].b);
  }
  g_n_spans = 0;
  return PH_COUNT;
}

extern "C" size_t tb_quantize_layer_workspace(const tb_layer_desc* desc, int with_r, int with_loss) {
  Plan p;
  // the larger of the two H_out cases, so that one query serves both
  size_t a = 0, b = 0;
  if (make_plan(desc, true, with_r != 0, with_loss != 0, nullptr, &p) == TB_OK) a = p.ws_total;
  if (make_plan(desc, false, with_r != 0, with_loss != 0, nullptr, &p) == TB_OK) b = p.ws_total;
  return a > b ? a : b;
}

extern "C" tb_status tb_quantize_layer(const tb_layer_desc* desc, const float* W, const float* H_in,
                                       const float* U_in, const float* H_out, const float* U_out,
                                       const float* R, const float* P, const float* C,
                                       unsigned char* codes, float* scales, int* zeros,
                                       unsigned char* cand, float* W_hat, double* W_comp, double* loss,
                                       tb_stats* stats, void* ws, size_t ws_bytes, void* stream) {
  if (!desc || !W || !H_in || !U_in || !codes || !scales || !zeros) return TB_ERR_INVALID_ARG;
  if ((H_out == nullptr) != (U_out == nullptr)) return TB_ERR_INVALID_ARG;
  const bool with_r = (R != nullptr);
  if (with_r != (P != nullptr) || with_r != (C != nullptr)) return TB_ERR_INVALID_ARG;
  if (!aligned(W, 16) || !aligned(H_in, 16) || !aligned(U_in, 16) || (P && !aligned(P, 16)))
    return TB_ERR_INVALID_ARG;
  Plan p;
  TB_TRY(make_plan(desc, H_out != nullptr, with_r, loss != nullptr, nullptr, &p));
  if (!ws || !aligned(ws, 256) || ws_bytes < p.ws_total) return TB_ERR_WORKSPACE;
  TB_TRY(make_plan(desc, H_out != nullptr, with_r, loss != nullptr, ws, &p));
  cudaStream_t st = as_stream(stream);
  const int d = p.d;
  const long long n_all = (long long)p.d_out * d;
  const long long dd = (long long)d * d;

  {
    PhaseScope ph(PH_SETUP, st);
    if (stats) TB_CUDA_CHECK(cudaMemsetAsync(stats, 0, sizeof(tb_stats), st));
    k_widen<<<ew_blocks(n_all), 256, 0, st>>>(W, p.Wt, n_all);
    TB_LAUNCH_CHECK();
    if (p.T) {
      k_comp_matrices<<<dim3(p.S, p.H), 128, 0, st>>>(U_out, p.T, p.dh, p.g, p.S);
      TB_LAUNCH_CHECK();
    }
  }
  if (!p.adaptive && !p.dynamic) {
    // fixed grid: every row, once, from the original weights
    PhaseScope ph(PH_GRID, st);
    RowMap all{p.dh, p.dh, 0};
    TB_TRY(run_grid(p, H_in, scales, zeros, cand, all, p.d_out, st));
  }

  for (int step = 0; step < p.S; ++step) {
    const int i0 = step * p.g, M = p.H * p.g;
    RowMap rm{p.g, p.dh, i0};
    if (p.adaptive) {
      PhaseScope ph(PH_GRID, st);
      TB_TRY(run_grid(p, H_in, scales, zeros, cand, rm, M, st));
    }
    {
      PhaseScope ph(PH_SWEEP, st);
      if (with_r) {  // the snapshot W0 as a contiguous GEMM operand of the propagated-error term
        k_gather<<<ew_blocks((long long)M * d), 256, 0, st>>>(p.Wt, p.W0c, nullptr, rm, M, d);
        TB_LAUNCH_CHECK();
      }
      if (p.dynamic)
        TB_TRY(run_sweep_dynamic(p, H_in, U_in, P, codes, scales, zeros, cand, stats, rm, M, st));
      else
        TB_TRY(run_sweep_rows(p, U_in, P, codes, zeros, stats, rm, M, st));
    }
    const int nrem = p.dh - i0 - p.g;
    if (!p.has_hout || nrem <= 0) continue;
    PhaseScope ph_comp(PH_COMP, st);
    k_residual<<<ew_blocks((long long)M * d), 256, 0, st>>>(p.Wt, codes, p.sD, zeros, p.E, rm, M, d,
                                                            p.seg, p.ng);
    TB_LAUNCH_CHECK();
    if (with_r) {
      // E <- E - W0 (R H_in^{-1})   (Proposition 3.2)
      GemmP g = gemm_params();
      const int units = (p.n_hin == 1) ? 1 : p.H;
      g.A = p.W0c;
      g.a_m = d;
      g.a_k = 1;
      g.B = C;
      g.b_k = d;
      g.b_n = 1;
      g.C = p.E;
      g.ldc = d;
      g.M = M / units;
      g.N = d;
      g.K = d;
      g.n_batch = units;
      g.a_batch = (long long)g.M * d;
      g.c_batch = (long long)g.M * d;
      g.b_batch = (units > 1) ? dd : 0;
      g.alpha = -1.0;
      g.beta = 1.0;
      TB_TRY((gemm_launch<double, float, double, double, false, true>(g, st)));
    }
    {
      // W~[rem rows of every head] -= T_i E   (Propositions 3.1 / 3.2; Algorithm 1, update step)
      GemmP g = gemm_params();
      g.A = p.T + (long long)step * p.dh * p.g;
      g.a_m = p.g;
      g.a_k = 1;
      g.a_batch = (long long)p.S * p.dh * p.g;
      g.B = p.E;
      g.b_k = d;
      g.b_n = 1;
      g.b_batch = (long long)p.g * d;
      g.C = p.Wt + (long long)(i0 + p.g) * d;
      g.ldc = d;
      g.c_batch = (long long)p.dh * d;
      g.M = nrem;
      g.N = d;
      g.K = p.g;
      g.n_batch = p.H;
      g.alpha = -1.0;
      g.beta = 1.0;
      TB_TRY((gemm_launch<double, double, double, double, false, true>(g, st)));
    }
  }

  // A group's rows are never written after they have been taken, and the rows of later groups only by
  // the compensation of the groups before them: after the loop row r of W~ is what the sweep saw.
  if (W_comp)
    TB_CUDA_CHECK(cudaMemcpyAsync(W_comp, p.Wt, (size_t)n_all * sizeof(double), cudaMemcpyDeviceToDevice, st));

  // ---- coordinate descent on the scales (Algorithm 3) ----
  if (p.cd) {
    PhaseScope ph(PH_CD, st);
    const int units = (p.n_hin == 1) ? 1 : p.H;
    k_cd_prep<<<ew_blocks(n_all), 256, 0, st>>>(W, codes, p.sD, zeros, p.Dq, p.Wb, p.d_out, d, p.seg,
                                               p.ng);
    TB_LAUNCH_CHECK();
    for (long long r0 = 0; r0 < p.d_out; r0 += p.cd_rows) {
      const long long rows = (p.d_out - r0 < p.cd_rows) ? (p.d_out - r0) : p.cd_rows;
      // Dm = (Q - W) H_in (+ W R); Yw = blockwise Wbar H_in.  With one H_in per head the
      // batch is whole heads and the products run head by head.
      const bool heads_together = p.yw_tensor && units > 1;   // per-head H_in on the tensor-core path
      const int hunits = heads_together ? (int)(rows / p.dh) : 1;
      const long long rows_per_prod = (units > 1 && !heads_together) ? p.dh : rows;
      for (long long q0 = 0; q0 < rows; q0 += rows_per_prod) {
        const long long rr = r0 + q0;
        const float* Hh = H_in + ((units > 1) ? (rr / p.dh) * dd : 0);
        if (p.yw_tensor)  // also splits H_in into its bf16 pieces on the first batch
          TB_TRY(yw_tensor(reinterpret_cast<float*>(p.Yw), codes + rr * d, zeros + rr * p.ng, Hh, p.WbT, p.Hp,
                           r0 == 0 || with_r || units > 1, rows, d, p.seg, p.ng, hunits,
                           st));  // with R the pieces of R replace H_in's below
        GemmP g = gemm_params();
        g.A = p.Dq + rr * d;
        g.a_m = d;
        g.a_k = 1;
        g.B = Hh;
        g.b_k = d;
        g.b_n = 1;
        g.C = p.Dm + rr * d;
        g.ldc = d;
        g.M = (int)rows_per_prod;
        g.N = d;
        g.K = d;
        if (p.dm_tensor) {
          // the pieces of (Q - W), transposed, live in this batch's rows of the W~ buffer (free by now,
          // and overwritten by G = H_out Dm only after the product)
          __nv_bfloat16* DqT = reinterpret_cast<__nv_bfloat16*>(p.Wt + rr * d);
          TB_TRY(split3_transpose(p.Dq + rr * d, DqT, rows, d, st));
          TB_TRY(gemm_split_presplit(p.Dm + rr * d, d, DqT, p.Hp, rows, d, d, false, st, hunits));
        } else {
          TB_TRY((gemm_launch<double, float, double, double, false, true>(g, st)));
        }
        if (with_r && p.dm_tensor) {
          // Dm += W R through the same split-bf16 product; the pieces of R take the place of H_in's
          __nv_bfloat16* WT = reinterpret_cast<__nv_bfloat16*>(p.Wt + rr * d);
          TB_TRY(split3_transpose(W + rr * d, WT, rows, d, st));
          TB_TRY(split3(R + ((units > 1) ? (rr / p.dh) * dd : 0), p.Hp, dd * hunits, st));
          TB_TRY(gemm_split_presplit(p.Dm + rr * d, d, WT, p.Hp, rows, d, d, true, st, hunits));
        } else if (with_r) {
          GemmP h = g;
          h.A = W + rr * d;
          h.B = R + ((units > 1) ? (rr / p.dh) * dd : 0);
          h.beta = 1.0;
          TB_TRY((gemm_launch<float, float, double, double, false, true>(h, st)));
        }
        if (!p.yw_tensor) {
          GemmP y = gemm_params();
          y.A = p.Wb + rr * d;
          y.a_m = d;
          y.a_k = 1;
          y.a_batch = p.seg;
          y.B = Hh;
          y.b_k = d;
          y.b_n = 1;
          y.b_batch = (long long)p.seg * d;
          y.C = p.Yw + q0 * p.ng * d;
          y.ldc = (long long)p.ng * d;
          y.c_batch = d;
          y.M = (int)rows_per_prod;
          y.N = d;
          y.K = p.seg;
          y.n_batch = p.ng;
          TB_TRY((gemm_launch<float, float, double, double, false, true>(y, st)));
        }
      }
      if (p.has_hout) {
        // rows of a head are coupled through H_out: one CTA per head walks them in order
        const int heads_b = (int)(rows / p.dh);
        const long long nb_el = rows * d;
        CdHeadP hp;
        hp.G = p.Wt + r0 * d;      // W~ is no longer needed: its buffer holds G = H_out Dm
        hp.Uacc = p.Dq + r0 * d;   // (Q - W) has been consumed by the product above
        hp.Yw = p.Yw;
        hp.Wb = p.Wb + r0 * d;
        hp.Hout = H_out + (r0 / p.dh) * (long long)p.dh * p.dh;
        hp.sD = p.sD + r0 * p.ng;
        hp.d = d;
        hp.seg = p.seg;
        hp.ng = p.ng;
        hp.dh = p.dh;
        hp.uw = (p.seg % 128 == 0) ? 128 : (p.seg <= 128 ? p.seg : 32);
        // CTAs per head: whole groups per CTA, and no more CTAs than the GPU holds at once
        int csize = 8;
        while (csize > 1 && ((p.ng % csize) || (long long)heads_b * csize > 148)) csize >>= 1;
        hp.csize = csize;
        const int n_units = (p.ng / csize) * (p.seg / hp.uw);
        const size_t sm_head =
            ((size_t)n_units * (p.ng + 1) + 2 * (size_t)p.ng * p.ng + 3 * (size_t)p.ng) * sizeof(double);
        if (sm_head > 200 * 1024) return TB_ERR_UNSUPPORTED;
        static bool conf_head[64] = {false}, conf_head2[64] = {false};
        auto cd_head_kern = p.yw_tensor ? k_cd_head<float> : k_cd_head<double>;
        if (p.yw_tensor)
          TB_TRY(allow_smem(k_cd_head<float>, 200 * 1024, conf_head));
        else
          TB_TRY(allow_smem(k_cd_head<double>, 200 * 1024, conf_head2));
        // column-parallel pass where a CTA's columns fit two per thread and the chain fits a warp
        const int c_cnt = (p.ng / csize) * p.seg;
        const bool by_cols = (p.ng <= CDC_MAXG) && (c_cnt <= 2 * CDC_THREADS) && (p.seg % 2 == 0) && (d % 2 == 0) &&
                             ((size_t)d * sizeof(float) <= 48 * 1024);
        CdColP cp2;
        cp2.G = hp.G;
        cp2.Uacc = hp.Uacc;
        cp2.Yw = hp.Yw;
        cp2.Wb = hp.Wb;
        cp2.Hout = hp.Hout;
        cp2.Amat = p.Amat;
        cp2.sD = hp.sD;
        cp2.d = d;
        cp2.seg = p.seg;
        cp2.ng = p.ng;
        cp2.dh = p.dh;
        cp2.csize = csize;
        if (by_cols) {
          if (p.yw_tensor)
            k_cd_amat<float><<<(unsigned)rows, 256, (size_t)d * sizeof(float), st>>>(p.Yw, hp.Wb, p.Amat, d, p.seg, p.ng);
          else
            k_cd_amat<double><<<(unsigned)rows, 256, (size_t)d * sizeof(float), st>>>(p.Yw, hp.Wb, p.Amat, d, p.seg, p.ng);
          TB_LAUNCH_CHECK();
        }
        for (int it = 0; it < p.cd_iters; ++it) {
          GemmP g = gemm_params();  // G = H_out Dm, head by head
          g.A = hp.Hout;
          g.a_m = p.dh;
          g.a_k = 1;
          g.a_batch = (long long)p.dh * p.dh;
          g.B = p.Dm + r0 * d;
          g.b_k = d;
          g.b_n = 1;
          g.b_batch = (long long)p.dh * d;
          g.C = hp.G;
          g.ldc = d;
          g.c_batch = (long long)p.dh * d;
          g.M = p.dh;
          g.N = d;
          g.K = p.dh;
          g.n_batch = heads_b;
          TB_TRY((gemm_launch<float, double, double, double, false, true>(g, st)));
          cudaLaunchConfig_t cfg = {};
          cfg.gridDim = dim3((unsigned)(heads_b * csize));
          cfg.blockDim = dim3(by_cols ? CDC_THREADS : CDH_THREADS);
          cfg.dynamicSmemBytes = by_cols ? 0 : sm_head;
          cfg.stream = st;
          cudaLaunchAttribute attr[1];
          attr[0].id = cudaLaunchAttributeClusterDimension;
          attr[0].val.clusterDim.x = (unsigned)csize;
          attr[0].val.clusterDim.y = 1;
          attr[0].val.clusterDim.z = 1;
          cfg.attrs = attr;
          cfg.numAttrs = 1;
          if (by_cols) {
            if (p.yw_tensor)
              TB_CUDA_CHECK(cudaLaunchKernelEx(&cfg, k_cd_head_cols<float>, cp2));
            else
              TB_CUDA_CHECK(cudaLaunchKernelEx(&cfg, k_cd_head_cols<double>, cp2));
          } else {
            TB_CUDA_CHECK(cudaLaunchKernelEx(&cfg, cd_head_kern, hp));
          }
          TB_LAUNCH_CHECK();
          k_axpy<<<ew_blocks(nb_el), 256, 0, st>>>(p.Dm + r0 * d, hp.Uacc, nb_el);
          TB_LAUNCH_CHECK();
        }
        continue;
      }
      // H_out = I: rows are independent, every row is its own line of one row
      CdP cp;
      cp.Dm = p.Dm + r0 * d;
      cp.Yw = p.Yw;
      cp.Wb = p.Wb + r0 * d;
      cp.sD = p.sD + r0 * p.ng;
      cp.n0 = p.n0;
      cp.Amat = p.Amat;
      cp.d = d;
      cp.seg = p.seg;
      cp.ng = p.ng;
      cp.Hout = nullptr;
      cp.dh = 1;
      cp.lines_per_head = 1;
      cp.j0 = 0;
      const int lines = (int)rows;
      // columns per CTA: whole groups, about 512 columns
      int gpc = 512 / p.seg;
      if (gpc < 1) gpc = 1;
      if (gpc > p.ng) gpc = p.ng;
      cp.groups_per_cta = gpc;
      const int xctas = (p.ng + gpc - 1) / gpc;
      const size_t sm_stats = ((size_t)gpc * (p.seg / 32) * (p.ng + 1) + cp.dh) * sizeof(double);
      size_t sm_upd = ((size_t)2 * p.ng + (size_t)p.ng * p.ng) * sizeof(double);
      cp.a_in_smem = 1;
      if (sm_upd > 200 * 1024) {
        sm_upd = (size_t)2 * p.ng * sizeof(double);
        cp.a_in_smem = 0;
      }
      static bool conf_stats[64] = {false}, conf_upd[64] = {false};
      static bool conf_stats_f[64] = {false}, conf_upd_f[64] = {false};
      TB_TRY(allow_smem(k_cd_row_stats<double>, 200 * 1024, conf_stats));
      TB_TRY(allow_smem(k_cd_row_update<double>, 200 * 1024, conf_upd));
      TB_TRY(allow_smem(k_cd_row_stats<float>, 200 * 1024, conf_stats_f));
      TB_TRY(allow_smem(k_cd_row_update<float>, 200 * 1024, conf_upd_f));
      const size_t ysz = p.yw_tensor ? sizeof(float) : sizeof(double);
      if (sm_stats > 200 * 1024) return TB_ERR_UNSUPPORTED;
      for (int it = 0; it < p.cd_iters; ++it) {
        for (int l0 = 0; l0 < lines; l0 += 65535) {
          const int nl = (lines - l0 < 65535) ? (lines - l0) : 65535;
          CdP cq = cp;  // advance every per-line pointer by l0 rows
          cq.Dm = cp.Dm + (long long)l0 * d;
          cq.Yw = static_cast<const char*>(cp.Yw) + (size_t)l0 * p.ng * d * ysz;
          cq.Wb = cp.Wb + (long long)l0 * d;
          cq.sD = cp.sD + (long long)l0 * p.ng;
          cq.n0 = cp.n0 + (long long)l0 * p.ng;
          cq.Amat = cp.Amat + (long long)l0 * p.ng * p.ng;
          if (p.yw_tensor) {
            k_cd_row_stats<float><<<dim3(xctas, nl), 256, sm_stats, st>>>(cq);
            TB_LAUNCH_CHECK();
            k_cd_row_update<float><<<dim3(xctas, nl), 256, sm_upd, st>>>(cq);
          } else {
            k_cd_row_stats<double><<<dim3(xctas, nl), 256, sm_stats, st>>>(cq);
            TB_LAUNCH_CHECK();
            k_cd_row_update<double><<<dim3(xctas, nl), 256, sm_upd, st>>>(cq);
          }
          TB_LAUNCH_CHECK();
        }
      }
    }
  }

  {
    PhaseScope ph(PH_OUTPUT, st);
    k_dequant<<<ew_blocks(n_all), 256, 0, st>>>(codes, p.sD, zeros, W_hat, scales, p.d_out, d, p.seg,
                                               p.ng);
    TB_LAUNCH_CHECK();
  }

  // ---- loss of the proofs of Propositions 3.1 / 3.2 ----
  if (loss) {
    PhaseScope ph(PH_LOSS, st);
    const int units = (p.n_hin == 1) ? 1 : p.H;
    k_cd_prep<<<ew_blocks(n_all), 256, 0, st>>>(W, codes, p.sD, zeros, p.Dq, nullptr, p.d_out, d,
                                               p.seg, p.ng);
    TB_LAUNCH_CHECK();
    GemmP g = gemm_params();
    g.A = p.Dq;
    g.a_m = d;
    g.a_k = 1;
    g.B = H_in;
    g.b_k = d;
    g.b_n = 1;
    g.C = p.Dm;
    g.ldc = d;
    g.M = p.d_out / units;
    g.N = d;
    g.K = d;
    g.n_batch = units;
    g.a_batch = g.c_batch = (long long)g.M * d;
    g.b_batch = (units > 1) ? dd : 0;
    // Z = dW H_in (+ 2 W R).  After the scale refinement without R the buffer Dm already holds
    // dW H_in for the final scales (it was kept current through the pass), so the product is skipped.
    // With R the pass keeps Dm = dW H_in + W R, so only one more W R is missing.
    const bool dm_is_current = p.cd;
    if (!dm_is_current && p.loss_tensor && units == 1) {
      __nv_bfloat16* DqT = reinterpret_cast<__nv_bfloat16*>(p.Wt);  // W~ is no longer needed
      TB_TRY(split3_transpose(p.Dq, DqT, p.d_out, d, st));
      TB_TRY(split3(H_in, p.Hp, dd, st));
      TB_TRY(gemm_split_presplit(p.Dm, d, DqT, p.Hp, p.d_out, d, d, false, st));
    } else if (!dm_is_current && p.loss_tensor) {
      // one H_in per head: a batch of heads per launch, every head against its own pieces
      for (int h0 = 0; h0 < p.H; h0 += p.loss_heads) {
        const int nb = (p.H - h0 < p.loss_heads) ? (p.H - h0) : p.loss_heads;
        const long long rr = (long long)h0 * p.dh, rows = (long long)nb * p.dh;
        __nv_bfloat16* DqT = reinterpret_cast<__nv_bfloat16*>(p.Wt + rr * d);  // W~ is no longer needed
        TB_TRY(split3_transpose(p.Dq + rr * d, DqT, rows, d, st));
        TB_TRY(split3(H_in + (long long)h0 * dd, p.Hp, dd * nb, st));
        TB_TRY(gemm_split_presplit(p.Dm + rr * d, d, DqT, p.Hp, rows, d, d, false, st, nb));
      }
    } else if (!dm_is_current) {
      TB_TRY((gemm_launch<double, float, double, double, false, true>(g, st)));
    }
    if (with_r && (p.loss_tensor || (dm_is_current && p.dm_tensor)) && units == 1) {
      __nv_bfloat16* WT = reinterpret_cast<__nv_bfloat16*>(p.Wt);  // W~ is no longer needed
      TB_TRY(split3_transpose(W, WT, p.d_out, d, st));
      TB_TRY(split3(R, p.Hp, dd, st));
      TB_TRY(gemm_split_presplit(p.Dm, d, WT, p.Hp, p.d_out, d, d, true, st));
      if (!dm_is_current) TB_TRY(gemm_split_presplit(p.Dm, d, WT, p.Hp, p.d_out, d, d, true, st));  // 2 W R
    } else if (with_r) {
      GemmP h = g;
      h.A = W;
      h.B = R;
      h.alpha = dm_is_current ? 1.0 : 2.0;
      h.beta = 1.0;
      TB_TRY((gemm_launch<float, float, double, double, false, true>(h, st)));
    }
    // loss_h = tr(H_out,h Z_h dW_h^T) = sum over the head's entries of (H_out,h Z_h) .* dW_h: a product
    // with d_in columns (many tiles) and an elementwise reduction, instead of a d_head x d_head product
    // whose contraction runs over d_in on a handful of tiles.
    const double* lhs = p.Dm;
    if (p.has_hout) {
      GemmP q = gemm_params();
      q.A = H_out;
      q.a_m = p.dh;
      q.a_k = 1;
      q.a_batch = (long long)p.dh * p.dh;
      q.B = p.Dm;  // Z
      q.b_k = d;
      q.b_n = 1;
      q.b_batch = (long long)p.dh * d;
      q.C = p.Wt;  // W~ is no longer needed
      q.ldc = d;
      q.c_batch = (long long)p.dh * d;
      q.M = p.dh;
      q.N = d;
      q.K = p.dh;
      q.n_batch = p.H;
      TB_TRY((gemm_launch<float, double, double, double, false, true>(q, st)));
      lhs = p.Wt;
    }
    const int chunks = (p.dh + 31) / 32;
    k_loss_identity_partial<<<dim3(chunks, p.H), 256, 0, st>>>(lhs, p.Dq, p.G2, p.dh, d, chunks);
    TB_LAUNCH_CHECK();
    k_loss_identity_final<<<p.H, 32, 0, st>>>(p.G2, loss, chunks);
    TB_LAUNCH_CHECK();
  }
  return TB_OK;
}
