// Deviation correlation R += alpha (X - Xfp)^T X (Algorithm 1, deviation step) for bf16
// activations on the 5th-generation tensor cores.
//
// D = X - Xfp is formed in float (exact whenever the two values differ by less than
// 2^16 in magnitude ratio) and split into two bf16 pieces, D = D1 + D2: the pieces
// hold 16 significant bits, which is all of D unless x and xfp differ by more than a
// factor 256 in magnitude (then the relative error of that element is below 2^-17).
// Products of bf16 values are exact in float, so R = alpha (D1^T X + D2^T X) is
// rounded only by the float accumulation, organised as in the Hessian kernel: 2048
// contraction steps at a time in one of two TMEM buffers, drained into float
// running sums by the epilogue warps while the tensor cores fill the other.  The
// two pieces are stacked along the token axis, [D1; D2], next to [X; X], so that
// the product is one long contraction per tile.  One CTA owns a 128 x 256 tile of
// R for the whole contraction: fixed summation order, no atomics.
//
// Operand layout, pipeline, warp roles and the bounded waits are those of
// tb_syrk_tc.cu (TMA boxes of 64 tokens x 64 columns with the 128-byte swizzle =
// MN-major SWIZZLE_128B operands; warps 0-7 epilogue, warp 8 TMA producer, warp 9
// MMA issuer).  No cluster launch; every CTA issues its own loads.
#include "tb_common.cuh"
#include "tb_tma.cuh"

namespace tb {

enum {
  XC_BM = 128,
  XC_BN = 256,
  XC_BK = 64,
  XC_STAGES = 4,
  XC_CHUNK = 32,
  XC_BOX_BYTES = 64 * 64 * 2,
  XC_A_BYTES = 2 * XC_BOX_BYTES,
  XC_B_BYTES = 4 * XC_BOX_BYTES,
  XC_STAGE_BYTES = XC_A_BYTES + XC_B_BYTES,
  XC_THREADS = 320,
  XC_SMEM = XC_STAGES * XC_STAGE_BYTES + 1024 + 256,
  XC_PIECES = 2
};

__device__ int g_xc_error = 0;

// Dp[p][t][c] = piece p of X[t][c] - Xfp[t][c] for t < n_tok, 0 for n_tok <= t < ntp
__global__ void k_deviation_split(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ Xfp,
                                  __nv_bfloat16* __restrict__ Dp, long long n_tok, long long ntp, int d) {
  const long long n = ntp * d, n_in = n_tok * d;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    __nv_bfloat16 p1 = __float2bfloat16_rn(0.0f), p2 = p1;
    if (i < n_in) {
      const float dv = __bfloat162float(X[i]) - __bfloat162float(Xfp[i]);
      p1 = __float2bfloat16_rn(dv);
      p2 = __float2bfloat16_rn(dv - __bfloat162float(p1));
    }
    Dp[i] = p1;
    Dp[n + i] = p2;
  }
}

__global__ void __launch_bounds__(XC_THREADS, 1)
    k_cross_tc(float* __restrict__ R, const __grid_constant__ CUtensorMap dmap, const __grid_constant__ CUtensorMap xmap,
               int ntp, int d, int n_tiles, float alpha) {
  extern __shared__ unsigned char xc_smem_raw[];
  const uint32_t raw = smem_u32(xc_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = xc_smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + XC_STAGES * XC_STAGE_BYTES);
  // bars[0..3] full, [4..7] empty, [8..9] acc_full, [10..11] acc_empty; then tmem slot, abort flag
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (4 + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (8 + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (10 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < XC_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 8);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int stages_per_piece = ntp / XC_BK;            // ntp is a multiple of 64
  const int n_stages = XC_PIECES * stages_per_piece;   // the stacked contraction [D1; D2] x [X; X]
  const int n_blocks = (d + XC_BN - 1) / XC_BN;        // tile t -> (mi, nj) = (t / n_blocks, t % n_blocks)

  if (warp == 8) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        const int m0 = (t / n_blocks) * XC_BM, n0 = (t % n_blocks) * XC_BN;
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % XC_STAGES;
          const uint32_t ph = (it / XC_STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, &g_xc_error)) break;
          mbar_expect_tx(full_bar(s), XC_STAGE_BYTES);
          const uint32_t sa = base + s * XC_STAGE_BYTES, sb = sa + XC_A_BYTES;
          const int ka = st * XC_BK;                              // row of the stacked pieces
          const int kb = (st % stages_per_piece) * XC_BK;         // token of X (rows past n_tok read as zero)
#pragma unroll
          for (int j = 0; j < 2; ++j) tma_load_2d(sa + j * XC_BOX_BYTES, &dmap, m0 + 64 * j, ka, full_bar(s));
#pragma unroll
          for (int j = 0; j < 4; ++j) tma_load_2d(sb + j * XC_BOX_BYTES, &xmap, n0 + 64 * j, kb, full_bar(s));
        }
      }
    }
  } else if (warp == 9) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_mn(128, 256);
      uint32_t it = 0, chunk_it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int in_chunk = st % XC_CHUNK;
          const int b = chunk_it & 1;
          if (in_chunk == 0) {
            if (!mbar_wait(acce_bar(b), ((chunk_it >> 1) & 1u) ^ 1u, abort_flag, &g_xc_error)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          const int s = it % XC_STAGES;
          const uint32_t ph = (it / XC_STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, &g_xc_error)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + s * XC_STAGE_BYTES, sb = sa + XC_A_BYTES;
          const uint32_t tmem_d = tmem_base + (uint32_t)b * XC_BN;
#pragma unroll
          for (int kk = 0; kk < XC_BK / 16; ++kk) {
            const uint64_t adesc = smem_desc_mn_sw128(sa + kk * 2048);
            const uint64_t bdesc = smem_desc_mn_sw128(sb + kk * 2048);
            umma_bf16(tmem_d, adesc, bdesc, idesc, (in_chunk > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(s));
          if (in_chunk == XC_CHUNK - 1 || st == n_stages - 1) {
            umma_commit(accf_bar(b));
            ++chunk_it;
          }
        }
      }
    }
  } else {
    // ---------------- epilogue warps 0-7 ----------------
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    uint32_t chunk_it = 0;
    for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
      const int m0 = (t / n_blocks) * XC_BM, n0 = (t % n_blocks) * XC_BN;
      float run[128];
#pragma unroll
      for (int i = 0; i < 128; ++i) run[i] = 0.0f;
      bool ok = true;
      for (int st0 = 0; st0 < n_stages && ok; st0 += XC_CHUNK, ++chunk_it) {
        const int b = chunk_it & 1;
        ok = mbar_wait(accf_bar(b), (chunk_it >> 1) & 1u, abort_flag, &g_xc_error);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * XC_BN + hf * 128);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(taddr + c * 32, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int i = 0; i < 32; ++i) run[c * 32 + i] += __uint_as_float(r[i]);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(b));
      }
      if (ok) {
        const int gm = m0 + row;
        if (gm < d) {
          float* rrow = R + (long long)gm * d;
#pragma unroll
          for (int i = 0; i < 128; ++i) {
            const int gn = n0 + hf * 128 + i;
            if (gn < d) rrow[gn] = fmaf(alpha, run[i], rrow[gn]);
          }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

static long long padded_tokens(long long n_tok) { return (n_tok + XC_BK - 1) / XC_BK * XC_BK; }

// bytes of scratch for the two pieces of the deviation
size_t cross_bf16_workspace(long long n_tok, int d) {
  return (size_t)XC_PIECES * (size_t)padded_tokens(n_tok) * (size_t)d * sizeof(__nv_bfloat16);
}

tb_status cross_bf16_tensor(float* R, const __nv_bfloat16* X, const __nv_bfloat16* Xfp, long long n_tok, int d,
                            float alpha, void* ws, cudaStream_t st) {
  const long long ntp = padded_tokens(n_tok);
  if (XC_PIECES * ntp > 0x7fffffffll) return TB_ERR_UNSUPPORTED;
  __nv_bfloat16* Dp = static_cast<__nv_bfloat16*>(ws);
  k_deviation_split<<<148 * 8, 256, 0, st>>>(X, Xfp, Dp, n_tok, ntp, d);
  TB_LAUNCH_CHECK();
  CUtensorMap dmap, xmap;
  TB_TRY(make_map_2d(&dmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, sizeof(__nv_bfloat16), Dp, (unsigned long long)d,
                     (unsigned long long)(XC_PIECES * ntp), 64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  TB_TRY(make_map_2d(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, sizeof(__nv_bfloat16), X, (unsigned long long)d,
                     (unsigned long long)n_tok, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  const int n_tiles = ((d + XC_BM - 1) / XC_BM) * ((d + XC_BN - 1) / XC_BN);
  int dev = 0, sms = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  TB_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  static bool configured[64] = {false};
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!configured[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_cross_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)XC_SMEM));
    configured[dev] = true;
  }
  // as many CTAs as fill the rounds of tiles evenly (the same number of rounds as with every SM: fewer CTAs
  // asking L2 at once, and less power, for the same time or less)
  const int rounds_of_tiles = (int)((n_tiles + sms - 1) / (sms > 0 ? sms : 1));
  const int grid = (int)((n_tiles + rounds_of_tiles - 1) / (rounds_of_tiles > 0 ? rounds_of_tiles : 1));
  k_cross_tc<<<grid, XC_THREADS, XC_SMEM, st>>>(R, dmap, xmap, (int)ntp, d, n_tiles, alpha);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

int cross_error_read_clear() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_xc_error, sizeof(int)) != cudaSuccess) return -1;
  if (v) {
    int z = 0;
    cudaMemcpyToSymbol(g_xc_error, &z, sizeof(int));
  }
  return v;
}

}  // namespace tb
