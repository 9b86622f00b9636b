// Hessian accumulation H += X^T X for bf16 activations on the 5th-generation
// tensor cores (tcgen05.mma, accumulators in tensor memory, operands staged by
// TMA).  Products of bf16 values are exact in float, so the only rounding is
// the float accumulation, which is kept short: the tensor cores accumulate
// 2048 tokens at a time into one of two TMEM buffers; the epilogue warps drain
// the finished buffer into float registers (round-to-nearest adds) while the
// tensor cores fill the other one.  One CTA owns a 128 x 256 tile of H for the
// whole token range, so the sum into H has a fixed order and needs no atomics.
//
// X is token-major [n_tok][d]: both operands of X^T X have the token index
// (the contraction index K) as the strided one, i.e. they are "MN-major".  A
// TMA box of 64 tokens x 64 columns lands in shared memory as 64 rows of
// 128 bytes with the 128-byte swizzle, which is the canonical MN-major
// SWIZZLE_128B operand layout: 8 rows of 128 B form one swizzle atom, atoms
// repeat every 1024 B along K (stride byte offset) and every 8192 B (one box)
// along M / N (leading byte offset).
//
// Warp roles (320 threads): warps 0-7 epilogue (warp w reads TMEM lanes
// 32 (w % 4) .. +31, columns 128 (w / 4) .. +127), warp 8 TMA producer, warp 9
// MMA issuer.  Every wait on an mbarrier is bounded; when a bound runs out the
// kernel raises a device error word, leaves its loops, frees its tensor memory
// and returns.
#include "tb_common.cuh"
#include "tb_tma.cuh"

namespace tb {

enum {
  TC_BM = 128,
  TC_BN = 256,
  TC_BK = 64,          // tokens per pipeline stage
  TC_STAGES = 4,
  TC_CHUNK = 32,       // stages per TMEM accumulation (2048 tokens)
  TC_BOX_BYTES = 64 * 64 * 2,
  TC_A_BYTES = 2 * TC_BOX_BYTES,
  TC_B_BYTES = 4 * TC_BOX_BYTES,
  TC_STAGE_BYTES = TC_A_BYTES + TC_B_BYTES,
  TC_THREADS = 320,
  TC_SMEM = TC_STAGES * TC_STAGE_BYTES + 1024 /*alignment*/ + 256 /*barriers*/
};

__device__ int g_tc_error = 0;

__global__ void __launch_bounds__(TC_THREADS, 1)
    k_syrk_tc(float* __restrict__ H, const __grid_constant__ CUtensorMap xmap, int n_tok, int d, int n_tiles) {
  extern __shared__ unsigned char tc_smem_raw[];
  // 1024-byte aligned stage buffers, then the barriers
  const uint32_t raw = smem_u32(tc_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = tc_smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + TC_STAGES * TC_STAGE_BYTES);
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
    for (int s = 0; s < TC_STAGES; ++s) {
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

  const int n_stages = (n_tok + TC_BK - 1) / TC_BK;
  const int m_blocks = (d + TC_BM - 1) / TC_BM;

  // tile t -> (mi, nj): row block mi has the column blocks nj = 0 .. mi / 2
  auto tile_of = [&](int t, int& mi, int& nj) {
    int acc = 0;
    for (mi = 0; mi < m_blocks; ++mi) {
      const int cnt = mi / 2 + 1;
      if (t < acc + cnt) {
        nj = t - acc;
        return;
      }
      acc += cnt;
    }
    mi = m_blocks - 1;
    nj = 0;
  };

  if (warp == 8) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        int mi, nj;
        tile_of(t, mi, nj);
        const int m0 = mi * TC_BM, n0 = nj * TC_BN;
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % TC_STAGES;
          const uint32_t ph = (it / TC_STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, &g_tc_error)) break;
          mbar_expect_tx(full_bar(s), TC_STAGE_BYTES);
          const uint32_t sa = base + s * TC_STAGE_BYTES, sb = sa + TC_A_BYTES;
          const int k0 = st * TC_BK;
#pragma unroll
          for (int j = 0; j < 2; ++j) tma_load_2d(sa + j * TC_BOX_BYTES, &xmap, m0 + 64 * j, k0, full_bar(s));
#pragma unroll
          for (int j = 0; j < 4; ++j) tma_load_2d(sb + j * TC_BOX_BYTES, &xmap, n0 + 64 * j, k0, full_bar(s));
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
          const int in_chunk = st % TC_CHUNK;
          const int b = chunk_it & 1;
          if (in_chunk == 0) {
            // the accumulator buffer must have been drained by the epilogue warps
            if (!mbar_wait(acce_bar(b), ((chunk_it >> 1) & 1u) ^ 1u, abort_flag, &g_tc_error)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          const int s = it % TC_STAGES;
          const uint32_t ph = (it / TC_STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, &g_tc_error)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + s * TC_STAGE_BYTES, sb = sa + TC_A_BYTES;
          const uint32_t tmem_d = tmem_base + (uint32_t)b * TC_BN;
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk) {
            const uint64_t adesc = smem_desc_mn_sw128(sa + kk * 2048);
            const uint64_t bdesc = smem_desc_mn_sw128(sb + kk * 2048);
            umma_bf16(tmem_d, adesc, bdesc, idesc, (in_chunk > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(s));  // the stage may be refilled once these MMAs have read it
          if (in_chunk == TC_CHUNK - 1 || st == n_stages - 1) {
            umma_commit(accf_bar(b));  // the chunk's accumulator is complete
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
      int mi, nj;
      tile_of(t, mi, nj);
      const int m0 = mi * TC_BM, n0 = nj * TC_BN;
      // The running sums start from the values already in H and are stored back at the end, so that
      // accumulating the tokens over several calls (split at multiples of 2048 tokens) performs
      // exactly the additions of one call over all of them.
      float run[128];
      const int gm = m0 + row;
      float* hrow = H + (long long)gm * d;
#pragma unroll
      for (int i = 0; i < 128; ++i) {
        const int gn = n0 + hf * 128 + i;
        run[i] = (gm < d && gn < d && gn < m0 + TC_BM) ? hrow[gn] : 0.0f;
      }
      bool ok = true;
      for (int st0 = 0; st0 < n_stages && ok; st0 += TC_CHUNK, ++chunk_it) {
        const int b = chunk_it & 1;
        ok = mbar_wait(accf_bar(b), (chunk_it >> 1) & 1u, abort_flag, &g_tc_error);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * TC_BN + hf * 128);
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
      if (ok && gm < d) {
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          const int gn = n0 + hf * 128 + i;
          // column blocks strictly above the diagonal block are filled by the mirror pass
          if (gn < d && gn < m0 + TC_BM) hrow[gn] = run[i];
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

// H += X^T X for bf16 X on the tensor cores: tiles on or below the diagonal
// (128-row blocks x 256-column blocks); the caller mirrors the rest.
tb_status syrk_bf16_tensor_pair(float* H, const __nv_bfloat16* X, long long n_tok, int d, cudaStream_t st);

tb_status syrk_bf16_tensor(float* H, const __nv_bfloat16* X, long long n_tok, int d, cudaStream_t st) {
  if (n_tok > 0x7fffffffll) return TB_ERR_UNSUPPORTED;
  // From 6144 columns on, 256 x 256 tiles on CTA pairs (measured: 11 % faster at 8192 columns, level at 5120
  // and 6144; below that the single-CTA tiles win by 3-10 %).
  if (d >= 6144) return syrk_bf16_tensor_pair(H, X, n_tok, d, st);
  CUtensorMap map;
  TB_TRY(make_map_2d(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, sizeof(__nv_bfloat16), X, (unsigned long long)d,
                     (unsigned long long)n_tok, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  const int m_blocks = (d + TC_BM - 1) / TC_BM;
  int n_tiles = 0;
  for (int mi = 0; mi < m_blocks; ++mi) n_tiles += mi / 2 + 1;
  int dev = 0, sms = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  TB_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  static bool configured[64] = {false};
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!configured[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_syrk_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM));
    configured[dev] = true;
  }
  // as many CTAs as fill the rounds of tiles evenly (the same number of rounds as with every SM)
  const int rounds = (n_tiles + sms - 1) / (sms > 0 ? sms : 1);
  const int grid = (n_tiles + rounds - 1) / rounds;
  k_syrk_tc<<<grid, TC_THREADS, TC_SMEM, st>>>(H, map, (int)n_tok, d, n_tiles);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

}  // namespace tb

// 0, or 1 once a bounded wait inside a tensor-core kernel has run out (sticky until read).
namespace tb {
int sweep_error_read_clear();  // the same word of the column-sweep kernel (tb_quantize.cu)
int yw_error_read_clear();     // and of the tensor-core product of the scale refinement (tb_gemm_tc.cu)
int cross_error_read_clear();  // and of the deviation correlation (tb_cross_tc.cu)
int pair_error_read_clear();   // and of the CTA-pair form of the Hessian kernel (tb_syrk_tc2.cu)
}

// One CTA waits on an mbarrier at which nothing ever arrives, through the same bounded wait the
// tensor-core kernels use, with the given cycle budget: the wait must give up, raise the device
// error word and let the kernel return.
namespace tb {
__global__ void k_bounded_wait_probe(long long budget_cycles, int* __restrict__ gave_up) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, &g_tc_error, budget_cycles);
  __syncthreads();
  if (threadIdx.x == 0 && gave_up) *gave_up = ok ? 0 : 1;
}
}  // namespace tb

extern "C" tb_status tb_selftest_bounded_wait(long long budget_cycles, int* gave_up, void* stream) {
  if (budget_cycles < 0 || budget_cycles > 200000000ll) return TB_ERR_INVALID_ARG;  // at most ~0.1 s
  tb::k_bounded_wait_probe<<<1, 64, 0, tb::as_stream(stream)>>>(budget_cycles, gave_up);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

extern "C" int tb_device_error_flag(void) {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, tb::g_tc_error, sizeof(int)) != cudaSuccess) return -1;
  if (v) {
    int z = 0;
    cudaMemcpyToSymbol(tb::g_tc_error, &z, sizeof(int));
  }
  const int w = tb::sweep_error_read_clear();
  const int y = tb::yw_error_read_clear();
  const int x = tb::cross_error_read_clear();
  const int q = tb::pair_error_read_clear();
  if (w < 0 || y < 0 || x < 0 || q < 0) return -1;
  return (v || w || y || x || q) ? 1 : 0;
}
