// Blockwise product Yw[r][g][:] = Wbar[r, G_g] H_in[G_g, :] of the scale refinement
// (Algorithm 3: one row of products per scale) on the 5th-generation tensor cores.
//
// Wbar = W_int - z holds small integers, exact in bf16.  H_in (float) is split
// exactly into three bf16 pieces, H = H1 + H2 + H3 (8 + 8 + 8 mantissa bits), so
// every product Wbar * H_p is exact in float and the only rounding is the float
// accumulation of 3 * |G_g| terms per output in tensor memory.  The result is
// stored in float: it feeds coefficients and small corrections of the
// refinement, where a relative error of a few 1e-7 is three orders of magnitude
// below the tolerance on the scales.
//
// Both operands are MN-major (the contraction index is the strided one): Wbar is
// written transposed, [d_in][rows], by the preparation kernel, H_in's pieces are
// [d_in][d_in] row-major.  Same machinery as the Hessian kernel: TMA boxes of
// 64 x 64 with the 128-byte swizzle, mbarrier ring, tcgen05.mma kind::f16 with
// accumulators in TMEM, two accumulator buffers so that the epilogue of one tile
// overlaps the MMAs of the next.  Warps 0-7 epilogue, warp 8 TMA producer, warp 9
// MMA issuer.  Every mbarrier wait is bounded.
#include "tb_common.cuh"
#include "tb_tma.cuh"

namespace tb {

enum {
  YT_BM = 128,
  YT_BN = 128,
  YT_BK = 128,                        // a whole quantization group per product
  YT_STAGES = 2,
  YT_BOX = 64 * 64 * 2,
  YT_A_BYTES = 4 * YT_BOX,            // Wbar^T: 128 k x 128 rows
  YT_B_BYTES = 3 * 4 * YT_BOX,        // three pieces of H_in: 128 k x 128 columns each
  YT_STAGE_OUT = 8 * 32 * 33 * 4,     // epilogue staging, one 32 x 33 float tile per warp
  YT_THREADS = 320,
  YT_SMEM = YT_B_BYTES + YT_STAGES * YT_A_BYTES + YT_STAGE_OUT + 1024 + 256
};

__device__ int g_yt_error = 0;

// H (float) -> three bf16 pieces with H = p1 + p2 + p3 exactly (for finite normal values)
__global__ void k_split3(const float* __restrict__ H, __nv_bfloat16* __restrict__ out, long long n) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const float x = H[i];
    const __nv_bfloat16 p1 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(p1);
    const __nv_bfloat16 p2 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(p2);
    out[i] = p1;
    out[n + i] = p2;
    out[2 * n + i] = __float2bfloat16_rn(r2);
  }
}

// WbT[k][r] = code[r][k] - z[r][group(k)] as bf16 (exact), tiled transpose
__global__ void k_wbar_transpose(const unsigned char* __restrict__ codes, const int* __restrict__ z,
                                 __nv_bfloat16* __restrict__ WbT, long long rows, int d, int seg, int ng) {
  __shared__ float tile[32][33];
  const long long r0 = (long long)blockIdx.y * 32;
  const int k0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const long long r = r0 + i;
    const int k = k0 + threadIdx.x;
    tile[i][threadIdx.x] = (r < rows) ? (float)((int)codes[r * d + k] - z[r * ng + k / seg]) : 0.0f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int k = k0 + i;
    const long long r = r0 + threadIdx.x;
    if (r < rows) WbT[(long long)k * rows + r] = __float2bfloat16_rn(tile[threadIdx.x][i]);
  }
}

__global__ void __launch_bounds__(YT_THREADS, 1)
    k_yw_tc(float* __restrict__ Yw, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            int rows, int d, int seg, int ng, int n_units, int hunits, int rows_per_hunit) {
  extern __shared__ unsigned char yt_raw[];
  const uint32_t raw = smem_u32(yt_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = yt_raw + (base - raw);
  const uint32_t sb = base;                      // H_in pieces of the unit: [3][2 k-halves][2 n-halves] boxes
  const uint32_t sa0 = base + YT_B_BYTES;        // Wbar^T ring: [stage][2 k-halves][2 row-halves] boxes
  float* stage = reinterpret_cast<float*>(gen_base + YT_B_BYTES + YT_STAGES * YT_A_BYTES);  // [8 warps][32][33]
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + YT_B_BYTES + YT_STAGES * YT_A_BYTES + YT_STAGE_OUT);
  // bars[0..1] a_full, [2..3] a_empty, [4] b_full, [5] b_empty, [6..7] acc_full, [8..9] acc_empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto afull_bar = [&](int s) { return bar0 + 8u * s; };
  auto aempty_bar = [&](int s) { return bar0 + 8u * (2 + s); };
  const uint32_t bfull_bar = bar0 + 8u * 4, bempty_bar = bar0 + 8u * 5;
  auto accf_bar = [&](int b) { return bar0 + 8u * (6 + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (8 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < YT_STAGES; ++s) {
      mbar_init(afull_bar(s), 1);
      mbar_init(aempty_bar(s), 1);
    }
    mbar_init(bfull_bar, 1);
    mbar_init(bempty_bar, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 8);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // hunits > 1: every block of rows_per_hunit rows (a head; a multiple of 128) has its own H_in, whose
  // pieces are stacked [piece][head][k]; the units then also run over the heads
  const int m_tiles = (rows_per_hunit + YT_BM - 1) / YT_BM, n_tilesN = (d + YT_BN - 1) / YT_BN;
  const int units_per_head = ng * n_tilesN;
  const int khalves = seg / 64;  // 1 or 2 boxes of 64 contraction steps per group
  // unit u -> (group g, column tile nj): the unit's slice of H_in stays in shared memory while
  // the row tiles stream through
  if (warp == 8) {
    if (lane == 0) {
      uint32_t it = 0, unit_it = 0;
      for (int u = blockIdx.x; u < n_units && !*abort_flag; u += gridDim.x, ++unit_it) {
        const int hu = u / units_per_head, ur = u % units_per_head;
        const int g = ur / n_tilesN, nj = ur % n_tilesN;
        const int n0 = nj * YT_BN, k00 = g * seg;
        if (!mbar_wait(bempty_bar, (unit_it & 1u) ^ 1u, abort_flag, &g_yt_error)) break;
        mbar_expect_tx(bfull_bar, 3u * khalves * 2u * YT_BOX);
#pragma unroll
        for (int pc = 0; pc < 3; ++pc)
          for (int kh = 0; kh < khalves; ++kh)
#pragma unroll
            for (int j = 0; j < 2; ++j)
              tma_load_2d(sb + ((pc * 2 + kh) * 2 + j) * YT_BOX, &map_b, n0 + 64 * j,
                          (pc * hunits + hu) * d + k00 + 64 * kh, bfull_bar);
        bool ok = true;
        for (int mi = 0; mi < m_tiles; ++mi, ++it) {
          const int s = it % YT_STAGES;
          const uint32_t ph = (it / YT_STAGES) & 1u;
          if (!mbar_wait(aempty_bar(s), ph ^ 1u, abort_flag, &g_yt_error)) {
            ok = false;
            break;
          }
          mbar_expect_tx(afull_bar(s), khalves * 2u * YT_BOX);
          const uint32_t sa = sa0 + s * YT_A_BYTES;
          for (int kh = 0; kh < khalves; ++kh)
#pragma unroll
            for (int j = 0; j < 2; ++j)
              tma_load_2d(sa + (kh * 2 + j) * YT_BOX, &map_a, hu * rows_per_hunit + mi * YT_BM + 64 * j, k00 + 64 * kh,
                          afull_bar(s));
        }
        if (!ok) break;
      }
    }
  } else if (warp == 9) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_mn(YT_BM, YT_BN);
      uint32_t it = 0, unit_it = 0;
      for (int u = blockIdx.x; u < n_units && !*abort_flag; u += gridDim.x, ++unit_it) {
        if (!mbar_wait(bfull_bar, unit_it & 1u, abort_flag, &g_yt_error)) break;
        bool ok = true;
        for (int mi = 0; mi < m_tiles; ++mi, ++it) {
          const int b = it & 1;
          if (!mbar_wait(acce_bar(b), ((it >> 1) & 1u) ^ 1u, abort_flag, &g_yt_error)) {
            ok = false;
            break;
          }
          const int s = it % YT_STAGES;
          const uint32_t ph = (it / YT_STAGES) & 1u;
          if (!mbar_wait(afull_bar(s), ph, abort_flag, &g_yt_error)) {
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t tmem_d = tmem_base + (uint32_t)b * YT_BN;
          const uint32_t sa = sa0 + s * YT_A_BYTES;
          for (int kk = 0; kk < 4 * khalves; ++kk) {
            const uint32_t koff = (uint32_t)(kk >> 2) * 2 * YT_BOX + (uint32_t)(kk & 3) * 2048;
            const uint64_t adesc = smem_desc_mn_sw128(sa + koff);
#pragma unroll
            for (int pc = 0; pc < 3; ++pc) {
              const uint64_t bdesc = smem_desc_mn_sw128(sb + pc * 4 * YT_BOX + koff);
              umma_bf16(tmem_d, adesc, bdesc, idesc, (kk > 0 || pc > 0) ? 1u : 0u);
            }
          }
          umma_commit(aempty_bar(s));
          umma_commit(accf_bar(b));
        }
        if (!ok) break;
        umma_commit(bempty_bar);  // every product of the unit has read its H_in slice
      }
    }
  } else {
    // epilogue warps 0-7: TMEM lanes 32 (w % 4) .., columns 64 (w / 4) ..; a warp turns its
    // 32 x 32 pieces through shared memory so that every store covers one 128-byte row piece
    const int q = warp & 3, hf = warp >> 2;
    float* st = stage + warp * (32 * 33);
    uint32_t it = 0;
    for (int u = blockIdx.x; u < n_units && !*abort_flag; u += gridDim.x) {
      const int hu = u / units_per_head, ur = u % units_per_head;
      const int g = ur / n_tilesN, nj = ur % n_tilesN;
      bool ok = true;
      for (int mi = 0; mi < m_tiles; ++mi, ++it) {
        const int b = it & 1;
        if (!mbar_wait(accf_bar(b), (it >> 1) & 1u, abort_flag, &g_yt_error)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * YT_BN + hf * 64);
        uint32_t r0[32], r1[32];
        tmem_ld_32x32(taddr, r0);
        tmem_ld_32x32(taddr + 32, r1);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(b));   // the accumulator may be overwritten
        const long long gr0 = (long long)hu * rows_per_hunit + (long long)mi * YT_BM + q * 32;
        const int gc0 = nj * YT_BN + hf * 64;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
#pragma unroll
          for (int i = 0; i < 32; ++i) st[lane * 33 + i] = __uint_as_float(c == 0 ? r0[i] : r1[i]);
          __syncwarp();
          const int gc = gc0 + 32 * c + lane;
          if (gc < d) {
#pragma unroll 8
            for (int r = 0; r < 32; ++r)
              if (gr0 + r < rows) Yw[((gr0 + r) * ng + g) * (long long)d + gc] = st[r * 33 + lane];
          }
          __syncwarp();
        }
      }
      if (!ok) break;
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// The same product for groups wider than 128 columns: the H_in pieces stream through the
// ring together with Wbar^T, 64 contraction steps per stage (no slice stays resident).
enum {
  YS_BK = 64,
  YS_STAGES = 3,
  YS_A_BYTES = 2 * YT_BOX,            // Wbar^T: 64 k x 128 rows
  YS_B_BYTES = 3 * 2 * YT_BOX,        // three pieces of H_in: 64 k x 128 columns each
  YS_STAGE_BYTES = YS_A_BYTES + YS_B_BYTES,
  YS_SMEM = YS_STAGES * YS_STAGE_BYTES + 1024 + 256
};

__global__ void __launch_bounds__(YT_THREADS, 1)
    k_yw_tc_stream(float* __restrict__ Yw, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            int rows, int d, int seg, int ng, int n_tiles) {
  extern __shared__ unsigned char ys_raw[];
  const uint32_t raw = smem_u32(ys_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = ys_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + YS_STAGES * YS_STAGE_BYTES);
  // bars[0..2] full, [3..5] empty, [6..7] acc_full, [8..9] acc_empty; then tmem slot, abort flag
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (3 + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (6 + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (8 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < YS_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 8);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int n_stages = seg / YS_BK;                       // stages per tile
  const int m_tiles = (rows + YT_BM - 1) / YT_BM, n_tilesN = (d + YT_BN - 1) / YT_BN;
  // tile t -> (group g, row tile mi, column tile nj), column tiles innermost
  auto tile_of = [&](int t, int& g, int& mi, int& nj) {
    nj = t % n_tilesN;
    mi = (t / n_tilesN) % m_tiles;
    g = t / (n_tilesN * m_tiles);
  };

  if (warp == 8) {
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        int g, mi, nj;
        tile_of(t, g, mi, nj);
        const int m0 = mi * YT_BM, n0 = nj * YT_BN, k00 = g * seg;
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % YS_STAGES;
          const uint32_t ph = (it / YS_STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, &g_yt_error)) break;
          mbar_expect_tx(full_bar(s), YS_STAGE_BYTES);
          const uint32_t sa = base + s * YS_STAGE_BYTES, sb = sa + YS_A_BYTES;
          const int k0 = k00 + st * YS_BK;
#pragma unroll
          for (int j = 0; j < 2; ++j) tma_load_2d(sa + j * YT_BOX, &map_a, m0 + 64 * j, k0, full_bar(s));
#pragma unroll
          for (int pc = 0; pc < 3; ++pc)
#pragma unroll
            for (int j = 0; j < 2; ++j)
              tma_load_2d(sb + (pc * 2 + j) * YT_BOX, &map_b, n0 + 64 * j, pc * d + k0, full_bar(s));
        }
      }
    }
  } else if (warp == 9) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_mn(YT_BM, YT_BN);
      uint32_t it = 0, tile_it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x, ++tile_it) {
        const int b = tile_it & 1;
        if (!mbar_wait(acce_bar(b), ((tile_it >> 1) & 1u) ^ 1u, abort_flag, &g_yt_error)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + (uint32_t)b * YT_BN;
        bool ok = true;
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % YS_STAGES;
          const uint32_t ph = (it / YS_STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, &g_yt_error)) {
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + s * YS_STAGE_BYTES, sb = sa + YS_A_BYTES;
#pragma unroll
          for (int kk = 0; kk < YS_BK / 16; ++kk) {
            const uint64_t adesc = smem_desc_mn_sw128(sa + kk * 2048);
#pragma unroll
            for (int pc = 0; pc < 3; ++pc) {
              const uint64_t bdesc = smem_desc_mn_sw128(sb + pc * 2 * YT_BOX + kk * 2048);
              umma_bf16(tmem_d, adesc, bdesc, idesc, (st > 0 || kk > 0 || pc > 0) ? 1u : 0u);
            }
          }
          umma_commit(empty_bar(s));
        }
        if (!ok) break;
        umma_commit(accf_bar(b));
      }
    }
  } else {
    // epilogue warps 0-7: TMEM lanes 32 (w % 4) .., columns 64 (w / 4) ..
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    uint32_t tile_it = 0;
    for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x, ++tile_it) {
      int g, mi, nj;
      tile_of(t, g, mi, nj);
      const int b = tile_it & 1;
      if (!mbar_wait(accf_bar(b), (tile_it >> 1) & 1u, abort_flag, &g_yt_error)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * YT_BN + hf * 64);
      uint32_t r0[32], r1[32];
      tmem_ld_32x32(taddr, r0);
      tmem_ld_32x32(taddr + 32, r1);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar(b));   // the accumulator may be overwritten
      const long long gr = (long long)mi * YT_BM + row;
      const int gc = nj * YT_BN + hf * 64;
      if (gr < rows) {
        float* dst = Yw + (gr * ng + g) * (long long)d + gc;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          if (gc + i + 3 < d)
            *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(r0[i]), __uint_as_float(r0[i + 1]),
                                                              __uint_as_float(r0[i + 2]), __uint_as_float(r0[i + 3]));
          if (gc + 32 + i + 3 < d)
            *reinterpret_cast<float4*>(dst + 32 + i) = make_float4(__uint_as_float(r1[i]), __uint_as_float(r1[i + 1]),
                                                                   __uint_as_float(r1[i + 2]), __uint_as_float(r1[i + 3]));
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// Yw (float, [rows][ng][d]) from the codes; WbT ([d][rows] bf16) and Hp ([3][d][d] bf16) are scratch.
// Requires seg % 64 == 0, d % 8 == 0, rows % 8 == 0.
tb_status yw_tensor(float* Yw, const unsigned char* codes, const int* zeros, const float* H_in, __nv_bfloat16* WbT,
                    __nv_bfloat16* Hp, bool split_h, long long rows, int d, int seg, int ng, int hunits,
                    cudaStream_t st) {
  const long long dd = (long long)d * d;
  if (hunits > 1 && (seg > 128 || (rows / hunits) % YT_BM || rows % hunits)) return TB_ERR_UNSUPPORTED;
  if (split_h) {
    k_split3<<<148 * 8, 256, 0, st>>>(H_in, Hp, dd * hunits);
    TB_LAUNCH_CHECK();
  }
  k_wbar_transpose<<<dim3(d / 32, (unsigned)((rows + 31) / 32)), dim3(32, 8), 0, st>>>(codes, zeros, WbT, rows, d, seg, ng);
  TB_LAUNCH_CHECK();
  CUtensorMap map_a, map_b;
  TB_TRY(make_map_2d(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, WbT, (unsigned long long)rows, (unsigned long long)d,
                     64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  TB_TRY(make_map_2d(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Hp, (unsigned long long)d,
                     (unsigned long long)3 * hunits * d, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  const int m_tiles = (int)((rows + YT_BM - 1) / YT_BM), n_tilesN = (d + YT_BN - 1) / YT_BN;
  const bool resident = (seg <= 128);  // the group's slice of H_in fits next to the Wbar^T ring
  const long long n_tiles = resident ? (long long)n_tilesN * ng * hunits   // units: one (head, group, column tile) each
                                     : (long long)m_tiles * n_tilesN * ng;
  if (n_tiles > 0x7fffffffll) return TB_ERR_UNSUPPORTED;
  int dev = 0, sms = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  TB_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  static bool configured[64] = {false};
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!configured[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_yw_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)YT_SMEM));
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_yw_tc_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)YS_SMEM));
    configured[dev] = true;
  }
  // as many CTAs as fill the rounds of tiles evenly (the same number of rounds as with every SM: fewer CTAs
  // asking L2 at once, and less power, for the same time or less)
  const int rounds_of_tiles = (int)((n_tiles + sms - 1) / (sms > 0 ? sms : 1));
  const int grid = (int)((n_tiles + rounds_of_tiles - 1) / (rounds_of_tiles > 0 ? rounds_of_tiles : 1));
  if (resident)
    k_yw_tc<<<grid, YT_THREADS, YT_SMEM, st>>>(Yw, map_a, map_b, (int)rows, d, seg, ng, (int)n_tiles, hunits,
                                               (int)(rows / hunits));
  else
    k_yw_tc_stream<<<grid, YT_THREADS, YS_SMEM, st>>>(Yw, map_a, map_b, (int)rows, d, seg, ng, (int)n_tiles);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

// ---------------------------------------------------------------------------
// C (double, [M][ldc]) = A B for float A [M][K] and float B [K][N], both split
// exactly into three bf16 pieces; the six piece products that matter to float
// accuracy (1*1, 1*2, 2*1, 1*3, 3*1, 2*2) run on tcgen05 with float
// accumulation in TMEM over 128 contraction steps at a time, and the chunks are
// summed in double by the epilogue warps.  Used for G Hsum of the H_out build
// (Table 1).  A arrives transposed and split, AT [3][K][M]; B split, [3][K][N].
// ---------------------------------------------------------------------------
enum {
  GS_BM = 128,
  GS_BN = 128,
  GS_BK = 32,
  GS_STAGES = 4,
  GS_CHUNK = 4,                       // stages per TMEM accumulation (128 contraction steps)
  GS_BOX = 32 * 64 * 2,
  GS_A_BYTES = 3 * 2 * GS_BOX,
  GS_B_BYTES = 3 * 2 * GS_BOX,
  GS_STAGE_BYTES = GS_A_BYTES + GS_B_BYTES,
  GS_SMEM = GS_STAGES * GS_STAGE_BYTES + 1024 + 256
};

// AT[p][k][m] = piece p of A[m][k]; a double input keeps its leading 24 bits
template <typename TA>
__global__ void k_split3_transpose(const TA* __restrict__ A, __nv_bfloat16* __restrict__ AT, long long M, int K) {
  __shared__ TA tile[32][33];
  const long long m0 = (long long)blockIdx.y * 32;
  const int k0 = blockIdx.x * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const long long m = m0 + i;
    const int k = k0 + threadIdx.x;
    tile[i][threadIdx.x] = (m < M && k < K) ? A[m * K + k] : (TA)0;
  }
  __syncthreads();
  const long long plane = (long long)K * M;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int k = k0 + i;
    const long long m = m0 + threadIdx.x;
    if (m < M && k < K) {
      const TA x = tile[threadIdx.x][i];
      const __nv_bfloat16 p1 = __float2bfloat16_rn((float)x);
      const TA r1 = x - (TA)__bfloat162float(p1);  // exact in TA
      const __nv_bfloat16 p2 = __float2bfloat16_rn((float)r1);
      const long long o = (long long)k * M + m;
      AT[o] = p1;
      AT[plane + o] = p2;
      AT[2 * plane + o] = __float2bfloat16_rn((float)(r1 - (TA)__bfloat162float(p2)));
    }
  }
}

__global__ void __launch_bounds__(YT_THREADS, 1)
    k_gsplit_tc(double* __restrict__ C, long long ldc, const __grid_constant__ CUtensorMap map_a,
                const __grid_constant__ CUtensorMap map_b, int M, int N, int K, int n_tiles, int accumulate, int hunits,
                int rows_per_hunit) {
  extern __shared__ unsigned char gs_raw[];
  const uint32_t raw = smem_u32(gs_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen_base = gs_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + GS_STAGES * GS_STAGE_BYTES);
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
    for (int s = 0; s < GS_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 8);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int n_stages = (K + GS_BK - 1) / GS_BK;
  const int n_tilesN = (N + GS_BN - 1) / GS_BN;

  if (warp == 8) {
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        const int m0 = (t / n_tilesN) * GS_BM, n0 = (t % n_tilesN) * GS_BN;
        const int hu = (hunits > 1) ? m0 / rows_per_hunit : 0;  // the block of rows (head) whose B this tile multiplies
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % GS_STAGES;
          const uint32_t ph = (it / GS_STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, &g_yt_error)) break;
          mbar_expect_tx(full_bar(s), GS_STAGE_BYTES);
          const uint32_t sa = base + s * GS_STAGE_BYTES, sb = sa + GS_A_BYTES;
          const int k0 = st * GS_BK;
#pragma unroll
          for (int pc = 0; pc < 3; ++pc)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              tma_load_2d(sa + (pc * 2 + j) * GS_BOX, &map_a, m0 + 64 * j, pc * K + k0, full_bar(s));
              tma_load_2d(sb + (pc * 2 + j) * GS_BOX, &map_b, n0 + 64 * j, (pc * hunits + hu) * K + k0, full_bar(s));
            }
        }
      }
    }
  } else if (warp == 9) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_mn(GS_BM, GS_BN);
      uint32_t it = 0, chunk_it = 0;
      for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int in_chunk = st % GS_CHUNK;
          const int b = chunk_it & 1;
          if (in_chunk == 0) {
            if (!mbar_wait(acce_bar(b), ((chunk_it >> 1) & 1u) ^ 1u, abort_flag, &g_yt_error)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          const int s = it % GS_STAGES;
          const uint32_t ph = (it / GS_STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, &g_yt_error)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + s * GS_STAGE_BYTES, sb = sa + GS_A_BYTES;
          const uint32_t tmem_d = tmem_base + (uint32_t)b * GS_BN;
          bool first = (in_chunk == 0);
#pragma unroll
          for (int kk = 0; kk < GS_BK / 16; ++kk) {
            // piece pairs (a, b): 1*1, 1*2, 2*1, 1*3, 3*1, 2*2
            const int pa[6] = {0, 0, 1, 0, 2, 1}, pb[6] = {0, 1, 0, 2, 0, 1};
#pragma unroll
            for (int i = 0; i < 6; ++i) {
              const uint64_t adesc = smem_desc_mn_sw128(sa + pa[i] * 2 * GS_BOX + kk * 2048, GS_BOX);
              const uint64_t bdesc = smem_desc_mn_sw128(sb + pb[i] * 2 * GS_BOX + kk * 2048, GS_BOX);
              umma_bf16(tmem_d, adesc, bdesc, idesc, first ? 0u : 1u);
              first = false;
            }
          }
          umma_commit(empty_bar(s));
          if (in_chunk == GS_CHUNK - 1 || st == n_stages - 1) {
            umma_commit(accf_bar(b));
            ++chunk_it;
          }
        }
      }
    }
  } else {
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    uint32_t chunk_it = 0;
    for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
      const int m0 = (t / n_tilesN) * GS_BM, n0 = (t % n_tilesN) * GS_BN;
      double run[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) run[i] = 0.0;
      bool ok = true;
      for (int st0 = 0; st0 < n_stages && ok; st0 += GS_CHUNK, ++chunk_it) {
        const int b = chunk_it & 1;
        ok = mbar_wait(accf_bar(b), (chunk_it >> 1) & 1u, abort_flag, &g_yt_error);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * GS_BN + hf * 64);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(taddr + c * 32, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int i = 0; i < 32; ++i) run[c * 32 + i] += (double)__uint_as_float(r[i]);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(b));
      }
      if (ok) {
        const long long gm = (long long)m0 + row;
        if (gm < M) {
          double* dst = C + gm * ldc + n0 + hf * 64;
#pragma unroll
          for (int i = 0; i < 64; i += 2)
            if (n0 + hf * 64 + i + 1 < N) {
              double2 v = make_double2(run[i], run[i + 1]);
              if (accumulate) {
                const double2 old = *reinterpret_cast<const double2*>(dst + i);
                v.x += old.x;
                v.y += old.y;
              }
              *reinterpret_cast<double2*>(dst + i) = v;
            }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// C (+)= A B (double result) from operands already split: AT [3][K][M], Bp [3][K][N].
// Requires M % 8 == 0, N % 8 == 0, K % 32 == 0.
// hunits > 1: every block of M / hunits rows (a multiple of 128) multiplies its own B, Bp stacked [3][hunits][K][N].
tb_status gemm_split_presplit(double* C, long long ldc, const __nv_bfloat16* AT, const __nv_bfloat16* Bp, long long M,
                              int N, int K, bool accumulate, cudaStream_t st, int hunits) {
  if (hunits > 1 && (M % hunits || (M / hunits) % GS_BM)) return TB_ERR_UNSUPPORTED;
  CUtensorMap map_a, map_b;
  TB_TRY(make_map_2d(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, AT, (unsigned long long)M, (unsigned long long)3 * K,
                     64, 32, CU_TENSOR_MAP_SWIZZLE_128B));
  TB_TRY(make_map_2d(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bp, (unsigned long long)N,
                     (unsigned long long)3 * hunits * K, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B));
  const long long n_tiles = ((M + GS_BM - 1) / GS_BM) * (long long)((N + GS_BN - 1) / GS_BN);
  if (n_tiles > 0x7fffffffll) return TB_ERR_UNSUPPORTED;
  int dev = 0, sms = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  TB_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  static bool configured[64] = {false};
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!configured[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_gsplit_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GS_SMEM));
    configured[dev] = true;
  }
  // as many CTAs as fill the rounds of tiles evenly (the same number of rounds as with every SM: fewer CTAs
  // asking L2 at once, and less power, for the same time or less)
  const int rounds_of_tiles = (int)((n_tiles + sms - 1) / (sms > 0 ? sms : 1));
  const int grid = (int)((n_tiles + rounds_of_tiles - 1) / (rounds_of_tiles > 0 ? rounds_of_tiles : 1));
  k_gsplit_tc<<<grid, YT_THREADS, GS_SMEM, st>>>(C, ldc, map_a, map_b, (int)M, N, K, (int)n_tiles, accumulate ? 1 : 0,
                                                 hunits, (int)(M / hunits));
  TB_LAUNCH_CHECK();
  return TB_OK;
}

// Bp[p][i] = piece p of B[i]
tb_status split3(const float* B, __nv_bfloat16* Bp, long long n, cudaStream_t st) {
  k_split3<<<148 * 8, 256, 0, st>>>(B, Bp, n);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

tb_status split3_transpose(const float* A, __nv_bfloat16* AT, long long M, int K, cudaStream_t st) {
  k_split3_transpose<float><<<dim3((K + 31) / 32, (unsigned)((M + 31) / 32)), dim3(32, 8), 0, st>>>(A, AT, M, K);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

tb_status split3_transpose(const double* A, __nv_bfloat16* AT, long long M, int K, cudaStream_t st) {
  k_split3_transpose<double><<<dim3((K + 31) / 32, (unsigned)((M + 31) / 32)), dim3(32, 8), 0, st>>>(A, AT, M, K);
  TB_LAUNCH_CHECK();
  return TB_OK;
}

// C = A B (double result) through split bf16 pieces; AT ([3][K][M]) and Bp ([3][K][N]) are scratch.
tb_status gemm_split_tensor(double* C, long long ldc, const float* A, const float* B, __nv_bfloat16* AT,
                            __nv_bfloat16* Bp, long long M, int N, int K, cudaStream_t st) {
  TB_TRY(split3(B, Bp, (long long)K * N, st));
  TB_TRY(split3_transpose(A, AT, M, K, st));
  return gemm_split_presplit(C, ldc, AT, Bp, M, N, K, false, st, 1);
}

int yw_error_read_clear() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_yt_error, sizeof(int)) != cudaSuccess) return -1;
  if (v) {
    int z = 0;
    cudaMemcpyToSymbol(g_yt_error, &z, sizeof(int));
  }
  return v;
}

}  // namespace tb
