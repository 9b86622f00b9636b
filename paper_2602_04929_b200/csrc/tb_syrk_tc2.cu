// Hessian accumulation H += X^T X for bf16 activations, CTA-pair form: two CTAs of a cluster share
// one 256 x 256 tile of H (tcgen05.mma with cta_group::2).  CTA r of the pair stages the 128
// columns of X that make its rows of the tile (operand A) and its half of the 256 columns that
// make the tile's columns (operand B); the tensor cores of both SMs read both halves of B, so each
// SM fetches 32 KB per 64 tokens for its 128 x 256 share where the single-CTA kernel fetches 48 KB for
// a 128 x 256 tile: a third less operand traffic from L2 per flop.  Everything else is as in the
// single-CTA kernel: 2048 tokens per accumulation in one of two TMEM buffers, drained into float
// registers by the epilogue warps while the other buffer fills, one owner per tile for the whole
// token range, the same additions in the same order.
//
// Roles per CTA (320 threads): warps 0-7 epilogue, warp 8 TMA producer, warp 9 the MMA issuer (CTA 0
// only: one thread issues the MMAs of the pair).  The loads of both CTAs are counted at CTA 0's stage
// barrier (the cta_group::2 form of the TMA load may name a barrier of the partner CTA; no load is shared
// between CTAs).  A tcgen05.commit of CTA 0 arrives at the same barrier offset in both CTAs; the
// epilogue warps of CTA 1 release an accumulator buffer by a remote arrive.  Barriers that are completed
// from the partner CTA are polled (test_wait) rather than waited on with a suspending try_wait.
// Every wait is bounded; a wait that gives up raises the device error word, and both CTAs still
// meet at the closing cluster barrier and free their tensor memory.
#include "tb_common.cuh"
#include "tb_tma.cuh"

namespace tb {

enum {
  T2_BK = 64,           // tokens per pipeline stage
  T2_STAGES = 6,
  T2_CHUNK = 32,        // stages per TMEM accumulation (2048 tokens)
  T2_BOX_BYTES = 64 * 64 * 2,
  T2_A_BYTES = 2 * T2_BOX_BYTES,
  T2_B_BYTES = 2 * T2_BOX_BYTES,
  T2_STAGE_BYTES = T2_A_BYTES + T2_B_BYTES,
  T2_THREADS = 320,
  T2_SMEM = T2_STAGES * T2_STAGE_BYTES + 1024 /*alignment*/ + 512 /*barriers*/
};

__device__ int g_pair_error = 0;

__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives, once the MMAs issued so far have completed, at the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"((unsigned short)3)
               : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted at a barrier that may live in the other
// CTA of the pair (`bar` is a shared::cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bounded wait that polls without suspending: for barriers completed from the other CTA of the pair
// (a remote arrive, or a commit sent to both CTAs).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_poll(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* device_error_word) {
  if (mbar_test_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_test_wait(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > MBAR_WAIT_BUDGET) {
      *abort_flag = 1;
      atomicExch(device_error_word, 1);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(T2_THREADS, 1)
    k_syrk_tc_pair(float* __restrict__ H, const __grid_constant__ CUtensorMap xmap, int n_tok, int d, int n_tiles) {
  extern __shared__ unsigned char t2_smem_raw[];
  const uint32_t raw = smem_u32(t2_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;   // the same offset in both CTAs (same kernel, same layout)
  unsigned char* gen_base = t2_smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + T2_STAGES * T2_STAGE_BYTES);
  // full[S]: the TMA bytes of both CTAs, counted in CTA 0; empty[S], accf[2]: signalled in both CTAs by the
  // commits of CTA 0; acce[2]: in CTA 0, the epilogue warps of both CTAs arrive
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4 * T2_STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (T2_STAGES + s); };
  auto accf_bar = [&](int b) { return bar0 + 8u * (3 * T2_STAGES + b); };
  auto acce_bar = [&](int b) { return bar0 + 8u * (3 * T2_STAGES + 2 + b); };

  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < T2_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), 1);
      mbar_init(acce_bar(b), 16);  // one arrival per epilogue warp of either CTA
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_barrier();  // both CTAs' barriers are initialised before anything arrives at them from outside
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int n_stages = (n_tok + T2_BK - 1) / T2_BK;
  const int m_blocks = (d + 255) / 256;
  // tile t -> (mi, nj): row block mi (256 rows) has the column blocks nj = 0 .. mi
  auto tile_of = [&](int t, int& mi, int& nj) {
    int acc = 0;
    for (mi = 0; mi < m_blocks; ++mi) {
      if (t < acc + mi + 1) {
        nj = t - acc;
        return;
      }
      acc += mi + 1;
    }
    mi = m_blocks - 1;
    nj = 0;
  };

  if (warp == 8) {
    // ---------------- TMA producer (both CTAs: own rows of A, own half of B) ----------------
    if (lane == 0) {
      uint32_t it = 0;
      for (int t = pair; t < n_tiles && !*abort_flag; t += n_pairs) {
        int mi, nj;
        tile_of(t, mi, nj);
        const int m0 = mi * 256 + 128 * (int)rank, n0 = nj * 256 + 128 * (int)rank;
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int s = it % T2_STAGES;
          const uint32_t ph = (it / T2_STAGES) & 1u;
          if (!mbar_poll(empty_bar(s), ph ^ 1u, abort_flag, &g_pair_error)) break;
          // both CTAs' bytes are counted at CTA 0's barrier, which expects the two stages
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * T2_STAGE_BYTES);
          const uint32_t fb = map_to_rank(full_bar(s), 0);
          const uint32_t sa = base + s * T2_STAGE_BYTES, sb = sa + T2_A_BYTES;
          const int k0 = st * T2_BK;
#pragma unroll
          for (int j = 0; j < 2; ++j) tma_load_2d_pair(sa + j * T2_BOX_BYTES, &xmap, m0 + 64 * j, k0, fb);
#pragma unroll
          for (int j = 0; j < 2; ++j) tma_load_2d_pair(sb + j * T2_BOX_BYTES, &xmap, n0 + 64 * j, k0, fb);
        }
      }
    }
  } else if (warp == 9 && rank == 1) {
    // nothing to do in CTA 1: CTA 0 issues the MMAs of the pair
  } else if (warp == 9) {
    // ---------------- MMA issuer (CTA 0) ----------------
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_mn(256, 256);
      uint32_t it = 0, chunk_it = 0;
      for (int t = pair; t < n_tiles && !*abort_flag; t += n_pairs) {
        for (int st = 0; st < n_stages; ++st, ++it) {
          const int in_chunk = st % T2_CHUNK;
          const int b = chunk_it & 1;
          if (in_chunk == 0) {
            // the accumulator buffer must have been drained by the epilogue warps of both CTAs
            if (!mbar_poll(acce_bar(b), ((chunk_it >> 1) & 1u) ^ 1u, abort_flag, &g_pair_error)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          const int s = it % T2_STAGES;
          const uint32_t ph = (it / T2_STAGES) & 1u;
          if (!mbar_poll(full_bar(s), ph, abort_flag, &g_pair_error)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = base + s * T2_STAGE_BYTES, sb = sa + T2_A_BYTES;
          const uint32_t tmem_d = tmem_base + (uint32_t)b * 256u;
#pragma unroll
          for (int kk = 0; kk < T2_BK / 16; ++kk) {
            const uint64_t adesc = smem_desc_mn_sw128(sa + kk * 2048);
            const uint64_t bdesc = smem_desc_mn_sw128(sb + kk * 2048);
            umma_bf16_pair(tmem_d, adesc, bdesc, idesc, (in_chunk > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(s));  // both CTAs may refill the stage once these MMAs have read it
          if (in_chunk == T2_CHUNK - 1 || st == n_stages - 1) {
            umma_commit_pair(accf_bar(b));  // the chunk's accumulator is complete in both CTAs
            ++chunk_it;
          }
        }
      }
    }
  } else {
    // ---------------- epilogue warps 0-7 (own 128 rows of the tile, all 256 columns) ----------------
    const int q = warp & 3, hf = warp >> 2;
    const int row = q * 32 + lane;
    uint32_t chunk_it = 0;
    for (int t = pair; t < n_tiles && !*abort_flag; t += n_pairs) {
      int mi, nj;
      tile_of(t, mi, nj);
      const int m0 = mi * 256 + 128 * (int)rank, n0 = nj * 256;
      // running sums start from H and go back at the end (so calls split at multiples of 2048 tokens add
      // up exactly like one call); entries right of this CTA's 128-wide diagonal block belong to the mirror pass
      float run[128];
      const int gm = m0 + row;
      float* hrow = H + (long long)gm * d;
#pragma unroll
      for (int i = 0; i < 128; ++i) {
        const int gn = n0 + hf * 128 + i;
        run[i] = (gm < d && gn < d && gn < m0 + 128) ? hrow[gn] : 0.0f;
      }
      bool ok = true;
      for (int st0 = 0; st0 < n_stages && ok; st0 += T2_CHUNK, ++chunk_it) {
        const int b = chunk_it & 1;
        int okw = 1;
        if (lane == 0) okw = mbar_poll(accf_bar(b), (chunk_it >> 1) & 1u, abort_flag, &g_pair_error) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, okw, 0) != 0;
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * 256 + hf * 128);
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
        if (lane == 0) {
          if (rank == 0)
            mbar_arrive(acce_bar(b));
          else
            mbar_arrive_remote(map_to_rank(acce_bar(b), 0));
        }
      }
      if (ok && gm < d) {
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          const int gn = n0 + hf * 128 + i;
          if (gn < d && gn < m0 + 128) hrow[gn] = run[i];
        }
      }
    }
  }

  // nobody leaves while the other CTA may still signal into this one or read its shared memory
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_barrier();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

int pair_error_read_clear() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_pair_error, sizeof(int)) != cudaSuccess) return -1;
  if (v) {
    int z = 0;
    cudaMemcpyToSymbol(g_pair_error, &z, sizeof(int));
  }
  return v;
}

// H += X^T X for bf16 X, 256 x 256 tiles on or below the diagonal, one per CTA pair.
tb_status syrk_bf16_tensor_pair(float* H, const __nv_bfloat16* X, long long n_tok, int d, cudaStream_t st) {
  if (n_tok > 0x7fffffffll) return TB_ERR_UNSUPPORTED;
  CUtensorMap map;
  TB_TRY(make_map_2d(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, sizeof(__nv_bfloat16), X, (unsigned long long)d,
                     (unsigned long long)n_tok, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B));
  const int m_blocks = (d + 255) / 256;
  const int n_tiles = m_blocks * (m_blocks + 1) / 2;
  int dev = 0, sms = 0;
  TB_CUDA_CHECK(cudaGetDevice(&dev));
  TB_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  static bool configured[64] = {false};
  if (dev < 0 || dev >= 64) return TB_ERR_CUDA;
  if (!configured[dev]) {
    TB_CUDA_CHECK(cudaFuncSetAttribute(k_syrk_tc_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T2_SMEM));
    configured[dev] = true;
  }
  // as many pairs as fill the rounds evenly: 528 tiles on 74 pairs take 8 rounds, the last one with 10 tiles;
  // 66 pairs take the same 8 rounds and leave 16 SMs (and their share of the power budget) to other work
  const int max_pairs = sms / 2 > 0 ? sms / 2 : 1;
  const int rounds = (n_tiles + max_pairs - 1) / max_pairs;
  const int pairs = (n_tiles + rounds - 1) / rounds;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(T2_THREADS);
  cfg.dynamicSmemBytes = T2_SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  TB_CUDA_CHECK(cudaLaunchKernelEx(&cfg, k_syrk_tc_pair, H, map, (int)n_tok, d, n_tiles));
  TB_LAUNCH_CHECK();
  return TB_OK;
}

}  // namespace tb
