// Bit-packed storage of the integer weights W_int in {0 .. 2^b - 1} (Section 2.1:
// Q = diag(s) W_int) and the fused unpack + dequantize + compare.
//
// Format: every row is a little-endian bit stream, code j of the row in bits
// [j b, (j + 1) b) counted from the least significant bit of 32-bit word 0; rows
// are d_in * b / 32 words long (d_in is a multiple of 32, so rows end on a word
// boundary).  A code may straddle two words when b does not divide 32.
//
// Both kernels are pure data movement: one thread handles 32 consecutive codes of
// a row, i.e. two 16-byte loads (or stores) of codes and b whole words of the
// stream; a warp covers 1024 consecutive codes, so the code side is fully
// coalesced and the word side is contiguous per warp.
#include "tb_common.cuh"

namespace tb {

template <int BITS>
__global__ void __launch_bounds__(256) k_pack_codes(const unsigned char* __restrict__ codes,
                                                    unsigned int* __restrict__ packed, long long n_groups) {
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < n_groups;
       g += (long long)gridDim.x * blockDim.x) {
    const uint4* src = reinterpret_cast<const uint4*>(codes + g * 32);
    const uint4 a = src[0], b = src[1];
    const unsigned int w8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    unsigned long long acc = 0;   // bits of the stream not yet written
    int have = 0;
    unsigned int* dst = packed + g * BITS;
    int o = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const unsigned int c = (w8[i >> 2] >> (8 * (i & 3))) & ((1u << BITS) - 1u);
      acc |= (unsigned long long)c << have;
      have += BITS;
      if (have >= 32) {
        dst[o++] = (unsigned int)acc;
        acc >>= 32;
        have -= 32;
      }
    }
  }
}

struct UnpackP {
  const unsigned int* packed;
  const float* scales;
  const int* zeros;
  unsigned char* codes_out;
  float* what_out;
  const unsigned char* codes_ref;
  const float* what_ref;
  unsigned long long* mismatch;  // [0] codes that differ from codes_ref, [1] values beyond tol of what_ref
  long long n_groups;
  int d_in, seg, ng;
  float tol;
};

template <int BITS>
__global__ void __launch_bounds__(256) k_unpack_dequant(UnpackP p) {
  unsigned long long bad_codes = 0, bad_vals = 0;
  const int groups_per_row = p.d_in / 32;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < p.n_groups;
       g += (long long)gridDim.x * blockDim.x) {
    const long long row = g / groups_per_row;
    const int col0 = (int)(g % groups_per_row) * 32;
    // 32 columns lie in one column group (groups are multiples of 32 columns)
    const long long so = row * p.ng + col0 / p.seg;
    const float s = p.scales[so];
    const int z = p.zeros[so];
    const unsigned int* src = p.packed + g * BITS;
    unsigned long long acc = 0;
    int have = 0, o = 0;
    unsigned int out8[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    float vals[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      if (have < BITS) {
        acc |= (unsigned long long)src[o++] << have;
        have += 32;
      }
      const unsigned int c = (unsigned int)acc & ((1u << BITS) - 1u);
      acc >>= BITS;
      have -= BITS;
      out8[i >> 2] |= c << (8 * (i & 3));
      vals[i] = s * (float)((int)c - z);
    }
    const long long e0 = g * 32;
    if (p.codes_out) {
      uint4* dst = reinterpret_cast<uint4*>(p.codes_out + e0);
      dst[0] = make_uint4(out8[0], out8[1], out8[2], out8[3]);
      dst[1] = make_uint4(out8[4], out8[5], out8[6], out8[7]);
    }
    if (p.codes_ref) {
      const uint4* ref = reinterpret_cast<const uint4*>(p.codes_ref + e0);
      const uint4 a = ref[0], b = ref[1];
      const unsigned int r8[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const unsigned int x = r8[i] ^ out8[i];
        bad_codes += ((x & 0xffu) != 0) + ((x & 0xff00u) != 0) + ((x & 0xff0000u) != 0) + ((x & 0xff000000u) != 0);
      }
    }
    if (p.what_out) {
      float4* dst = reinterpret_cast<float4*>(p.what_out + e0);
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[i] = make_float4(vals[4 * i], vals[4 * i + 1], vals[4 * i + 2], vals[4 * i + 3]);
    }
    if (p.what_ref) {
      const float4* ref = reinterpret_cast<const float4*>(p.what_ref + e0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 r = ref[i];
        const float rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float v = vals[4 * i + k];
          // !(<=) so that a NaN on either side counts as a deviation
          if (!(fabsf(v - rr[k]) <= p.tol * fabsf(rr[k]))) ++bad_vals;
        }
      }
    }
  }
  if (p.mismatch) {
    bad_codes = __reduce_add_sync(0xffffffffu, (unsigned)bad_codes);
    bad_vals = __reduce_add_sync(0xffffffffu, (unsigned)bad_vals);
    if ((threadIdx.x & 31) == 0) {
      if (bad_codes) atomicAdd(&p.mismatch[0], bad_codes);
      if (bad_vals) atomicAdd(&p.mismatch[1], bad_vals);
    }
  }
}

static int pack_blocks(long long n_groups) {
  long long b = (n_groups + 255) / 256;
  if (b > 148 * 8) b = 148 * 8;
  return (int)(b < 1 ? 1 : b);
}

}  // namespace tb

using namespace tb;

extern "C" size_t tb_packed_bytes(int d_out, int d_in, int bits) {
  if (d_out <= 0 || d_in <= 0 || (d_in % 32) || bits < 2 || bits > 8) return 0;
  return (size_t)d_out * (size_t)(d_in / 32) * (size_t)bits * sizeof(unsigned int);
}

extern "C" tb_status tb_pack_codes(const unsigned char* codes, int d_out, int d_in, int bits, unsigned int* packed,
                                   void* stream) {
  if (!codes || !packed || d_out <= 0 || d_in <= 0 || bits < 2 || bits > 8) return TB_ERR_INVALID_ARG;
  if (d_in % 32) return TB_ERR_UNSUPPORTED;
  if (!aligned(codes, 16) || !aligned(packed, 4)) return TB_ERR_INVALID_ARG;
  const long long n_groups = (long long)d_out * (d_in / 32);
  cudaStream_t st = as_stream(stream);
  const int nb = pack_blocks(n_groups);
  switch (bits) {
    case 2: k_pack_codes<2><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    case 3: k_pack_codes<3><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    case 4: k_pack_codes<4><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    case 5: k_pack_codes<5><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    case 6: k_pack_codes<6><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    case 7: k_pack_codes<7><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
    default: k_pack_codes<8><<<nb, 256, 0, st>>>(codes, packed, n_groups); break;
  }
  TB_LAUNCH_CHECK();
  return TB_OK;
}

extern "C" tb_status tb_unpack_dequant(const unsigned int* packed, const float* scales, const int* zeros, int d_out,
                                       int d_in, int bits, int quant_group, unsigned char* codes_out,
                                       float* W_hat_out, const unsigned char* codes_ref, const float* W_hat_ref,
                                       float tol, unsigned long long* mismatch, void* stream) {
  if (!packed || !scales || !zeros || d_out <= 0 || d_in <= 0 || bits < 2 || bits > 8) return TB_ERR_INVALID_ARG;
  if (quant_group < 0 || (quant_group > 0 && d_in % quant_group)) return TB_ERR_INVALID_ARG;
  if ((d_in % 32) || (quant_group > 0 && quant_group % 32)) return TB_ERR_UNSUPPORTED;
  if ((codes_ref || W_hat_ref) && !mismatch) return TB_ERR_INVALID_ARG;
  if (!(tol >= 0.0f)) return TB_ERR_INVALID_ARG;
  if (!aligned(packed, 4) || !aligned(codes_out, 16) || !aligned(codes_ref, 16) || !aligned(W_hat_out, 16) ||
      !aligned(W_hat_ref, 16))
    return TB_ERR_INVALID_ARG;
  UnpackP p;
  p.packed = packed;
  p.scales = scales;
  p.zeros = zeros;
  p.codes_out = codes_out;
  p.what_out = W_hat_out;
  p.codes_ref = codes_ref;
  p.what_ref = W_hat_ref;
  p.mismatch = mismatch;
  p.n_groups = (long long)d_out * (d_in / 32);
  p.d_in = d_in;
  p.seg = quant_group > 0 ? quant_group : d_in;
  p.ng = d_in / p.seg;
  p.tol = tol;
  cudaStream_t st = as_stream(stream);
  if (mismatch) TB_CUDA_CHECK(cudaMemsetAsync(mismatch, 0, 2 * sizeof(unsigned long long), st));
  const int nb = pack_blocks(p.n_groups);
  switch (bits) {
    case 2: k_unpack_dequant<2><<<nb, 256, 0, st>>>(p); break;
    case 3: k_unpack_dequant<3><<<nb, 256, 0, st>>>(p); break;
    case 4: k_unpack_dequant<4><<<nb, 256, 0, st>>>(p); break;
    case 5: k_unpack_dequant<5><<<nb, 256, 0, st>>>(p); break;
    case 6: k_unpack_dequant<6><<<nb, 256, 0, st>>>(p); break;
    case 7: k_unpack_dequant<7><<<nb, 256, 0, st>>>(p); break;
    default: k_unpack_dequant<8><<<nb, 256, 0, st>>>(p); break;
  }
  TB_LAUNCH_CHECK();
  return TB_OK;
}
