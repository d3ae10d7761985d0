// NF4 quantiser for the frozen weight of the quantised-LoRA regime (Section 4.5, Q+LoRA; 4-bit NormalFloat of
// Dettmers et al. 2023).  Storage format of this library:
//   * blocks of 64 consecutive elements along d_in;  absmax[b, o] = max |W[o, 64 b .. 64 b + 63]|  (float32,
//     block-major [d_in / 64, d_out], so that the scales of consecutive rows are contiguous)
//   * code = number of midpoints between neighbouring NF4 levels that lie strictly below x = w / absmax (float32),
//     i.e. the nearest level, the lower one on a tie; an all-zero block has absmax 0 and code 7 (level 0)
//   * byte k of a row of `codes` [d_out, d_in / 2] holds element 2k in its low nibble, element 2k + 1 in its high nibble
// Quantiser: one warp per block, a lane owns two neighbouring elements, i.e. one output byte.
// Expander (codes + scales -> bf16 weight, every element bf16(level * absmax): one float32 product, one rounding): a
// thread turns 4 code bytes into 8 bf16 (16 bytes), so a warp reads 128 contiguous code bytes and writes 512 contiguous
// bytes; the level table sits in shared memory once per lane (no bank conflicts for arbitrary codes).
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace lora {

namespace {

__device__ __constant__ float c_nf4_quant_levels[16] = {
    -1.0f, -0.6961928009986877f, -0.5250730514526367f, -0.39491748809814453f,
    -0.28444138169288635f, -0.18477343022823334f, -0.09105003625154495f, 0.0f,
    0.07958029955625534f, 0.16093020141124725f, 0.24611230194568634f, 0.33791524171829224f,
    0.44070982933044434f, 0.5626170039176941f, 0.7229568362236023f, 1.0f};

__device__ __forceinline__ unsigned nf4_code(float x) {
  unsigned c = 0;
#pragma unroll
  for (int k = 0; k < 15; ++k) {
    const float mid = __fmul_rn(__fadd_rn(c_nf4_quant_levels[k], c_nf4_quant_levels[k + 1]), 0.5f);
    c += (x > mid) ? 1u : 0u;
  }
  return c;
}

__global__ void __launch_bounds__(256) lora_nf4_quantize_kernel(const __nv_bfloat16* __restrict__ W, long long d_out, long long d_in,
                                                                uint8_t* __restrict__ codes, float* __restrict__ absmax) {
  const long long n_blocks_row = d_in / kNf4Block;
  const long long warp_id = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp_id >= d_out * n_blocks_row) return;
  const long long o = warp_id / n_blocks_row, b = warp_id - o * n_blocks_row;
  const __nv_bfloat162 w2 = *reinterpret_cast<const __nv_bfloat162*>(W + o * d_in + b * kNf4Block + 2 * lane);
  const float w0 = __low2float(w2), w1 = __high2float(w2);
  float m = fmaxf(fabsf(w0), fabsf(w1));
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
  unsigned c0 = 7u, c1 = 7u;
  if (m > 0.f) {
    c0 = nf4_code(__fdiv_rn(w0, m));
    c1 = nf4_code(__fdiv_rn(w1, m));
  }
  codes[o * (d_in / 2) + b * (kNf4Block / 2) + lane] = static_cast<uint8_t>(c0 | (c1 << 4));
  if (lane == 0) absmax[b * d_out + o] = m;
}

// Expands the window rows [o0, o0 + n_rows) x columns [c0, c0 + n_cols) of the quantised weight into W (row pitch ld_w
// elements, row 0 / column 0 of W = weight element (o0, c0)); the whole weight is the window (0, d_out, 0, d_in).
__global__ void __launch_bounds__(256) lora_nf4_dequantize_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ absmax,
                                                                  long long d_out, long long d_in, long long o0, long long n_rows,
                                                                  long long c0, long long n_cols, long long ld_w,
                                                                  __nv_bfloat16* __restrict__ W) {
  __shared__ float lut[16 * 32];
  pdl_launch_dependents();
  for (int b = threadIdx.x; b < 16 * 32; b += blockDim.x) lut[b] = c_nf4_quant_levels[b >> 5];
  __syncthreads();
  pdl_wait();
  const float* lut_lane = lut + (threadIdx.x & 31);
  const long long words_full = d_in / 8;                        // code words of a whole weight row
  const int words_row = static_cast<int>(n_cols / 8);           // 4 code bytes = 8 elements per thread and step
  const long long word0 = c0 / 8;
  // a block walks whole rows (no index division); a thread fetches up to four code words (t, t + 256, ...) and their
  // scales before it converts any of them, so that four loads per thread are in flight
  for (long long o = blockIdx.x; o < n_rows; o += gridDim.x) {
    const uint32_t* crow = codes + (o0 + o) * words_full + word0;
    uint4* wrow = reinterpret_cast<uint4*>(W + o * ld_w);
    for (int base = 0; base < words_row; base += 4 * blockDim.x) {
      uint32_t cw[4];
      float scale[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int wcol = base + k * blockDim.x + threadIdx.x;
        cw[k] = wcol < words_row ? __ldg(crow + wcol) : 0u;
        scale[k] = wcol < words_row ? __ldg(absmax + ((word0 + wcol) >> 3) * d_out + o0 + o) : 0.f;   // 8 words = one block
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int wcol = base + k * blockDim.x + threadIdx.x;
        if (wcol >= words_row) continue;
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float lo = lut_lane[((cw[k] >> (8 * j)) & 0xFu) << 5];
          const float hi = lut_lane[((cw[k] >> (8 * j + 4)) & 0xFu) << 5];
          w[j] = pack_bf16x2(lo * scale[k], hi * scale[k]);
        }
        wrow[wcol] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
}

}  // namespace

cudaError_t launch_nf4_dequantize_window(const uint8_t* codes, const float* absmax, long long d_out, long long d_in, long long o0,
                                         long long n_rows, long long c0, long long n_cols, __nv_bfloat16* W, long long ld_w,
                                         int num_sms, cudaStream_t stream) {
  long long blocks = n_rows;
  const long long cap = static_cast<long long>(num_sms > 0 ? num_sms : 148) * 16;
  if (blocks > cap) blocks = cap;
  return launch_pdl(lora_nf4_dequantize_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream,
                    reinterpret_cast<const uint32_t*>(codes), absmax, d_out, d_in, o0, n_rows, c0, n_cols, ld_w, W);
}

cudaError_t launch_nf4_dequantize(const uint8_t* codes, const float* absmax, long long d_out, long long d_in, __nv_bfloat16* W,
                                  int num_sms, cudaStream_t stream) {
  return launch_nf4_dequantize_window(codes, absmax, d_out, d_in, 0, d_out, 0, d_in, W, d_in, num_sms, stream);
}

cudaError_t launch_nf4_quantize(const __nv_bfloat16* W, long long d_out, long long d_in, uint8_t* codes, float* absmax,
                                cudaStream_t stream) {
  const long long warps = d_out * (d_in / kNf4Block);
  const long long blocks = (warps * 32 + 255) / 256;
  lora_nf4_quantize_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(W, d_out, d_in, codes, absmax);
  return cudaGetLastError();
}

}  // namespace lora
