// 8-bit storage of expert rows for the host link: FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa
// bits, no infinities, largest finite value 448) with one fp32 scale per row.
//
//     scale = max|w| / 448   (1 for an all-zero row)        code = e4m3(w / scale), round to nearest even, saturating
//     w'    = bf16(value(code) * scale)
//
// The paper names bit-width adaptation only as the earlier route to cheaper expert offloading (Section 2.3,
// Section 5); this is that route applied to the packed expert rows: an expert crosses the host link in half the
// bytes and is widened back to bf16 on the device, in the slot the layer kernels read.
// The encoder and decoder below are written from the format's definition.
#include <algorithm>

#include "common.cuh"

namespace cosmoe {
namespace {

constexpr float kE4M3Max = 448.0f;

// fp32 -> E4M3 code.  |x| >= 2^-6: the fp32 mantissa is cut to 3 bits with round-to-nearest-even on the bit
// pattern (a carry runs into the exponent as it should).  Below: multiples of 2^-9.
__device__ __forceinline__ uint32_t e4m3_encode(float x) {
  const uint32_t b = __float_as_uint(x);
  const uint32_t sign = (b >> 24) & 0x80u;
  const float a = fabsf(x);
  if (!(a == a)) return 0x7fu;
  if (a >= kE4M3Max) return sign | 0x7eu;
  if (a < 0.015625f) return sign | (uint32_t)__float2int_rn(a * 512.0f);  // 0..8 steps of 2^-9; 8 is 2^-6 = code 0x08
  const uint32_t ab = b & 0x7fffffffu;
  const uint32_t r = (ab + 0x7ffffu + ((ab >> 20) & 1u)) >> 20;  // (biased exponent << 3) | mantissa
  const uint32_t code = r - ((127u - 7u) << 3);
  return sign | (code > 0x7eu ? 0x7eu : code);
}
__device__ __forceinline__ float e4m3_decode(uint32_t c) {
  const uint32_t e = (c >> 3) & 15u, m = c & 7u;
  const float mag = e == 0u ? (float)m * 0.001953125f : __uint_as_float(((e + 120u) << 23) | (m << 20));
  return (c & 0x80u) ? -mag : mag;
}

// One warp per row of n bf16 values (n a multiple of 8).
__global__ void fp8_quantize_kernel(const uint4* __restrict__ w, long long rows, int n, uint2* __restrict__ codes,
                                    float* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const long long row = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  if (row >= rows) return;
  const int chunks = n >> 3;
  const uint4* src = w + row * chunks;
  float amax = 0.f;
  for (int c = lane; c < chunks; c += 32) {
    float f[8];
    unpack8(__ldg(src + c), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float scale = amax > 0.f ? __fdiv_rn(amax, kE4M3Max) : 1.0f;
  if (lane == 0) scales[row] = scale;
  for (int c = lane; c < chunks; c += 32) {
    float f[8];
    unpack8(__ldg(src + c), f);
    uint32_t q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = e4m3_encode(__fdiv_rn(f[i], scale));
    uint2 o;
    o.x = q[0] | (q[1] << 8) | (q[2] << 16) | (q[3] << 24);
    o.y = q[4] | (q[5] << 8) | (q[6] << 16) | (q[7] << 24);
    codes[row * chunks + c] = o;
  }
}

// 8 codes per thread -> 8 bf16 values.
__global__ void fp8_dequant_kernel(const uint2* __restrict__ codes, const float* __restrict__ scales, long long rows, int n,
                                   uint4* __restrict__ w) {
  const int chunks = n >> 3;
  const long long total = rows * chunks;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long row = i / chunks;
    const float s = __ldg(scales + row);
    const uint2 c = __ldg(codes + i);
    float f[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      f[j] = e4m3_decode((c.x >> (8 * j)) & 0xffu) * s;
      f[4 + j] = e4m3_decode((c.y >> (8 * j)) & 0xffu) * s;
    }
    uint4 o;
    o.x = pack_bf16x2(f[0], f[1]), o.y = pack_bf16x2(f[2], f[3]);
    o.z = pack_bf16x2(f[4], f[5]), o.w = pack_bf16x2(f[6], f[7]);
    w[i] = o;
  }
}

}  // namespace

int launch_fp8_dequant(const void* codes, const float* scales, long long rows, int n, void* w, cudaStream_t s) {
  const long long total = rows * (n >> 3);
  if (total <= 0) return MOE_OK;
  const int grid = (int)std::min<long long>((total + 255) / 256, 148 * 16);
  fp8_dequant_kernel<<<grid, 256, 0, s>>>((const uint2*)codes, scales, rows, n, (uint4*)w);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

}  // namespace cosmoe

using namespace cosmoe;

extern "C" {

int moe_fp8_quantize_rows(const void* w, int64_t rows, int32_t n, void* codes, float* scales, void* stream) {
  if (!w || !codes || !scales || rows < 0 || n <= 0) return MOE_ERR_INVALID_ARG;
  if (n % 8 || (((uintptr_t)w | (uintptr_t)codes) & 15u)) return MOE_ERR_UNSUPPORTED;
  if (rows == 0) return MOE_OK;
  const long long blocks = (rows * 32 + 255) / 256;
  if (blocks > 0x7fffffffll) return MOE_ERR_UNSUPPORTED;
  fp8_quantize_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((const uint4*)w, rows, n, (uint2*)codes, scales);
  MOE_CUDA_TRY(cudaGetLastError());
  return MOE_OK;
}

int moe_fp8_dequantize_rows(const void* codes, const float* scales, int64_t rows, int32_t n, void* w, void* stream) {
  if (!w || !codes || !scales || rows < 0 || n <= 0) return MOE_ERR_INVALID_ARG;
  if (n % 8 || (((uintptr_t)w | (uintptr_t)codes) & 15u)) return MOE_ERR_UNSUPPORTED;
  return launch_fp8_dequant(codes, scales, rows, n, w, (cudaStream_t)stream);
}

}  // extern "C"
