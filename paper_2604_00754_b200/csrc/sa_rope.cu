// Rotary position embedding with ORIGINAL token positions (the paper applies RoPE to Q and K
// before the shuffle: Sec. 4.2, attention paragraph of App. B).  This file holds the table of
// angles and the stand-alone pass over a tensor; the forward kernels can apply the same
// rotation inside their row gather (sa_forward_rope), which saves this pass.
//
// Layout of the rotation: dimension c of the first half of a head is paired with dimension
// c + d/2; token t turns the pair by t * base^(-2c/d).
#include "sa_common.cuh"

namespace sa {
namespace {

__global__ void rope_table_kernel(int n, int half, double log2_base_over_half, float* cs,
                                  float* sn) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)n * half) return;
  const int t = (int)(i / half), c = (int)(i % half);
  // base^(-2c/d) = 2^(-c * log2(base) / half), in double: the angle reaches n radians
  const double ang = (double)t * exp2(-(double)c * log2_base_over_half);
  double s, co;
  sincos(ang, &s, &co);
  cs[i] = (float)co;
  sn[i] = (float)s;
}

// One thread per 8 consecutive dimensions of the first half of a row and their partners.
// General form (any even d, any dtype): element by element.
template <typename T>
__global__ void rope_apply_kernel(const T* __restrict__ x, T* __restrict__ out, int B, int H,
                                  int n, int d, int64_t s0, int64_t s1, int64_t s2,
                                  const float* __restrict__ cs, const float* __restrict__ sn,
                                  float sign) {
  const int half = d / 2, groups = (half + 7) / 8;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)B * H * n * groups) return;
  const int g = (int)(i % groups);
  const int64_t row = i / groups;
  const int t = (int)(row % n), h = (int)((row / n) % H), b = (int)(row / ((int64_t)n * H));
  const int64_t off = b * s0 + h * s1 + (int64_t)t * s2;
  for (int c = 8 * g; c < min(8 * g + 8, half); ++c) {
    const float co = cs[(int64_t)t * half + c], si = sign * sn[(int64_t)t * half + c];
    const float x1 = to_f32(x[off + c]), x2 = to_f32(x[off + c + half]);
    out[off + c] = from_f32<T>(fmaf(x1, co, -x2 * si));
    out[off + c + half] = from_f32<T>(fmaf(x2, co, x1 * si));
  }
}

// bf16 with d a multiple of 16: the same arithmetic with 16-byte accesses (8 dimensions of
// each half per thread; consecutive threads take consecutive pieces of a row).  HBM-bound: one
// read and one write of the tensor.
__global__ void __launch_bounds__(256)
rope_apply_bf16_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ out,
                       int B, int H, int n, int d, int64_t s0, int64_t s1, int64_t s2,
                       const float* __restrict__ cs, const float* __restrict__ sn, float sign) {
  const int half = d / 2, groups = half / 8;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)B * H * n * groups) return;
  const int g = (int)(i % groups);
  const int64_t row = i / groups;
  const int t = (int)(row % n), h = (int)((row / n) % H), b = (int)(row / ((int64_t)n * H));
  const int64_t off = b * s0 + h * s1 + (int64_t)t * s2 + 8 * g;
  const uint4 a1 = *reinterpret_cast<const uint4*>(x + off);
  const uint4 a2 = *reinterpret_cast<const uint4*>(x + off + half);
  const float4 c0 = *reinterpret_cast<const float4*>(cs + (int64_t)t * half + 8 * g);
  const float4 c1 = *reinterpret_cast<const float4*>(cs + (int64_t)t * half + 8 * g + 4);
  const float4 q0 = *reinterpret_cast<const float4*>(sn + (int64_t)t * half + 8 * g);
  const float4 q1 = *reinterpret_cast<const float4*>(sn + (int64_t)t * half + 8 * g + 4);
  const float co[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  const float si[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
  const __nv_bfloat162* h1 = reinterpret_cast<const __nv_bfloat162*>(&a1);
  const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&a2);
  uint4 o1, o2;
  __nv_bfloat162* r1 = reinterpret_cast<__nv_bfloat162*>(&o1);
  __nv_bfloat162* r2 = reinterpret_cast<__nv_bfloat162*>(&o2);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float2 x1 = __bfloat1622float2(h1[k]), x2 = __bfloat1622float2(h2[k]);
    const float s_lo = sign * si[2 * k], s_hi = sign * si[2 * k + 1];
    r1[k] = __floats2bfloat162_rn(fmaf(x1.x, co[2 * k], -x2.x * s_lo),
                                  fmaf(x1.y, co[2 * k + 1], -x2.y * s_hi));
    r2[k] = __floats2bfloat162_rn(fmaf(x2.x, co[2 * k], x1.x * s_lo),
                                  fmaf(x2.y, co[2 * k + 1], x1.y * s_hi));
  }
  *reinterpret_cast<uint4*>(out + off) = o1;
  *reinterpret_cast<uint4*>(out + off + half) = o2;
}

}  // namespace

cudaError_t launch_rope_apply(const void* x, void* out, int B, int H, int n, int d,
                              const int64_t s[3], int dtype, const float* cs, const float* sn,
                              bool inverse, cudaStream_t st) {
  const int64_t total = (int64_t)B * H * n * ((d / 2 + 7) / 8);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  const float sign = inverse ? -1.f : 1.f;
  if (dtype == SA_BF16 && d % 16 == 0)
    rope_apply_bf16_kernel<<<blocks, 256, 0, st>>>(
        (const __nv_bfloat16*)x, (__nv_bfloat16*)out, B, H, n, d, s[0], s[1], s[2], cs, sn, sign);
  else if (dtype == SA_BF16)
    rope_apply_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(
        (const __nv_bfloat16*)x, (__nv_bfloat16*)out, B, H, n, d, s[0], s[1], s[2], cs, sn, sign);
  else
    rope_apply_kernel<float><<<blocks, 256, 0, st>>>((const float*)x, (float*)out, B, H, n, d,
                                                     s[0], s[1], s[2], cs, sn, sign);
  bump_launches();
  return cudaGetLastError();
}

}  // namespace sa

extern "C" sa_status sa_rope_table(int32_t n, int32_t d, double base, float* rope_cos,
                                   float* rope_sin, sa_stream_t stream) {
  using namespace sa;
  if (n < 1 || d < 2 || d % 2 != 0 || !(base > 0.0) || !rope_cos || !rope_sin)
    return SA_ERR_INVALID_ARG;
  const int half = d / 2;
  const int64_t total = (int64_t)n * half;
  rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      n, half, log2(base) / half, rope_cos, rope_sin);
  bump_launches();
  return cudaGetLastError() == cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
