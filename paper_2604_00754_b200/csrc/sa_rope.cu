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

}  // namespace

cudaError_t launch_rope_apply(const void* x, void* out, int B, int H, int n, int d,
                              const int64_t s[3], int dtype, const float* cs, const float* sn,
                              bool inverse, cudaStream_t st) {
  const int64_t total = (int64_t)B * H * n * ((d / 2 + 7) / 8);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  const float sign = inverse ? -1.f : 1.f;
  if (dtype == SA_BF16)
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
