// Operand preparation of the 3xTF32 path: an fp32 matrix is split into two tf32-representable
// planes, hi = x rounded to tf32 (10 mantissa bits, round to nearest) and lo = x - hi (exact in
// fp32, then rounded to tf32), so that x = hi + lo up to 2^-22 |x|.  The tensor-core kernel then
// accumulates X_hi W_hi + X_hi W_lo + X_lo W_hi in fp32; the dropped lo * lo term is 2^-22 relative.
// Layout of the result: [batch][rows][2 * k_plane], the hi plane in columns [0, k_plane) and the lo
// plane in [k_plane, 2 k_plane); k_plane = K rounded up to 32 (one 128-byte k-block), the padding
// is zero.  HBM-bound: 4 bytes read and 8 written per element.
#include "fgr_internal.h"

namespace fgr {
namespace {

__device__ __forceinline__ float to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}

__global__ void __launch_bounds__(256) split_tf32_kernel(const float* __restrict__ src, float* __restrict__ dst, int batch,
                                                         int rows, int K, long long ld, long long bs, int k_plane) {
  const int groups = k_plane / 4;                       // float4 groups per row of a plane
  const long long total = (long long)batch * rows * groups;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int g = (int)(i % groups);
    const long long r = i / groups;                     // bt * rows + row
    const int bt = (int)(r / rows), row = (int)(r % rows);
    const int k = 4 * g;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (k < K) v = *reinterpret_cast<const float4*>(src + (long long)bt * bs + (long long)row * ld + k);   // K % 4 == 0
    float4 hi, lo;
    hi.x = to_tf32(v.x); hi.y = to_tf32(v.y); hi.z = to_tf32(v.z); hi.w = to_tf32(v.w);
    lo.x = to_tf32(v.x - hi.x); lo.y = to_tf32(v.y - hi.y); lo.z = to_tf32(v.z - hi.z); lo.w = to_tf32(v.w - hi.w);
    float* out = dst + r * (2LL * k_plane) + k;
    *reinterpret_cast<float4*>(out) = hi;
    *reinterpret_cast<float4*>(out + k_plane) = lo;
  }
}

}  // namespace

cudaError_t launch_split_tf32(const float* src, float* dst, int batch, int rows, int K, long long ld, long long bs,
                              int k_plane, cudaStream_t stream) {
  const long long total = (long long)batch * rows * (k_plane / 4);
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  split_tf32_kernel<<<(unsigned)blocks, 256, 0, stream>>>(src, dst, batch, rows, K, ld, bs, k_plane);
  return cudaGetLastError();
}

}  // namespace fgr
