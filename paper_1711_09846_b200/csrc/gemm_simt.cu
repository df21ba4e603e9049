// Member-batched GEMM on the plain FP32 ALUs: C[m][n] = sum_k A(m,k) B(n,k).
//
// This is the path for fp32 populations (1e-5 parity with a float64 reference
// rules out TF32) and for the skinny layers of bf16 populations (widths of 1, 2
// or 10, ragged shapes) that do not fill a tensor-core tile.  Operands are float
// or bfloat16, accumulation is float, one 64x64 output tile per CTA, 4x4 outputs
// per thread, K in slices of 16 staged through shared memory.
#include "pbt_common.cuh"

namespace pbt {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }

template <typename T, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(256) k_gemm_simt(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int member = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const T* __restrict__ A = reinterpret_cast<const T*>(g.A) + member * g.strideA;
  const T* __restrict__ B = reinterpret_cast<const T*>(g.B) + member * g.strideB;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < (BM * BK) / 256; ++i) {
      const int idx = tid + i * 256;
      int mm, kk;
      if (A_MN) { mm = idx % BM; kk = idx / BM; } else { kk = idx % BK; mm = idx / BK; }
      const int gm = m0 + mm, gk = k0 + kk;
      float v = 0.f;
      if (gm < g.M && gk < g.K) v = to_f<T>(A_MN ? A[(long long)gk * g.lda + gm] : A[(long long)gm * g.lda + gk]);
      As[kk][mm] = v;
    }
#pragma unroll
    for (int i = 0; i < (BN * BK) / 256; ++i) {
      const int idx = tid + i * 256;
      int nn, kk;
      if (B_MN) { nn = idx % BN; kk = idx / BN; } else { kk = idx % BK; nn = idx / BK; }
      const int gn = n0 + nn, gk = k0 + kk;
      float v = 0.f;
      if (gn < g.N && gk < g.K) v = to_f<T>(B_MN ? B[(long long)gk * g.ldb + gn] : B[(long long)gn * g.ldb + gk]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * TM]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * TN]);
      const float a[TM] = {a4.x, a4.y, a4.z, a4.w};
      const float b[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  const float* bias = g.bias ? g.bias + member * g.strideBias : nullptr;
  const T* mask = g.mask ? reinterpret_cast<const T*>(g.mask) + member * g.strideMask : nullptr;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int gm = m0 + ty * TM + i;
    if (gm >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int gn = n0 + tx * TN + j;
      if (gn >= g.N) continue;
      float v = acc[i][j];
      if (bias) v += bias[gn];
      if (g.relu) v = fmaxf(v, 0.f);
      if (mask && !(to_f<T>(mask[(long long)gm * g.ldmask + gn]) > 0.f)) v = 0.f;
      const long long ci = member * g.strideC + (long long)gm * g.ldc + gn;
      if (g.out_dtype == kBF16) reinterpret_cast<bf16*>(g.C)[ci] = __float2bfloat16_rn(v);
      else reinterpret_cast<float*>(g.C)[ci] = v;
    }
  }
}

template <typename T>
static cudaError_t launch_t(const GemmArgs& g, cudaStream_t s) {
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  if (!g.a_mn && !g.b_mn) k_gemm_simt<T, false, false><<<grid, 256, 0, s>>>(g);
  else if (!g.a_mn && g.b_mn) k_gemm_simt<T, false, true><<<grid, 256, 0, s>>>(g);
  else if (g.a_mn && g.b_mn) k_gemm_simt<T, true, true><<<grid, 256, 0, s>>>(g);
  else k_gemm_simt<T, true, false><<<grid, 256, 0, s>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return cudaSuccess;
  return g.in_dtype == kBF16 ? launch_t<bf16>(g, s) : launch_t<float>(g, s);
}

}  // namespace pbt
