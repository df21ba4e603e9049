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
  pdl_prologue();
  // double-buffered k-slabs: the global loads of slab k+1 are in flight (in registers) while slab k is multiplied
  __shared__ float As[2][BK][BM + 4];
  __shared__ float Bs[2][BK][BN + 4];
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
  constexpr int kPerThread = (BM * BK) / 256;
  float ra[kPerThread], rb[kPerThread];

  auto load_slab = [&](int k0) {
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int idx = tid + i * 256;
      int mm, kk;
      if (A_MN) { mm = idx % BM; kk = idx / BM; } else { kk = idx % BK; mm = idx / BK; }
      const int gm = m0 + mm;
      int gk = k0 + kk;
      ra[i] = (gm < g.M && gk < g.K) ? to_f<T>(A_MN ? A[(long long)gk * g.lda + gm] : A[(long long)gm * g.lda + gk]) : 0.f;
      int nn;
      if (B_MN) { nn = idx % BN; kk = idx / BN; } else { kk = idx % BK; nn = idx / BK; }
      const int gn = n0 + nn;
      gk = k0 + kk;
      rb[i] = (gn < g.N && gk < g.K) ? to_f<T>(B_MN ? B[(long long)gk * g.ldb + gn] : B[(long long)gn * g.ldb + gk]) : 0.f;
    }
  };
  auto store_slab = [&](int buf) {
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int idx = tid + i * 256;
      int mm, kk;
      if (A_MN) { mm = idx % BM; kk = idx / BM; } else { kk = idx % BK; mm = idx / BK; }
      As[buf][kk][mm] = ra[i];
      int nn;
      if (B_MN) { nn = idx % BN; kk = idx / BN; } else { kk = idx % BK; nn = idx / BK; }
      Bs[buf][kk][nn] = rb[i];
    }
  };

  if (g.K > 0) {
    load_slab(0);
    store_slab(0);
  }
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < g.K; k0 += BK, buf ^= 1) {
    const bool more = k0 + BK < g.K;
    if (more) load_slab(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * TM]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * TN]);
      const float a[TM] = {a4.x, a4.y, a4.z, a4.w};
      const float b[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) store_slab(buf ^ 1);
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

// The same K order and multiply-add order (bit-identical results) for GEMMs whose tiles are all interior
// (M, N multiples of 64, K of 16) with 4-element-aligned operands: every thread moves one or two 4-element vectors
// of each operand per K slice through pointers that advance by a constant, and writes its outputs as vectors.
// In the general kernel above the per-element index arithmetic and bounds checks of the slice loads were 46 % of
// the instructions issued, and issue was the limit (FMA pipe 43-46 % busy on the 128 x 512 x 512 layers of the
// fp32 population).
template <typename T>
__device__ __forceinline__ float4 ld4(const T* p);
template <>
__device__ __forceinline__ float4 ld4<float>(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
template <>
__device__ __forceinline__ float4 ld4<bf16>(const bf16* p) {
  const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}

template <typename T, bool A_MN, bool B_MN, int TMV>
__global__ void __launch_bounds__(256) k_gemm_simt_interior(GemmArgs g) {
  // TMV = 4: 64 x 64 tile, 4 x 4 outputs per thread.  TMV = 8: 128 x 64 tile, 8 x 4 outputs per thread (fewer
  // shared-memory reads per multiply-add; for GEMMs with enough 128-row tiles to go round).
  constexpr int BMV = 16 * TMV, AV = TMV / 4;   // tile rows; vectors of A a thread moves per K slice
  pdl_prologue();
  __shared__ __align__(16) float As[2][BK][BMV + 4];
  __shared__ __align__(16) float Bs[2][BK][BN + 4];
  const int member = blockIdx.z;
  const int m0 = blockIdx.y * BMV, n0 = blockIdx.x * BN;
  const int tid = threadIdx.x;
  // a warp covers 8 x 4 threads, so that its shared-memory reads per k are one 128-byte row segment of B and 64 (128)
  // bytes of A: two (three) wavefronts
  const int lane = tid & 31, warp = tid >> 5;
  const int tx = (lane & 7) + 8 * (warp & 1), ty = (lane >> 3) + 4 * (warp >> 1);
  // K-major operand: the slice is rows x 16 k, a thread takes row tid / 4 (+ 64), k (tid % 4) * 4 .. + 3.
  // MN-major operand: the slice is 16 k x columns, a thread takes columns (tid % (columns / 4)) * 4 .. + 3 of
  // k = tid / (columns / 4) (+ 8 when the slice has 128 columns).
  constexpr int AVW = BMV / 4;   // vectors per k row of an MN-major A slice
  const T* pa = reinterpret_cast<const T*>(g.A) + member * g.strideA +
                (A_MN ? (long long)(tid / AVW) * g.lda + m0 + (tid % AVW) * 4 : (long long)(m0 + (tid >> 2)) * g.lda + (tid & 3) * 4);
  const T* pb = reinterpret_cast<const T*>(g.B) + member * g.strideB +
                (B_MN ? (long long)(tid >> 4) * g.ldb + n0 + (tid & 15) * 4 : (long long)(n0 + (tid >> 2)) * g.ldb + (tid & 3) * 4);
  const long long step_a = A_MN ? (long long)BK * g.lda : BK, step_b = B_MN ? (long long)BK * g.ldb : BK;
  const long long second_a = A_MN ? (long long)(256 / AVW) * g.lda : 64ll * g.lda;   // the thread's second vector of A
  float acc[TMV][TN];
#pragma unroll
  for (int i = 0; i < TMV; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
  float4 ra[AV], rb;
  auto load_slab = [&]() {
#pragma unroll
    for (int v = 0; v < AV; ++v) ra[v] = ld4<T>(pa + v * second_a);
    rb = ld4<T>(pb);
    pa += step_a; pb += step_b;
  };
  auto store_slab = [&](int buf) {
#pragma unroll
    for (int v = 0; v < AV; ++v) {
      if (A_MN) {
        *reinterpret_cast<float4*>(&As[buf][tid / AVW + v * (256 / AVW)][(tid % AVW) * 4]) = ra[v];
      } else {
        const int kq = (tid & 3) * 4, mm = (tid >> 2) + 64 * v;
        As[buf][kq][mm] = ra[v].x; As[buf][kq + 1][mm] = ra[v].y; As[buf][kq + 2][mm] = ra[v].z; As[buf][kq + 3][mm] = ra[v].w;
      }
    }
    if (B_MN) {
      *reinterpret_cast<float4*>(&Bs[buf][tid >> 4][(tid & 15) * 4]) = rb;
    } else {
      const int kq = (tid & 3) * 4, nn = tid >> 2;
      Bs[buf][kq][nn] = rb.x; Bs[buf][kq + 1][nn] = rb.y; Bs[buf][kq + 2][nn] = rb.z; Bs[buf][kq + 3][nn] = rb.w;
    }
  };
  load_slab();
  store_slab(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < g.K; k0 += BK, buf ^= 1) {
    const bool more = k0 + BK < g.K;
    if (more) load_slab();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TMV];
#pragma unroll
      for (int v = 0; v < AV; ++v) {
        const float4 a4 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * TMV + 4 * v]);
        a[4 * v] = a4.x; a[4 * v + 1] = a4.y; a[4 * v + 2] = a4.z; a[4 * v + 3] = a4.w;
      }
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * TN]);
      const float b[TN] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < TMV; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) store_slab(buf ^ 1);
    __syncthreads();
  }

  const int gn = n0 + tx * TN;
  float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
  if (g.bias) bv = __ldg(reinterpret_cast<const float4*>(g.bias + member * g.strideBias + gn));
  const T* mask = g.mask ? reinterpret_cast<const T*>(g.mask) + member * g.strideMask : nullptr;
#pragma unroll
  for (int i = 0; i < TMV; ++i) {
    const int gm = m0 + ty * TMV + i;
    float4 v = make_float4(acc[i][0] + bv.x, acc[i][1] + bv.y, acc[i][2] + bv.z, acc[i][3] + bv.w);
    if (!g.bias) v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    if (g.relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
    if (mask) {
      const float4 mk = ld4<T>(mask + (long long)gm * g.ldmask + gn);
      if (!(mk.x > 0.f)) v.x = 0.f;
      if (!(mk.y > 0.f)) v.y = 0.f;
      if (!(mk.z > 0.f)) v.z = 0.f;
      if (!(mk.w > 0.f)) v.w = 0.f;
    }
    const long long ci = member * g.strideC + (long long)gm * g.ldc + gn;
    if (g.out_dtype == kBF16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(g.C) + ci) =
          make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + ci) = v;
    }
  }
}

template <typename T>
static bool simt_interior_ok(const GemmArgs& g) {
  const size_t ev = sizeof(T) * 4, cv = (g.out_dtype == kBF16 ? 2 : 4) * 4;
  auto al = [](const void* p, size_t a) { return ((uintptr_t)p % a) == 0; };
  return g.M % BM == 0 && g.N % BN == 0 && g.K % BK == 0 && g.K > 0 && !g.a_rowoff && !g.b_rowoff &&
         g.lda % 4 == 0 && g.ldb % 4 == 0 && g.ldc % 4 == 0 && g.strideA % 4 == 0 && g.strideB % 4 == 0 && g.strideC % 4 == 0 &&
         al(g.A, ev) && al(g.B, ev) && al(g.C, cv) &&
         (!g.bias || (al(g.bias, 16) && g.strideBias % 4 == 0)) &&
         (!g.mask || (al(g.mask, ev) && g.ldmask % 4 == 0 && g.strideMask % 4 == 0));
}

// ---------------------------------------------------------------------------
// Skinny shapes (a dimension of 16 or less: one-, two- and ten-wide output layers, two-wide inputs).
// The 64x64 tile kernel above spends its time in shared-memory round trips there; these three kernels
// read every operand once, coalesced, and reduce in a fixed order.
// ---------------------------------------------------------------------------
constexpr int kSkinny = 16;

__device__ __forceinline__ float epilogue_one(const GemmArgs& g, int member, int m, int n, float v, int in_is_bf16) {
  if (g.bias) v += g.bias[member * g.strideBias + n];
  if (g.relu) v = fmaxf(v, 0.f);
  if (g.mask) {
    const long long mi = member * g.strideMask + (long long)m * g.ldmask + n;
    const float mv = in_is_bf16 ? __bfloat162float(reinterpret_cast<const bf16*>(g.mask)[mi])
                                : reinterpret_cast<const float*>(g.mask)[mi];
    if (!(mv > 0.f)) v = 0.f;
  }
  return v;
}
__device__ __forceinline__ void store_one(const GemmArgs& g, int member, int m, int n, float v) {
  const long long ci = member * g.strideC + (long long)m * g.ldc + n;
  if (g.out_dtype == kBF16) reinterpret_cast<bf16*>(g.C)[ci] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(g.C)[ci] = v;
}

// N <= NT <= 16, A K-major: one warp per output row, lanes stride over K, shuffle reduction.
template <typename T, bool B_MN, int NT>
__global__ void __launch_bounds__(256) k_gemm_rowdot(GemmArgs g) {
  pdl_prologue();
  const int member = blockIdx.y, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (m >= g.M) return;
  const T* __restrict__ A = reinterpret_cast<const T*>(g.A) + member * g.strideA + (long long)m * g.lda;
  const T* __restrict__ B = reinterpret_cast<const T*>(g.B) + member * g.strideB;
  float acc[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n] = 0.f;
#pragma unroll 4
  for (int k = lane; k < g.K; k += 32) {
    const float a = to_f<T>(A[k]);
#pragma unroll
    for (int n = 0; n < NT; ++n)
      if (NT == 1 || n < g.N) acc[n] = fmaf(a, to_f<T>(B_MN ? B[(long long)k * g.ldb + n] : B[(long long)n * g.ldb + k]), acc[n]);
  }
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    float v = acc[n];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == n && n < g.N) store_one(g, member, m, n, epilogue_one(g, member, m, n, v, sizeof(T) == 2));
  }
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& w, float* f) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) { f[2 * j] = __uint_as_float(u[j] << 16); f[2 * j + 1] = __uint_as_float(u[j] & 0xFFFF0000u); }
}

// The row-dot kernel for bf16 operands that are both K-major with K a multiple of 8: a lane takes 8 consecutive k
// per trip with one 16-byte load per operand row.  The scalar form above is bound by instruction issue (address
// arithmetic, conversion and one multiply-add per 2-byte load); this one issues about a third as many.
// A warp works on RPW rows at a time, so that every 16-byte load of a B row serves RPW rows of A and RPW + NT loads
// are in flight per trip; the sum of a row is formed in the same order whatever RPW is.
template <int NT, int RPW>
__global__ void __launch_bounds__(256) k_gemm_rowdot_bf16x8(GemmArgs g) {
  pdl_prologue();
  const int member = blockIdx.y, lane = threadIdx.x & 31;
  const int m0 = (blockIdx.x * 8 + (threadIdx.x >> 5)) * RPW;
  if (m0 >= g.M) return;
  const bf16* __restrict__ A = reinterpret_cast<const bf16*>(g.A) + member * g.strideA;
  const bf16* __restrict__ B = reinterpret_cast<const bf16*>(g.B) + member * g.strideB;
  float acc[RPW][NT];
#pragma unroll
  for (int r = 0; r < RPW; ++r)
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[r][n] = 0.f;
#pragma unroll 2
  for (int k = lane * 8; k < g.K; k += 256) {
    float a[RPW][8];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const int m = m0 + r < g.M ? m0 + r : g.M - 1;      // rows past the end repeat the last row and are not stored
      unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(A + (long long)m * g.lda + k)), a[r]);
    }
    const bf16* bk = B + k;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      float b[8];
      unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(bk + (long long)n * g.ldb)), b);
#pragma unroll
      for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[r][n] = fmaf(a[r][j], b[j], acc[r][n]);
    }
  }
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      float v = acc[r][n];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == n && m0 + r < g.M) store_one(g, member, m0 + r, n, epilogue_one(g, member, m0 + r, n, v, 1));
    }
  }
}

static bool rowdot_vec_ok(const GemmArgs& g) {
  return g.in_dtype == kBF16 && !g.a_mn && !g.b_mn && g.N <= kSkinny && g.K % 8 == 0 && g.K >= 64 && g.lda % 8 == 0 &&
         g.ldb % 8 == 0 && g.strideA % 8 == 0 && g.strideB % 8 == 0 && (((uintptr_t)g.A | (uintptr_t)g.B) & 15) == 0 &&
         g.batch <= 65535;
}
// one instantiation per width: no predicated-off columns in the inner loop
template <int NT>
static void launch_rowdot_vec_n(const GemmArgs& g, cudaStream_t s) {
  constexpr int RPW = NT <= 4 ? 4 : 2;
  if (g.M >= 8 * RPW)
    launch_with(dim3((g.M + 8 * RPW - 1) / (8 * RPW), g.batch), 256, 0, s)(k_gemm_rowdot_bf16x8<NT, RPW>, g);
  else
    launch_with(dim3((g.M + 7) / 8, g.batch), 256, 0, s)(k_gemm_rowdot_bf16x8<NT, 1>, g);
}
static void launch_rowdot_vec(const GemmArgs& g, cudaStream_t s) {
  switch (g.N) {
    case 1: launch_rowdot_vec_n<1>(g, s); break;   case 2: launch_rowdot_vec_n<2>(g, s); break;
    case 3: launch_rowdot_vec_n<3>(g, s); break;   case 4: launch_rowdot_vec_n<4>(g, s); break;
    case 5: launch_rowdot_vec_n<5>(g, s); break;   case 6: launch_rowdot_vec_n<6>(g, s); break;
    case 7: launch_rowdot_vec_n<7>(g, s); break;   case 8: launch_rowdot_vec_n<8>(g, s); break;
    case 9: launch_rowdot_vec_n<9>(g, s); break;   case 10: launch_rowdot_vec_n<10>(g, s); break;
    case 11: launch_rowdot_vec_n<11>(g, s); break; case 12: launch_rowdot_vec_n<12>(g, s); break;
    case 13: launch_rowdot_vec_n<13>(g, s); break; case 14: launch_rowdot_vec_n<14>(g, s); break;
    case 15: launch_rowdot_vec_n<15>(g, s); break; default: launch_rowdot_vec_n<16>(g, s); break;
  }
}

// Both operands MN-major (weight gradients), the short one of M, N at most ST <= 16: thread per index of the
// long dimension, 16 slices of K per block combined in a fixed order.  LONG_A: M is the long dimension, else N.
template <typename T, bool LONG_A, int ST>
__global__ void __launch_bounds__(512) k_gemm_colacc(GemmArgs g) {
  pdl_prologue();
  __shared__ float red[16][32][ST + 1];
  const int member = blockIdx.y, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int L = LONG_A ? g.M : g.N, S = LONG_A ? g.N : g.M;
  const long long ldx = LONG_A ? g.lda : g.ldb, ldy = LONG_A ? g.ldb : g.lda;
  const T* __restrict__ X = reinterpret_cast<const T*>(LONG_A ? g.A : g.B) + member * (LONG_A ? g.strideA : g.strideB);
  const T* __restrict__ Y = reinterpret_cast<const T*>(LONG_A ? g.B : g.A) + member * (LONG_A ? g.strideB : g.strideA);
  const int l = blockIdx.x * 32 + tx;
  float acc[ST];
#pragma unroll
  for (int s = 0; s < ST; ++s) acc[s] = 0.f;
  if (l < L) {
#pragma unroll 4
    for (int k = ty; k < g.K; k += 16) {
      const float x = to_f<T>(X[(long long)k * ldx + l]);
#pragma unroll
      for (int s = 0; s < ST; ++s)
        if (ST == 1 || s < S) acc[s] = fmaf(x, to_f<T>(Y[(long long)k * ldy + s]), acc[s]);
    }
  }
#pragma unroll
  for (int s = 0; s < ST; ++s) red[ty][tx][s] = acc[s];
  __syncthreads();
  if (ty == 0 && l < L) {
#pragma unroll
    for (int s = 0; s < ST; ++s) {
      if (s < S) {
        float v = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) v += red[j][tx][s];
        const int m = LONG_A ? l : s, n = LONG_A ? s : l;
        store_one(g, member, m, n, epilogue_one(g, member, m, n, v, sizeof(T) == 2));
      }
    }
  }
}

// The column-accumulate kernel for bf16 operands with the long dimension a multiple of 8: a thread owns 8
// consecutive indices of the long dimension (one 16-byte load per batch row), 16 threads cover 128 of them, and the
// block's 16 slices of K are combined in a fixed order, one short index at a time through 8 KB of shared memory.
// LG = lane groups per block (LG * 8 indices of the long dimension), 256 / LG slices of K: 16 x 16 when that gives
// enough blocks to fill the GPU, 8 x 32 (half as many indices per block, twice the blocks) for small populations.
template <bool LONG_A, int ST, int LG>
__global__ void __launch_bounds__(256) k_gemm_colacc_bf16x8(GemmArgs g) {
  pdl_prologue();
  constexpr int KS = 256 / LG, W = LG * 8;
  __shared__ float red[KS][W + 4];
  const int member = blockIdx.y, lg = threadIdx.x % LG, ks = threadIdx.x / LG;
  const int L = LONG_A ? g.M : g.N;
  const long long ldx = LONG_A ? g.lda : g.ldb, ldy = LONG_A ? g.ldb : g.lda;
  const bf16* __restrict__ X = reinterpret_cast<const bf16*>(LONG_A ? g.A : g.B) + member * (LONG_A ? g.strideA : g.strideB);
  const bf16* __restrict__ Y = reinterpret_cast<const bf16*>(LONG_A ? g.B : g.A) + member * (LONG_A ? g.strideB : g.strideA);
  const int l0 = blockIdx.x * W + lg * 8;
  float acc[8][ST];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int t = 0; t < ST; ++t) acc[j][t] = 0.f;
  if (l0 < L) {
    // short widths leave registers for more loads in flight: a block's 16 slices of K are walked by 8 warps only
#pragma unroll(ST <= 2 ? 8 : (ST <= 4 ? 4 : 2))
    for (int k = ks; k < g.K; k += KS) {
      float x[8];
      unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(X + (long long)k * ldx + l0)), x);
      const bf16* yk = Y + (long long)k * ldy;
#pragma unroll
      for (int t = 0; t < ST; ++t) {
        const float y = __bfloat162float(yk[t]);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j][t] = fmaf(x[j], y, acc[j][t]);
      }
    }
  }
  const int l = blockIdx.x * W + threadIdx.x;
#pragma unroll
  for (int t = 0; t < ST; ++t) {
#pragma unroll
    for (int j = 0; j < 8; ++j) red[ks][lg * 8 + j] = acc[j][t];
    __syncthreads();
    if (threadIdx.x < W && l < L) {
      float v = 0.f;
#pragma unroll
      for (int q = 0; q < KS; ++q) v += red[q][threadIdx.x];
      const int m = LONG_A ? l : t, n = LONG_A ? t : l;
      store_one(g, member, m, n, epilogue_one(g, member, m, n, v, 1));
    }
    __syncthreads();
  }
}

template <bool LONG_A, int ST>
static void launch_colacc_vec_n(const GemmArgs& g, int L, cudaStream_t s) {
  if ((long long)((L + 127) / 128) * g.batch >= 296)
    launch_with(dim3((L + 127) / 128, g.batch), 256, 0, s)(k_gemm_colacc_bf16x8<LONG_A, ST, 16>, g);
  else
    launch_with(dim3((L + 63) / 64, g.batch), 256, 0, s)(k_gemm_colacc_bf16x8<LONG_A, ST, 8>, g);
}
template <bool LONG_A>
static bool launch_colacc_vec(const GemmArgs& g, cudaStream_t s) {
  const int L = LONG_A ? g.M : g.N, S = LONG_A ? g.N : g.M;
  const long long ldx = LONG_A ? g.lda : g.ldb, sx = LONG_A ? g.strideA : g.strideB;
  const void* X = LONG_A ? g.A : g.B;
  if (g.in_dtype != kBF16 || L % 8 != 0 || L < 64 || ldx % 8 != 0 || sx % 8 != 0 || ((uintptr_t)X & 15) || g.batch > 65535)
    return false;
  switch (S) {   // one instantiation per width: no predicated-off columns in the inner loop
    case 1: launch_colacc_vec_n<LONG_A, 1>(g, L, s); break;   case 2: launch_colacc_vec_n<LONG_A, 2>(g, L, s); break;
    case 3: launch_colacc_vec_n<LONG_A, 3>(g, L, s); break;   case 4: launch_colacc_vec_n<LONG_A, 4>(g, L, s); break;
    case 5: launch_colacc_vec_n<LONG_A, 5>(g, L, s); break;   case 6: launch_colacc_vec_n<LONG_A, 6>(g, L, s); break;
    case 7: launch_colacc_vec_n<LONG_A, 7>(g, L, s); break;   case 8: launch_colacc_vec_n<LONG_A, 8>(g, L, s); break;
    case 9: launch_colacc_vec_n<LONG_A, 9>(g, L, s); break;   case 10: launch_colacc_vec_n<LONG_A, 10>(g, L, s); break;
    case 11: launch_colacc_vec_n<LONG_A, 11>(g, L, s); break; case 12: launch_colacc_vec_n<LONG_A, 12>(g, L, s); break;
    case 13: launch_colacc_vec_n<LONG_A, 13>(g, L, s); break; case 14: launch_colacc_vec_n<LONG_A, 14>(g, L, s); break;
    case 15: launch_colacc_vec_n<LONG_A, 15>(g, L, s); break; case 16: launch_colacc_vec_n<LONG_A, 16>(g, L, s); break;
    default: return false;
  }
  return true;
}

// K <= 16: every output element is a short dot product.  A thread owns one column n: it keeps B(n, 0..K-1) in
// registers and walks kSmallKRows rows of A, whose values every thread of the block reads alike (broadcast).
constexpr int kSmallKRows = 32;
template <typename T>
__global__ void __launch_bounds__(256) k_gemm_smallk(GemmArgs g) {
  pdl_prologue();
  const int member = blockIdx.z, m0 = blockIdx.y * kSmallKRows;
  const int n = blockIdx.x * 256 + threadIdx.x;
  __shared__ float As[kSmallKRows][kSkinny];
  const T* __restrict__ A = reinterpret_cast<const T*>(g.A) + member * g.strideA;
  const T* __restrict__ B = reinterpret_cast<const T*>(g.B) + member * g.strideB;
  for (int i = threadIdx.x; i < kSmallKRows * g.K; i += 256) {
    const int r = i / g.K, k = i % g.K, m = m0 + r;
    As[r][k] = m < g.M ? to_f<T>(g.a_mn ? A[(long long)k * g.lda + m] : A[(long long)m * g.lda + k]) : 0.f;
  }
  __syncthreads();
  if (n >= g.N) return;
  float b[kSkinny];
#pragma unroll
  for (int k = 0; k < kSkinny; ++k)
    b[k] = k < g.K ? to_f<T>(g.b_mn ? B[(long long)k * g.ldb + n] : B[(long long)n * g.ldb + k]) : 0.f;
  const int rows = min(kSmallKRows, g.M - m0);
  for (int r = 0; r < rows; ++r) {
    float v = 0.f;
#pragma unroll
    for (int k = 0; k < kSkinny; ++k)
      if (k < g.K) v = fmaf(As[r][k], b[k], v);
    store_one(g, member, m0 + r, n, epilogue_one(g, member, m0 + r, n, v, sizeof(T) == 2));
  }
}

// The same for bf16 operands and output with N a multiple of 8: a thread produces 8 consecutive columns
// of a row (16-byte loads of the weights and of the ReLU mask, one 16-byte store), the block's threads are spread
// over the 32 rows x N / 8 column groups of its slab.  Same multiply-add order per element as the kernel above.
template <bool B_MN>
__global__ void __launch_bounds__(256) k_gemm_smallk_bf16x8(GemmArgs g) {
  pdl_prologue();
  constexpr int KV = kSkinny;
  const int member = blockIdx.z, m0 = blockIdx.y * kSmallKRows;
  __shared__ float As[kSmallKRows][KV];
  const bf16* __restrict__ A = reinterpret_cast<const bf16*>(g.A) + member * g.strideA;
  const bf16* __restrict__ B = reinterpret_cast<const bf16*>(g.B) + member * g.strideB;
  for (int i = threadIdx.x; i < kSmallKRows * KV; i += 256) {
    const int r = i / KV, k = i % KV, m = m0 + r;
    As[r][k] = (m < g.M && k < g.K) ? __bfloat162float(g.a_mn ? A[(long long)k * g.lda + m] : A[(long long)m * g.lda + k]) : 0.f;
  }
  __syncthreads();
  const int groups = g.N >> 3;
  const int rows = min(kSmallKRows, g.M - m0);
  const float* bias = g.bias ? g.bias + member * g.strideBias : nullptr;
  const bf16* mask = g.mask ? reinterpret_cast<const bf16*>(g.mask) + member * g.strideMask : nullptr;
  bf16* C = reinterpret_cast<bf16*>(g.C) + member * g.strideC;
  const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll 2
  for (int idx = blockIdx.x * 256 + threadIdx.x; idx < rows * groups; idx += gridDim.x * 256) {
    const int r = idx / groups, n = (idx % groups) << 3;
    const int m = m0 + r;
    float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < KV; ++k) {
      if (k < g.K) {
        float b[8];
        if (B_MN) {
          const uint4 w = __ldg(reinterpret_cast<const uint4*>(B + (long long)k * g.ldb + n));
          const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) { b[2 * j] = __uint_as_float(u[j] << 16); b[2 * j + 1] = __uint_as_float(u[j] & 0xFFFF0000u); }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) b[j] = __bfloat162float(B[(long long)(n + j) * g.ldb + k]);
        }
        const float a = As[r][k];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = fmaf(a, b[j], v[j]);
      }
    }
    if (bias) {
      const float4 b0 = __ldg(reinterpret_cast<const float4*>(bias + n)), b1 = __ldg(reinterpret_cast<const float4*>(bias + n + 4));
      v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w; v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
    }
    if (g.relu) {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = fmaxf(v[j], 0.f);
    }
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      o[j] = *reinterpret_cast<uint32_t*>(&t);
    }
    if (mask) {
      const uint4 mk = __ldg(reinterpret_cast<const uint4*>(mask + (long long)m * g.ldmask + n));
      const uint32_t mu[4] = {mk.x, mk.y, mk.z, mk.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) o[j] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mu[j]), zero2);
    }
    *reinterpret_cast<uint4*>(C + (long long)m * g.ldc + n) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// The same for fp32 operands and output with N a multiple of 4: a thread produces 4 consecutive columns of a row
// (16-byte loads of the weights and of the ReLU mask, one 16-byte store).  The one-column-per-thread kernel above
// took 19 us for the data gradient of the fp32 population's one-wide output layer (128 x 512 outputs per member):
// 32 rows in sequence per thread, scalar mask loads and stores.  Same multiply-add order per element.
template <bool B_MN>
__global__ void __launch_bounds__(256) k_gemm_smallk_f32x4(GemmArgs g) {
  pdl_prologue();
  constexpr int KV = kSkinny;
  const int member = blockIdx.z, m0 = blockIdx.y * kSmallKRows;
  __shared__ float As[kSmallKRows][KV];
  const float* __restrict__ A = reinterpret_cast<const float*>(g.A) + member * g.strideA;
  const float* __restrict__ B = reinterpret_cast<const float*>(g.B) + member * g.strideB;
  for (int i = threadIdx.x; i < kSmallKRows * KV; i += 256) {
    const int r = i / KV, k = i % KV, m = m0 + r;
    As[r][k] = (m < g.M && k < g.K) ? (g.a_mn ? A[(long long)k * g.lda + m] : A[(long long)m * g.lda + k]) : 0.f;
  }
  __syncthreads();
  const int groups = g.N >> 2;
  const int rows = min(kSmallKRows, g.M - m0);
  const float* bias = g.bias ? g.bias + member * g.strideBias : nullptr;
  const float* mask = g.mask ? reinterpret_cast<const float*>(g.mask) + member * g.strideMask : nullptr;
  float* C = reinterpret_cast<float*>(g.C) + member * g.strideC;
#pragma unroll 2
  for (int idx = blockIdx.x * 256 + threadIdx.x; idx < rows * groups; idx += gridDim.x * 256) {
    const int r = idx / groups, n = (idx % groups) << 2;
    const int m = m0 + r;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < KV; ++k) {
      if (k < g.K) {
        float4 b;
        if (B_MN) b = __ldg(reinterpret_cast<const float4*>(B + (long long)k * g.ldb + n));
        else b = make_float4(B[(long long)n * g.ldb + k], B[(long long)(n + 1) * g.ldb + k], B[(long long)(n + 2) * g.ldb + k],
                             B[(long long)(n + 3) * g.ldb + k]);
        const float a = As[r][k];
        v[0] = fmaf(a, b.x, v[0]); v[1] = fmaf(a, b.y, v[1]); v[2] = fmaf(a, b.z, v[2]); v[3] = fmaf(a, b.w, v[3]);
      }
    }
    if (bias) {
      const float4 b0 = __ldg(reinterpret_cast<const float4*>(bias + n));
      v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
    }
    if (g.relu) {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = fmaxf(v[j], 0.f);
    }
    if (mask) {
      const float4 mk = __ldg(reinterpret_cast<const float4*>(mask + (long long)m * g.ldmask + n));
      if (!(mk.x > 0.f)) v[0] = 0.f;
      if (!(mk.y > 0.f)) v[1] = 0.f;
      if (!(mk.z > 0.f)) v[2] = 0.f;
      if (!(mk.w > 0.f)) v[3] = 0.f;
    }
    *reinterpret_cast<float4*>(C + (long long)m * g.ldc + n) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

static bool smallk_f32x4_ok(const GemmArgs& g) {
  if (g.in_dtype != kF32 || g.out_dtype != kF32 || g.K < 1 || g.K > kSkinny || g.N % 4 != 0 || g.N < 4) return false;
  if (g.ldc % 4 || g.strideC % 4 || ((uintptr_t)g.C & 15)) return false;
  if (g.b_mn && (g.ldb % 4 || g.strideB % 4 || ((uintptr_t)g.B & 15))) return false;
  if (g.mask && (g.ldmask % 4 || g.strideMask % 4 || ((uintptr_t)g.mask & 15))) return false;
  if (g.bias && (g.strideBias % 4 || ((uintptr_t)g.bias & 15))) return false;
  return (g.M + kSmallKRows - 1) / kSmallKRows <= 65535 && g.batch <= 65535;
}

// The same product for K <= 10 (a critic's two-wide input layer, the data gradient of a one-, two- or ten-wide
// output layer) with
// the roles turned around: a thread keeps the weights and the bias of ITS 8 columns in registers and walks down the
// rows, so that per output vector there is one small broadcast load of the row's K inputs, K x 8 multiply-adds,
// the mask load and one 16-byte store, with four rows in flight.  A block covers all columns (up to 2048) and
// kRowsPerLane rows per row lane.  Same multiply-add order per element as the kernels above.
constexpr int kRowsPerLane = 16;
constexpr int kTinyK = 10;   // K up to which a thread keeps its 8 columns' weights in registers
template <bool B_MN, int KK>
__global__ void __launch_bounds__(256) k_gemm_tinyk_bf16x8(GemmArgs g) {
  pdl_prologue();
  const int member = blockIdx.z;
  const int groups = g.N >> 3;
  const int tpr = groups < 256 ? groups : 256;          // threads across one row
  const int lanes = 256 / tpr;                          // rows worked on at a time
  const int cg = threadIdx.x % tpr, rl = threadIdx.x / tpr;
  if (rl >= lanes) return;
  const int n = (blockIdx.x * tpr + cg) << 3;
  if (n >= g.N) return;
  const bf16* __restrict__ A = reinterpret_cast<const bf16*>(g.A) + member * g.strideA;
  const bf16* __restrict__ B = reinterpret_cast<const bf16*>(g.B) + member * g.strideB;
  float b[KK][8], bias[8];
#pragma unroll
  for (int k = 0; k < KK; ++k) {
    if (B_MN) {
      unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(B + (long long)k * g.ldb + n)), b[k]);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) b[k][j] = __bfloat162float(B[(long long)(n + j) * g.ldb + k]);
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) bias[j] = g.bias ? g.bias[member * g.strideBias + n + j] : 0.f;
  const bf16* mask = g.mask ? reinterpret_cast<const bf16*>(g.mask) + member * g.strideMask : nullptr;
  bf16* C = reinterpret_cast<bf16*>(g.C) + member * g.strideC;
  const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
  const int m_begin = blockIdx.y * (lanes * kRowsPerLane) + rl;
  const int m_end = min(g.M, (int)(blockIdx.y + 1) * (lanes * kRowsPerLane));
#pragma unroll 4
  for (int m = m_begin; m < m_end; m += lanes) {
    float a[KK];
#pragma unroll
    for (int k = 0; k < KK; ++k) a[k] = __bfloat162float(A[(long long)m * g.lda + k]);
    float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < KK; ++k)
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = fmaf(a[k], b[k][j], v[j]);
    if (g.bias) {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] += bias[j];
    }
    if (g.relu) {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = fmaxf(v[j], 0.f);
    }
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      o[j] = *reinterpret_cast<uint32_t*>(&t);
    }
    if (mask) {
      const uint4 mk = __ldg(reinterpret_cast<const uint4*>(mask + (long long)m * g.ldmask + n));
      const uint32_t mu[4] = {mk.x, mk.y, mk.z, mk.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) o[j] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mu[j]), zero2);
    }
    *reinterpret_cast<uint4*>(C + (long long)m * g.ldc + n) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

template <bool B_MN>
static void launch_tinyk(const GemmArgs& g, cudaStream_t s) {
  const int groups = g.N >> 3, tpr = groups < 256 ? groups : 256, lanes = 256 / tpr;
  const dim3 grid((groups + tpr - 1) / tpr, (g.M + lanes * kRowsPerLane - 1) / (lanes * kRowsPerLane), g.batch);
  switch (g.K) {
    case 1: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 1>, g); break;
    case 2: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 2>, g); break;
    case 3: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 3>, g); break;
    case 4: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 4>, g); break;
    case 5: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 5>, g); break;
    case 6: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 6>, g); break;
    case 7: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 7>, g); break;
    case 8: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 8>, g); break;
    case 9: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 9>, g); break;
    default: launch_with(grid, 256, 0, s)(k_gemm_tinyk_bf16x8<B_MN, 10>, g); break;
  }
}

static bool smallk_vec_ok(const GemmArgs& g) {
  if (g.in_dtype != kBF16 || g.out_dtype != kBF16 || g.K < 1 || g.K > kSkinny || g.N % 8 != 0) return false;
  if (g.ldc % 8 || g.strideC % 8 || ((uintptr_t)g.C & 15)) return false;
  if (g.b_mn && (g.ldb % 8 || g.strideB % 8 || ((uintptr_t)g.B & 15))) return false;
  if (g.mask && (g.ldmask % 8 || g.strideMask % 8 || ((uintptr_t)g.mask & 15))) return false;
  if (g.bias && (g.strideBias % 4 || ((uintptr_t)g.bias & 15))) return false;
  return (g.M + kSmallKRows - 1) / kSmallKRows <= 65535 && g.batch <= 65535;
}

template <typename T, bool B_MN>
static void launch_rowdot(const GemmArgs& g, cudaStream_t s) {
  dim3 grid((g.M + 7) / 8, g.batch);
  if (g.N == 1) launch_with(grid, 256, 0, s)(k_gemm_rowdot<T, B_MN, 1>, g);
  else if (g.N == 2) launch_with(grid, 256, 0, s)(k_gemm_rowdot<T, B_MN, 2>, g);
  else if (g.N <= 4) launch_with(grid, 256, 0, s)(k_gemm_rowdot<T, B_MN, 4>, g);
  else if (g.N <= 8) launch_with(grid, 256, 0, s)(k_gemm_rowdot<T, B_MN, 8>, g);
  else launch_with(grid, 256, 0, s)(k_gemm_rowdot<T, B_MN, 16>, g);
}
template <typename T, bool LONG_A>
static void launch_colacc(const GemmArgs& g, cudaStream_t s) {
  const int L = LONG_A ? g.M : g.N, S = LONG_A ? g.N : g.M;
  dim3 grid((L + 31) / 32, g.batch);
  if (S == 1) launch_with(grid, 512, 0, s)(k_gemm_colacc<T, LONG_A, 1>, g);
  else if (S == 2) launch_with(grid, 512, 0, s)(k_gemm_colacc<T, LONG_A, 2>, g);
  else if (S <= 4) launch_with(grid, 512, 0, s)(k_gemm_colacc<T, LONG_A, 4>, g);
  else if (S <= 8) launch_with(grid, 512, 0, s)(k_gemm_colacc<T, LONG_A, 8>, g);
  else launch_with(grid, 512, 0, s)(k_gemm_colacc<T, LONG_A, 16>, g);
}

template <typename T>
static bool launch_skinny(const GemmArgs& g, cudaStream_t s) {
  if (smallk_vec_ok(g) && g.K <= kTinyK && !g.a_mn && g.N >= 8 &&
      (long long)((g.M + kRowsPerLane - 1) / kRowsPerLane) <= 65535) {
    if (g.b_mn) launch_tinyk<true>(g, s);
    else launch_tinyk<false>(g, s);
    return true;
  }
  if (smallk_vec_ok(g)) {
    const int per_slab = kSmallKRows * (g.N / 8);
    const dim3 grid((per_slab + 255) / 256 > 8 ? 8 : (per_slab + 255) / 256, (g.M + kSmallKRows - 1) / kSmallKRows, g.batch);
    if (g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_smallk_bf16x8<true>, g);
    else launch_with(grid, 256, 0, s)(k_gemm_smallk_bf16x8<false>, g);
    return true;
  }
  if (smallk_f32x4_ok(g)) {
    const int per_slab = kSmallKRows * (g.N / 4);
    const dim3 grid((per_slab + 255) / 256 > 8 ? 8 : (per_slab + 255) / 256, (g.M + kSmallKRows - 1) / kSmallKRows, g.batch);
    if (g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_smallk_f32x4<true>, g);
    else launch_with(grid, 256, 0, s)(k_gemm_smallk_f32x4<false>, g);
    return true;
  }
  if (g.K <= kSkinny && g.K > 0 && (g.M + kSmallKRows - 1) / kSmallKRows <= 65535 && g.batch <= 65535) {
    launch_with(dim3((g.N + 255) / 256, (g.M + kSmallKRows - 1) / kSmallKRows, g.batch), 256, 0, s)(k_gemm_smallk<T>, g);
    return true;
  }
  if (rowdot_vec_ok(g)) {
    launch_rowdot_vec(g, s);
    return true;
  }
  if (g.N <= kSkinny && !g.a_mn) {
    if (g.b_mn) launch_rowdot<T, true>(g, s);
    else launch_rowdot<T, false>(g, s);
    return true;
  }
  if (g.a_mn && g.b_mn && g.N <= kSkinny) {
    if (!launch_colacc_vec<true>(g, s)) launch_colacc<T, true>(g, s);
    return true;
  }
  if (g.a_mn && g.b_mn && g.M <= kSkinny) {
    if (!launch_colacc_vec<false>(g, s)) launch_colacc<T, false>(g, s);
    return true;
  }
  return false;
}

template <typename T>
static cudaError_t launch_t(const GemmArgs& g, cudaStream_t s) {
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  if (simt_interior_ok<T>(g)) {
    // 128 x 64 tiles when they still go round the SMs (both tiles add in the same order: the choice, which depends on
    // the number of members, does not change a bit of the result)
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool tall = g.M % 128 == 0 && (long long)(g.M / 128) * grid.x * g.batch * 5 >= (long long)sms * 4;
    if (tall) {
      grid.y = g.M / 128;
      if (!g.a_mn && !g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, false, false, 8>, g);
      else if (!g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, false, true, 8>, g);
      else if (g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, true, true, 8>, g);
      else launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, true, false, 8>, g);
      return cudaGetLastError();
    }
    if (!g.a_mn && !g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, false, false, 4>, g);
    else if (!g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, false, true, 4>, g);
    else if (g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, true, true, 4>, g);
    else launch_with(grid, 256, 0, s)(k_gemm_simt_interior<T, true, false, 4>, g);
    return cudaGetLastError();
  }
  if (!g.a_mn && !g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt<T, false, false>, g);
  else if (!g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt<T, false, true>, g);
  else if (g.a_mn && g.b_mn) launch_with(grid, 256, 0, s)(k_gemm_simt<T, true, true>, g);
  else launch_with(grid, 256, 0, s)(k_gemm_simt<T, true, false>, g);
  return cudaGetLastError();
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return cudaSuccess;
  if (g.in_dtype == kBF16 ? launch_skinny<bf16>(g, s) : launch_skinny<float>(g, s)) return cudaGetLastError();
  return g.in_dtype == kBF16 ? launch_t<bf16>(g, s) : launch_t<float>(g, s);
}

}  // namespace pbt
