// Fused per-member optimiser kernels: theta <- step(theta | h) (Eq. 2), the
// update part.  One pass over the member-major slabs; every member reads its own
// learning rate / momentum / beta1 / weight decay from its row of H.
//
// HBM-bound by construction.  Adam moves, per parameter, 16 B in (master, m, v,
// gradient) and 14 B out (master, m, v, bf16 shadow); SGD-momentum 12 B in and
// 8 B out (+2 B shadow for bf16 populations).  All streams are accessed as
// 16-byte vectors, two per thread per stream, fully coalesced.
#include "pbt_common.cuh"

namespace pbt {

constexpr int kOptThreads = 256;
constexpr int kOptVecPerThread = 2;                              // float4 per stream per thread per iteration
constexpr int kOptTile = kOptThreads * kOptVecPerThread * 4;     // elements per block iteration

// v <- mu v + g ; theta <- theta - lr v
__global__ void __launch_bounds__(kOptThreads) k_sgdm(OptArgs a) {
  pdl_prologue();
  const int m = blockIdx.y;
  const float* Hrow = a.H + (long long)m * a.nh_stride;
  const float lr = hp(Hrow, a.slot_lr, a.const_lr);
  const float mu = hp(Hrow, a.slot_momentum, a.const_momentum);
  const long long base = (long long)m * a.p_pad + a.begin;
  float* w = a.w32 + base;
  float* v = a.opt1 + base;
  const float* g = a.grad + base;
  bf16* w16 = a.w16 ? a.w16 + base : nullptr;
  for (long long t0 = (long long)blockIdx.x * kOptTile; t0 < a.count; t0 += (long long)gridDim.x * kOptTile) {
#pragma unroll
    for (int j = 0; j < kOptVecPerThread; ++j) {
      const long long i = t0 + ((long long)j * kOptThreads + threadIdx.x) * 4;
      if (i < a.count) {
        const float4 gw = ld_stream(g + i), ww = ld_stream(w + i), vv = ld_stream(v + i);
        float4 nv, nw;
        nv.x = __fmaf_rn(mu, vv.x, gw.x); nv.y = __fmaf_rn(mu, vv.y, gw.y);
        nv.z = __fmaf_rn(mu, vv.z, gw.z); nv.w = __fmaf_rn(mu, vv.w, gw.w);
        nw.x = __fmaf_rn(-lr, nv.x, ww.x); nw.y = __fmaf_rn(-lr, nv.y, ww.y);
        nw.z = __fmaf_rn(-lr, nv.z, ww.z); nw.w = __fmaf_rn(-lr, nv.w, ww.w);
        st_stream(v + i, nv);
        st_stream(w + i, nw);
        if (w16) st_bf16x4(w16 + i, nw);
      }
    }
  }
}

// m <- b1 m + (1-b1) g ; v <- b2 v + (1-b2) g^2 ;
// theta <- theta - lr (m / (1-c1)) / (sqrt(v / (1-c2)) + eps) - lr wd theta,
// c1, c2 = running products of the betas including this step.
__global__ void __launch_bounds__(kOptThreads) k_adam(OptArgs a) {
  pdl_prologue();
  const int m = blockIdx.y;
  const float* Hrow = a.H + (long long)m * a.nh_stride;
  const float lr = hp(Hrow, a.slot_lr, a.const_lr);
  const float b1 = hp(Hrow, a.slot_beta1, a.const_beta1);
  const float wd = hp(Hrow, a.slot_wd, a.const_wd);
  const float b2 = a.const_beta2, eps = a.const_eps;
  const float c1 = __fmul_rn(a.scalars[m * PBT_N_SCALARS + a.scalar_base + 0], b1);
  const float c2 = __fmul_rn(a.scalars[m * PBT_N_SCALARS + a.scalar_base + 1], b2);
  const float inv_bc1 = 1.f / (1.f - c1), inv_bc2 = 1.f / (1.f - c2);
  const float omb1 = 1.f - b1, omb2 = 1.f - b2, lrwd = lr * wd;
  const long long base = (long long)m * a.p_pad + a.begin;
  float* w = a.w32 + base;
  float* m1 = a.opt1 + base;
  float* m2 = a.opt2 + base;
  const float* g = a.grad + base;
  bf16* w16 = a.w16 ? a.w16 + base : nullptr;
  for (long long t0 = (long long)blockIdx.x * kOptTile; t0 < a.count; t0 += (long long)gridDim.x * kOptTile) {
    float4 gw[kOptVecPerThread], ww[kOptVecPerThread], aa[kOptVecPerThread], bb[kOptVecPerThread];
#pragma unroll
    for (int j = 0; j < kOptVecPerThread; ++j) {
      const long long i = t0 + ((long long)j * kOptThreads + threadIdx.x) * 4;
      if (i < a.count) {
        gw[j] = ld_stream(g + i); ww[j] = ld_stream(w + i);
        aa[j] = ld_stream(m1 + i); bb[j] = ld_stream(m2 + i);
      }
    }
#pragma unroll
    for (int j = 0; j < kOptVecPerThread; ++j) {
      const long long i = t0 + ((long long)j * kOptThreads + threadIdx.x) * 4;
      if (i < a.count) {
        float4 nw;
        nw.x = adam_one(ww[j].x, aa[j].x, bb[j].x, gw[j].x, b1, omb1, b2, omb2, inv_bc1, inv_bc2, lr, eps, lrwd);
        nw.y = adam_one(ww[j].y, aa[j].y, bb[j].y, gw[j].y, b1, omb1, b2, omb2, inv_bc1, inv_bc2, lr, eps, lrwd);
        nw.z = adam_one(ww[j].z, aa[j].z, bb[j].z, gw[j].z, b1, omb1, b2, omb2, inv_bc1, inv_bc2, lr, eps, lrwd);
        nw.w = adam_one(ww[j].w, aa[j].w, bb[j].w, gw[j].w, b1, omb1, b2, omb2, inv_bc1, inv_bc2, lr, eps, lrwd);
        st_stream(m1 + i, aa[j]);
        st_stream(m2 + i, bb[j]);
        st_stream(w + i, nw);
        if (w16) st_bf16x4(w16 + i, nw);
      }
    }
  }
}

// ms <- rho ms + (1-rho) g^2 ; theta <- theta - lr g / (sqrt(ms) + eps)
__global__ void __launch_bounds__(kOptThreads) k_rmsprop(OptArgs a) {
  pdl_prologue();
  const int m = blockIdx.y;
  const float* Hrow = a.H + (long long)m * a.nh_stride;
  const float lr = hp(Hrow, a.slot_lr, a.const_lr);
  const float rho = a.const_beta2, omr = 1.f - a.const_beta2, eps = a.const_eps;
  const long long base = (long long)m * a.p_pad + a.begin;
  float* w = a.w32 + base;
  float* ms = a.opt1 + base;
  const float* g = a.grad + base;
  bf16* w16 = a.w16 ? a.w16 + base : nullptr;
  for (long long t0 = (long long)blockIdx.x * kOptTile; t0 < a.count; t0 += (long long)gridDim.x * kOptTile) {
#pragma unroll
    for (int j = 0; j < kOptVecPerThread; ++j) {
      const long long i = t0 + ((long long)j * kOptThreads + threadIdx.x) * 4;
      if (i < a.count) {
        const float4 gw = ld_stream(g + i), ww = ld_stream(w + i), vv = ld_stream(ms + i);
        float4 nv, nw;
        nv.x = __fmaf_rn(rho, vv.x, omr * gw.x * gw.x); nv.y = __fmaf_rn(rho, vv.y, omr * gw.y * gw.y);
        nv.z = __fmaf_rn(rho, vv.z, omr * gw.z * gw.z); nv.w = __fmaf_rn(rho, vv.w, omr * gw.w * gw.w);
        nw.x = ww.x - lr * __fdividef(gw.x, sqrtf(nv.x) + eps); nw.y = ww.y - lr * __fdividef(gw.y, sqrtf(nv.y) + eps);
        nw.z = ww.z - lr * __fdividef(gw.z, sqrtf(nv.z) + eps); nw.w = ww.w - lr * __fdividef(gw.w, sqrtf(nv.w) + eps);
        st_stream(ms + i, nv);
        st_stream(w + i, nw);
        if (w16) st_bf16x4(w16 + i, nw);
      }
    }
  }
}

// after the Adam pass of a stack: store the advanced beta products
__global__ void k_adam_advance(OptArgs a) {
  pdl_prologue();
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= a.n_members) return;
  const float* Hrow = a.H + (long long)m * a.nh_stride;
  const float b1 = hp(Hrow, a.slot_beta1, a.const_beta1);
  float* sc = a.scalars + m * PBT_N_SCALARS + a.scalar_base;
  sc[0] = __fmul_rn(sc[0], b1);
  sc[1] = __fmul_rn(sc[1], a.const_beta2);
}

static unsigned opt_grid_x(const OptArgs& a) {
  long long tiles = (a.count + kOptTile - 1) / kOptTile;
  // enough blocks to fill 148 SMs several times over, but let big slabs loop
  long long per_member = (148ll * 8 + a.n_members - 1) / a.n_members;
  if (per_member < 1) per_member = 1;
  if (tiles > per_member) tiles = per_member;
  if (tiles < 1) tiles = 1;
  return (unsigned)tiles;
}

// theta <- theta - lr g (plain gradient descent: no optimiser state is read or written)
__global__ void __launch_bounds__(kOptThreads) k_sgd(OptArgs a) {
  pdl_prologue();
  const int m = blockIdx.y;
  const float lr = hp(a.H + (long long)m * a.nh_stride, a.slot_lr, a.const_lr);
  const long long base = (long long)m * a.p_pad + a.begin;
  float* w = a.w32 + base;
  const float* g = a.grad + base;
  bf16* w16 = a.w16 ? a.w16 + base : nullptr;
  for (long long t0 = (long long)blockIdx.x * kOptTile; t0 < a.count; t0 += (long long)gridDim.x * kOptTile) {
#pragma unroll
    for (int j = 0; j < kOptVecPerThread; ++j) {
      const long long i = t0 + ((long long)j * kOptThreads + threadIdx.x) * 4;
      if (i < a.count) {
        const float4 gw = ld_stream(g + i), ww = ld_stream(w + i);
        float4 nw;
        nw.x = __fmaf_rn(-lr, gw.x, ww.x); nw.y = __fmaf_rn(-lr, gw.y, ww.y);
        nw.z = __fmaf_rn(-lr, gw.z, ww.z); nw.w = __fmaf_rn(-lr, gw.w, ww.w);
        st_stream(w + i, nw);
        if (w16) st_bf16x4(w16 + i, nw);
      }
    }
  }
}

cudaError_t launch_sgd(const OptArgs& a, cudaStream_t s) {
  dim3 grid(opt_grid_x(a), a.n_members);
  launch_with(grid, kOptThreads, 0, s)(k_sgd, a);
  return cudaGetLastError();
}
cudaError_t launch_sgdm(const OptArgs& a, cudaStream_t s) {
  dim3 grid(opt_grid_x(a), a.n_members);
  launch_with(grid, kOptThreads, 0, s)(k_sgdm, a);
  return cudaGetLastError();
}
cudaError_t launch_rmsprop(const OptArgs& a, cudaStream_t s) {
  dim3 grid(opt_grid_x(a), a.n_members);
  launch_with(grid, kOptThreads, 0, s)(k_rmsprop, a);
  return cudaGetLastError();
}
cudaError_t launch_adam(const OptArgs& a, cudaStream_t s) {
  dim3 grid(opt_grid_x(a), a.n_members);
  launch_with(grid, kOptThreads, 0, s)(k_adam, a);
  return cudaGetLastError();
}
cudaError_t launch_adam_advance(const OptArgs& a, cudaStream_t s) {
  launch_with((a.n_members + 127) / 128, 128, 0, s)(k_adam_advance, a);
  return cudaGetLastError();
}

}  // namespace pbt
