// Small kernels of the training step: weight initialisation, batch windows,
// losses with their logit derivatives, bias gradients, evaluation reductions,
// the toy model.  All reductions run in a fixed order (no floating atomics), so
// a run is bit-reproducible.
#include "pbt_common.cuh"

namespace pbt {

// ---------------------------------------------------------------------------
// Initial weights: U(-a, a) from the init stream, one Philox call per 4 elements.
// Element idx of tensor `tensor_id` of member m uses
// philox(seed; m, idx >> 2, init stream, tensor_id).x[idx & 3].
// ---------------------------------------------------------------------------
__global__ void k_init_weights(float* __restrict__ w32, long long p_pad, long long w_off, long long count,
                               int tensor_id, float bound, uint64_t seed, int member_base) {
  pdl_prologue();
  const int m = blockIdx.y;
  const long long blk = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (blk * 4 >= count) return;
  const U4 r = philox4x32_10((uint32_t)(member_base + m), (uint32_t)blk, kStreamInit, (uint32_t)tensor_id, seed);
  float* dst = w32 + (long long)m * p_pad + w_off;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const long long idx = blk * 4 + j;
    if (idx < count) {
      const float u = __fsub_rn(__fmul_rn((float)(r.x[j] >> 8), 1.1920928955078125e-07f), 1.0f);
      dst[idx] = __fmul_rn(u, bound);
    }
  }
}

cudaError_t launch_init_weights(float* w32, long long p_pad, int n_members, long long w_off, int fan_out,
                                int fan_in, int tensor_id, float bound, uint64_t seed, int member_base, cudaStream_t s) {
  const long long count = (long long)fan_out * fan_in;
  const long long blocks4 = (count + 3) / 4;
  dim3 grid((unsigned)((blocks4 + 255) / 256), n_members);
  launch_with(grid, 256, 0, s)(k_init_weights, w32, p_pad, w_off, count, tensor_id, bound, seed, member_base);
  return cudaGetLastError();
}

__global__ void k_f32_to_bf16(const float* __restrict__ in, bf16* __restrict__ out, long long n) {
  pdl_prologue();
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += stride) out[i] = __float2bfloat16_rn(in[i]);
}

cudaError_t launch_f32_to_bf16(const float* in, bf16* out, long long n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  long long blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  launch_with((unsigned)blocks, 256, 0, s)(k_f32_to_bf16, in, out, n);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Training-batch window: rows [off, off + rows) of the pool, contiguous, so the
// copy is a flat byte range per member.
// ---------------------------------------------------------------------------
__global__ void k_gather_window(char* __restrict__ dst, long long dst_stride_bytes, long long dst_offset_bytes,
                                const char* __restrict__ pool, int row_bytes, int rows, int pool_rows, int block,
                                int word_index, uint64_t seed, const Counters* __restrict__ counters, StepClock clk) {
  pdl_prologue();
  if (counters->use_supplied_batch) return;
  const int m = blockIdx.y;
  const U4 r = philox4x32_10((uint32_t)(clk.member_base + m), (uint32_t)clk.t[m], kStreamBatch, (uint32_t)block, seed);
  const uint32_t n_win = (uint32_t)((pool_rows - rows) / 128 + 1);
  const long long off = 128ll * (long long)(((uint64_t)r.x[word_index] * n_win) >> 32);
  const long long bytes = (long long)rows * row_bytes;
  const char* src = pool + off * row_bytes;
  char* d = dst + (long long)m * dst_stride_bytes + dst_offset_bytes;
  const long long n16 = bytes / 16;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long nthreads = (long long)gridDim.x * blockDim.x;
  if ((((uintptr_t)src | (uintptr_t)d) & 15) == 0) {
    const int4* s4 = reinterpret_cast<const int4*>(src);
    int4* d4 = reinterpret_cast<int4*>(d);
    for (long long i = tid; i < n16; i += nthreads) d4[i] = __ldg(s4 + i);
    for (long long i = n16 * 16 + tid; i < bytes; i += nthreads) d[i] = src[i];
  } else {
    for (long long i = tid; i < bytes; i += nthreads) d[i] = src[i];
  }
}

__global__ void k_window_offsets(int* __restrict__ off, int rows, int pool_rows, int n_members, int block, int word_index,
                                 uint64_t seed, StepClock clk) {
  pdl_prologue();
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= n_members) return;
  const U4 r = philox4x32_10((uint32_t)(clk.member_base + m), (uint32_t)clk.t[m], kStreamBatch, (uint32_t)block, seed);
  const uint32_t n_win = (uint32_t)((pool_rows - rows) / 128 + 1);
  off[m] = (int)(128ll * (long long)(((uint64_t)r.x[word_index] * n_win) >> 32));
}

cudaError_t launch_window_offsets(int* off, int rows, int pool_rows, int n_members, int block, int word_index,
                                  uint64_t seed, StepClock clk, cudaStream_t s) {
  launch_with((n_members + 127) / 128, 128, 0, s)(k_window_offsets, off, rows, pool_rows, n_members, block, word_index, seed, clk);
  return cudaGetLastError();
}

cudaError_t launch_gather_window(char* dst, long long dst_stride_bytes, long long dst_offset_bytes,
                                 const char* pool, int row_bytes, int rows, int pool_rows, int n_members,
                                 int block, int word_index, uint64_t seed, const Counters* counters,
                                 StepClock clk, cudaStream_t s) {
  const long long bytes = (long long)rows * row_bytes;
  long long blocks = (bytes / 16 + 255) / 256;
  if (blocks < 1) blocks = 1;
  if (blocks > 64) blocks = 64;
  dim3 grid((unsigned)blocks, n_members);
  launch_with(grid, 256, 0, s)(k_gather_window, dst, dst_stride_bytes, dst_offset_bytes, pool, row_bytes, rows, pool_rows,
                                       block, word_index, seed, counters, clk);
  return cudaGetLastError();
}

template <typename TD>
__global__ void k_copy_rows(TD* __restrict__ dst, long long dst_ld, long long dst_stride,
                            const float* __restrict__ src, long long src_ld, long long src_stride, int rows,
                            int cols) {
  pdl_prologue();
  const int m = blockIdx.y;
  const long long total = (long long)rows * cols;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / cols, c = i % cols;
    const float v = src[m * src_stride + r * src_ld + c];
    if constexpr (sizeof(TD) == 2) dst[m * dst_stride + r * dst_ld + c] = __float2bfloat16_rn(v);
    else dst[m * dst_stride + r * dst_ld + c] = v;
  }
}

cudaError_t launch_copy_rows(void* dst, int dst_dtype, long long dst_ld, long long dst_stride, const float* src,
                             long long src_ld, long long src_stride, int rows, int cols, int n_members,
                             cudaStream_t s) {
  const long long total = (long long)rows * cols;
  long long blocks = (total + 255) / 256;
  if (blocks > 32) blocks = 32;
  dim3 grid((unsigned)blocks, n_members);
  if (dst_dtype == kBF16)
    launch_with(grid, 256, 0, s)(k_copy_rows<bf16>, (bf16*)dst, dst_ld, dst_stride, src, src_ld, src_stride, rows, cols);
  else
    launch_with(grid, 256, 0, s)(k_copy_rows<float>, (float*)dst, dst_ld, dst_stride, src, src_ld, src_stride, rows, cols);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Losses: one warp per (member, row).  Writes the row's loss and, when asked,
// dL/dz of the batch-mean loss in the operand type.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float load_as_float(const void* p, int dtype, long long i) {
  return dtype == kBF16 ? __bfloat162float(reinterpret_cast<const bf16*>(p)[i])
                        : reinterpret_cast<const float*>(p)[i];
}
__device__ __forceinline__ void store_from_float(void* p, int dtype, long long i, float v) {
  if (dtype == kBF16) reinterpret_cast<bf16*>(p)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[i] = v;
}
__device__ __forceinline__ float softplus_f(float x) { return fmaxf(x, 0.f) + log1pf(expf(-fabsf(x))); }
__device__ __forceinline__ float sigmoid_f(float x) {
  const float e = expf(-fabsf(x));
  return x >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
}

__global__ void k_loss_rows(LossArgs a) {
  pdl_prologue();
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.y;
  const int row = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const float* z = a.logits + m * a.stride_logits + (long long)row * a.ld_logits;
  const long long trow = (long long)row + (a.target_rowoff ? a.target_rowoff[m] : 0);   // row of the target matrix
  const long long dz_base = m * a.stride_dz + (long long)row * a.ld_dz;
  float loss = 0.f;
  if (a.kind == PBT_LOSS_MSE) {
    const float* y = reinterpret_cast<const float*>(a.target) + m * a.stride_target + trow * a.cols;
    float acc = 0.f;
    for (int c = lane; c < a.cols; c += 32) {
      const float d = z[c] - y[c];
      acc += d * d;
      if (a.dz) store_from_float(a.dz, a.dz_dtype, dz_base + c, 2.f * d * a.inv_batch);
    }
    loss = warp_sum(acc);
  } else if (a.kind == PBT_LOSS_CE_HARD || a.kind == PBT_LOSS_CE_SOFT) {
    float mx = -INFINITY;
    for (int c = lane; c < a.cols; c += 32) mx = fmaxf(mx, z[c]);
    mx = warp_max(mx);
    float se = 0.f;
    for (int c = lane; c < a.cols; c += 32) se += expf(z[c] - mx);
    se = warp_sum(se);
    const float lse = logf(se);
    const float inv_se = 1.f / se;
    if (a.kind == PBT_LOSS_CE_HARD) {
      const int label = reinterpret_cast<const int*>(a.target)[m * a.stride_target + trow];
      loss = lse - (z[label] - mx);
      if (a.dz)
        for (int c = lane; c < a.cols; c += 32) {
          const float p = expf(z[c] - mx) * inv_se;
          store_from_float(a.dz, a.dz_dtype, dz_base + c, (p - (c == label ? 1.f : 0.f)) * a.inv_batch);
        }
    } else {
      const long long tb = m * a.stride_target + trow * a.cols;
      float tsum = 0.f, tl = 0.f;
      for (int c = lane; c < a.cols; c += 32) {
        const float t = load_as_float(a.target, a.target_dtype, tb + c);
        tsum += t;
        tl += t * ((z[c] - mx) - lse);
      }
      tsum = warp_sum(tsum);
      loss = -warp_sum(tl);
      if (a.dz)
        for (int c = lane; c < a.cols; c += 32) {
          const float t = load_as_float(a.target, a.target_dtype, tb + c);
          const float p = expf(z[c] - mx) * inv_se;
          store_from_float(a.dz, a.dz_dtype, dz_base + c, (p * tsum - t) * a.inv_batch);
        }
    }
  } else if (a.kind == PBT_LOSS_WGAN_GP) {  // one critic value per row
    const float d = z[0];
    const int cls = row < a.n_real_rows ? 0 : (row < 2 * a.n_real_rows ? 1 : 2);
    if (a.dz && lane == 0)
      store_from_float(a.dz, a.dz_dtype, dz_base, cls == 0 ? -a.inv_batch : (cls == 1 ? a.inv_batch : 1.f));
    if (cls == 2) return;  // interpolate: its loss is the penalty, written once the input gradient is known
    loss = cls == 0 ? -d : d;
  } else {  // PBT_LOSS_GAN_LOGISTIC: one logit per row
    const float d = z[0];
    const bool real = row < a.n_real_rows;
    loss = real ? softplus_f(-d) : softplus_f(d);
    if (a.dz && lane == 0)
      store_from_float(a.dz, a.dz_dtype, dz_base, (real ? -sigmoid_f(-d) : sigmoid_f(d)) * a.inv_batch);
  }
  if (lane == 0) a.row_loss[(long long)m * a.rows + row] = loss;
}

// Cross-entropy against a bf16 target distribution for rows of 128 * ITERS logits (ITERS <= 8), one warp per row:
// the whole row and its targets are fetched with one batch of 16-byte / 8-byte loads per lane and stay in registers,
// so a row costs two memory latencies instead of one per loop trip (the generic kernel above is latency-bound:
// 29 us per row and warp on the 1024-wide output layer).  Same formulas, different summation order.
template <int ITERS>
__global__ void __launch_bounds__(256) k_loss_ce_soft_vec(LossArgs a) {
  pdl_prologue();
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.y;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= a.rows) return;
  const float4* z4 = reinterpret_cast<const float4*>(a.logits + m * a.stride_logits + (long long)row * a.ld_logits);
  const long long trow = (long long)row + (a.target_rowoff ? a.target_rowoff[m] : 0);
  const uint2* t2 = reinterpret_cast<const uint2*>(reinterpret_cast<const bf16*>(a.target) + m * a.stride_target + trow * a.cols);
  float4 z[ITERS];
  uint2 tp[ITERS];
#pragma unroll
  for (int k = 0; k < ITERS; ++k) z[k] = __ldg(z4 + lane + 32 * k);
#pragma unroll
  for (int k = 0; k < ITERS; ++k) tp[k] = __ldg(t2 + lane + 32 * k);
  float mx = -INFINITY;
#pragma unroll
  for (int k = 0; k < ITERS; ++k) mx = fmaxf(fmaxf(mx, fmaxf(z[k].x, z[k].y)), fmaxf(z[k].z, z[k].w));
  mx = warp_max(mx);
  float se = 0.f;
#pragma unroll
  for (int k = 0; k < ITERS; ++k) {
    z[k].x -= mx; z[k].y -= mx; z[k].z -= mx; z[k].w -= mx;
    se += (expf(z[k].x) + expf(z[k].y)) + (expf(z[k].z) + expf(z[k].w));
  }
  se = warp_sum(se);
  const float lse = logf(se);
  const float inv_se = 1.f / se;
  float tsum = 0.f, tl = 0.f;
#pragma unroll
  for (int k = 0; k < ITERS; ++k) {
    const float t0 = __uint_as_float(tp[k].x << 16), t1 = __uint_as_float(tp[k].x & 0xFFFF0000u);
    const float t3 = __uint_as_float(tp[k].y & 0xFFFF0000u), t2f = __uint_as_float(tp[k].y << 16);
    tsum += (t0 + t1) + (t2f + t3);
    tl += (t0 * (z[k].x - lse) + t1 * (z[k].y - lse)) + (t2f * (z[k].z - lse) + t3 * (z[k].w - lse));
  }
  tsum = warp_sum(tsum);
  const float loss = -warp_sum(tl);
  if (a.dz) {
    uint2* d2 = reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(a.dz) + m * a.stride_dz + (long long)row * a.ld_dz);
#pragma unroll
    for (int k = 0; k < ITERS; ++k) {
      const float t0 = __uint_as_float(tp[k].x << 16), t1 = __uint_as_float(tp[k].x & 0xFFFF0000u);
      const float t3 = __uint_as_float(tp[k].y & 0xFFFF0000u), t2f = __uint_as_float(tp[k].y << 16);
      const float g0 = (expf(z[k].x) * inv_se * tsum - t0) * a.inv_batch, g1 = (expf(z[k].y) * inv_se * tsum - t1) * a.inv_batch;
      const float g2 = (expf(z[k].z) * inv_se * tsum - t2f) * a.inv_batch, g3 = (expf(z[k].w) * inv_se * tsum - t3) * a.inv_batch;
      __nv_bfloat162 lo = __floats2bfloat162_rn(g0, g1), hi = __floats2bfloat162_rn(g2, g3);
      uint2 o;
      o.x = *reinterpret_cast<uint32_t*>(&lo); o.y = *reinterpret_cast<uint32_t*>(&hi);
      d2[lane + 32 * k] = o;
    }
  }
  if (lane == 0) a.row_loss[(long long)m * a.rows + row] = loss;
}

static bool launch_ce_soft_vec(const LossArgs& a, cudaStream_t s) {
  if (a.kind != PBT_LOSS_CE_SOFT || a.target_dtype != kBF16 || a.cols % 128 != 0 || a.cols > 1024 || a.cols < 128) return false;
  if (a.dz && (a.dz_dtype != kBF16 || a.ld_dz % 4 != 0 || a.stride_dz % 4 != 0 || ((uintptr_t)a.dz & 7))) return false;
  if (a.ld_logits % 4 != 0 || a.stride_logits % 4 != 0 || ((uintptr_t)a.logits & 15)) return false;
  if (a.stride_target % 4 != 0 || ((uintptr_t)a.target & 7)) return false;
  dim3 grid((a.rows + 7) / 8, a.n_members);
  switch (a.cols / 128) {
    case 1: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<1>, a); break;
    case 2: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<2>, a); break;
    case 3: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<3>, a); break;
    case 4: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<4>, a); break;
    case 5: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<5>, a); break;
    case 6: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<6>, a); break;
    case 7: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<7>, a); break;
    default: launch_with(grid, 256, 0, s)(k_loss_ce_soft_vec<8>, a); break;
  }
  return true;
}

cudaError_t launch_loss_rows(const LossArgs& a, cudaStream_t s) {
  if (launch_ce_soft_vec(a, s)) return cudaGetLastError();
  const int warps = 8;
  dim3 grid((a.rows + warps - 1) / warps, a.n_members);
  launch_with(grid, warps * 32, 0, s)(k_loss_rows, a);
  return cudaGetLastError();
}

// block-wide sum in a fixed order: thread t adds elements t, t+256, ...; then a tree over shared memory
template <typename T>
__device__ __forceinline__ T block_sum_256(T v, T* sh) {
  sh[threadIdx.x] = v;
  __syncthreads();
#pragma unroll
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  const T r = sh[0];
  __syncthreads();
  return r;
}

__global__ void k_reduce_rows(const float* __restrict__ row_loss, int rows, float scale, void* out,
                              int out_is_double, int out_stride) {
  pdl_prologue();
  __shared__ double sh[256];
  const int m = blockIdx.x;
  double acc = 0.0;
  for (int r = threadIdx.x; r < rows; r += 256) acc += (double)row_loss[(long long)m * rows + r];
  const double total = block_sum_256<double>(acc, sh);
  if (threadIdx.x == 0) {
    const float v = (float)total * scale;
    if (out_is_double) reinterpret_cast<double*>(out)[(long long)m * out_stride] = (double)v;
    else reinterpret_cast<float*>(out)[(long long)m * out_stride] = v;
  }
}

cudaError_t launch_reduce_rows(const float* row_loss, int rows, int n_members, float scale, void* out,
                               int out_is_double, int out_stride, cudaStream_t s) {
  launch_with(n_members, 256, 0, s)(k_reduce_rows, row_loss, rows, scale, out, out_is_double, out_stride);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Bias gradient: column sums of dZ.  Block = 32 columns x 8 row-lanes.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void k_bias_grad(const T* __restrict__ dz, long long ld, long long stride, int rows, int cols,
                            float* __restrict__ out, long long out_stride) {
  pdl_prologue();
  __shared__ float sh[8][33];
  const int m = blockIdx.y;
  const int c = blockIdx.x * 32 + threadIdx.x;
  float acc = 0.f;
  if (c < cols) {
    const T* p = dz + m * stride + c;
    for (int r = threadIdx.y; r < rows; r += 8) {
      if constexpr (sizeof(T) == 2) acc += __bfloat162float(p[(long long)r * ld]);
      else acc += p[(long long)r * ld];
    }
  }
  sh[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.y == 0 && c < cols) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) t += sh[j][threadIdx.x];
    out[m * out_stride + c] = t;
  }
}

// bf16 deltas with 16-byte alignment: a lane reads 8 columns per row, a warp 512 contiguous bytes; warp w adds rows
// w, w + 8, ... and the eight partial sums are combined in order, exactly like the scalar kernel above (same bits).
__global__ void __launch_bounds__(256) k_bias_grad_bf16x8(const bf16* __restrict__ dz, long long ld, long long stride, int rows,
                                                          int cols, float* __restrict__ out, long long out_stride) {
  pdl_prologue();
  __shared__ float sh[8][256 + 8];
  const int m = blockIdx.y, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c0 = blockIdx.x * 256 + lane * 8;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c0 < cols) {
    const bf16* p = dz + m * stride + c0;
#pragma unroll 4
    for (int r = w; r < rows; r += 8) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + (long long)r * ld));
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[2 * j] += __uint_as_float(u[j] << 16);
        acc[2 * j + 1] += __uint_as_float(u[j] & 0xFFFF0000u);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) sh[w][lane * 8 + j] = acc[j];
  __syncthreads();
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c < cols) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) t += sh[j][threadIdx.x];
    out[m * out_stride + c] = t;
  }
}

// The same sums for populations whose layers are too narrow to fill the GPU with one block per 256 columns: a block
// owns 64 columns, 8 threads x 16 bytes across and 32 row lanes down (a warp reads 4 rows x 128 contiguous bytes),
// every thread keeps 8 loads in flight, and the 32 partial sums of a column are combined in a fixed order.
__global__ void __launch_bounds__(256) k_bias_grad_bf16x8_tall(const bf16* __restrict__ dz, long long ld, long long stride,
                                                               int rows, int cols, float* __restrict__ out,
                                                               long long out_stride) {
  pdl_prologue();
  __shared__ float sh[32][64 + 1];
  const int m = blockIdx.y, cl = threadIdx.x & 7, rl = threadIdx.x >> 3;
  const int c0 = blockIdx.x * 64 + cl * 8;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c0 < cols) {
    const bf16* p = dz + m * stride + c0;
#pragma unroll 8
    for (int r = rl; r < rows; r += 32) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + (long long)r * ld));
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[2 * j] += __uint_as_float(u[j] << 16);
        acc[2 * j + 1] += __uint_as_float(u[j] & 0xFFFF0000u);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) sh[rl][cl * 8 + j] = acc[j];
  __syncthreads();
  const int c = blockIdx.x * 64 + threadIdx.x;
  if (threadIdx.x < 64 && c < cols) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) t += sh[j][threadIdx.x];
    out[m * out_stride + c] = t;
  }
}

// Column sums of a narrow matrix (one-, two- or ten-wide output layers): one block per member, thread t adds rows
// t, t + 256, ..., then the 256 partial sums of a column are combined in a fixed order (warp shuffles, then warps).
template <typename T>
__global__ void __launch_bounds__(256) k_bias_grad_narrow(const T* __restrict__ dz, long long ld, long long stride, int rows,
                                                          int cols, float* __restrict__ out, long long out_stride) {
  pdl_prologue();
  __shared__ float sh[8][16];
  const int m = blockIdx.x, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const T* p = dz + m * stride;
  float acc[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) acc[c] = 0.f;
  for (int r = threadIdx.x; r < rows; r += 256) {
#pragma unroll
    for (int c = 0; c < 16; ++c)
      if (c < cols) {
        if constexpr (sizeof(T) == 2) acc[c] += __bfloat162float(p[(long long)r * ld + c]);
        else acc[c] += p[(long long)r * ld + c];
      }
  }
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    if (c < cols) {
      float v = acc[c];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) sh[w][c] = v;
    }
  }
  __syncthreads();
  if (threadIdx.x < cols) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) t += sh[j][threadIdx.x];
    out[m * out_stride + threadIdx.x] = t;
  }
}

cudaError_t launch_bias_grad(const void* dz, int dz_dtype, long long ld, long long stride, int rows, int cols,
                             float* out, long long out_stride, int n_members, cudaStream_t s) {
  // the wide kernel has one block per 256 columns and member: only when that fills the GPU twice over
  if (dz_dtype == kBF16 && cols % 8 == 0 && (long long)((cols + 255) / 256) * n_members >= 296 && ld % 8 == 0 &&
      stride % 8 == 0 && ((uintptr_t)dz & 15) == 0) {
    dim3 grid((cols + 255) / 256, n_members);
    launch_with(grid, 256, 0, s)(k_bias_grad_bf16x8, (const bf16*)dz, ld, stride, rows, cols, out, out_stride);
    return cudaGetLastError();
  }
  if (dz_dtype == kBF16 && cols % 8 == 0 && cols >= 64 && rows >= 64 && ld % 8 == 0 && stride % 8 == 0 &&
      ((uintptr_t)dz & 15) == 0) {
    dim3 grid((cols + 63) / 64, n_members);
    launch_with(grid, 256, 0, s)(k_bias_grad_bf16x8_tall, (const bf16*)dz, ld, stride, rows, cols, out, out_stride);
    return cudaGetLastError();
  }
  if (cols <= 16 && rows >= 256) {
    if (dz_dtype == kBF16)
      launch_with(n_members, 256, 0, s)(k_bias_grad_narrow<bf16>, (const bf16*)dz, ld, stride, rows, cols, out, out_stride);
    else
      launch_with(n_members, 256, 0, s)(k_bias_grad_narrow<float>, (const float*)dz, ld, stride, rows, cols, out, out_stride);
    return cudaGetLastError();
  }
  dim3 grid((cols + 31) / 32, n_members), block(32, 8);
  if (dz_dtype == kBF16)
    launch_with(grid, block, 0, s)(k_bias_grad<bf16>, (const bf16*)dz, ld, stride, rows, cols, out, out_stride);
  else
    launch_with(grid, block, 0, s)(k_bias_grad<float>, (const float*)dz, ld, stride, rows, cols, out, out_stride);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Toy model (Figure 2): ascend 1.2 - sum_i h_i theta_i^2; evaluate 1.2 - sum_i theta_i^2.
// Explicitly rounded operations (no fused multiply-add) so the CPU reproduces every bit.
// ---------------------------------------------------------------------------
__global__ void k_toy_step(double* theta, const double* __restrict__ H, int n_members, int dim, double eta) {
  pdl_prologue();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_members * dim) return;
  const int m = i / dim, k = i % dim;
  const double h = H[m * PBT_MAX_NH + k];
  const double g = __dmul_rn(__dmul_rn(-2.0, h), theta[i]);
  theta[i] = __dadd_rn(theta[i], __dmul_rn(eta, g));
}

__global__ void k_toy_eval(const double* __restrict__ theta, double* fitness, int n_members, int dim) {
  pdl_prologue();
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= n_members) return;
  double s = 0.0;
  for (int k = 0; k < dim; ++k) s = __dadd_rn(s, __dmul_rn(theta[m * dim + k], theta[m * dim + k]));
  fitness[m] = __dsub_rn(1.2, s);
}

cudaError_t launch_toy_step(double* theta, const double* H, int n_members, int dim, double eta, cudaStream_t s) {
  const int n = n_members * dim;
  launch_with((n + 127) / 128, 128, 0, s)(k_toy_step, theta, H, n_members, dim, eta);
  return cudaGetLastError();
}
cudaError_t launch_toy_eval(const double* theta, double* fitness, int n_members, int dim, cudaStream_t s) {
  launch_with((n_members + 127) / 128, 128, 0, s)(k_toy_eval, theta, fitness, n_members, dim);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Energy distance of n generated 2-D points to the eight-mode unit ring.
// Block b of member m handles points i in [b*256, b*256+256) against all j.
// ---------------------------------------------------------------------------
constexpr int kEdBlock = 256;
int energy_partial_count(int n) { return 2 * ((n + kEdBlock - 1) / kEdBlock); }

__global__ void k_energy_partial(const float* __restrict__ x, long long stride, int n, double* __restrict__ partial) {
  pdl_prologue();
  __shared__ float2 tile[kEdBlock];
  __shared__ double sh[256];
  const int m = blockIdx.y;
  const float2* xm = reinterpret_cast<const float2*>(x + m * stride);
  const int i = blockIdx.x * kEdBlock + threadIdx.x;
  const bool valid = i < n;
  const float2 xi = valid ? xm[i] : make_float2(0.f, 0.f);
  double within = 0.0;
  for (int j0 = 0; j0 < n; j0 += kEdBlock) {
    const int j = j0 + threadIdx.x;
    tile[threadIdx.x] = j < n ? xm[j] : make_float2(0.f, 0.f);
    __syncthreads();
    const int cnt = min(kEdBlock, n - j0);
    float acc = 0.f;
    for (int t = 0; t < cnt; ++t) {
      const float dx = xi.x - tile[t].x, dy = xi.y - tile[t].y;
      acc += sqrtf(dx * dx + dy * dy);
    }
    within += (double)acc;
    __syncthreads();
  }
  double cross = 0.0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    double sn, cs;
    sincospi(k * 0.25, &sn, &cs);
    const double dx = (double)xi.x - cs, dy = (double)xi.y - sn;
    cross += sqrt(dx * dx + dy * dy);
  }
  if (!valid) { within = 0.0; cross = 0.0; }
  const double w = block_sum_256<double>(within, sh);
  const double c = block_sum_256<double>(cross, sh);
  if (threadIdx.x == 0) {
    partial[((long long)m * gridDim.x + blockIdx.x) * 2 + 0] = w;
    partial[((long long)m * gridDim.x + blockIdx.x) * 2 + 1] = c;
  }
}

__global__ void k_energy_final(const double* __restrict__ partial, int nblocks, int n, float* fitness) {
  pdl_prologue();
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= (int)gridDim.x * (int)blockDim.x) return;
  double within = 0.0, cross = 0.0;
  for (int b = 0; b < nblocks; ++b) {
    within += partial[((long long)m * nblocks + b) * 2 + 0];
    cross += partial[((long long)m * nblocks + b) * 2 + 1];
  }
  double modes = 0.0;
  for (int a = 0; a < 8; ++a)
    for (int b = 0; b < 8; ++b) {
      double sa, ca, sb, cb;
      sincospi(a * 0.25, &sa, &ca);
      sincospi(b * 0.25, &sb, &cb);
      modes += sqrt((ca - cb) * (ca - cb) + (sa - sb) * (sa - sb));
    }
  const double e = 2.0 * cross / ((double)n * 8.0) - within / ((double)n * (double)n) - modes / 64.0;
  fitness[m] = (float)(-e);
}

cudaError_t launch_energy_distance(const float* x, long long stride, int n, int n_members, double* partial,
                                   float* fitness, cudaStream_t s) {
  const int nblocks = (n + kEdBlock - 1) / kEdBlock;
  dim3 grid(nblocks, n_members);
  launch_with(grid, kEdBlock, 0, s)(k_energy_partial, x, stride, n, partial);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  launch_with(n_members, 1, 0, s)(k_energy_final, partial, nblocks, n, fitness);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// WGAN-GP (Section 4.3.1): interpolates between real and generated rows, and the
// penalty on the norm of the critic's input gradient with its derivative.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void k_gp_interp(T* __restrict__ x, long long stride, int B, int dim, int j, uint64_t seed, StepClock clk) {
  pdl_prologue();
  const int m = blockIdx.y;
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const U4 r = philox4x32_10((uint32_t)(clk.member_base + m), (uint32_t)clk.t[m], kStreamInterp,
                             (uint32_t)(j * 65536 + (b >> 2)), seed);
  // (w >> 9) + 1/2 has 24 significant bits, and so has its complement: both are exact in float
  const float e = ((float)(r.x[b & 3] >> 9) + 0.5f) * 1.1920928955078125e-07f;
  const float ome = 1.0f - e;
  T* xm = x + m * stride;
  for (int c = 0; c < dim; ++c) {
    float re, fa;
    if constexpr (sizeof(T) == 2) {
      re = __bfloat162float(xm[(long long)b * dim + c]);
      fa = __bfloat162float(xm[(long long)(B + b) * dim + c]);
      xm[(long long)(2 * B + b) * dim + c] = __float2bfloat16_rn(fmaf(e, re, ome * fa));
    } else {
      re = xm[(long long)b * dim + c];
      fa = xm[(long long)(B + b) * dim + c];
      xm[(long long)(2 * B + b) * dim + c] = fmaf(e, re, ome * fa);
    }
  }
}

cudaError_t launch_gp_interp(void* x, int dtype, long long stride, int B, int dim, int j, int n_members, uint64_t seed,
                             StepClock clk, cudaStream_t s) {
  dim3 grid((B + 127) / 128, n_members);
  if (dtype == kBF16) launch_with(grid, 128, 0, s)(k_gp_interp<bf16>, (bf16*)x, stride, B, dim, j, seed, clk);
  else launch_with(grid, 128, 0, s)(k_gp_interp<float>, (float*)x, stride, B, dim, j, seed, clk);
  return cudaGetLastError();
}

// one warp per (member, row)
__global__ void k_gp_penalty(const float* __restrict__ gx, long long gx_stride, int B, int dim, float lam,
                             float inv_batch, float* __restrict__ row_loss, int rows_total, int row_off, void* dv,
                             int dv_dtype, long long dv_stride) {
  pdl_prologue();
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.y;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= B) return;
  const float* g = gx + m * gx_stride + (long long)b * dim;
  float ss = 0.f;
  for (int c = lane; c < dim; c += 32) ss = fmaf(g[c], g[c], ss);
  ss = warp_sum(ss);
  const float nrm = sqrtf(ss);
  const float dev = nrm - 1.0f;
  if (lane == 0) row_loss[(long long)m * rows_total + row_off + b] = lam * dev * dev;
  const float scale = nrm > 0.f ? (2.0f * lam * inv_batch) * dev / nrm : 0.f;
  for (int c = lane; c < dim; c += 32) store_from_float(dv, dv_dtype, m * dv_stride + (long long)b * dim + c, scale * g[c]);
}

cudaError_t launch_gp_penalty(const float* gx, long long gx_stride, int B, int dim, float lam, float inv_batch,
                              float* row_loss, int rows_total, int row_off, void* dv, int dv_dtype,
                              long long dv_stride, int n_members, cudaStream_t s) {
  const int warps = 8;
  dim3 grid((B + warps - 1) / warps, n_members);
  launch_with(grid, warps * 32, 0, s)(k_gp_penalty, gx, gx_stride, B, dim, lam, inv_batch, row_loss, rows_total, row_off, dv,
                                           dv_dtype, dv_stride);
  return cudaGetLastError();
}

// every member of the window has taken one more step (Algorithm 1's t, counted per member)
__global__ void k_advance_step(Counters* c, long long* __restrict__ t, int n_members) {
  pdl_prologue();
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m < n_members) t[m] += 1;
  if (m == 0) c->use_supplied_batch = 0;
}
cudaError_t launch_advance_step(Counters* c, long long* t, int n_members, cudaStream_t s) {
  launch_with((n_members + 127) / 128, 128, 0, s)(k_advance_step, c, t, n_members);
  return cudaGetLastError();
}

}  // namespace pbt
