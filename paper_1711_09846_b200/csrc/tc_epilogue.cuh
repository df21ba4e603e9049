// Epilogue shared by the tensor-core GEMM kernels: one warp drains its 32-row quadrant of a 128 x BN fp32
// accumulator tile from tensor memory in 32-column chunks, transposes each chunk through padded shared memory
// and writes whole 128-byte lines with bias / ReLU / ReLU-mask / bf16 conversion fused.
#pragma once
#include "tc_common.cuh"

namespace pbt {
namespace tc {

constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kEpiPitch = 36;  // floats per row of the epilogue transpose buffer (16-byte aligned, conflict-free)

struct TcParams {
  int M, N, K, batch;
  int tiles_m, tiles_n, num_tiles, k_blocks;
  int a_mn, b_mn, a_batched, b_batched;
  void* C; long long ldc, strideC; int out_dtype;
  const float* bias; long long strideBias; int relu;
  const bf16* mask; long long ldmask, strideMask;
  int c_tma;             // the kernel was given a tensor map of C: interior tiles leave through bulk tensor stores
  Counters* counters;
  const int* a_rowoff;   // per-problem first row of the A / B operand inside a shared matrix (null: batched operand)
  const int* b_rowoff;
};


// tacc: TMEM address of (this warp's lane quadrant, first column of the accumulator); rows of the tile start at m0.
template <int BN, int NEPIW>
__device__ __forceinline__ void epilogue_tile(const TcParams& p, float* buf, uint32_t tacc, int member, int m0, int n0,
                                              int q, int half, int lane, bool vec_ok) {
  const int rsub = lane >> 3, cc = (lane & 7) * 4;   // phase 2: 4 rows x 8 column-quads per warp instruction
  const float* bias = p.bias ? p.bias + member * p.strideBias : nullptr;
  // The accumulator chunk for iteration c+1 is requested from tensor memory while chunk c is being
  // transposed and written out, and the ReLU-mask words are requested before the transpose, so that
  // neither latency sits on the warp's critical path.
  constexpr int kChunkStep = 32 * (NEPIW / 4);
  uint32_t r[32];
  // Interior tiles with bf16 output (the bulk of the forward and data-gradient GEMMs) take a path with no bounds
  // checks, pointers advanced by constant steps and the ReLU mask applied to the packed bf16 pairs: the epilogue
  // warps are bound by instruction issue, two warps per scheduler, so the instruction count per element is what
  // decides whether the epilogue hides behind a short main loop.
  if (vec_ok && p.out_dtype != kBF16 && !p.mask && m0 + kBM <= p.M && n0 + BN <= p.N) {
    // the same for fp32 output without a mask (logits, stored weight gradients)
    float* crow = reinterpret_cast<float*>(p.C) + member * p.strideC + (long long)(m0 + q * 32 + rsub) * p.ldc + n0 + cc;
    const long long cstep = 4 * p.ldc;
    tmem_ld32(tacc + half * 32, r);
#pragma unroll 1
    for (int c0 = half * 32; c0 < BN; c0 += kChunkStep) {
      tmem_ld_wait();
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<uint4*>(&buf[lane * kEpiPitch + j * 4]) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      if (c0 + kChunkStep < BN) tmem_ld32(tacc + c0 + kChunkStep, r);
      __syncwarp();
      float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bias) bv = __ldg(reinterpret_cast<const float4*>(bias + n0 + c0 + cc));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 a4 = *reinterpret_cast<const float4*>(&buf[(i * 4 + rsub) * kEpiPitch + cc]);
        if (bias) { a4.x += bv.x; a4.y += bv.y; a4.z += bv.z; a4.w += bv.w; }
        if (p.relu) { a4.x = fmaxf(a4.x, 0.f); a4.y = fmaxf(a4.y, 0.f); a4.z = fmaxf(a4.z, 0.f); a4.w = fmaxf(a4.w, 0.f); }
        *reinterpret_cast<float4*>(crow + c0 + i * cstep) = a4;
      }
    }
    return;
  }
  if (vec_ok && p.out_dtype == kBF16 && m0 + kBM <= p.M && n0 + BN <= p.N) {
    const long long row0 = m0 + q * 32 + rsub;
    bf16* crow = reinterpret_cast<bf16*>(p.C) + member * p.strideC + row0 * p.ldc + n0 + cc;
    const bf16* mrow = p.mask ? p.mask + member * p.strideMask + row0 * p.ldmask + n0 + cc : nullptr;
    const long long cstep = 4 * p.ldc, mstep = 4 * p.ldmask;
    const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
    tmem_ld32(tacc + half * 32, r);
#pragma unroll 1
    for (int c0 = half * 32; c0 < BN; c0 += kChunkStep) {
      uint2 mk[8];
      if (mrow) {
#pragma unroll
        for (int i = 0; i < 8; ++i) mk[i] = __ldg(reinterpret_cast<const uint2*>(mrow + c0 + i * mstep));
      }
      tmem_ld_wait();
      __syncwarp();  // the previous chunk's phase-2 reads of `buf` are complete
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<uint4*>(&buf[lane * kEpiPitch + j * 4]) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      if (c0 + kChunkStep < BN) tmem_ld32(tacc + c0 + kChunkStep, r);
      __syncwarp();
      float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bias) bv = __ldg(reinterpret_cast<const float4*>(bias + n0 + c0 + cc));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 a4 = *reinterpret_cast<const float4*>(&buf[(i * 4 + rsub) * kEpiPitch + cc]);
        if (bias) { a4.x += bv.x; a4.y += bv.y; a4.z += bv.z; a4.w += bv.w; }
        if (p.relu) { a4.x = fmaxf(a4.x, 0.f); a4.y = fmaxf(a4.y, 0.f); a4.z = fmaxf(a4.z, 0.f); a4.w = fmaxf(a4.w, 0.f); }
        __nv_bfloat162 t0 = __floats2bfloat162_rn(a4.x, a4.y);
        __nv_bfloat162 t1 = __floats2bfloat162_rn(a4.z, a4.w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t*>(&t0); o.y = *reinterpret_cast<uint32_t*>(&t1);
        if (mrow) {
          // keep an element where its mask value is > 0 (all-ones half-word), clear it otherwise (zero, negative, NaN)
          o.x &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[i].x), zero2);
          o.y &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[i].y), zero2);
        }
        *reinterpret_cast<uint2*>(crow + c0 + i * cstep) = o;
      }
    }
    return;
  }
  if (n0 + half * 32 < p.N) tmem_ld32(tacc + half * 32, r);
#pragma unroll 1
  for (int c0 = half * 32; c0 < BN; c0 += kChunkStep) {
    const int nbase = n0 + c0;
    if (nbase >= p.N) break;  // uniform across the warp
    const int col = nbase + cc;
    const bool full4 = vec_ok && col + 3 < p.N;
    uint2 mk[8];
    if (p.mask && full4) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int row = m0 + q * 32 + i * 4 + rsub;
        mk[i] = row < p.M ? __ldg(reinterpret_cast<const uint2*>(p.mask + member * p.strideMask + (long long)row * p.ldmask + col))
                          : make_uint2(0u, 0u);
      }
    }
    tmem_ld_wait();
    __syncwarp();  // the previous chunk's phase-2 reads of `buf` are complete
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<uint4*>(&buf[lane * kEpiPitch + j * 4]) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
    if (c0 + kChunkStep < BN && nbase + kChunkStep < p.N) tmem_ld32(tacc + c0 + kChunkStep, r);
    __syncwarp();
    {
      float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bias && col < p.N) {
        if (full4) bv = __ldg(reinterpret_cast<const float4*>(bias + col));
        else {
          bv.x = bias[col];
          if (col + 1 < p.N) bv.y = bias[col + 1];
          if (col + 2 < p.N) bv.z = bias[col + 2];
          if (col + 3 < p.N) bv.w = bias[col + 3];
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = i * 4 + rsub;
        const int row = m0 + q * 32 + rr;
        if (row >= p.M || col >= p.N) continue;
        const float4 a4 = *reinterpret_cast<const float4*>(&buf[rr * kEpiPitch + cc]);
        float v[4] = {a4.x + bv.x, a4.y + bv.y, a4.z + bv.z, a4.w + bv.w};
        if (p.relu) {
#pragma unroll
          for (int j = 0; j < 4; ++j) v[j] = fmaxf(v[j], 0.f);
        }
        if (p.mask) {
          const bf16* mp = p.mask + member * p.strideMask + (long long)row * p.ldmask + col;
          if (full4) {
            const uint32_t w[2] = {mk[i].x, mk[i].y};
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              // bf16 > 0  <=>  sign bit clear and magnitude non-zero
              const uint32_t lo = w[h2] & 0xFFFFu, hi = w[h2] >> 16;
              if (!(lo != 0 && lo < 0x8000u)) v[h2 * 2] = 0.f;
              if (!(hi != 0 && hi < 0x8000u)) v[h2 * 2 + 1] = 0.f;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (col + j < p.N && !(__bfloat162float(mp[j]) > 0.f)) v[j] = 0.f;
          }
        }
        const long long ci = member * p.strideC + (long long)row * p.ldc + col;
        if (p.out_dtype == kBF16) {
          bf16* cp = reinterpret_cast<bf16*>(p.C) + ci;
          if (full4) {
            __nv_bfloat162 t0 = __floats2bfloat162_rn(v[0], v[1]);
            __nv_bfloat162 t1 = __floats2bfloat162_rn(v[2], v[3]);
            uint2 o;
            o.x = *reinterpret_cast<uint32_t*>(&t0); o.y = *reinterpret_cast<uint32_t*>(&t1);
            *reinterpret_cast<uint2*>(cp) = o;
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) if (col + j < p.N) cp[j] = __float2bfloat16_rn(v[j]);
          }
        } else {
          float* cp = reinterpret_cast<float*>(p.C) + ci;
          if (full4) *reinterpret_cast<float4*>(cp) = make_float4(v[0], v[1], v[2], v[3]);
          else {
#pragma unroll
            for (int j = 0; j < 4; ++j) if (col + j < p.N) cp[j] = v[j];
          }
        }
      }
    }
}
}

// Interior tiles when a tensor map of C is available.  A thread's TMEM lane is a row of the tile, so after
// tcgen05.ld a thread holds 32 consecutive columns of ITS row: bias / ReLU / conversion / mask are applied in
// registers and the row segment goes, with the 128-byte swizzle of the tensor map (16-byte chunk index XOR row & 7,
// which also makes the warp's 16-byte shared-memory stores conflict-free), into a staging box of 32 rows x 128 bytes;
// one lane then issues a bulk tensor store of the box.  No transpose through shared memory and no per-thread global
// stores.  `stage` is this warp's 8 KB (two boxes, 1024-byte aligned): a box is rewritten only after the store that
// read it two boxes ago has finished reading.  bf16 output: a box is 64 columns (two 32-column chunks); fp32: 32.
// The accumulator is handed back to the MMA warp (one arrival per warp on the barrier at the shared::cluster
// address `handback`) as soon as its last chunk has left tensor memory, before that chunk is stored: when the
// contraction is short (K = 512 with fp32 output: the tile drains for longer than it is computed) the hand-back at
// the end of the tile was what the next-but-one tile waited for, and moving it gained 6 %.
__device__ __forceinline__ void release_accumulator(uint32_t handback, int lane) {
  tc_fence_before();
  __syncwarp();
  if (lane == 0) asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(handback) : "memory");
}
template <int BN, int NEPIW>
__device__ __forceinline__ void epilogue_tile_tma(const TcParams& p, const CUtensorMap* tmC, uint8_t* stage, uint32_t tacc,
                                                  int member, int m0, int n0, int q, int half, int lane,
                                                  uint32_t handback, uint32_t& boxes_used) {
  constexpr int kCols = BN / (NEPIW / 4);   // columns of the tile this warp drains
  constexpr int kChunks = kCols / 32;
  const int cbase = half * kCols;
  const float* bias = p.bias ? p.bias + member * p.strideBias + n0 + cbase : nullptr;
  const long long row = m0 + q * 32 + lane;
  const uint32_t sw = (uint32_t)(lane & 7);
  uint32_t r[32];
  tmem_ld32(tacc + cbase, r);
  if (p.out_dtype == kBF16) {
    const bf16* mrow = p.mask ? p.mask + member * p.strideMask + row * p.ldmask + n0 + cbase : nullptr;
    const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll 1
    for (int c = 0; c < kChunks; ++c) {
      uint4 mk[4];
      if (mrow) {
#pragma unroll
        for (int j = 0; j < 4; ++j) mk[j] = __ldg(reinterpret_cast<const uint4*>(mrow + c * 32) + j);
      }
      uint8_t* box = stage + (boxes_used & 1u) * 4096u;
      if ((c & 1) == 0) {
        if (lane == 0) tma_store_wait_read_but_one();
        __syncwarp();
      }
      tmem_ld_wait();
      uint32_t o[16];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float x0 = __uint_as_float(r[4 * j]), x1 = __uint_as_float(r[4 * j + 1]);
        float x2 = __uint_as_float(r[4 * j + 2]), x3 = __uint_as_float(r[4 * j + 3]);
        if (bias) {
          const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + c * 32) + j);   // same address in every lane
          x0 += bv.x; x1 += bv.y; x2 += bv.z; x3 += bv.w;
        }
        if (p.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); x2 = fmaxf(x2, 0.f); x3 = fmaxf(x3, 0.f); }
        __nv_bfloat162 t0 = __floats2bfloat162_rn(x0, x1), t1 = __floats2bfloat162_rn(x2, x3);
        o[2 * j] = *reinterpret_cast<uint32_t*>(&t0);
        o[2 * j + 1] = *reinterpret_cast<uint32_t*>(&t1);
      }
      if (c + 1 < kChunks) tmem_ld32(tacc + cbase + (c + 1) * 32, r);
      else release_accumulator(handback, lane);
      if (mrow) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          o[4 * j] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[j].x), zero2);
          o[4 * j + 1] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[j].y), zero2);
          o[4 * j + 2] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[j].z), zero2);
          o[4 * j + 3] &= __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&mk[j].w), zero2);
        }
      }
      const uint32_t hh = (uint32_t)(c & 1) * 4u;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<uint4*>(box + lane * 128 + (((hh + j) ^ sw) << 4)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
      if (c & 1) {
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_3d(tmC, box, n0 + cbase + (c - 1) * 32, m0 + q * 32, member);
          tma_store_commit();
        }
        ++boxes_used;
      }
    }
  } else {
#pragma unroll 1
    for (int c = 0; c < kChunks; ++c) {
      uint8_t* box = stage + (boxes_used & 1u) * 4096u;
      if (lane == 0) tma_store_wait_read_but_one();
      __syncwarp();
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                               __uint_as_float(r[4 * j + 3]));
        if (bias) {
          const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + c * 32) + j);
          v.x += bv.x; v.y += bv.y; v.z += bv.z; v.w += bv.w;
        }
        if (p.relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
        *reinterpret_cast<float4*>(box + lane * 128 + ((((uint32_t)j) ^ sw) << 4)) = v;
      }
      if (c + 1 < kChunks) tmem_ld32(tacc + cbase + (c + 1) * 32, r);
      else release_accumulator(handback, lane);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_3d(tmC, box, n0 + cbase + c * 32, m0 + q * 32, member);
        tma_store_commit();
      }
      ++boxes_used;
    }
  }
}

}  // namespace tc
}  // namespace pbt
