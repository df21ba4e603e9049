// Weight gradient and Adam update in one kernel (bf16 populations, sm_100a):
//   g[o][i]   = sum_b dZ[b][o] * a[b][i]            (tcgen05.mma, both operands MN-major, fp32 in TMEM)
//   theta[o][i], m, v  <- Adam(theta, m, v, g | the member's lr, beta1, weight decay)   (Eq. 2's update)
// The gradient goes from tensor memory straight into the update: it is never written to HBM (unless the
// caller asks for a copy), which removes 8 of the 34 bytes per parameter that a separate optimiser pass moves.
//
// The tile is computed TRANSPOSED, D[i][o] (128 inputs i x 256 outputs o, layer input as the A operand): a
// tensor-memory lane is then an index i, which is the contiguous direction of W[out][in] in memory, so that a
// warp's 32 lanes hold 32 consecutive floats of one weight row and a 32-column chunk of the accumulator is a box
// of 32 weight rows x 512 contiguous bytes.  (With lanes = weight rows the same chunk was 128 rows x 128 bytes;
// 128-byte pieces 8 KB apart cost about a tenth of the HBM bandwidth against 512-byte runs.)
//
// The update is HBM-bound (12 bytes in, 14 bytes out per parameter), so the kernel is organised around keeping
// ~100 KB of that traffic in flight per SM without holding it in registers:
//   warp 0       TMA producer for the GEMM operands (2-stage ring, the contraction over the batch is short)
//   warp 1       tensor-memory allocation + tcgen05.mma issue (128 x 256 tile, accumulator double-buffered)
//   warp 2       TMA loader for the optimiser state: per 32-column chunk of the tile one box of 32 weight rows x
//                128 floats each of master weights, first and second moment into a ring of two slots (row-major,
//                no swizzle: a warp reads and writes 128 consecutive bytes of a box row)
//   warp 3       TMA storer: when the sixteen update warps are done with a slot, stores the three boxes back in
//                place plus the bf16 shadow box, and hands the slot back to the loader once it has been read
//   warps 4..19  update: tcgen05.ld of 8 gradient columns (weight rows) of the thread's lane, Adam on the slot
// All mbarrier waits are bounded; on expiry PBT_ERR_TIMEOUT is recorded and every role leaves its loop.
#include <string.h>

#include "tc_common.cuh"

namespace pbt {

namespace {

using namespace tc;

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 2, kSlots = 2, kChunk = 32, kUpdWarps = 16;
constexpr int kColsPerWarp = kChunk / (kUpdWarps / 4);   // gradient columns one update thread handles per chunk
static_assert(kColsPerWarp == 4 || kColsPerWarp == 8 || kColsPerWarp == 16, "update warps per TMEM lane quadrant");
constexpr int kThreads = 32 * (4 + kUpdWarps);
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2, kStageBytes = kABytes + kBBytes;
constexpr int kBoxBytes = kBM * kChunk * 4;     // one fp32 state box
constexpr int kSlotBytes = 3 * kBoxBytes;       // master, m, v
constexpr int kW16Bytes = kBM * kChunk * 2;     // bf16 shadow box
constexpr int kSlotOffset = kStages * kStageBytes;
constexpr int kW16Offset = kSlotOffset + kSlots * kSlotBytes;
constexpr int kBarOffset = kW16Offset + kSlots * kW16Bytes;
constexpr int kSmemTotal = kBarOffset + 256 + 1024;
static_assert(kSmemTotal <= 232448, "shared memory budget of one CTA");

struct FusedParams {
  int M, N, K, batch;   // of the transposed product: M = layer inputs (tile rows / lanes), N = layer outputs
  int tiles_m, tiles_n, num_tiles, k_blocks;
  float* gout; long long ldc, strideC;  // optional copy of the gradient (may be null)
  Counters* counters;
  const int* in_rowoff;   // layer input taken from a shared pool: first batch row of each member (null: per-member buffer)
  OptArgs opt;
};

__device__ __forceinline__ void give_up(const FusedParams& p, volatile int* abort_flag, int site) {
  *abort_flag = 1;
  atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
  p.counters->status_info = site;
}

__global__ void __launch_bounds__(kThreads, 1)
k_wgrad_adam(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmM,
             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW16, const FusedParams p) {
  pdl_prologue();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kBarOffset);
  uint64_t* empty = full + kStages;
  uint64_t* tfull = empty + kStages;    // [2] accumulator ready
  uint64_t* tempty = tfull + 2;         // [2] accumulator drained
  uint64_t* sfull = tempty + 2;         // [kSlots] optimiser state landed
  uint64_t* sdone = sfull + kSlots;     // [kSlots] all update warps finished with the slot
  uint64_t* sempty = sdone + kSlots;    // [kSlots] slot stored and free again
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sempty + kSlots);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kTmemCols = 2 * kBN;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], kUpdWarps); }
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sfull[s], 1); mbar_init(&sdone[s], kUpdWarps); mbar_init(&sempty[s], 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int tiles_per_member = p.tiles_m * p.tiles_n;
  constexpr int kChunks = kBN / kChunk;

  if (warp == 0) {
    // ------------------------------ operand producer ------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
        const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * kBN;
        const int ra = p.in_rowoff ? p.in_rowoff[member] : 0, ca = p.in_rowoff ? 0 : member;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * kStageBytes;
          uint8_t* sb = sa + kABytes;
          mbar_expect_tx(&full[stage], kStageBytes);
#pragma unroll
          for (int j = 0; j < kBM / 64; ++j) tma_load_3d(sa + j * 8192, &tmA, &full[stage], m0 + j * 64, kb * kBK + ra, ca);
#pragma unroll
          for (int j = 0; j < kBN / 64; ++j) tma_load_3d(sb + j * 8192, &tmB, &full[stage], n0 + j * 64, kb * kBK, member);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) give_up(p, abort_flag, 11);
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                             ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
      uint32_t stage = 0, phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        if (!mbar_wait(&tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * kBN;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * kStageBytes), sb = sa + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16(tmem_d, smem_desc(sa + k * 2048, 8192, 1024), smem_desc(sb + k * 2048, 8192, 1024), idesc,
                      (kb | k) != 0 ? 1u : 0u);
          umma_commit(&empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(&tfull[acc]);
      }
      if (!ok) give_up(p, abort_flag, 12);
    }
  } else if (warp == 2) {
    // ------------------------------ optimiser-state loader ------------------------------
    if (lane == 0) {
      uint32_t slot = 0, sphase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
        const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * kBN;
        for (int c = 0; c < kChunks; ++c) {
          const int col = n0 + c * kChunk;
          if (col >= p.N) break;
          if (!mbar_wait(&sempty[slot], sphase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* box = smem + kSlotOffset + slot * kSlotBytes;
          mbar_expect_tx(&sfull[slot], kSlotBytes);
          tma_load_3d(box, &tmW, &sfull[slot], m0, col, member);
          tma_load_3d(box + kBoxBytes, &tmM, &sfull[slot], m0, col, member);
          tma_load_3d(box + 2 * kBoxBytes, &tmV, &sfull[slot], m0, col, member);
          if (++slot == kSlots) { slot = 0; sphase ^= 1; }
        }
      }
      if (!ok) give_up(p, abort_flag, 13);
    }
  } else if (warp == 3) {
    // ------------------------------ storer ------------------------------
    if (lane == 0) {
      uint32_t slot = 0, sphase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
        const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * kBN;
        for (int c = 0; c < kChunks; ++c) {
          const int col = n0 + c * kChunk;
          if (col >= p.N) break;
          if (!mbar_wait(&sdone[slot], sphase, abort_flag)) { ok = false; break; }
          const uint8_t* box = smem + kSlotOffset + slot * kSlotBytes;
          tma_store_3d(&tmW, box, m0, col, member);
          tma_store_3d(&tmM, box + kBoxBytes, m0, col, member);
          tma_store_3d(&tmV, box + 2 * kBoxBytes, m0, col, member);
          tma_store_3d(&tmW16, smem + kW16Offset + slot * kW16Bytes, m0, col, member);
          tma_store_commit();
          tma_store_wait_read();           // shared memory of the slot may be overwritten now
          mbar_arrive(&sempty[slot]);
          if (++slot == kSlots) { slot = 0; sphase ^= 1; }
        }
      }
      tma_store_wait_all();
      if (!ok) give_up(p, abort_flag, 14);
    }
  } else {
    // ------------------------------ update warps ------------------------------
    const int q = warp & 3;               // TMEM lane quadrant this warp may access
    const int half = (warp - 4) >> 2;     // which kColsPerWarp of the chunk's 32 columns
    const int rloc = q * 32 + lane;       // row of the tile handled by this thread
    uint32_t slot = 0, sphase = 0;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
      const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
      const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * kBN;
      const int acc = it & 1;
      if (!mbar_wait(&tfull[acc], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const float* Hrow = p.opt.H + (long long)member * p.opt.nh_stride;
      const float lr = hp(Hrow, p.opt.slot_lr, p.opt.const_lr);
      const float b1 = hp(Hrow, p.opt.slot_beta1, p.opt.const_beta1);
      const float wd = hp(Hrow, p.opt.slot_wd, p.opt.const_wd);
      const float b2 = p.opt.const_beta2, eps = p.opt.const_eps;
      const float c1 = __fmul_rn(p.opt.scalars[member * PBT_N_SCALARS + p.opt.scalar_base + 0], b1);
      const float c2 = __fmul_rn(p.opt.scalars[member * PBT_N_SCALARS + p.opt.scalar_base + 1], b2);
      const float inv_bc1 = 1.f / (1.f - c1), inv_bc2 = 1.f / (1.f - c2);
      const float omb1 = 1.f - b1, omb2 = 1.f - b2, lrwd = lr * wd;
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kBN + half * kColsPerWarp);
      uint32_t g[kColsPerWarp];
      tmem_ld_cols<kColsPerWarp>(tacc, g);
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        const int col0 = n0 + c * kChunk;
        if (col0 >= p.N) break;
        tmem_ld_wait();
        float gf[kColsPerWarp];
#pragma unroll
        for (int j = 0; j < kColsPerWarp; ++j) gf[j] = __uint_as_float(g[j]);
        const bool last = (c + 1 == kChunks) || (col0 + kChunk >= p.N);
        if (!last) {
          // next chunk's gradient while this one is applied
          tmem_ld_cols<kColsPerWarp>(tacc + (c + 1) * kChunk, g);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty[acc]);   // the accumulator can be reused by the MMA warp
        }
        if (!mbar_wait(&sfull[slot], sphase, abort_flag)) { ok = false; break; }
        // box row r (0..31) = weight row col0 + r, 128 floats = inputs m0 .. m0+127: this thread owns input rloc
        float* box = reinterpret_cast<float*>(smem + kSlotOffset + slot * kSlotBytes) + (half * kColsPerWarp) * kBM + rloc;
        bf16* w16 = reinterpret_cast<bf16*>(smem + kW16Offset + slot * kW16Bytes) + (half * kColsPerWarp) * kBM + rloc;
        constexpr int kBoxFloats = kBoxBytes / 4;
#pragma unroll
        for (int j = 0; j < kColsPerWarp; ++j) {
          const float w = box[j * kBM];
          float m1 = box[kBoxFloats + j * kBM];
          float m2 = box[2 * kBoxFloats + j * kBM];
          const float nw = adam_one(w, m1, m2, gf[j], b1, omb1, b2, omb2, inv_bc1, inv_bc2, lr, eps, lrwd);
          box[j * kBM] = nw;
          box[kBoxFloats + j * kBM] = m1;
          box[2 * kBoxFloats + j * kBM] = m2;
          w16[j * kBM] = __float2bfloat16_rn(nw);
        }
        if (p.gout) {
          const int in_idx = m0 + rloc;
          if (in_idx < p.M) {
#pragma unroll
            for (int j = 0; j < kColsPerWarp; ++j) {
              const int out_idx = col0 + half * kColsPerWarp + j;
              if (out_idx < p.N) p.gout[member * p.strideC + (long long)out_idx * p.ldc + in_idx] = gf[j];
            }
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sdone[slot]);
        if (++slot == kSlots) { slot = 0; sphase ^= 1; }
      }
    }
    if (!ok && lane == 0) give_up(p, abort_flag, 15);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

// g describes the weight-gradient GEMM (A = dZ, B = layer input, both MN-major bf16, M = out, N = in,
// K = batch rows); g.adam carries the slab pointers and the layer's offset; g.C, if not null, receives the gradient.
// The kernel computes the transposed product, so g's B operand is its A operand and g.N its M.
cudaError_t launch_wgrad_adam(const GemmArgs& g, Counters* counters, cudaStream_t s) {
  if (!g.adam || !g.a_mn || !g.b_mn || g.in_dtype != kBF16 || !g.adam->w16 || !g.adam->opt2) return cudaErrorInvalidValue;
  FusedParams p;
  memset(&p, 0, sizeof(p));
  p.M = g.N; p.N = g.M; p.K = g.K; p.batch = g.batch;
  p.tiles_m = (p.M + kBM - 1) / kBM;
  p.tiles_n = (p.N + kBN - 1) / kBN;
  p.num_tiles = p.tiles_m * p.tiles_n * g.batch;
  p.k_blocks = (g.K + kBK - 1) / kBK;
  p.gout = reinterpret_cast<float*>(g.C); p.ldc = g.ldc; p.strideC = g.strideC;
  p.counters = counters;
  p.opt = *g.adam;
  const OptArgs& o = *g.adam;
  CUtensorMap tmA, tmB, tmW, tmM, tmV, tmW16;
  const int ab = (g.batch > 1 && g.strideA != 0) ? g.batch : 1, bb = (g.batch > 1 && g.strideB != 0) ? g.batch : 1;
  // operand roles swapped (the layer input is the kernel's A); state boxes: kChunk weight rows x kBM inputs, row-major
  p.in_rowoff = g.b_rowoff;
  bool ok = make_map(&tmA, g.B, g.N, g.b_rowoff ? g.b_rows_total : g.K, g.ldb, g.b_rowoff ? 1 : bb, g.strideB, kBK) &&
            make_map(&tmB, g.A, g.M, g.K, g.lda, ab, g.strideA, kBK) &&
            make_map(&tmW, o.w32 + o.begin, g.N, g.M, g.ldc, g.batch, o.p_pad, kChunk, 4, kBM, 0) &&
            make_map(&tmM, o.opt1 + o.begin, g.N, g.M, g.ldc, g.batch, o.p_pad, kChunk, 4, kBM, 0) &&
            make_map(&tmV, o.opt2 + o.begin, g.N, g.M, g.ldc, g.batch, o.p_pad, kChunk, 4, kBM, 0) &&
            make_map(&tmW16, o.w16 + o.begin, g.N, g.M, g.ldc, g.batch, o.p_pad, kChunk, 2, kBM, 0);
  if (!ok) return cudaErrorInvalidValue;
  if (g.a_rowoff) return cudaErrorInvalidValue;   // only the layer input can come from a pool
  if (g.batch > 1 && (g.strideA == 0 || (g.strideB == 0 && !g.b_rowoff))) return cudaErrorInvalidValue;  // operands are per member here
  static DeviceSetup setup;
  int sms = 0;
  cudaError_t e = device_setup(&setup, k_wgrad_adam, kSmemTotal, &sms);
  if (e != cudaSuccess) return e;
  const int grid = p.num_tiles < sms ? p.num_tiles : sms;
  launch_with(grid, kThreads, kSmemTotal, s)(k_wgrad_adam, tmA, tmB, tmW, tmM, tmV, tmW16, p);
  return cudaGetLastError();
}

}  // namespace pbt
