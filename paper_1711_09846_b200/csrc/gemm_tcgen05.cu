// Member-batched bf16 GEMM on the 5th-generation tensor cores (sm_100a):
//   C[m][n] = sum_k A(m,k) * B(n,k),   one problem per population member,
// covering the forward (both operands K-major), data-gradient (B MN-major) and
// weight-gradient (both MN-major) contractions of the training step.
//
// Structure of one CTA (persistent, one per SM, static round-robin over tiles):
//   warp 0      TMA producer: 3-D tiled bulk-tensor loads (member = outer coordinate), 128-byte swizzle,
//               into a ring of shared-memory stages guarded by full/empty mbarriers; plain per-CTA loads
//   warp 1      allocates tensor memory, one elected lane issues tcgen05.mma (128 x BN x 16 per
//               instruction, fp32 accumulators in TMEM), tcgen05.commit frees the stage / publishes the tile
//   warps 2..9  epilogue (8 warps, two per TMEM lane quadrant): tcgen05.ld of the accumulator (double-buffered in TMEM, so the next
//               tile's main loop overlaps), a 32 x 32 transpose through padded shared memory so that global
//               accesses are whole 128-byte lines, then bias / ReLU / ReLU-mask / conversion
// Every mbarrier wait is bounded; on expiry the kernel records PBT_ERR_TIMEOUT in the device status
// word, all roles leave their loops, tensor memory is released and the kernel returns normally.
#include <string.h>

#include "tc_epilogue.cuh"

namespace pbt {

namespace {

using namespace tc;

template <int BN, int STAGES, int NEPIW>
struct Smem {
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = BN * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiOffset = STAGES * kStageBytes;
  static constexpr int kEpiBytesPerWarp = 32 * kEpiPitch * 4;
  static constexpr int kBarOffset = kEpiOffset + NEPIW * kEpiBytesPerWarp;
  static constexpr int kTotal = kBarOffset + 256 + 1024;  // barriers + slack for 1024-byte alignment
  static_assert(kTotal <= 232448, "shared memory budget of one CTA");
};

template <int BN, int STAGES, int EPI, int NEPIW>
__global__ void __launch_bounds__(64 + 32 * NEPIW, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcParams p) {
  pdl_prologue();
  using L = Smem<BN, STAGES, NEPIW>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;   // [2] accumulator ready for the epilogue
  uint64_t* tempty = tfull + 2;       // [2] accumulator drained
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kTmemCols = 2 * BN;  // 256 or 512: a power of two >= 32

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], NEPIW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const int member = tile / (p.tiles_m * p.tiles_n);
        const int rem = tile % (p.tiles_m * p.tiles_n);
        const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * BN;
        const int ca = p.a_batched ? member : 0, cb = p.b_batched ? member : 0;
        // a windowed operand is one shared matrix: the problem's rows start at its offset (slow coordinate)
        const int ra = p.a_rowoff ? p.a_rowoff[member] : 0, rb = p.b_rowoff ? p.b_rowoff[member] : 0;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * L::kStageBytes;
          uint8_t* sb = sa + L::kABytes;
          mbar_expect_tx(&full[stage], L::kStageBytes);
          const int k0 = kb * kBK;
          if (!p.a_mn) {
            tma_load_3d(sa, &tmA, &full[stage], k0, m0 + ra, ca);
          } else {
#pragma unroll
            for (int j = 0; j < kBM / 64; ++j) tma_load_3d(sa + j * 8192, &tmA, &full[stage], m0 + j * 64, k0 + ra, ca);
          }
          if (!p.b_mn) {
            tma_load_3d(sb, &tmB, &full[stage], k0, n0 + rb, cb);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_3d(sb + j * 8192, &tmB, &full[stage], n0 + j * 64, k0 + rb, cb);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
        p.counters->status_info = 1;
      }
      // drain: every stage this thread armed must have landed before the CTA may exit; the
      // consumer's commits are what flips `empty`, so wait (bounded) for the last STAGES of them
      for (int s = 0; s < STAGES && ok; ++s) {
        // a stage is idle once its `empty` phase matches the producer's next expectation
        if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
      uint32_t stage = 0, phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!mbar_wait(&tempty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // K-major: 16 elements of K are 32 bytes inside the swizzled 128-byte row; 8-row groups 1024 B apart.
            // MN-major: 16 rows of K are 2048 bytes; 64-element column blocks 8192 B apart, 8-row groups 1024 B.
            const uint64_t ad = p.a_mn ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
            const uint64_t bd = p.b_mn ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
            umma_bf16(tmem_d, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(&tfull[acc]);
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
        p.counters->status_info = 2;
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;            // TMEM lane quadrant this warp may access
    const int e = warp - 2;            // 0 .. NEPIW-1
    const int half = e >> 2;           // warps that share a quadrant interleave over the 32-column chunks
    float* buf = reinterpret_cast<float*>(smem + L::kEpiOffset + e * L::kEpiBytesPerWarp);
    int it = 0;
    bool ok = true;
    const int esz = p.out_dtype == kBF16 ? 2 : 4;
    const bool vec_ok = (((uintptr_t)p.C & 15) == 0) && ((p.ldc * esz) % 16 == 0) && ((p.strideC * esz) % 16 == 0) &&
                        (!p.mask || ((((uintptr_t)p.mask & 7) == 0) && (p.ldmask % 4 == 0) && (p.strideMask % 4 == 0))) &&
                        (!p.bias || ((((uintptr_t)p.bias & 15) == 0) && (p.strideBias % 4 == 0)));
    for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
      const int member = tile / (p.tiles_m * p.tiles_n);
      const int rem = tile % (p.tiles_m * p.tiles_n);
      const int m0 = (rem / p.tiles_n) * kBM, n0 = (rem % p.tiles_n) * BN;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!mbar_wait(&tfull[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      epilogue_tile<BN, NEPIW>(p, buf, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), member, m0, n0, q, half, lane, vec_ok);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[acc]);
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
      p.counters->status_info = 3;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

template <int BN, int STAGES, int EPI, int NEPIW>
cudaError_t launch_cfg(const CUtensorMap& tmA, const CUtensorMap& tmB, TcParams& p, cudaStream_t s) {
  using L = Smem<BN, STAGES, NEPIW>;
  static DeviceSetup setup;   // one per kernel instantiation
  int sms = 0;
  cudaError_t e = device_setup(&setup, k_gemm_tc<BN, STAGES, EPI, NEPIW>, L::kTotal, &sms);
  if (e != cudaSuccess) return e;
  p.tiles_n = (p.N + BN - 1) / BN;
  p.num_tiles = p.tiles_m * p.tiles_n * p.batch;
  const int grid = p.num_tiles < sms ? p.num_tiles : sms;
  launch_with(grid, 64 + 32 * NEPIW, L::kTotal, s)(k_gemm_tc<BN, STAGES, EPI, NEPIW>, tmA, tmB, p);
  return cudaGetLastError();
}

}  // namespace

// Self-test of the bounded wait every tensor-core kernel relies on: one CTA waits on a barrier that nothing ever
// signals; when the limit runs out it records PBT_ERR_TIMEOUT like the real kernels do and returns normally.
__global__ void k_selftest_bounded_wait(Counters* counters, uint32_t limit) {
  pdl_prologue();
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (!mbar_wait(&bar, 0, &abort_flag, limit)) {
      atomicCAS(&counters->status, 0, PBT_ERR_TIMEOUT);
      counters->status_info = 99;
    }
  }
}

cudaError_t launch_selftest_bounded_wait(Counters* counters, uint32_t limit, cudaStream_t s) {
  launch_with(1, 32, 0, s)(k_selftest_bounded_wait, counters, limit);
  return cudaGetLastError();
}

bool gemm_tc_supported(const GemmArgs& g) {
  if (g.in_dtype != kBF16) return false;
  if (g.M < 128 || g.K < 64 || g.batch < 1) return false;
  // Narrow outputs (a ten-wide logit layer): a 128-column tile whose B rows past N are out-of-range rows of the
  // tensor map and arrive as zeros, like the last tile of any ragged N.  Worth it when the ALU row-dot kernel would
  // be bound by unpacking and multiplying (5 or more columns) and the operand is long enough to stream.
  if (g.N < 128 && (g.N < 5 || g.a_mn || g.b_mn || g.K < 256)) return false;
  if (g.lda % 8 || g.ldb % 8) return false;
  if (g.batch > 1 && ((g.strideA != 0 && g.strideA % 8) || (g.strideB != 0 && g.strideB % 8))) return false;
  if (((uintptr_t)g.A & 15) || ((uintptr_t)g.B & 15)) return false;
  return encode_fn() != nullptr;
}

cudaError_t launch_gemm_tc(const GemmArgs& g, Counters* counters, cudaStream_t s) {
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.batch = g.batch;
  p.tiles_m = (g.M + kBM - 1) / kBM;
  p.k_blocks = (g.K + kBK - 1) / kBK;
  p.a_mn = g.a_mn; p.b_mn = g.b_mn;
  p.a_batched = (g.batch > 1 && g.strideA != 0 && !g.a_rowoff) ? 1 : 0;
  p.b_batched = (g.batch > 1 && g.strideB != 0 && !g.b_rowoff) ? 1 : 0;
  p.a_rowoff = g.a_rowoff; p.b_rowoff = g.b_rowoff;
  p.C = g.C; p.ldc = g.ldc; p.strideC = g.strideC; p.out_dtype = g.out_dtype;
  p.bias = g.bias; p.strideBias = g.strideBias; p.relu = g.relu;
  p.mask = reinterpret_cast<const bf16*>(g.mask); p.ldmask = g.ldmask; p.strideMask = g.strideMask;
  p.counters = counters;
  int BN = g.N >= 256 ? 256 : 128;
  if (BN == 256) {
    // Few tiles: 128-wide tiles when the 256-wide ones would leave most of the last wave idle (a wave of half tiles
    // costs a little over half a wave of full ones).  512 x 512 x 512 for 24 members: 192 wide tiles are 2 waves on
    // 148 SMs, 384 narrow ones 3 half-waves.
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long wide = (long long)p.tiles_m * ((g.N + 255) / 256) * g.batch;
    const long long narrow = (long long)p.tiles_m * ((g.N + 127) / 128) * g.batch;
    if (1.15 * (double)((narrow + sms - 1) / sms) < 2.0 * (double)((wide + sms - 1) / sms)) BN = 128;
  }
  CUtensorMap tmA, tmB;
  bool ok;
  // K-major operand: rows = M (or N), cols = K.  MN-major operand: rows = K, cols = M (or N), boxes of 64 x 64.
  // A windowed operand's map covers the whole shared matrix (its rows_total rows).
  const long long a_rows = g.a_rowoff ? g.a_rows_total : (g.a_mn ? g.K : g.M);
  const long long b_rows = g.b_rowoff ? g.b_rows_total : (g.b_mn ? g.K : g.N);
  if (!g.a_mn) ok = make_map(&tmA, g.A, g.K, a_rows, g.lda, p.a_batched ? g.batch : 1, g.strideA, kBM);
  else ok = make_map(&tmA, g.A, g.M, a_rows, g.lda, p.a_batched ? g.batch : 1, g.strideA, kBK);
  if (!ok) return cudaErrorInvalidValue;
  if (!g.b_mn) ok = make_map(&tmB, g.B, g.K, b_rows, g.ldb, p.b_batched ? g.batch : 1, g.strideB, BN);
  else ok = make_map(&tmB, g.B, g.N, b_rows, g.ldb, p.b_batched ? g.batch : 1, g.strideB, kBK);
  if (!ok) return cudaErrorInvalidValue;
  if (g.adam) return cudaErrorInvalidValue;  // the fused weight-gradient + Adam kernel has its own launcher
  // 8 epilogue warps (two per TMEM lane quadrant) keep the tile write-out and the ReLU-mask reads off the critical
  // path; a 3-stage operand ring is as fast as 4 stages here and leaves the shared memory for them
  if (BN == 256) return launch_cfg<256, 3, 0, 8>(tmA, tmB, p, s);
  return launch_cfg<128, 4, 0, 8>(tmA, tmB, p, s);
}

}  // namespace pbt
