// Member-batched bf16 GEMM with CTA pairs (tcgen05 cta_group::2): two CTAs of a cluster share one
// 256 x 256 output tile.  CTA r of the pair loads its own 128 rows of A and HALF of the B tile (128 of the 256
// columns of the output) into its shared memory; the leader CTA (rank 0) issues tcgen05.mma.cta_group::2, which
// reads A and the B halves from both CTAs' shared memory and accumulates rows [r*128, r*128+128) of the tile in
// CTA r's tensor memory.  Per SM that is 32 KB of operands per 64-deep k-block instead of 48 KB for the same
// flops, with plain per-CTA TMA loads.
//
// Synchronisation (all mbarrier waits bounded, as in the single-CTA kernel):
//   full[s]   lives in the leader; its producer announces the bytes of both CTAs and both CTAs' TMA loads
//             complete their bytes on it
//   empty[s]  one per CTA; the leader's MMA thread commits to both (the follower's through its cluster address)
//   tfull[a]  one per CTA, committed to both after the last k-block; tempty[a] lives in the leader and counts the
//             epilogue warps of both CTAs (the follower's arrive remotely)
// The cluster is synchronised after barrier initialisation and before exit.
#include <string.h>

#include "tc_epilogue.cuh"

namespace pbt {

namespace {

using namespace tc;

constexpr int kPN = 256;          // tile columns
constexpr int kPStages = 5;       // 32 KB per stage and CTA
constexpr int kPEpiW = 8;         // epilogue warps per CTA
constexpr int kPThreads = 64 + 32 * kPEpiW;
constexpr int kPABytes = kBM * kBK * 2, kPBBytes = (kPN / 2) * kBK * 2, kPStageBytes = kPABytes + kPBBytes;
constexpr int kPEpiOffset = kPStages * kPStageBytes;
constexpr int kPEpiBytesPerWarp = 8192;   // two staging boxes of 32 rows x 128 bytes (the transposing path uses 4.5 KB of it)
static_assert(kPEpiBytesPerWarp >= 32 * kEpiPitch * 4 && kPEpiOffset % 1024 == 0, "staging boxes are 1024-byte aligned");
constexpr int kPBarOffset = kPEpiOffset + kPEpiW * kPEpiBytesPerWarp;
constexpr int kPSmemTotal = kPBarOffset + 256 + 1024;
static_assert(kPSmemTotal <= 232448, "shared memory budget of one CTA");

// ---- cluster helpers ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes)
               : "memory");
}
// TMA load of this CTA's part of a pair tile; the bytes are accounted on the leader's barrier
__device__ __forceinline__ void tma_load_3d_pair(void* smem_dst, const CUtensorMap* map, uint32_t leader_bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at this shared::cluster address once the pair's MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
k_gemm_tc_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const TcParams p) {
  pdl_prologue();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kPBarOffset);   // used in the leader only
  uint64_t* empty = full + kPStages;                                    // per CTA
  uint64_t* tfull = empty + kPStages;                                   // per CTA
  uint64_t* tempty = tfull + 2;                                         // used in the leader only
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kTmemCols = 2 * kPN;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kPStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 2 * kPEpiW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers exist before anyone signals across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int tiles_per_member = p.tiles_m * p.tiles_n;   // tiles_m counts 256-row pair tiles

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int tile = pair; tile < p.num_tiles && ok; tile += n_pairs) {
        const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
        const int m0 = (rem / p.tiles_n) * (2 * kBM) + (int)rank * kBM;
        const int n0 = (rem % p.tiles_n) * kPN + (int)rank * (kPN / 2);
        const int ca = p.a_batched ? member : 0, cb = p.b_batched ? member : 0;
        const int ra = p.a_rowoff ? p.a_rowoff[member] : 0, rb = p.b_rowoff ? p.b_rowoff[member] : 0;   // row windows
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * kPStageBytes;
          uint8_t* sb = sa + kPABytes;
          const uint32_t lbar = map_to_cta(smem_u32(&full[stage]), 0);
          // the leader announces the bytes of both CTAs; the follower's loads simply complete on the leader's barrier
          // (it cannot run a phase ahead: its stage is handed back by the leader's commit for the previous phase)
          if (rank == 0) mbar_expect_tx(&full[stage], 2 * kPStageBytes);
          const int k0 = kb * kBK;
          if (!p.a_mn) {
            tma_load_3d_pair(sa, &tmA, lbar, k0, m0 + ra, ca);
          } else {
#pragma unroll
            for (int j = 0; j < kBM / 64; ++j) tma_load_3d_pair(sa + j * 8192, &tmA, lbar, m0 + j * 64, k0 + ra, ca);
          }
          if (!p.b_mn) {
            tma_load_3d_pair(sb, &tmB, lbar, k0, n0 + rb, cb);
          } else {
#pragma unroll
            for (int j = 0; j < kPN / 128; ++j) tma_load_3d_pair(sb + j * 8192, &tmB, lbar, n0 + j * 64, k0 + rb, cb);
          }
          if (++stage == kPStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
        p.counters->status_info = 21;
      }
      // drain: every commit the leader addressed to this CTA's `empty` barriers has landed before the CTA exits
      for (int s2 = 0; s2 < kPStages && ok; ++s2) {
        if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) break;
        if (++stage == kPStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only) ------------------------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                             ((uint32_t)(kPN >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24);
      uint32_t stage = 0, phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = pair; tile < p.num_tiles && ok; tile += n_pairs, ++it) {
        const int acc = it & 1;
        if (!mbar_wait(&tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * kPN;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * kPStageBytes);
          const uint32_t sb = sa + kPABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            const uint64_t ad = p.a_mn ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
            const uint64_t bd = p.b_mn ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
            umma_bf16_pair(tmem_d, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          const uint32_t eb = smem_u32(&empty[stage]);
          umma_commit_pair(map_to_cta(eb, 0));
          umma_commit_pair(map_to_cta(eb, 1));
          if (++stage == kPStages) { stage = 0; phase ^= 1; }
        }
        if (ok) {
          const uint32_t tb = smem_u32(&tfull[acc]);
          umma_commit_pair(map_to_cta(tb, 0));
          umma_commit_pair(map_to_cta(tb, 1));
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
        p.counters->status_info = 22;
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs, own 128 rows) ------------------------------
    const int q = warp & 3, e = warp - 2, half = e >> 2;
    uint8_t* stage = smem + kPEpiOffset + e * kPEpiBytesPerWarp;
    float* buf = reinterpret_cast<float*>(stage);
    uint32_t boxes_used = 0;
    int it = 0;
    bool ok = true;
    const int esz = p.out_dtype == kBF16 ? 2 : 4;
    const bool vec_ok = (((uintptr_t)p.C & 15) == 0) && ((p.ldc * esz) % 16 == 0) && ((p.strideC * esz) % 16 == 0) &&
                        (!p.mask || ((((uintptr_t)p.mask & 7) == 0) && (p.ldmask % 4 == 0) && (p.strideMask % 4 == 0))) &&
                        (!p.bias || ((((uintptr_t)p.bias & 15) == 0) && (p.strideBias % 4 == 0)));
    for (int tile = pair; tile < p.num_tiles && ok; tile += n_pairs, ++it) {
      const int member = tile / tiles_per_member, rem = tile % tiles_per_member;
      const int m0 = (rem / p.tiles_n) * (2 * kBM) + (int)rank * kBM, n0 = (rem % p.tiles_n) * kPN;
      const int acc = it & 1;
      if (!mbar_wait(&tfull[acc], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kPN);
      const uint32_t handback = map_to_cta(smem_u32(&tempty[acc]), 0);
      if (p.c_tma && m0 + kBM <= p.M && n0 + kPN <= p.N && (p.out_dtype == kBF16 || !p.mask)) {
        epilogue_tile_tma<kPN, kPEpiW>(p, &tmC, stage, tacc, member, m0, n0, q, half, lane, handback, boxes_used);
      } else {
        if (lane == 0) tma_store_wait_all();   // the transposing path reuses the staging memory
        __syncwarp();
        epilogue_tile<kPN, kPEpiW>(p, buf, tacc, member, m0, n0, q, half, lane, vec_ok);
        release_accumulator(handback, lane);
      }
    }
    if (lane == 0) tma_store_wait_all();     // the bulk stores have read the staging boxes and reached memory
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(&p.counters->status, 0, PBT_ERR_TIMEOUT);
      p.counters->status_info = 23;
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves while its partner may still signal its barriers or read its operands
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

}  // namespace

bool gemm_tc_pair_supported(const GemmArgs& g) {
  return gemm_tc_supported(g) && g.M >= 256 && g.N >= 256;
}

// Whether the pair kernel is the faster of the two tensor-core kernels for this problem.  Few tiles AND a short
// contraction (under four waves of pairs, under 12 k-blocks): the single-CTA kernel's shorter pipeline fills and
// drains faster (24 GAN pairs, 1024 x 512 x 512 per member: 23 -> 20 us per launch); longer contractions amortise the
// pair's set-up even on two waves (32 members of 256 x 1024 x 1024).
bool gemm_tc_pair_preferred(const GemmArgs& g) {
  if (!gemm_tc_pair_supported(g)) return false;
  const long long tiles = (long long)((g.M + 255) / 256) * ((g.N + 255) / 256) * g.batch;
  return tiles >= 296 || g.K >= 768;
}

cudaError_t launch_gemm_tc_pair(const GemmArgs& g, Counters* counters, cudaStream_t s) {
  if (g.adam) return cudaErrorInvalidValue;
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.M = g.M; p.N = g.N; p.K = g.K; p.batch = g.batch;
  p.tiles_m = (g.M + 2 * kBM - 1) / (2 * kBM);
  p.tiles_n = (g.N + kPN - 1) / kPN;
  p.num_tiles = p.tiles_m * p.tiles_n * g.batch;
  p.k_blocks = (g.K + kBK - 1) / kBK;
  p.a_mn = g.a_mn; p.b_mn = g.b_mn;
  p.a_batched = (g.batch > 1 && g.strideA != 0 && !g.a_rowoff) ? 1 : 0;
  p.b_batched = (g.batch > 1 && g.strideB != 0 && !g.b_rowoff) ? 1 : 0;
  p.a_rowoff = g.a_rowoff; p.b_rowoff = g.b_rowoff;
  p.C = g.C; p.ldc = g.ldc; p.strideC = g.strideC; p.out_dtype = g.out_dtype;
  p.bias = g.bias; p.strideBias = g.strideBias; p.relu = g.relu;
  p.mask = reinterpret_cast<const bf16*>(g.mask); p.ldmask = g.ldmask; p.strideMask = g.strideMask;
  p.counters = counters;
  CUtensorMap tmA, tmB;
  bool ok;
  const long long a_rows = g.a_rowoff ? g.a_rows_total : (g.a_mn ? g.K : g.M);   // a windowed operand: the whole pool
  const long long b_rows = g.b_rowoff ? g.b_rows_total : (g.b_mn ? g.K : g.N);
  if (!g.a_mn) ok = make_map(&tmA, g.A, g.K, a_rows, g.lda, p.a_batched ? g.batch : 1, g.strideA, kBM);
  else ok = make_map(&tmA, g.A, g.M, a_rows, g.lda, p.a_batched ? g.batch : 1, g.strideA, kBK);
  if (!ok) return cudaErrorInvalidValue;
  if (!g.b_mn) ok = make_map(&tmB, g.B, g.K, b_rows, g.ldb, p.b_batched ? g.batch : 1, g.strideB, kPN / 2);
  else ok = make_map(&tmB, g.B, g.N, b_rows, g.ldb, p.b_batched ? g.batch : 1, g.strideB, kBK);
  if (!ok) return cudaErrorInvalidValue;
  // C as a tensor map (boxes of 32 rows x 128 bytes, 128-byte swizzle) when its layout allows bulk stores
  CUtensorMap tmC;
  memset(&tmC, 0, sizeof(tmC));
  {
    const int esz = g.out_dtype == kBF16 ? 2 : 4;
    const bool mask_ok = !g.mask || ((((uintptr_t)g.mask) & 15) == 0 && g.ldmask % 8 == 0 && g.strideMask % 8 == 0);
    const bool bias_ok = !g.bias || ((((uintptr_t)g.bias) & 15) == 0 && g.strideBias % 4 == 0);
    if (mask_ok && bias_ok && (((uintptr_t)g.C) & 15) == 0 && (g.ldc * esz) % 16 == 0 && (g.strideC * esz) % 16 == 0 &&
        make_map(&tmC, g.C, g.N, g.M, g.ldc, g.batch, g.strideC, 32, esz, 128 / esz, 128))
      p.c_tma = 1;
  }
  static DeviceSetup setup;
  int sms = 0;
  cudaError_t e = device_setup(&setup, k_gemm_tc_pair, kPSmemTotal, &sms);
  if (e != cudaSuccess) return e;
  int pairs = sms / 2;
  if (pairs > p.num_tiles) pairs = p.num_tiles;
  launch_with(2 * pairs, kPThreads, kPSmemTotal, s)(k_gemm_tc_pair, tmA, tmB, tmC, p);
  return cudaGetLastError();
}

}  // namespace pbt
