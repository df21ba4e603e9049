// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "pbt.h"

namespace pbt {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11, Section 3.3), device + host.
// counter = (member, round_or_step, stream, block), key = (seed_lo, seed_hi)
// ---------------------------------------------------------------------------
enum PhiloxStream : uint32_t { kStreamExploit = 0, kStreamExplore = 1, kStreamBatch = 2, kStreamInit = 3, kStreamInterp = 4 };

struct U4 {
  uint32_t x[4];
};

__host__ __device__ inline U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint64_t seed) {
  const uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u, kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += kW0;
      k1 += kW1;
    }
    const uint64_t p0 = (uint64_t)kM0 * c0;
    const uint64_t p1 = (uint64_t)kM1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  U4 o;
  o.x[0] = c0; o.x[1] = c1; o.x[2] = c2; o.x[3] = c3;
  return o;
}

// ---------------------------------------------------------------------------
// Launching.  Every kernel of the library is launched through launch_with and begins with pdl_prologue().  When
// programmatic launches are switched on, the launch carries the programmatic-stream-serialization attribute: the
// grid may be scheduled while its predecessor in the stream drains, and its threads wait in griddepcontrol.wait
// until the predecessor has completed and its writes are visible, so the data dependences are exactly those of
// stream order.  No kernel triggers its successor early: a successor made resident ahead of time competes with the
// running kernel for the SM, and measured slower (C2 0.246 vs 0.227 ms per step).  With the implicit trigger at
// grid completion the gain over plain stream order inside a replayed CUDA graph is nil on this GPU (C2 0.226 vs
// 0.227 ms, C4 1.770 vs 1.758 ms per step), so plain stream order is the default and the attribute is opt-in
// (pbt_spec.programmatic_launches).
// ---------------------------------------------------------------------------
void set_serial_launches(bool serial);
bool serial_launches();

#ifdef __CUDACC__
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");   // returns at once unless launched with the attribute
}

struct LaunchCfg {
  dim3 grid, block;
  size_t smem;
  cudaStream_t stream;
  template <typename... KArgs, typename... Args>
  cudaError_t operator()(void (*kernel)(KArgs...), Args&&... args) const {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = serial_launches() ? 0 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(static_cast<Args&&>(args))...);
  }
};
inline LaunchCfg launch_with(dim3 grid, dim3 block, size_t smem, cudaStream_t stream) { return LaunchCfg{grid, block, smem, stream}; }
#endif

// ---------------------------------------------------------------------------
// Device-resident counters and status
// ---------------------------------------------------------------------------
struct Counters {
  long long reserved;  // (the members' step counts live in their own per-member array: see StepClock)
  long long round;   // ready points passed so far
  int status;        // 0, or a pbt_status set by a kernel (bounded wait expired, ...)
  int status_info;   // where it was set
  int use_supplied_batch;  // next step trains on rows supplied by the caller
  int max_level;           // copy passes minus one needed by the last ready point (tournament chains)
  // (the 32 bytes above are what pbt_grouped_gemm / pbt_selftest_bounded_wait callers provide; the rest exists
  // only inside a population's workspace)
  unsigned int bar_count;  // grid barrier of the multi-pass slab copy: arrivals of the current generation
  unsigned int bar_gen;    // ... and the generation
};

// Algorithm 1's t, counted per member (members may advance at their own pace).  Kernels that draw from the
// counter-based generator for "member m at its step t" get the step counts of the members they work on (t[i] belongs
// to the i-th member of the launch) and the population index of the launch's first member.
struct StepClock {
  const long long* t;
  int member_base;
};

// ---------------------------------------------------------------------------
// GEMM description: C[m][n] = sum_k A(m,k) * B(n,k), one problem per member.
// A_MN == false: A(m,k) = A[m*lda + k] (K contiguous); true: A(m,k) = A[k*lda + m].
// B likewise over (n,k).  Strides are in elements of the operand type.
// ---------------------------------------------------------------------------
enum DType : int { kF32 = 0, kBF16 = 1 };
struct OptArgs;

struct GemmArgs {
  int M, N, K, batch;
  int in_dtype;   // DType of A and B
  int out_dtype;  // DType of C
  const void* A; long long lda, strideA; int a_mn;
  const void* B; long long ldb, strideB; int b_mn;
  void* C; long long ldc, strideC;
  const float* bias; long long strideBias;  // added per column n (may be null)
  int relu;                                 // max(., 0) after the bias
  const void* mask; long long ldmask, strideMask;  // C *= (mask[m][n] > 0), operand type (may be null)
  // Weight-gradient GEMMs only (tensor-core path): when `adam` is set the epilogue applies the Adam update
  // to the member's slab in place (C[m][n] is the gradient of element adam->begin + m*ldc + n) and stores the
  // gradient itself only if C is not null.
  const struct OptArgs* adam;
  // Row windows (tensor-core kernels only): operand X is then ONE matrix of x_rows_total rows shared by all
  // problems (a data pool) and problem b uses the rows that start at x_rowoff[b] (device array, one int per
  // problem); strideX is ignored.  "Row" is the slow index of the stored matrix: m (or n) for a K-major operand,
  // k for an MN-major one.
  const int* a_rowoff; long long a_rows_total;
  const int* b_rowoff; long long b_rows_total;
};

// launchers (each enqueues on `s` and returns the CUDA error of the launch)
cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t s);
// tensor-core path; returns cudaErrorNotSupported when the shape does not qualify
bool gemm_tc_supported(const GemmArgs& g);
cudaError_t launch_gemm_tc(const GemmArgs& g, Counters* counters, cudaStream_t s);
// one CTA runs the kernels' bounded barrier wait on a barrier nobody signals, with `limit` polls
cudaError_t launch_selftest_bounded_wait(Counters* counters, uint32_t limit, cudaStream_t s);
// CTA-pair variant (256 x 256 tiles shared by two CTAs of a cluster) for shapes with M, N >= 256
bool gemm_tc_pair_supported(const GemmArgs& g);
bool gemm_tc_pair_preferred(const GemmArgs& g);   // the faster of the two tensor-core kernels for this problem?
cudaError_t launch_gemm_tc_pair(const GemmArgs& g, Counters* counters, cudaStream_t s);
// weight gradient with the Adam update applied in the same kernel (g.adam must be set; tensor-core shapes only)
cudaError_t launch_wgrad_adam(const GemmArgs& g, Counters* counters, cudaStream_t s);

struct OptArgs {
  int n_members;
  long long p_pad;           // slab stride in elements
  long long begin, count;    // element range of the stack inside each slab (multiples of 8)
  float* w32; float* opt1; float* opt2; const float* grad; bf16* w16;  // w16 may be null
  const float* H; int nh_stride;  // per-member hyperparameters (float), row stride
  int slot_lr, slot_momentum, slot_beta1, slot_wd;
  float const_lr, const_momentum, const_beta1, const_beta2, const_eps, const_wd;
  float* scalars; int scalar_base;   // scalars[m*PBT_N_SCALARS + scalar_base + {0,1}] = c1, c2
};
cudaError_t launch_sgd(const OptArgs& a, cudaStream_t s);
cudaError_t launch_sgdm(const OptArgs& a, cudaStream_t s);
cudaError_t launch_adam(const OptArgs& a, cudaStream_t s);
cudaError_t launch_rmsprop(const OptArgs& a, cudaStream_t s);
cudaError_t launch_adam_advance(const OptArgs& a, cudaStream_t s);

// ---- device helpers shared by the optimiser kernel and the fused weight-gradient epilogue ----
#ifdef __CUDACC__
__device__ __forceinline__ float hp(const float* __restrict__ Hrow, int slot, float fallback) {
  return slot >= 0 ? Hrow[slot] : fallback;
}

__device__ __forceinline__ float4 ld_stream(const float* p) {
  // read-once data: bypass L1 allocation
  float4 v;
  asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(float* p, float4 v) {
  asm volatile("st.global.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_bf16x4(bf16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&lo);
  u.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

// Every operation is an explicitly rounded intrinsic: the compiler's choice of where to contract a multiply and an add
// depends on the surrounding code, and the fused and the separate update must give identical bits.
__device__ __forceinline__ float adam_one(float w, float& m1, float& m2, float g, float b1, float omb1, float b2,
                                          float omb2, float inv_bc1, float inv_bc2, float lr, float eps,
                                          float lrwd) {
  m1 = __fmaf_rn(b1, m1, __fmul_rn(omb1, g));
  m2 = __fmaf_rn(b2, m2, __fmul_rn(__fmul_rn(omb2, g), g));
  const float mhat = __fmul_rn(m1, inv_bc1);
  const float vhat = __fmul_rn(m2, inv_bc2);
  // square root and reciprocal by the special-function unit (relative error about 2^-23 each): the update warps of
  // the fused kernel are bound by instruction issue, and the correctly rounded forms cost several times as many
  float root;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(vhat));
  const float upd = __fdividef(mhat, __fadd_rn(root, eps));
  return __fmaf_rn(-lrwd, w, __fmaf_rn(-lr, upd, w));
}

#endif  // __CUDACC__

struct SelectArgs {
  int n, nh, n_cut;
  int h_is_double;
  void* H;            // [n][PBT_MAX_NH] float or double
  void* fitness;      // [n] float or double
  int* src;           // [n]
  int* level;         // [n] copy pass of each recipient (0 unless its donor chain is longer)
  int rule;           // 0 truncation selection, 1 binary tournament, 2 t-test selection
  void* hist;         // [n][PBT_HISTORY] scores, oldest first (same type as fitness); t-test only
  int* hist_n;        // [n] valid entries per row
  double alpha;       // t-test significance level
  int explore_rule;   // 0 perturb, 1 resample from the prior
  uint32_t resample_thr;            // a slot is redrawn when its Philox word is below this
  int prior_kind[PBT_MAX_NH];
  double prior_a[PBT_MAX_NH], prior_b[PBT_MAX_NH];   // uniform: lo, hi; log-uniform: log lo, log hi
  Counters* counters;
  uint64_t seed;
  uint32_t ready_bits[32];          // bit i set: member i is ready (Algorithm 1) and may exploit at this ready point
  uint32_t perturb_mask, flags;
  double factor_lo, factor_hi;
  double clamp_lo[PBT_MAX_NH], clamp_hi[PBT_MAX_NH];
};
cudaError_t launch_select_explore(const SelectArgs& a, cudaStream_t s);
// append fitness[i] to row i of the score history (drop the oldest of PBT_HISTORY)
cudaError_t launch_history_push(const void* fitness, void* hist, int* hist_n, int n, int is_double, cudaStream_t s);

struct CopyArgs {
  int n;
  const int* src;
  const int* level;   // optional: only recipients with level[b] == want_level are copied in this launch
  int want_level;
  // up to 5 member-major arrays copied donor -> recipient; bytes per member, stride in bytes
  int n_arrays;
  char* base[5];
  long long stride_bytes[5];
  long long copy_bytes[5];  // multiples of 16
};
// After a selection over the whole (sharded) population: rows [base, base + n_local) of the global hyperparameter
// and fitness vectors become the shard's own, and the global copy map is translated: src_local[i] is the donor's
// local index if the donor of member base + i lives in this shard, i otherwise (the record arrives from outside).
cudaError_t launch_localize_selection(const int* src_global, const int* level_global, const void* H_global,
                                      const void* fit_global, int is_double, int base, int n_local, int* src_local,
                                      int* level_local, void* H_local, void* fit_local, cudaStream_t s);
cudaError_t launch_slab_copy(const CopyArgs& a, cudaStream_t s);
cudaError_t launch_copy_small(char* base, long long bytes, const int* src, int n, const int* level, int want_level,
                              cudaStream_t s);
// Every copy pass 0..counters->max_level in ONE launch (a.level must be set; a.want_level is ignored): the number of
// passes is read on the device, so the host never waits for the select kernel.  Between passes the blocks meet at a
// grid barrier (cooperative launch: all blocks are resident), whose wait is bounded: on expiry the kernel sets
// counters->status = PBT_ERR_TIMEOUT and returns.
cudaError_t launch_slab_copy_levels(const CopyArgs& a, Counters* counters, cudaStream_t s);
cudaError_t launch_copy_small_levels(char* base, long long bytes, const int* src, int n, const int* level,
                                     const Counters* counters, cudaStream_t s);

// misc kernels -------------------------------------------------------------
cudaError_t launch_init_weights(float* w32, long long p_pad, int n_members, long long w_off, int fan_out,
                                int fan_in, int tensor_id, float bound, uint64_t seed, int member_base, cudaStream_t s);
cudaError_t launch_f32_to_bf16(const float* in, bf16* out, long long n, cudaStream_t s);
// copy rows [off, off+rows) of a pool into dst + m*dst_stride_bytes (+ dst_offset_bytes) for every member;
// off = 128 * ((word * n_win) >> 32), word = philox(seed; m, step, batch stream, block).x[word_index]
// off[m] = first pool row of member m's training window for the current step (the rule of launch_gather_window)
cudaError_t launch_window_offsets(int* off, int rows, int pool_rows, int n_members, int block, int word_index,
                                  uint64_t seed, StepClock clk, cudaStream_t s);
cudaError_t launch_gather_window(char* dst, long long dst_stride_bytes, long long dst_offset_bytes,
                                 const char* pool, int row_bytes, int rows, int pool_rows, int n_members,
                                 int block, int word_index, uint64_t seed, const Counters* counters,
                                 StepClock clk, cudaStream_t s);
// strided row copy with optional conversion (float -> operand type), per member
cudaError_t launch_copy_rows(void* dst, int dst_dtype, long long dst_ld, long long dst_stride,
                             const float* src, long long src_ld, long long src_stride, int rows, int cols,
                             int n_members, cudaStream_t s);

struct LossArgs {
  int kind;        // pbt_loss
  int n_members, rows, cols;
  int n_real_rows; // GAN: rows < n_real_rows are labelled real; WGAN-GP: the next n_real_rows are generated rows and
                   // any rows after those are interpolates (dL/dz = 1, their loss is written by launch_gp_penalty)
  float inv_batch; // 1 / B  (scale of dL/dz and of the mean)
  const float* logits; long long ld_logits, stride_logits;
  const void* target; long long stride_target;   // elements of the target type; 0 = shared by all members
  const int* target_rowoff;                      // optional (device, one int per member): the member's targets are the
                                                 // rows of a shared pool that start here (stride_target is then 0)
  int target_dtype;                              // DType for MSE / CE_SOFT targets (MSE is always float)
  void* dz; int dz_dtype; long long ld_dz, stride_dz;   // may be null (eval)
  float* row_loss;   // [n_members][rows]
};
cudaError_t launch_loss_rows(const LossArgs& a, cudaStream_t s);
// out[m*out_stride] = scale * sum_r row_loss[m][r], fixed summation order
cudaError_t launch_reduce_rows(const float* row_loss, int rows, int n_members, float scale, void* out,
                               int out_is_double, int out_stride, cudaStream_t s);
cudaError_t launch_bias_grad(const void* dz, int dz_dtype, long long ld, long long stride, int rows, int cols,
                             float* out, long long out_stride, int n_members, cudaStream_t s);
cudaError_t launch_toy_step(double* theta, const double* H, int n_members, int dim, double eta, cudaStream_t s);
cudaError_t launch_toy_eval(const double* theta, double* fitness, int n_members, int dim, cudaStream_t s);
// fitness[m] = -(energy distance between x[m][n][2] and the eight-mode unit ring)
cudaError_t launch_energy_distance(const float* x, long long stride, int n, int n_members, double* partial,
                                   float* fitness, cudaStream_t s);
int energy_partial_count(int n);  // doubles of scratch per member
// WGAN-GP (Section 4.3.1).  x holds, per member, rows [0,B) real, [B,2B) generated; writes rows [2B,3B):
// xhat_b = eps_b real_b + (1 - eps_b) fake_b, eps_b from the interpolation stream at (member, step, block j*65536 + b/4)
cudaError_t launch_gp_interp(void* x, int dtype, long long stride, int B, int dim, int j, int n_members, uint64_t seed,
                             StepClock clk, cudaStream_t s);
// gx[m][b][dim] = grad_x D(xhat_b).  row_loss[m][row_off + b] = lam (||gx_b|| - 1)^2 (row stride rows_total) and
// dv[m][b][:] = (2 lam / B)(||gx_b|| - 1) / ||gx_b|| * gx_b (zero where the norm is zero), in the operand type
cudaError_t launch_gp_penalty(const float* gx, long long gx_stride, int B, int dim, float lam, float inv_batch,
                              float* row_loss, int rows_total, int row_off, void* dv, int dv_dtype,
                              long long dv_stride, int n_members, cudaStream_t s);
cudaError_t launch_advance_step(Counters* c, long long* t, int n_members, cudaStream_t s);

}  // namespace pbt
