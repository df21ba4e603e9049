// Host side of the library: the C ABI of pbt.h, the member-major layout of the
// population in the caller's workspace, and the lockstep schedule of one
// training step / evaluation / ready point as a sequence of kernel launches.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <utility>
#include <vector>

#include "pbt_common.cuh"

using namespace pbt;

namespace {

thread_local char g_err[512] = "";

struct Layer {
  int in, out;
  long long w_off, b_off;  // element offsets inside a member's padded slab
};
struct Stack {
  int nl;
  Layer L[PBT_MAX_LAYERS];
  long long begin, count;  // padded element range of the stack inside the slab
  int rows_cap;            // rows the activation buffers can hold
};

enum KClass { kGemm = 0, kOpt, kLoss, kCopy, kSelect, kOther, kFused, kNumClasses };
const char* const kClassNames[kNumClasses] = {"gemm", "optimizer", "loss", "copy", "select", "other", "wgrad_adam"};

struct ProfRec {
  int cls;
  cudaEvent_t a, b;
};

}  // namespace

struct pbt_handle {
  pbt_spec spec;
  pbt_data data;
  cudaStream_t stream;
  // Launches go to `ls`: the handle's stream, except while a backward pass has forked work to `side` (a second
  // stream the handle owns; every fork is joined back before the pass returns).  side == nullptr: never fork.
  cudaStream_t ls, side;
  cudaEvent_t ev_fork, ev_join;
  bool side_pending;   // side-stream work not yet joined
  uint64_t seed;
  int N, ns, nh;
  bool toy, gan, is_bf16;
  int cdt;      // DType of GEMM operands
  int esz;      // bytes of one operand element
  long long P, P_pad;
  Stack st[2];
  int max_width, dz_rows_cap, rowloss_cap;
  // device state (all inside the caller's workspace)
  float *W32, *O1, *O2, *G;
  bf16* W16;
  float* scalars;
  void* H;        // [N][PBT_MAX_NH] float (double for the toy)
  void* fitness;  // [N] float (double for the toy)
  int* src;
  int* level;        // [N] copy pass of each recipient at the last ready point
  void* hist;        // [N][PBT_HISTORY] scores for t-test selection, same type as fitness
  int* hist_n;       // [N]
  Counters* counters;
  long long* tm;     // [N] every member's own step count (Algorithm 1's t)
  // sharded populations: the whole population's selection inputs and outputs (n_global entries each)
  void* g_fit; void* g_H; int* g_src; int* g_level;
  void* g_hist; int* g_hist_n; bool g_hist_set;   // t-test selection: the whole population's score histories
  int member_base;   // population index of the first member the pointers below refer to (0 unless a window is open)
  float* last_loss;  // [N][2]
  double* theta;     // toy: [N][nh]
  void* act[2][PBT_MAX_LAYERS];  // input of layer l of stack s: [N][rows_cap][in_l]
  float* logits[2];              // [N][rows_cap][out_last]
  void* dz[2];                   // ping-pong deltas [N][dz_rows_cap][max_width]
  // WGAN-GP only: the critic's deltas of every layer are kept until its weight gradients, which need the
  // penalty's second chain, can be formed: gp_dz[l] is [N][3 batch][out_l]; gp_gx is the input gradient [N][batch][d]
  void* gp_dz[PBT_MAX_LAYERS];
  float* gp_gx;
  bool wgan;
  // MLP populations whose first layer runs on the tensor cores read their training rows straight from the data
  // pools (TMA row windows) instead of gathering them first: win_off[m] is member m's first pool row this step
  int* win_off;
  bool direct_pool;
  bool supplied_next;   // the next step trains on rows the caller put into act[0][0] / ybatch
  void* ybatch;
  long long ybatch_stride;  // elements of the target type per member
  // second copy of the training-row buffers: host batches are uploaded here on a copy stream while the step
  // on the current buffers runs (pbt_prefetch_host_batch / pbt_step_prefetched)
  void* act0_alt;
  void* ybatch_alt;
  cudaStream_t copy_stream;
  cudaEvent_t ev_copied, ev_release;   // ev_release: see pbt_step_prefetched
  bool prefetched;
  long long pf_steps;  // prefetched steps taken so far
  float* row_loss;
  double* ed_partial;
  size_t workspace_bytes;
  // bookkeeping
  int64_t launches;
  bool profiling;
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> event_pool;
  std::vector<float> host_loss;  // staging for pbt_step_host
  double prof_ms[kNumClasses];
  int64_t prof_n[kNumClasses];
  cudaGraphExec_t step_graph;
  int64_t graph_nodes;  // kernels in one captured step
  bool graph_failed;
  char err[512];
};

namespace {

int fail(pbt_t* p, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  snprintf(g_err, sizeof(g_err), "%s", buf);
  if (p) snprintf(p->err, sizeof(p->err), "%s", buf);
  return code;
}

}  // namespace
namespace pbt {
void set_last_error(const char* msg) { snprintf(g_err, sizeof(g_err), "%s", msg); }
namespace {
bool g_serial_launches = true;
}
void set_serial_launches(bool serial) { g_serial_launches = serial; }
bool serial_launches() { return g_serial_launches; }
}  // namespace pbt
namespace {

#define CU(p, expr)                                                                                   \
  do {                                                                                                \
    cudaError_t e_ = (expr);                                                                          \
    if (e_ != cudaSuccess) return fail(p, PBT_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_));     \
  } while (0)

const int kOne = 1;   // source of small asynchronous host-to-device copies: must outlive the call

long long pad32(long long n) { return (n + 31) / 32 * 32; }
size_t align256(size_t n) { return (n + 255) / 256 * 256; }

int validate(const pbt_spec* s) {
  if (!s) return fail(nullptr, PBT_ERR_INVALID_ARG, "spec is NULL");
  if (s->n_members < 1 || s->n_members > 1024) return fail(nullptr, PBT_ERR_INVALID_ARG, "n_members must be in [1, 1024]");
  if (s->nh < 0 || s->nh > PBT_MAX_NH) return fail(nullptr, PBT_ERR_INVALID_ARG, "nh must be in [0, %d]", PBT_MAX_NH);
  if (s->trunc_num < 0 || s->trunc_den < 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "bad truncation fraction");
  if (s->exploit_rule < 0 || s->exploit_rule > 2) return fail(nullptr, PBT_ERR_INVALID_ARG, "unknown exploit rule");
  if (s->explore_rule != 0 && s->explore_rule != 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "unknown explore rule");
  if (s->exploit_rule == 2 && !(s->ttest_alpha > 0.0 && s->ttest_alpha < 1.0))
    return fail(nullptr, PBT_ERR_INVALID_ARG, "ttest_alpha must lie in (0, 1)");
  if (s->explore_rule == 1) {
    if (!(s->resample_prob >= 0.0 && s->resample_prob <= 1.0)) return fail(nullptr, PBT_ERR_INVALID_ARG, "resample_prob must lie in [0, 1]");
    for (int k = 0; k < s->nh; ++k) {
      const int kind = s->prior_kind[k];
      if (kind < PBT_PRIOR_FIXED || kind > PBT_PRIOR_LOG_UNIFORM) return fail(nullptr, PBT_ERR_INVALID_ARG, "unknown prior kind");
      if (kind != PBT_PRIOR_FIXED && !(s->prior_lo[k] <= s->prior_hi[k])) return fail(nullptr, PBT_ERR_INVALID_ARG, "prior range is empty");
      if (kind == PBT_PRIOR_LOG_UNIFORM && !(s->prior_lo[k] > 0.0)) return fail(nullptr, PBT_ERR_INVALID_ARG, "log-uniform prior needs lo > 0");
    }
  }
  const int slots[5] = {s->slot_lr, s->slot_lr_d, s->slot_momentum, s->slot_beta1, s->slot_wd};
  for (int i = 0; i < 5; ++i)
    if (slots[i] < -1 || slots[i] >= s->nh) return fail(nullptr, PBT_ERR_INVALID_ARG, "hyperparameter slot out of range");
  if (s->backward_streams < 0 || s->backward_streams > 2)
    return fail(nullptr, PBT_ERR_INVALID_ARG, "backward_streams must be 0 (automatic), 1 or 2");
  if (s->member_base < 0 || s->n_global < 0 || s->n_global > 1024 ||
      (s->n_global == 0 && s->member_base != 0) || (s->n_global > 0 && s->member_base + s->n_members > s->n_global))
    return fail(nullptr, PBT_ERR_INVALID_ARG, "member_base / n_global do not describe a shard of a population of at most 1024 members");
  if (s->model == PBT_TOY_QUADRATIC) {
    if (s->dtype != PBT_FP64_TOY) return fail(nullptr, PBT_ERR_UNSUPPORTED, "the toy model runs in fp64 only");
    if (s->nh < 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "toy model needs nh >= 1");
    return PBT_OK;
  }
  if (s->model != PBT_MLP && s->model != PBT_GAN_PAIR) return fail(nullptr, PBT_ERR_INVALID_ARG, "unknown model");
  if (s->dtype != PBT_FP32 && s->dtype != PBT_BF16_FP32MASTER)
    return fail(nullptr, PBT_ERR_UNSUPPORTED, "networks run in fp32 or bf16 with fp32 masters");
  if (s->optimizer != PBT_OPT_SGD_PLAIN && s->optimizer != PBT_OPT_SGDM && s->optimizer != PBT_OPT_ADAM &&
      s->optimizer != PBT_OPT_RMSPROP)
    return fail(nullptr, PBT_ERR_UNSUPPORTED, "network optimiser must be plain SGD, SGD-momentum, RMSProp or Adam");
  const int ns = s->model == PBT_GAN_PAIR ? 2 : 1;
  for (int k = 0; k < ns; ++k) {
    if (s->n_layers[k] < 1 || s->n_layers[k] > PBT_MAX_LAYERS) return fail(nullptr, PBT_ERR_INVALID_ARG, "n_layers out of range");
    for (int l = 0; l <= s->n_layers[k]; ++l)
      if (s->widths[k][l] < 1 || s->widths[k][l] > 65536) return fail(nullptr, PBT_ERR_INVALID_ARG, "layer width out of range");
  }
  if (s->batch < 1 || s->eval_batch < 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "batch sizes must be positive");
  if (s->pool_rows < s->batch) return fail(nullptr, PBT_ERR_INVALID_ARG, "pool smaller than one batch");
  if (s->model == PBT_GAN_PAIR) {
    if (s->loss != PBT_LOSS_GAN_LOGISTIC && s->loss != PBT_LOSS_WGAN_GP)
      return fail(nullptr, PBT_ERR_UNSUPPORTED, "GAN pairs use the logistic losses or WGAN-GP");
    if (s->loss == PBT_LOSS_WGAN_GP && !(s->gp_lambda >= 0.0)) return fail(nullptr, PBT_ERR_INVALID_ARG, "gp_lambda must be >= 0");
    if (s->widths[1][0] != s->widths[0][s->n_layers[0]]) return fail(nullptr, PBT_ERR_INVALID_ARG, "discriminator input != generator output");
    if (s->widths[1][s->n_layers[1]] != 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "discriminator must end in one logit");
    if (s->widths[0][s->n_layers[0]] != 2) return fail(nullptr, PBT_ERR_UNSUPPORTED, "GAN evaluation (energy distance to the ring) is two-dimensional");
    if (s->gan_d_steps < 1 || s->gan_d_steps > 64) return fail(nullptr, PBT_ERR_INVALID_ARG, "gan_d_steps out of range");
    if (s->optimizer != PBT_OPT_ADAM) return fail(nullptr, PBT_ERR_UNSUPPORTED, "GAN pairs use Adam");
  } else {
    if (s->loss != PBT_LOSS_MSE && s->loss != PBT_LOSS_CE_HARD && s->loss != PBT_LOSS_CE_SOFT)
      return fail(nullptr, PBT_ERR_UNSUPPORTED, "MLP loss must be MSE or cross-entropy");
  }
  return PBT_OK;
}

// Fills the layout-dependent fields of h and assigns workspace pointers starting at base
// (base may be NULL: sizes only).  Returns the bytes needed.
size_t plan(pbt_handle* h, char* base) {
  const pbt_spec& s = h->spec;
  h->N = s.n_members;
  h->nh = s.nh;
  h->toy = s.model == PBT_TOY_QUADRATIC;
  h->gan = s.model == PBT_GAN_PAIR;
  h->is_bf16 = s.dtype == PBT_BF16_FP32MASTER;
  h->cdt = h->is_bf16 ? kBF16 : kF32;
  h->esz = h->is_bf16 ? 2 : 4;
  h->ns = h->toy ? 0 : (h->gan ? 2 : 1);
  h->wgan = h->gan && s.loss == PBT_LOSS_WGAN_GP;
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    char* p = base ? base + off : nullptr;
    off += align256(bytes);
    return p;
  };
  const size_t N = h->N;
  h->counters = (Counters*)take(sizeof(Counters));
  h->tm = (long long*)take(N * sizeof(long long));
  h->member_base = s.member_base;
  h->g_fit = h->g_H = nullptr; h->g_src = h->g_level = nullptr;
  h->g_hist = nullptr; h->g_hist_n = nullptr;
  if (s.n_global > 0) {
    const size_t G = s.n_global;
    h->g_fit = take(G * sizeof(double));
    h->g_H = take(G * PBT_MAX_NH * sizeof(double));
    h->g_src = (int*)take(G * sizeof(int));
    h->g_level = (int*)take(G * sizeof(int));
    h->g_hist = take(G * PBT_HISTORY * sizeof(double));
    h->g_hist_n = (int*)take(G * sizeof(int));
  }
  h->src = (int*)take(N * sizeof(int));
  h->level = (int*)take(N * sizeof(int));
  h->H = take(N * PBT_MAX_NH * sizeof(double));
  h->fitness = take(N * sizeof(double));
  h->hist = take(N * PBT_HISTORY * sizeof(double));
  h->hist_n = (int*)take(N * sizeof(int));
  h->last_loss = (float*)take(N * 2 * sizeof(float));
  h->scalars = (float*)take(N * PBT_N_SCALARS * sizeof(float));
  h->win_off = (int*)take(N * sizeof(int));
  h->direct_pool = false;
  if (h->toy) {
    h->P = s.nh;
    h->P_pad = s.nh;
    h->theta = (double*)take(N * s.nh * sizeof(double));
    h->workspace_bytes = off;
    return off;
  }
  long long p = 0, flat = 0;
  h->max_width = 1;
  for (int k = 0; k < h->ns; ++k) {
    Stack& st = h->st[k];
    st.nl = s.n_layers[k];
    st.begin = p;
    for (int l = 0; l < st.nl; ++l) {
      Layer& L = st.L[l];
      L.in = s.widths[k][l];
      L.out = s.widths[k][l + 1];
      L.w_off = p;
      p += pad32((long long)L.in * L.out);
      L.b_off = p;
      p += pad32(L.out);
      flat += (long long)L.in * L.out + L.out;
      if (L.in > h->max_width) h->max_width = L.in;
      if (L.out > h->max_width) h->max_width = L.out;
    }
    st.count = p - st.begin;
  }
  h->P = flat;
  h->P_pad = p;
  if (h->gan) {
    h->st[0].rows_cap = s.batch > s.eval_batch ? s.batch : s.eval_batch;
    h->st[1].rows_cap = (h->wgan ? 3 : 2) * s.batch;   // real, generated (and interpolated) rows
    h->dz_rows_cap = 2 * s.batch;
  } else {
    h->st[0].rows_cap = s.batch > s.eval_batch ? s.batch : s.eval_batch;
    h->dz_rows_cap = s.batch;
  }
  h->rowloss_cap = h->dz_rows_cap > s.eval_batch ? h->dz_rows_cap : s.eval_batch;
  if (h->wgan && h->rowloss_cap < 3 * s.batch) h->rowloss_cap = 3 * s.batch;
  const size_t slab = (size_t)h->P_pad * sizeof(float);
  h->W32 = (float*)take(N * slab);
  h->O1 = (float*)take(N * slab);
  h->O2 = s.optimizer == PBT_OPT_ADAM ? (float*)take(N * slab) : nullptr;
  h->G = (float*)take(N * slab);
  h->W16 = h->is_bf16 ? (bf16*)take(N * (size_t)h->P_pad * 2) : nullptr;
  for (int k = 0; k < h->ns; ++k) {
    Stack& st = h->st[k];
    for (int l = 0; l < st.nl; ++l) {
      // layer 0 of an MLP / generator only ever holds training rows (evaluation reads the held-out set in place)
      const int rows = (l == 0 && k == 0) ? s.batch : st.rows_cap;
      h->act[k][l] = take(N * (size_t)rows * st.L[l].in * h->esz);
    }
    h->logits[k] = (float*)take(N * (size_t)st.rows_cap * st.L[st.nl - 1].out * sizeof(float));
  }
  for (int i = 0; i < 2; ++i) h->dz[i] = take(N * (size_t)h->dz_rows_cap * h->max_width * h->esz);
  h->gp_gx = nullptr;
  if (h->wgan) {
    for (int l = 0; l < h->st[1].nl; ++l) h->gp_dz[l] = take(N * (size_t)3 * s.batch * h->st[1].L[l].out * h->esz);
    h->gp_gx = (float*)take(N * (size_t)s.batch * h->st[1].L[0].in * sizeof(float));
  }
  if (!h->gan) {
    const int out = h->st[0].L[h->st[0].nl - 1].out;
    if (s.loss == PBT_LOSS_MSE) h->ybatch_stride = (long long)s.batch * out;
    else if (s.loss == PBT_LOSS_CE_HARD) h->ybatch_stride = s.batch;
    else h->ybatch_stride = (long long)s.batch * out;
    const size_t tsz = s.loss == PBT_LOSS_CE_SOFT ? h->esz : 4;
    h->ybatch_stride = (h->ybatch_stride * tsz + 15) / 16 * 16 / tsz;
    h->ybatch = take(N * (size_t)h->ybatch_stride * tsz);
    h->ybatch_alt = take(N * (size_t)h->ybatch_stride * tsz);
    h->act0_alt = take(N * (size_t)s.batch * h->st[0].L[0].in * h->esz);
  } else {
    h->ybatch = nullptr;
    h->ybatch_alt = nullptr;
    h->act0_alt = nullptr;
    h->ybatch_stride = 0;
  }
  if (!h->gan && h->is_bf16) {
    const Layer& L0 = h->st[0].L[0];
    h->direct_pool = s.batch >= 128 && s.batch % 64 == 0 && L0.in >= 128 && L0.out >= 128 && L0.in % 8 == 0 &&
                     L0.out % 8 == 0 && h->data.x_pool && (((uintptr_t)h->data.x_pool) & 15) == 0 &&
                     h->data.y_pool && (((uintptr_t)h->data.y_pool) & 15) == 0;
  }
  h->row_loss = (float*)take(N * (size_t)h->rowloss_cap * sizeof(float));
  h->ed_partial = h->gan ? (double*)take(N * (size_t)energy_partial_count(s.eval_batch) * sizeof(double)) : nullptr;
  h->workspace_bytes = off;
  return off;
}

long long act_stride(const pbt_handle* h, int k, int l) {
  const Stack& st = h->st[k];
  const int rows = (l == 0 && k == 0) ? h->spec.batch : st.rows_cap;
  return (long long)rows * st.L[l].in;
}
long long logits_stride(const pbt_handle* h, int k) {
  const Stack& st = h->st[k];
  return (long long)st.rows_cap * st.L[st.nl - 1].out;
}
long long dz_stride(const pbt_handle* h) { return (long long)h->dz_rows_cap * h->max_width; }

StepClock clock(const pbt_handle* h) { return StepClock{h->tm, h->member_base}; }

// A member window: for the duration of a subset step the handle's per-member STATE pointers refer to members
// [first, first + count) only, so that every launch of the step machinery covers just those members.  The scratch
// buffers (activations, deltas, row losses, window offsets) are not shifted: the window uses their first `count`
// member slots.  Kernels that need a member's population index (counter-based draws) add member_base.
struct MemberWindow {
  int N, member_base;
  float *W32, *O1, *O2, *G, *scalars, *last_loss;
  bf16* W16;
  void* H;
  double* theta;
  long long* tm;
};

MemberWindow open_window(pbt_handle* h, int first, int count) {
  MemberWindow w{h->N, h->member_base, h->W32, h->O1, h->O2, h->G, h->scalars, h->last_loss, h->W16, h->H, h->theta, h->tm};
  const size_t f = (size_t)first;
  if (h->W32) h->W32 += f * h->P_pad;
  if (h->O1) h->O1 += f * h->P_pad;
  if (h->O2) h->O2 += f * h->P_pad;
  if (h->G) h->G += f * h->P_pad;
  if (h->W16) h->W16 += f * h->P_pad;
  h->scalars += f * PBT_N_SCALARS;
  h->last_loss += f * 2;
  h->H = (char*)h->H + f * PBT_MAX_NH * (h->toy ? 8 : 4);
  if (h->theta) h->theta += f * h->nh;
  h->tm += f;
  h->N = count;
  h->member_base += first;
  return w;
}

void close_window(pbt_handle* h, const MemberWindow& w) {
  h->N = w.N; h->member_base = w.member_base;
  h->W32 = w.W32; h->O1 = w.O1; h->O2 = w.O2; h->G = w.G; h->scalars = w.scalars; h->last_loss = w.last_loss;
  h->W16 = w.W16; h->H = w.H; h->theta = w.theta; h->tm = w.tm;
}

// ----- launch bookkeeping -----------------------------------------------------
cudaEvent_t get_event(pbt_handle* h) {
  if (!h->event_pool.empty()) {
    cudaEvent_t e = h->event_pool.back();
    h->event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct LaunchScope {
  pbt_handle* h;
  int cls;
  cudaEvent_t a, b;
  LaunchScope(pbt_handle* h_, int cls_) : h(h_), cls(cls_), a(nullptr), b(nullptr) {
    h->launches++;
    if (h->profiling) {
      a = get_event(h);
      b = get_event(h);
      cudaEventRecord(a, h->ls);
    }
  }
  ~LaunchScope() {
    if (h->profiling) {
      cudaEventRecord(b, h->ls);
      h->prof.push_back(ProfRec{cls, a, b});
    }
  }
};

#define LAUNCH(h, cls, expr)                                                                        \
  do {                                                                                              \
    cudaError_t e_;                                                                                 \
    {                                                                                               \
      LaunchScope scope_(h, cls);                                                                   \
      e_ = (expr);                                                                                  \
    }                                                                                               \
    if (e_ != cudaSuccess) return fail(h, PBT_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_));   \
  } while (0)

int gemm(pbt_handle* h, const GemmArgs& g) {
  if (g.adam) {
    LAUNCH(h, kFused, launch_wgrad_adam(g, h->counters, h->ls));
  } else if (gemm_tc_pair_preferred(g)) {
    LAUNCH(h, kGemm, launch_gemm_tc_pair(g, h->counters, h->ls));
  } else if (gemm_tc_supported(g)) {
    LAUNCH(h, kGemm, launch_gemm_tc(g, h->counters, h->ls));
  } else {
    if (g.a_rowoff || g.b_rowoff) return fail(h, PBT_ERR_UNSUPPORTED, "row-window operands need a tensor-core shape");
    LAUNCH(h, kGemm, launch_gemm_simt(g, h->ls));
  }
  return PBT_OK;
}

// Work enqueued between fork_side() and the matching join_side() may be sent to the side stream by wrapping it in
// a SideScope: it then depends on everything in the handle's stream up to the fork, and everything enqueued in
// the handle's stream after the join depends on it.  In a stream capture the two become parallel branches of the
// graph.  The side stream is in order, so the work of successive forks never overlaps itself.
bool fork_side(pbt_handle* h) {
  if (!h->side || h->profiling) return false;   // per-launch timing wants every launch alone on the GPU
  cudaEventRecord(h->ev_fork, h->stream);
  cudaStreamWaitEvent(h->side, h->ev_fork, 0);
  h->side_pending = true;
  return true;
}
void join_side(pbt_handle* h) {
  cudaEventRecord(h->ev_join, h->side);
  cudaStreamWaitEvent(h->stream, h->ev_join, 0);
  h->side_pending = false;
}
struct SideScope {
  pbt_handle* h;
  SideScope(pbt_handle* h_, bool on) : h(h_) { if (on) h->ls = h->side; }
  ~SideScope() { h->ls = h->stream; }
};

const void* weights(const pbt_handle* h, long long off) {
  return h->is_bf16 ? (const void*)(h->W16 + off) : (const void*)(h->W32 + off);
}

// z_l = a_{l-1} W_l^T + b_l, ReLU on hidden layers; the last layer's output goes to logits[k] in fp32
// With in_rowoff the input rows of member m are rows in_rowoff[m].. of `in`, a pool of in_rows_total rows.
int forward(pbt_handle* h, int k, int rows, const void* in, long long in_stride, const int* in_rowoff = nullptr,
            long long in_rows_total = 0) {
  const Stack& st = h->st[k];
  for (int l = 0; l < st.nl; ++l) {
    const Layer& L = st.L[l];
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = rows; g.N = L.out; g.K = L.in; g.batch = h->N;
    g.in_dtype = h->cdt;
    g.A = l == 0 ? in : h->act[k][l];
    g.lda = L.in;
    g.strideA = l == 0 ? in_stride : act_stride(h, k, l);
    if (l == 0 && in_rowoff) { g.a_rowoff = in_rowoff; g.a_rows_total = in_rows_total; g.strideA = 0; }
    g.B = weights(h, L.w_off); g.ldb = L.in; g.strideB = h->P_pad;
    g.bias = h->W32 + L.b_off; g.strideBias = h->P_pad;
    if (l + 1 < st.nl) {
      g.C = h->act[k][l + 1]; g.ldc = L.out; g.strideC = act_stride(h, k, l + 1);
      g.out_dtype = h->cdt; g.relu = 1;
    } else {
      g.C = h->logits[k]; g.ldc = L.out; g.strideC = logits_stride(h, k);
      g.out_dtype = kF32; g.relu = 0;
    }
    int rc = gemm(h, g);
    if (rc) return rc;
  }
  return PBT_OK;
}

void fill_opt_args(pbt_handle* h, OptArgs* a, int slot_lr, int scalar_base) {
  const pbt_spec& s = h->spec;
  memset(a, 0, sizeof(*a));
  a->n_members = h->N; a->p_pad = h->P_pad;
  a->w32 = h->W32; a->opt1 = h->O1; a->opt2 = h->O2; a->grad = h->G; a->w16 = h->W16;
  a->H = (const float*)h->H; a->nh_stride = PBT_MAX_NH;
  a->slot_lr = slot_lr; a->slot_momentum = s.slot_momentum; a->slot_beta1 = s.slot_beta1; a->slot_wd = s.slot_wd;
  a->const_lr = (float)s.const_lr; a->const_momentum = (float)s.const_momentum; a->const_beta1 = (float)s.const_beta1;
  a->const_beta2 = (float)s.const_beta2; a->const_eps = (float)s.const_eps; a->const_wd = (float)s.const_wd;
  a->scalars = h->scalars; a->scalar_base = scalar_base;
}

// dC = (dZ_l W_l) [* (mask > 0)]: the data gradient of layer l of stack k for `rows` rows per member.
int dgrad(pbt_handle* h, int k, int l, int rows, const void* dz, long long dz_stride, void* out, long long out_stride,
          int out_dtype, const void* mask, long long mask_stride) {
  const Layer& L = h->st[k].L[l];
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.M = rows; g.N = L.in; g.K = L.out; g.batch = h->N;
  g.in_dtype = h->cdt; g.out_dtype = out_dtype;
  g.A = dz; g.lda = L.out; g.strideA = dz_stride;
  g.B = weights(h, L.w_off); g.ldb = L.in; g.strideB = h->P_pad; g.b_mn = 1;
  g.C = out; g.ldc = L.in; g.strideC = out_stride;
  if (mask) { g.mask = mask; g.ldmask = L.in; g.strideMask = mask_stride; }
  return gemm(h, g);
}

// dW_l = dZ_l^T a_{l-1} over `rows` rows and db_l = column sums of the first `bias_rows` rows of dZ_l.
// Layers whose weight gradient runs on the tensor cores get their Adam update inside that GEMM's epilogue
// (the caller must have finished every read of the layer's old weights); fused[l] records it.
int wgrad_layer(pbt_handle* h, int k, int l, int rows, int bias_rows, const void* dz, long long dz_stride,
                const void* in, long long in_stride, const OptArgs& opt, bool* fused, const int* in_rowoff = nullptr,
                long long in_rows_total = 0, bool forked = false, bool gemm_on_side = true, bool* bias_done = nullptr) {
  // forked: the caller has forked the side stream where dz was complete; the bias gradient goes there, and so
  // does an unfused weight gradient if gemm_on_side (a fused one stays in the handle's stream, behind the data
  // gradient that reads the old weights)
  const pbt_spec& s = h->spec;
  const Layer& L = h->st[k].L[l];
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.M = L.out; g.N = L.in; g.K = rows; g.batch = h->N;
  g.in_dtype = h->cdt; g.out_dtype = kF32;
  g.A = dz; g.lda = L.out; g.strideA = dz_stride; g.a_mn = 1;
  g.B = in; g.ldb = L.in; g.strideB = in_stride; g.b_mn = 1;
  if (in_rowoff) { g.b_rowoff = in_rowoff; g.b_rows_total = in_rows_total; g.strideB = 0; }
  g.C = h->G + L.w_off; g.ldc = L.in; g.strideC = h->P_pad;
  OptArgs lopt = opt;
  if (s.fuse_adam && s.optimizer == PBT_OPT_ADAM && gemm_tc_supported(g)) {
    lopt.begin = L.w_off; lopt.count = (long long)L.in * L.out;
    g.adam = &lopt;
    if (!s.keep_grad) g.C = nullptr;
    fused[l] = true;
  }
  {
    SideScope side(h, forked && gemm_on_side && !g.adam);
    int rc = gemm(h, g);
    if (rc) return rc;
  }
  SideScope side(h, forked);
  LAUNCH(h, kLoss, launch_bias_grad(dz, h->cdt, L.out, dz_stride, bias_rows, L.out, h->G + L.b_off, h->P_pad, h->N, h->ls));
  if (forked && bias_done && g.adam) {
    // the layer's weights are updated by the fused launch: its bias vector is the whole of what is left, nothing
    // in the backward pass reads it, and its gradient is complete in this stream: update it here, off the
    // critical path, instead of in a launch of its own after the pass
    const Stack& st = h->st[k];
    OptArgs a = opt;
    a.begin = L.b_off;
    a.count = (l + 1 < st.nl ? st.L[l + 1].w_off : st.begin + st.count) - L.b_off;
    LAUNCH(h, kOpt, launch_adam(a, h->ls));
    bias_done[l] = true;
  }
  return PBT_OK;
}

// element-wise optimiser over what the fused epilogues did not cover (biases, skinny layers, SGD-momentum,
// RMSProp); adjacent slab ranges are merged into one launch
int finish_optimizer(pbt_handle* h, int k, const bool* fused, const OptArgs& opt, const bool* bias_done = nullptr) {
  const pbt_spec& s = h->spec;
  const Stack& st = h->st[k];
  long long rb = -1, re = -1;
  auto flush = [&]() -> int {
    if (rb < 0) return PBT_OK;
    OptArgs a = opt;
    a.begin = rb; a.count = re - rb;
    rb = re = -1;
    if (s.optimizer == PBT_OPT_SGD_PLAIN) { LAUNCH(h, kOpt, launch_sgd(a, h->stream)); }
    else if (s.optimizer == PBT_OPT_SGDM) { LAUNCH(h, kOpt, launch_sgdm(a, h->stream)); }
    else if (s.optimizer == PBT_OPT_RMSPROP) { LAUNCH(h, kOpt, launch_rmsprop(a, h->stream)); }
    else { LAUNCH(h, kOpt, launch_adam(a, h->stream)); }
    return PBT_OK;
  };
  for (int l = 0; l < st.nl; ++l) {
    const Layer& L = st.L[l];
    const long long w_end = L.b_off, b_end = l + 1 < st.nl ? st.L[l + 1].w_off : st.begin + st.count;
    if (!fused[l]) {
      if (rb < 0) rb = L.w_off;
      re = w_end;
    } else {
      int rc = flush();
      if (rc) return rc;
    }
    if (bias_done && bias_done[l]) {
      int rc = flush();
      if (rc) return rc;
      continue;
    }
    if (rb < 0) rb = L.b_off;
    re = b_end;
  }
  int rc = flush();
  if (rc) return rc;
  if (s.optimizer == PBT_OPT_ADAM) LAUNCH(h, kOther, launch_adam_advance(opt, h->stream));
  return PBT_OK;
}

// dW_l = dZ_l^T a_{l-1}, db_l = column sums of dZ_l, dZ_{l-1} = (dZ_l W_l) * [a_{l-1} > 0].
// dZ of the last layer is in h->dz[*cur]; on return *cur names the buffer written last.
// With need_wgrad the optimiser update of the stack is part of this pass: a layer's fused update runs
// after the layer's data gradient has read the old weights.
int backward(pbt_handle* h, int k, int rows, const void* in, long long in_stride, bool need_wgrad,
             bool need_input_grad, int* cur, int slot_lr, int scalar_base, const int* in_rowoff = nullptr,
             long long in_rows_total = 0) {
  const Stack& st = h->st[k];
  const long long dzs = dz_stride(h);
  OptArgs opt;
  fill_opt_args(h, &opt, slot_lr, scalar_base);
  bool fused[PBT_MAX_LAYERS] = {false}, bias_done[PBT_MAX_LAYERS] = {false};
  for (int l = st.nl - 1; l >= 0; --l) {
    const void* dz = h->dz[*cur];
    bool wrote_dgrad = false;
    // dz is complete here: what else reads it may run beside the data gradient; it is joined before the next
    // layer's data gradient overwrites dz
    const bool forked = need_wgrad && fork_side(h);
    if (l > 0 || need_input_grad) {
      int rc = dgrad(h, k, l, rows, dz, dzs, h->dz[1 - *cur], dzs, h->cdt, l > 0 ? h->act[k][l] : nullptr,
                     l > 0 ? act_stride(h, k, l) : 0);
      if (rc) return rc;
      wrote_dgrad = true;
    }
    if (need_wgrad) {
      int rc = wgrad_layer(h, k, l, rows, rows, dz, dzs, l == 0 ? in : h->act[k][l],
                           l == 0 ? in_stride : act_stride(h, k, l), opt, fused, l == 0 ? in_rowoff : nullptr,
                           in_rows_total, forked, wrote_dgrad, bias_done);
      if (forked) join_side(h);
      if (rc) return rc;
    }
    if (wrote_dgrad) *cur = 1 - *cur;
  }
  if (!need_wgrad) return PBT_OK;
  return finish_optimizer(h, k, fused, opt, bias_done);
}

int loss_and_dz(pbt_handle* h, int k, int rows, int n_real, const void* target, long long target_stride,
                bool want_dz, int dz_buf, float scale, void* out, int out_stride, const int* target_rowoff = nullptr) {
  const pbt_spec& s = h->spec;
  const Stack& st = h->st[k];
  LossArgs a;
  memset(&a, 0, sizeof(a));
  a.kind = s.loss; a.n_members = h->N; a.rows = rows; a.cols = st.L[st.nl - 1].out;
  a.n_real_rows = n_real; a.inv_batch = 1.0f / (float)s.batch;
  a.logits = h->logits[k]; a.ld_logits = a.cols; a.stride_logits = logits_stride(h, k);
  a.target = target; a.stride_target = target_stride; a.target_rowoff = target_rowoff;
  a.target_dtype = s.loss == PBT_LOSS_CE_SOFT ? h->cdt : kF32;
  a.dz = want_dz ? h->dz[dz_buf] : nullptr; a.dz_dtype = h->cdt; a.ld_dz = a.cols; a.stride_dz = dz_stride(h);
  a.row_loss = h->row_loss;
  LAUNCH(h, kLoss, launch_loss_rows(a, h->stream));
  // With deltas wanted, a backward pass follows that waits for the deltas only: the reduction of the row losses to
  // the member's loss runs beside it (joined with the pass's first join, at the latest when the step ends; the
  // next writer of row_loss is a later loss kernel in the handle's stream, behind that join).
  SideScope side(h, want_dz && fork_side(h));
  LAUNCH(h, kLoss, launch_reduce_rows(h->row_loss, rows, h->N, scale, out, 0, out_stride, h->ls));
  return PBT_OK;
}

size_t target_row_bytes(const pbt_handle* h) {
  const pbt_spec& s = h->spec;
  const int out = h->st[0].L[h->st[0].nl - 1].out;
  if (s.loss == PBT_LOSS_MSE) return (size_t)out * 4;
  if (s.loss == PBT_LOSS_CE_HARD) return 4;
  return (size_t)out * h->esz;
}

int step_mlp(pbt_handle* h) {
  const pbt_spec& s = h->spec;
  const Stack& st = h->st[0];
  const int in = st.L[0].in;
  if (h->direct_pool && !h->supplied_next) {
    // the first layer's forward and weight-gradient GEMMs and the loss read the window of each member in place
    LAUNCH(h, kCopy, launch_window_offsets(h->win_off, s.batch, s.pool_rows, h->N, 0, 0, h->seed, clock(h), h->stream));
    int rc = forward(h, 0, s.batch, h->data.x_pool, 0, h->win_off, s.pool_rows);
    if (rc) return rc;
    rc = loss_and_dz(h, 0, s.batch, s.batch, h->data.y_pool, 0, true, 0, 1.0f / s.batch, h->last_loss, 2, h->win_off);
    if (rc) return rc;
    int cur = 0;
    return backward(h, 0, s.batch, h->data.x_pool, 0, true, false, &cur, s.slot_lr, 0, h->win_off, s.pool_rows);
  }
  LAUNCH(h, kCopy, launch_gather_window((char*)h->act[0][0], act_stride(h, 0, 0) * h->esz, 0, (const char*)h->data.x_pool,
                                        in * h->esz, s.batch, s.pool_rows, h->N, 0, 0, h->seed, h->counters, clock(h), h->stream));
  const size_t trb = target_row_bytes(h);
  const size_t tsz = s.loss == PBT_LOSS_CE_SOFT ? h->esz : 4;
  // the targets are needed by the loss only: their gather runs beside the forward pass
  const bool forked = fork_side(h);
  {
    SideScope side(h, forked);
    LAUNCH(h, kCopy, launch_gather_window((char*)h->ybatch, h->ybatch_stride * tsz, 0, (const char*)h->data.y_pool, (int)trb,
                                          s.batch, s.pool_rows, h->N, 0, 0, h->seed, h->counters, clock(h), h->ls));
  }
  int rc = forward(h, 0, s.batch, h->act[0][0], act_stride(h, 0, 0));
  if (forked) join_side(h);
  if (rc) return rc;
  rc = loss_and_dz(h, 0, s.batch, s.batch, h->ybatch, h->ybatch_stride, true, 0, 1.0f / s.batch, h->last_loss, 2);
  if (rc) return rc;
  int cur = 0;
  return backward(h, 0, s.batch, h->act[0][0], act_stride(h, 0, 0), true, false, &cur, s.slot_lr, 0);
}

// Section 4.3.1: K discriminator updates, then one generator update.
int step_gan(pbt_handle* h) {
  const pbt_spec& s = h->spec;
  const int B = s.batch;
  const int zdim = h->st[0].L[0].in, xdim = h->st[1].L[0].in;
  const long long d_in_stride = act_stride(h, 1, 0);
  int rc;
  for (int j = 0; j <= s.gan_d_steps; ++j) {
    const bool d_phase = j < s.gan_d_steps;
    // the real rows are needed by the discriminator only: their gather runs beside the generator's forward pass
    const bool forked = d_phase && fork_side(h);
    if (d_phase) {
      SideScope side(h, forked);
      LAUNCH(h, kCopy, launch_gather_window((char*)h->act[1][0], d_in_stride * h->esz, 0, (const char*)h->data.x_pool,
                                            xdim * h->esz, B, s.pool_rows, h->N, j, 0, h->seed, h->counters, clock(h), h->ls));
    }
    LAUNCH(h, kCopy, launch_gather_window((char*)h->act[0][0], act_stride(h, 0, 0) * h->esz, 0, (const char*)h->data.z_pool,
                                          zdim * h->esz, B, s.pool_rows, h->N, j, 1, h->seed, h->counters, clock(h), h->stream));
    rc = forward(h, 0, B, h->act[0][0], act_stride(h, 0, 0));
    if (forked) join_side(h);
    if (rc) return rc;
    // generated samples become discriminator input rows (after the real rows in a discriminator update)
    char* fake_dst = (char*)h->act[1][0] + (d_phase ? (size_t)B * xdim * h->esz : 0);
    LAUNCH(h, kCopy, launch_copy_rows(fake_dst, h->cdt, xdim, d_in_stride, h->logits[0], xdim, logits_stride(h, 0), B, xdim,
                                      h->N, h->stream));
    const int rows = d_phase ? 2 * B : B;
    rc = forward(h, 1, rows, h->act[1][0], d_in_stride);
    if (rc) return rc;
    rc = loss_and_dz(h, 1, rows, B, nullptr, 0, true, 0, 1.0f / B, h->last_loss + (d_phase ? 1 : 0), 2);
    if (rc) return rc;
    int cur = 0;
    if (d_phase) {
      rc = backward(h, 1, rows, h->act[1][0], d_in_stride, true, false, &cur, s.slot_lr_d, 2);
      if (rc) return rc;
    } else {
      rc = backward(h, 1, rows, h->act[1][0], d_in_stride, false, true, &cur, s.slot_lr_d, 2);
      if (rc) return rc;
      rc = backward(h, 0, B, h->act[0][0], act_stride(h, 0, 0), true, false, &cur, s.slot_lr, 0);
      if (rc) return rc;
    }
  }
  return PBT_OK;
}

// Section 4.3.1 with the paper's own objective (WGAN-GP): K critic updates, then one generator update on
// L_G = -mean D(G(z)).  A critic update sends three row blocks per member through the critic: real rows,
// generated rows and their interpolates xhat.  Back-propagation of all three is one chain of data-gradient
// GEMMs over 3B rows (the interpolates start from dD/dD = 1, so their deltas u_l are the factors of the input
// gradient grad_x D(xhat) = u_0 W_0).  The penalty's gradient with respect to W_l is u_l^T dv_l with a second,
// forward-running chain dv_0 = d(penalty)/d(grad_x D), dv_{l+1} = (dv_l W_l^T) * [a_{l+1}(xhat) > 0].  dv_l
// overwrites the interpolates' rows of layer l's input, which nothing reads any more (each element is the
// ReLU mask of exactly the element that replaces it, read by the thread that then writes it), so that ONE
// weight-gradient GEMM over 3B rows gives  dZ_l^T a_{l-1} (real, generated rows) + u_l^T dv_l.
int step_wgan(pbt_handle* h) {
  const pbt_spec& s = h->spec;
  const int B = s.batch;
  const Stack& G = h->st[0];
  const Stack& D = h->st[1];
  const int zdim = G.L[0].in, xdim = D.L[0].in;
  const long long d_in_stride = act_stride(h, 1, 0);
  const float lam = (float)s.gp_lambda;
  int rc;
  for (int j = 0; j < s.gan_d_steps; ++j) {
    LAUNCH(h, kCopy, launch_gather_window((char*)h->act[1][0], d_in_stride * h->esz, 0, (const char*)h->data.x_pool,
                                          xdim * h->esz, B, s.pool_rows, h->N, j, 0, h->seed, h->counters, clock(h), h->stream));
    LAUNCH(h, kCopy, launch_gather_window((char*)h->act[0][0], act_stride(h, 0, 0) * h->esz, 0, (const char*)h->data.z_pool,
                                          zdim * h->esz, B, s.pool_rows, h->N, j, 1, h->seed, h->counters, clock(h), h->stream));
    rc = forward(h, 0, B, h->act[0][0], act_stride(h, 0, 0));
    if (rc) return rc;
    LAUNCH(h, kCopy, launch_copy_rows((char*)h->act[1][0] + (size_t)B * xdim * h->esz, h->cdt, xdim, d_in_stride, h->logits[0],
                                      xdim, logits_stride(h, 0), B, xdim, h->N, h->stream));
    LAUNCH(h, kOther, launch_gp_interp(h->act[1][0], h->cdt, d_in_stride, B, xdim, j, h->N, h->seed, clock(h), h->stream));
    rc = forward(h, 1, 3 * B, h->act[1][0], d_in_stride);
    if (rc) return rc;
    // deltas of the last layer for all 3B rows; losses of the real and generated rows
    {
      LossArgs a;
      memset(&a, 0, sizeof(a));
      a.kind = PBT_LOSS_WGAN_GP; a.n_members = h->N; a.rows = 3 * B; a.cols = 1;
      a.n_real_rows = B; a.inv_batch = 1.0f / (float)B;
      a.logits = h->logits[1]; a.ld_logits = 1; a.stride_logits = logits_stride(h, 1);
      a.dz = h->gp_dz[D.nl - 1]; a.dz_dtype = h->cdt; a.ld_dz = 1; a.stride_dz = 3ll * B;
      a.row_loss = h->row_loss;
      LAUNCH(h, kLoss, launch_loss_rows(a, h->stream));
    }
    for (int l = D.nl - 1; l >= 1; --l) {
      rc = dgrad(h, 1, l, 3 * B, h->gp_dz[l], 3ll * B * D.L[l].out, h->gp_dz[l - 1], 3ll * B * D.L[l].in, h->cdt,
                 h->act[1][l], act_stride(h, 1, l));
      if (rc) return rc;
    }
    // grad_x D(xhat) = u_0 W_0 (kept in fp32), then the penalty and the start of its chain, dv_0, over xhat
    rc = dgrad(h, 1, 0, B, (const char*)h->gp_dz[0] + (size_t)2 * B * D.L[0].out * h->esz, 3ll * B * D.L[0].out, h->gp_gx,
               (long long)B * xdim, kF32, nullptr, 0);
    if (rc) return rc;
    LAUNCH(h, kLoss, launch_gp_penalty(h->gp_gx, (long long)B * xdim, B, xdim, lam, 1.0f / (float)B, h->row_loss, 3 * B, 2 * B,
                                       (char*)h->act[1][0] + (size_t)2 * B * xdim * h->esz, h->cdt, d_in_stride, h->N,
                                       h->stream));
    LAUNCH(h, kLoss, launch_reduce_rows(h->row_loss, 3 * B, h->N, 1.0f / (float)B, h->last_loss + 1, 0, 2, h->stream));
    for (int l = 0; l + 1 < D.nl; ++l) {
      const Layer& L = D.L[l];
      GemmArgs g;
      memset(&g, 0, sizeof(g));
      g.M = B; g.N = L.out; g.K = L.in; g.batch = h->N;
      g.in_dtype = h->cdt; g.out_dtype = h->cdt;
      g.A = (const char*)h->act[1][l] + (size_t)2 * B * L.in * h->esz; g.lda = L.in; g.strideA = act_stride(h, 1, l);
      g.B = weights(h, L.w_off); g.ldb = L.in; g.strideB = h->P_pad;
      g.C = (char*)h->act[1][l + 1] + (size_t)2 * B * L.out * h->esz; g.ldc = L.out; g.strideC = act_stride(h, 1, l + 1);
      g.mask = g.C; g.ldmask = L.out; g.strideMask = g.strideC;
      rc = gemm(h, g);
      if (rc) return rc;
    }
    OptArgs opt;
    fill_opt_args(h, &opt, s.slot_lr_d, 2);
    bool fused[PBT_MAX_LAYERS] = {false}, bias_done[PBT_MAX_LAYERS] = {false};
    // every layer's deltas are complete: the weight and bias gradients of all layers are independent launches
    const bool forked = fork_side(h);
    for (int l = D.nl - 1; l >= 0; --l) {
      rc = wgrad_layer(h, 1, l, 3 * B, 2 * B, h->gp_dz[l], 3ll * B * D.L[l].out, h->act[1][l], act_stride(h, 1, l), opt, fused,
                       nullptr, 0, forked, (l & 1) != 0, bias_done);
      if (rc) break;
    }
    if (forked) join_side(h);
    if (rc) return rc;
    rc = finish_optimizer(h, 1, fused, opt, bias_done);
    if (rc) return rc;
  }
  // generator update
  LAUNCH(h, kCopy, launch_gather_window((char*)h->act[0][0], act_stride(h, 0, 0) * h->esz, 0, (const char*)h->data.z_pool,
                                        zdim * h->esz, B, s.pool_rows, h->N, s.gan_d_steps, 1, h->seed, h->counters, clock(h), h->stream));
  rc = forward(h, 0, B, h->act[0][0], act_stride(h, 0, 0));
  if (rc) return rc;
  LAUNCH(h, kCopy, launch_copy_rows(h->act[1][0], h->cdt, xdim, d_in_stride, h->logits[0], xdim, logits_stride(h, 0), B, xdim,
                                    h->N, h->stream));
  rc = forward(h, 1, B, h->act[1][0], d_in_stride);
  if (rc) return rc;
  rc = loss_and_dz(h, 1, B, B, nullptr, 0, true, 0, 1.0f / B, h->last_loss, 2);
  if (rc) return rc;
  int cur = 0;
  rc = backward(h, 1, B, h->act[1][0], d_in_stride, false, true, &cur, s.slot_lr_d, 2);
  if (rc) return rc;
  return backward(h, 0, B, h->act[0][0], act_stride(h, 0, 0), true, false, &cur, s.slot_lr, 0);
}

int one_step(pbt_handle* h) {
  int rc;
  if (h->toy) {
    LAUNCH(h, kOpt, launch_toy_step(h->theta, (const double*)h->H, h->N, h->nh, h->spec.toy_eta, h->stream));
  } else if (h->wgan) {
    rc = step_wgan(h);
    if (rc) return rc;
  } else if (h->gan) {
    rc = step_gan(h);
    if (rc) return rc;
  } else {
    rc = step_mlp(h);
    if (rc) return rc;
  }
  if (h->side_pending) join_side(h);
  LAUNCH(h, kOther, launch_advance_step(h->counters, h->tm, h->N, h->stream));
  h->supplied_next = false;
  return PBT_OK;
}

int check_device_status(pbt_handle* h) {
  Counters c;
  CU(h, cudaMemcpyAsync(&c, h->counters, sizeof(c), cudaMemcpyDeviceToHost, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  if (c.status != 0) return fail(h, c.status, "a kernel reported status %d (site %d)", c.status, c.status_info);
  return PBT_OK;
}

int refresh_shadow(pbt_handle* h, int member) {
  if (!h->is_bf16) return PBT_OK;
  const long long off = (long long)member * h->P_pad;
  LAUNCH(h, kOther, launch_f32_to_bf16(h->W32 + off, h->W16 + off, h->P_pad, h->stream));
  return PBT_OK;
}

}  // namespace

// ------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------
extern "C" {

const char* pbt_last_error(const pbt_t* p) { return p ? p->err : g_err; }

int pbt_query_workspace(const pbt_spec* spec, size_t* bytes) {
  if (!bytes) return fail(nullptr, PBT_ERR_INVALID_ARG, "bytes is NULL");
  int rc = validate(spec);
  if (rc) return rc;
  pbt_handle* h = new pbt_handle();
  h->spec = *spec;
  *bytes = plan(h, nullptr);
  delete h;
  return PBT_OK;
}

int pbt_param_count(const pbt_spec* spec, int64_t* count) {
  if (!count) return fail(nullptr, PBT_ERR_INVALID_ARG, "count is NULL");
  int rc = validate(spec);
  if (rc) return rc;
  pbt_handle* h = new pbt_handle();
  h->spec = *spec;
  plan(h, nullptr);
  *count = h->P;
  delete h;
  return PBT_OK;
}

int pbt_create(pbt_t** out, const pbt_spec* spec, const double* init_hparams, uint64_t seed, const pbt_data* data,
               void* workspace, size_t workspace_bytes, void* stream) {
  if (!out) return fail(nullptr, PBT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  int rc = validate(spec);
  if (rc) return rc;
  if (spec->nh > 0 && !init_hparams) return fail(nullptr, PBT_ERR_INVALID_ARG, "init_hparams is NULL");
  if (spec->model != PBT_TOY_QUADRATIC) {
    if (!data) return fail(nullptr, PBT_ERR_INVALID_ARG, "data is NULL");
    if (!data->x_pool || !data->x_eval) return fail(nullptr, PBT_ERR_INVALID_ARG, "x_pool / x_eval missing");
    if (spec->model == PBT_MLP && (!data->y_pool || !data->y_eval)) return fail(nullptr, PBT_ERR_INVALID_ARG, "y_pool / y_eval missing");
    if (spec->model == PBT_GAN_PAIR && !data->z_pool) return fail(nullptr, PBT_ERR_INVALID_ARG, "z_pool missing");
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return fail(nullptr, PBT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  }
  pbt_handle* h = new pbt_handle();
  h->spec = *spec;
  if (data) h->data = *data;
  h->stream = (cudaStream_t)stream;
  h->ls = h->stream;
  h->side = nullptr;
  h->side_pending = false;
  h->seed = seed;
  h->step_graph = nullptr;
  const size_t need = plan(h, nullptr);
  if (!workspace || ((uintptr_t)workspace & 255) != 0 || workspace_bytes < need) {
    delete h;
    return fail(nullptr, PBT_ERR_WORKSPACE, "workspace must be 256-byte aligned and hold %zu bytes (got %zu)", need, workspace_bytes);
  }
  plan(h, (char*)workspace);
  auto bail = [&](int code) {
    snprintf(g_err, sizeof(g_err), "%s", h->err);
    delete h;
    return code;
  };
#define CREATE_CU(expr)                                                                              \
  do {                                                                                               \
    cudaError_t e_ = (expr);                                                                         \
    if (e_ != cudaSuccess) { fail(h, PBT_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); return bail(PBT_ERR_CUDA); } \
  } while (0)
  // zero the persistent state (everything up to and including the gradient slabs); activations need no clearing
  const size_t state_bytes = h->toy ? need : (size_t)((char*)(h->is_bf16 ? (void*)(h->W16 + (size_t)h->N * h->P_pad) : (void*)(h->G + (size_t)h->N * h->P_pad)) - (char*)workspace);
  CREATE_CU(cudaMemsetAsync(workspace, 0, state_bytes, h->stream));
  // hyperparameters and scalars
  {
    std::vector<double> Hd((size_t)h->N * PBT_MAX_NH, 0.0);
    std::vector<float> Hf((size_t)h->N * PBT_MAX_NH, 0.f);
    for (int m = 0; m < h->N; ++m)
      for (int k = 0; k < h->nh; ++k) {
        Hd[(size_t)m * PBT_MAX_NH + k] = init_hparams[(size_t)m * h->nh + k];
        Hf[(size_t)m * PBT_MAX_NH + k] = (float)init_hparams[(size_t)m * h->nh + k];
      }
    if (h->toy) CREATE_CU(cudaMemcpyAsync(h->H, Hd.data(), Hd.size() * 8, cudaMemcpyHostToDevice, h->stream));
    else CREATE_CU(cudaMemcpyAsync(h->H, Hf.data(), Hf.size() * 4, cudaMemcpyHostToDevice, h->stream));
    std::vector<float> ones((size_t)h->N * PBT_N_SCALARS, 1.f);
    CREATE_CU(cudaMemcpyAsync(h->scalars, ones.data(), ones.size() * 4, cudaMemcpyHostToDevice, h->stream));
    std::vector<int> ident(h->N);
    for (int m = 0; m < h->N; ++m) ident[m] = m;
    CREATE_CU(cudaMemcpyAsync(h->src, ident.data(), ident.size() * 4, cudaMemcpyHostToDevice, h->stream));
    if (h->toy) {
      std::vector<double> th((size_t)h->N * h->nh);
      for (int m = 0; m < h->N; ++m)
        for (int k = 0; k < h->nh; ++k) th[(size_t)m * h->nh + k] = spec->toy_theta0[k];
      CREATE_CU(cudaMemcpyAsync(h->theta, th.data(), th.size() * 8, cudaMemcpyHostToDevice, h->stream));
    }
    CREATE_CU(cudaStreamSynchronize(h->stream));  // the host vectors above go out of scope
  }
  if (!h->toy) {
    for (int k = 0; k < h->ns; ++k)
      for (int l = 0; l < h->st[k].nl; ++l) {
        const Layer& L = h->st[k].L[l];
        const float bound = (float)sqrt(6.0 / (double)L.in);
        CREATE_CU(launch_init_weights(h->W32, h->P_pad, h->N, L.w_off, L.out, L.in, k * PBT_MAX_LAYERS + l, bound, seed, h->member_base, h->stream));
      }
    if (h->is_bf16) CREATE_CU(launch_f32_to_bf16(h->W32, h->W16, (long long)h->N * h->P_pad, h->stream));
  }
  {
    if (spec->backward_streams != 1 && h->stream != nullptr && !h->toy) {
      CREATE_CU(cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking));
      CREATE_CU(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
      CREATE_CU(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
    }
  }
#undef CREATE_CU
  h->err[0] = 0;
  h->host_loss.assign((size_t)h->N * 2, 0.f);
  *out = h;
  return PBT_OK;
}

int pbt_destroy(pbt_t* p) {
  if (!p) return PBT_OK;
  if (p->step_graph) cudaGraphExecDestroy(p->step_graph);
  if (p->copy_stream) {
    cudaStreamSynchronize(p->copy_stream);
    cudaEventDestroy(p->ev_copied);
    cudaEventDestroy(p->ev_release);
    cudaStreamDestroy(p->copy_stream);
  }
  if (p->side) {
    cudaStreamSynchronize(p->side);
    cudaEventDestroy(p->ev_fork);
    cudaEventDestroy(p->ev_join);
    cudaStreamDestroy(p->side);
  }
  for (auto& r : p->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  for (auto e : p->event_pool) cudaEventDestroy(e);
  delete p;
  return PBT_OK;
}

int pbt_step(pbt_t* p, int k) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  set_serial_launches(p->spec.programmatic_launches == 0);
  if (k < 0) return fail(p, PBT_ERR_INVALID_ARG, "k must be >= 0");
  p->launches = 0;
  // Small populations are launch-bound: replay one captured step as a CUDA graph.  Capture needs a
  // non-default stream and no per-launch event records.
  if (k > 0 && p->supplied_next && p->direct_pool) {
    // the captured step reads the pools; the caller's rows are consumed by one step of the other form
    int rc = one_step(p);
    if (rc) return rc;
    --k;
  }
  const bool want_graph = !p->profiling && !p->graph_failed && p->stream != nullptr && k > 0;
  if (want_graph && !p->step_graph) {
    cudaGraph_t graph = nullptr;
    if (cudaStreamBeginCapture(p->stream, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
      const int64_t before = p->launches;
      int rc = one_step(p);
      cudaError_t e = cudaStreamEndCapture(p->stream, &graph);
      p->graph_nodes = p->launches - before;
      p->launches = before;
      if (rc == PBT_OK && e == cudaSuccess && graph &&
          cudaGraphInstantiate(&p->step_graph, graph, 0) == cudaSuccess) {
        // ready
      } else {
        p->step_graph = nullptr;
        p->graph_failed = true;
        cudaGetLastError();
      }
      if (graph) cudaGraphDestroy(graph);
    } else {
      p->graph_failed = true;
      cudaGetLastError();
    }
  }
  if (want_graph && p->step_graph) {
    for (int i = 0; i < k; ++i) CU(p, cudaGraphLaunch(p->step_graph, p->stream));
    p->launches = (int64_t)k * p->graph_nodes;
    return PBT_OK;
  }
  for (int i = 0; i < k; ++i) {
    int rc = one_step(p);
    if (rc) return rc;
  }
  return PBT_OK;
}

int pbt_step_subset(pbt_t* p, const uint8_t* active_host, int k) {
  if (!p || !active_host) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  set_serial_launches(p->spec.programmatic_launches == 0);
  if (k < 0) return fail(p, PBT_ERR_INVALID_ARG, "k must be >= 0");
  if (p->supplied_next) return fail(p, PBT_ERR_STATE, "a caller-supplied batch is pending: it belongs to a step of the whole population");
  p->launches = 0;
  // one pass of the step machinery per maximal run of consecutive active members
  int m = 0;
  while (m < p->N) {
    if (!active_host[m]) { ++m; continue; }
    int e = m;
    while (e < p->N && active_host[e]) ++e;
    const MemberWindow w = open_window(p, m, e - m);
    int rc = PBT_OK;
    for (int i = 0; i < k && rc == PBT_OK; ++i) rc = one_step(p);
    close_window(p, w);
    if (rc) return rc;
    m = e;
  }
  return PBT_OK;
}

// t-test selection compares the last PBT_HISTORY scores of two members: every evaluation is appended
static int record_scores(pbt_t* p) {
  if (p->spec.exploit_rule != 2) return PBT_OK;
  LAUNCH(p, kOther, launch_history_push(p->fitness, p->hist, p->hist_n, p->N, p->toy ? 1 : 0, p->stream));
  return PBT_OK;
}

int pbt_eval(pbt_t* p) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  set_serial_launches(p->spec.programmatic_launches == 0);
  p->launches = 0;
  const pbt_spec& s = p->spec;
  if (p->toy) {
    LAUNCH(p, kLoss, launch_toy_eval(p->theta, (double*)p->fitness, p->N, p->nh, p->stream));
    return record_scores(p);
  }
  int rc = forward(p, 0, s.eval_batch, p->data.x_eval, 0);
  if (rc) return rc;
  if (p->gan) {
    LAUNCH(p, kLoss, launch_energy_distance(p->logits[0], logits_stride(p, 0), s.eval_batch, p->N, p->ed_partial,
                                            (float*)p->fitness, p->stream));
    p->launches++;  // the launcher issues two kernels
    return record_scores(p);
  }
  LossArgs a;
  memset(&a, 0, sizeof(a));
  const Stack& st = p->st[0];
  a.kind = s.loss; a.n_members = p->N; a.rows = s.eval_batch; a.cols = st.L[st.nl - 1].out;
  a.n_real_rows = s.eval_batch; a.inv_batch = 1.0f / (float)s.eval_batch;
  a.logits = p->logits[0]; a.ld_logits = a.cols; a.stride_logits = logits_stride(p, 0);
  a.target = p->data.y_eval; a.stride_target = 0;
  a.target_dtype = s.loss == PBT_LOSS_CE_SOFT ? p->cdt : kF32;
  a.dz = nullptr; a.row_loss = p->row_loss;
  LAUNCH(p, kLoss, launch_loss_rows(a, p->stream));
  LAUNCH(p, kLoss, launch_reduce_rows(p->row_loss, s.eval_batch, p->N, -1.0f / (float)s.eval_batch, p->fitness, 0, 1, p->stream));
  return record_scores(p);
}

int pbt_exploit_explore(pbt_t* p) { return pbt_exploit_explore_ready(p, nullptr); }

// the arguments of the selection / explore kernel for a population of n members whose records are the given arrays
static void fill_select_args(pbt_t* p, SelectArgs* out, int n, const uint8_t* ready_host, void* H, void* fitness, int* src,
                             int* level, int* n_cut_out) {
  const pbt_spec& s = p->spec;
  SelectArgs& a = *out;
  memset(&a, 0, sizeof(a));
  for (int i = 0; i < n; ++i)
    if (!ready_host || ready_host[i]) a.ready_bits[i >> 5] |= 1u << (i & 31);
  a.n = n; a.nh = p->nh;
  int n_cut = 0;
  if (n >= 2) {
    long long c = ((long long)n * s.trunc_num) / s.trunc_den;
    if (c < 1) c = 1;
    if (c > n / 2) c = n / 2;
    n_cut = (int)c;
  }
  a.n_cut = n_cut;
  *n_cut_out = n_cut;
  a.h_is_double = p->toy ? 1 : 0;
  a.H = H; a.fitness = fitness; a.src = src; a.level = level; a.counters = p->counters; a.seed = p->seed;
  a.rule = s.exploit_rule;
  a.hist = p->hist; a.hist_n = p->hist_n; a.alpha = s.ttest_alpha;
  a.explore_rule = s.explore_rule;
  if (s.explore_rule == 1) {
    long long thr = (long long)(s.resample_prob * 4294967296.0);
    a.resample_thr = (uint32_t)(thr < 0 ? 0 : (thr > 0xFFFFFFFFll ? 0xFFFFFFFFll : thr));
    for (int k = 0; k < PBT_MAX_NH; ++k) {
      a.prior_kind[k] = k < p->nh ? s.prior_kind[k] : PBT_PRIOR_FIXED;
      const bool lg = a.prior_kind[k] == PBT_PRIOR_LOG_UNIFORM;
      a.prior_a[k] = lg ? log(s.prior_lo[k]) : s.prior_lo[k];
      a.prior_b[k] = lg ? log(s.prior_hi[k]) : s.prior_hi[k];
    }
  }
  a.perturb_mask = s.perturb_mask; a.flags = s.flags;
  a.factor_lo = s.factor_lo; a.factor_hi = s.factor_hi;
  for (int k = 0; k < PBT_MAX_NH; ++k) { a.clamp_lo[k] = s.clamp_lo[k]; a.clamp_hi[k] = s.clamp_hi[k]; }
}

// the member-major arrays a slab copy moves (weights, optimiser state, shadow, Adam's running products)
static void fill_copy_arrays(pbt_t* p, CopyArgs* c) {
  auto add = [&](void* base, long long stride, long long bytes) {
    if (!base) return;
    c->base[c->n_arrays] = (char*)base; c->stride_bytes[c->n_arrays] = stride; c->copy_bytes[c->n_arrays] = bytes;
    c->n_arrays++;
  };
  if (p->toy) return;
  const long long slab = p->P_pad * 4;
  add(p->W32, slab, slab);
  add(p->O1, slab, slab);
  add(p->O2, slab, slab);
  add(p->W16, p->P_pad * 2, p->P_pad * 2);
  add(p->scalars, PBT_N_SCALARS * 4, PBT_N_SCALARS * 4);
}

int pbt_exploit_explore_ready(pbt_t* p, const uint8_t* ready_host) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  set_serial_launches(p->spec.programmatic_launches == 0);
  p->launches = 0;
  const pbt_spec& s = p->spec;
  if (s.n_global > 0 && s.n_global != p->N)
    return fail(p, PBT_ERR_STATE, "a shard of a larger population takes its ready points through pbt_exploit_explore_global");
  SelectArgs a;
  int n_cut = 0;
  fill_select_args(p, &a, p->N, ready_host, p->H, p->fitness, p->src, p->level, &n_cut);
  LAUNCH(p, kSelect, launch_select_explore(a, p->stream));
  if (!(s.flags & PBT_COPY_WEIGHTS) || p->N < 2 || (s.exploit_rule == 0 && n_cut == 0)) return PBT_OK;
  // Truncation: donors are never recipients, one parallel copy pass.  Tournament, t-test: a donor may be a recipient
  // too; recipients are copied in passes (deepest readers first) so that every copy reads the donor's record
  // as it was before this ready point.  The number of passes stays on the device: one launch walks them all.
  CopyArgs c;
  memset(&c, 0, sizeof(c));
  c.n = p->N; c.src = p->src;
  c.level = s.exploit_rule != 0 ? p->level : nullptr;
  fill_copy_arrays(p, &c);
  if (p->toy) {
    // nh doubles per member: tiny, and not a multiple of 16 bytes in general
    if (s.exploit_rule != 0)
      LAUNCH(p, kCopy, launch_copy_small_levels((char*)p->theta, (long long)p->nh * 8, p->src, p->N, p->level, p->counters, p->stream));
    else
      LAUNCH(p, kCopy, launch_copy_small((char*)p->theta, (long long)p->nh * 8, p->src, p->N, nullptr, 0, p->stream));
  } else if (s.exploit_rule != 0) {
    LAUNCH(p, kCopy, launch_slab_copy_levels(c, p->counters, p->stream));
  } else {
    LAUNCH(p, kCopy, launch_slab_copy(c, p->stream));
  }
  return PBT_OK;
}

int pbt_exploit_explore_global(pbt_t* p, double* fit_g, double* H_g, const uint8_t* ready_g, int32_t* src_out,
                               int32_t* level_out, int32_t* n_levels_out) {
  if (!p || !fit_g || !H_g || !src_out || !level_out || !n_levels_out) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  const pbt_spec& s = p->spec;
  if (s.n_global <= 0) return fail(p, PBT_ERR_STATE, "the handle was not created as a shard (n_global = 0)");
  if (s.exploit_rule == 2 && !p->g_hist_set)
    return fail(p, PBT_ERR_STATE, "t-test selection needs the whole population's score histories: call pbt_set_global_history first");
  set_serial_launches(s.programmatic_launches == 0);
  p->launches = 0;
  const int G = s.n_global;
  // the whole population's p and h, in the element type of the handle's own records
  std::vector<double> Hd((size_t)G * PBT_MAX_NH, 0.0);
  std::vector<float> Hf((size_t)G * PBT_MAX_NH, 0.f), ff(G);
  for (int m = 0; m < G; ++m) {
    ff[m] = (float)fit_g[m];
    for (int k = 0; k < p->nh; ++k) {
      Hd[(size_t)m * PBT_MAX_NH + k] = H_g[(size_t)m * p->nh + k];
      Hf[(size_t)m * PBT_MAX_NH + k] = (float)H_g[(size_t)m * p->nh + k];
    }
  }
  if (p->toy) {
    CU(p, cudaMemcpyAsync(p->g_fit, fit_g, (size_t)G * 8, cudaMemcpyHostToDevice, p->stream));
    CU(p, cudaMemcpyAsync(p->g_H, Hd.data(), Hd.size() * 8, cudaMemcpyHostToDevice, p->stream));
  } else {
    CU(p, cudaMemcpyAsync(p->g_fit, ff.data(), (size_t)G * 4, cudaMemcpyHostToDevice, p->stream));
    CU(p, cudaMemcpyAsync(p->g_H, Hf.data(), Hf.size() * 4, cudaMemcpyHostToDevice, p->stream));
  }
  SelectArgs a;
  int n_cut = 0;
  fill_select_args(p, &a, G, ready_g, p->g_H, p->g_fit, p->g_src, p->g_level, &n_cut);
  if (s.exploit_rule == 2) { a.hist = p->g_hist; a.hist_n = p->g_hist_n; }
  LAUNCH(p, kSelect, launch_select_explore(a, p->stream));
  LAUNCH(p, kSelect, launch_localize_selection(p->g_src, p->g_level, p->g_H, p->g_fit, p->toy ? 1 : 0, s.member_base, p->N,
                                               p->src, p->level, p->H, p->fitness, p->stream));
  if (s.exploit_rule == 2) {
    // a copy moved the donor's score history with it (inside the global arrays): take this shard's rows back
    const size_t esz = p->toy ? 8 : 4;
    CU(p, cudaMemcpyAsync(p->hist, (const char*)p->g_hist + (size_t)s.member_base * PBT_HISTORY * esz,
                          (size_t)p->N * PBT_HISTORY * esz, cudaMemcpyDeviceToDevice, p->stream));
    CU(p, cudaMemcpyAsync(p->hist_n, p->g_hist_n + s.member_base, (size_t)p->N * 4, cudaMemcpyDeviceToDevice, p->stream));
    p->g_hist_set = false;
  }
  Counters cnt;
  CU(p, cudaMemcpyAsync(&cnt, p->counters, sizeof(cnt), cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaMemcpyAsync(src_out, p->g_src, (size_t)G * 4, cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaMemcpyAsync(level_out, p->g_level, (size_t)G * 4, cudaMemcpyDeviceToHost, p->stream));
  if (p->toy) {
    CU(p, cudaMemcpyAsync(fit_g, p->g_fit, (size_t)G * 8, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaMemcpyAsync(Hd.data(), p->g_H, Hd.size() * 8, cudaMemcpyDeviceToHost, p->stream));
  } else {
    CU(p, cudaMemcpyAsync(ff.data(), p->g_fit, (size_t)G * 4, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaMemcpyAsync(Hf.data(), p->g_H, Hf.size() * 4, cudaMemcpyDeviceToHost, p->stream));
  }
  CU(p, cudaStreamSynchronize(p->stream));
  if (cnt.status != 0) return fail(p, cnt.status, "a kernel reported status %d (site %d)", cnt.status, cnt.status_info);
  for (int m = 0; m < G; ++m) {
    if (!p->toy) fit_g[m] = ff[m];
    for (int k = 0; k < p->nh; ++k)
      H_g[(size_t)m * p->nh + k] = p->toy ? Hd[(size_t)m * PBT_MAX_NH + k] : (double)Hf[(size_t)m * PBT_MAX_NH + k];
  }
  const bool copies = (s.flags & PBT_COPY_WEIGHTS) && G >= 2 && !(s.exploit_rule == 0 && n_cut == 0);
  if (!copies) {
    // no weights move: report an empty copy map so that the caller's exchange has nothing to do
    for (int m = 0; m < G; ++m) { src_out[m] = m; level_out[m] = 0; }
    *n_levels_out = 0;
    return PBT_OK;
  }
  *n_levels_out = (s.exploit_rule == 0 ? 0 : cnt.max_level) + 1;
  return PBT_OK;
}

int pbt_set_global_history(pbt_t* p, const double* hist, const int32_t* count) {
  if (!p || !hist || !count) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  const pbt_spec& s = p->spec;
  if (s.n_global <= 0) return fail(p, PBT_ERR_STATE, "the handle was not created as a shard (n_global = 0)");
  const int G = s.n_global;
  for (int m = 0; m < G; ++m)
    if (count[m] < 0 || count[m] > PBT_HISTORY) return fail(p, PBT_ERR_INVALID_ARG, "history count out of range");
  const size_t n = (size_t)G * PBT_HISTORY;
  std::vector<float> hf(n);
  for (size_t i = 0; i < n; ++i) hf[i] = (float)hist[i];
  if (p->toy) CU(p, cudaMemcpyAsync(p->g_hist, hist, n * 8, cudaMemcpyHostToDevice, p->stream));
  else CU(p, cudaMemcpyAsync(p->g_hist, hf.data(), n * 4, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaMemcpyAsync(p->g_hist_n, count, (size_t)G * 4, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  p->g_hist_set = true;
  return PBT_OK;
}

int pbt_copy_members_level(pbt_t* p, int level) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  if (level < 0) return fail(p, PBT_ERR_INVALID_ARG, "level must be >= 0");
  if (!(p->spec.flags & PBT_COPY_WEIGHTS) || p->N < 2) return PBT_OK;
  set_serial_launches(p->spec.programmatic_launches == 0);
  p->launches = 0;
  if (p->toy) {
    LAUNCH(p, kCopy, launch_copy_small((char*)p->theta, (long long)p->nh * 8, p->src, p->N, p->level, level, p->stream));
    return PBT_OK;
  }
  CopyArgs c;
  memset(&c, 0, sizeof(c));
  c.n = p->N; c.src = p->src; c.level = p->level; c.want_level = level;
  fill_copy_arrays(p, &c);
  LAUNCH(p, kCopy, launch_slab_copy(c, p->stream));
  return PBT_OK;
}

int pbt_member_slabs(pbt_t* p, int member, void** ptrs, size_t* bytes, int32_t* count) {
  if (!p || !ptrs || !bytes || !count) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (member < 0 || member >= p->N) return fail(p, PBT_ERR_INVALID_ARG, "member out of range");
  int n = 0;
  if (p->toy) {
    ptrs[n] = p->theta + (size_t)member * p->nh; bytes[n++] = (size_t)p->nh * 8;
  } else {
    const size_t off = (size_t)member * p->P_pad;
    ptrs[n] = p->W32 + off; bytes[n++] = (size_t)p->P_pad * 4;
    ptrs[n] = p->O1 + off; bytes[n++] = (size_t)p->P_pad * 4;
    if (p->O2) { ptrs[n] = p->O2 + off; bytes[n++] = (size_t)p->P_pad * 4; }
    if (p->W16) { ptrs[n] = p->W16 + off; bytes[n++] = (size_t)p->P_pad * 2; }
    ptrs[n] = p->scalars + (size_t)member * PBT_N_SCALARS; bytes[n++] = PBT_N_SCALARS * 4;
  }
  *count = n;
  return PBT_OK;
}

int pbt_get_state(pbt_t* p, int member, pbt_state_view* v) {
  if (!p || !v) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (member < 0 || member >= p->N) return fail(p, PBT_ERR_INVALID_ARG, "member out of range");
  std::vector<float> sc(PBT_N_SCALARS);
  Counters c;
  if (p->toy) {
    if (v->w) CU(p, cudaMemcpyAsync(v->w, p->theta + (size_t)member * p->nh, p->nh * 8, cudaMemcpyDeviceToHost, p->stream));
  } else {
    struct { void* host; const float* dev; } parts[4] = {{v->w, p->W32}, {v->opt1, p->O1}, {v->opt2, p->O2}, {v->grad, p->G}};
    for (auto& part : parts) {
      if (!part.host) continue;
      float* dst = (float*)part.host;
      if (!part.dev) {  // no second moment for SGD-momentum: report zeros
        memset(dst, 0, (size_t)p->P * 4);
        continue;
      }
      const float* slab = part.dev + (size_t)member * p->P_pad;
      for (int k = 0; k < p->ns; ++k)
        for (int l = 0; l < p->st[k].nl; ++l) {
          const Layer& L = p->st[k].L[l];
          const size_t nw = (size_t)L.in * L.out;
          CU(p, cudaMemcpyAsync(dst, slab + L.w_off, nw * 4, cudaMemcpyDeviceToHost, p->stream));
          dst += nw;
          CU(p, cudaMemcpyAsync(dst, slab + L.b_off, (size_t)L.out * 4, cudaMemcpyDeviceToHost, p->stream));
          dst += L.out;
        }
    }
  }
  CU(p, cudaMemcpyAsync(sc.data(), p->scalars + (size_t)member * PBT_N_SCALARS, PBT_N_SCALARS * 4, cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaMemcpyAsync(&c, p->counters, sizeof(c), cudaMemcpyDeviceToHost, p->stream));
  long long tstep = 0;
  CU(p, cudaMemcpyAsync(&tstep, p->tm + member, 8, cudaMemcpyDeviceToHost, p->stream));
  double hd[PBT_MAX_NH];
  float hf[PBT_MAX_NH];
  double fd = 0;
  float ff = 0;
  if (p->toy) {
    CU(p, cudaMemcpyAsync(hd, (double*)p->H + (size_t)member * PBT_MAX_NH, sizeof(hd), cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaMemcpyAsync(&fd, (double*)p->fitness + member, 8, cudaMemcpyDeviceToHost, p->stream));
  } else {
    CU(p, cudaMemcpyAsync(hf, (float*)p->H + (size_t)member * PBT_MAX_NH, sizeof(hf), cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaMemcpyAsync(&ff, (float*)p->fitness + member, 4, cudaMemcpyDeviceToHost, p->stream));
  }
  CU(p, cudaStreamSynchronize(p->stream));
  if (c.status != 0) return fail(p, c.status, "a kernel reported status %d (site %d)", c.status, c.status_info);
  if (v->scalars) for (int i = 0; i < PBT_N_SCALARS; ++i) v->scalars[i] = sc[i];
  if (v->hparams) for (int k = 0; k < p->nh; ++k) v->hparams[k] = p->toy ? hd[k] : (double)hf[k];
  if (v->fitness) *v->fitness = p->toy ? fd : (double)ff;
  if (v->step) *v->step = tstep;
  if (v->round) *v->round = c.round;
  return PBT_OK;
}

int pbt_set_state(pbt_t* p, int member, const pbt_state_view* v) {
  if (!p || !v) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (member < 0 || member >= p->N) return fail(p, PBT_ERR_INVALID_ARG, "member out of range");
  if (p->toy) {
    if (v->w) CU(p, cudaMemcpyAsync(p->theta + (size_t)member * p->nh, v->w, p->nh * 8, cudaMemcpyHostToDevice, p->stream));
  } else {
    struct { const void* host; float* dev; } parts[3] = {{v->w, p->W32}, {v->opt1, p->O1}, {v->opt2, p->O2}};
    for (auto& part : parts) {
      if (!part.host || !part.dev) continue;
      const float* srcp = (const float*)part.host;
      float* slab = part.dev + (size_t)member * p->P_pad;
      for (int k = 0; k < p->ns; ++k)
        for (int l = 0; l < p->st[k].nl; ++l) {
          const Layer& L = p->st[k].L[l];
          const size_t nw = (size_t)L.in * L.out;
          CU(p, cudaMemcpyAsync(slab + L.w_off, srcp, nw * 4, cudaMemcpyHostToDevice, p->stream));
          srcp += nw;
          CU(p, cudaMemcpyAsync(slab + L.b_off, srcp, (size_t)L.out * 4, cudaMemcpyHostToDevice, p->stream));
          srcp += L.out;
        }
    }
    if (v->w) {
      int rc = refresh_shadow(p, member);
      if (rc) return rc;
    }
  }
  float sc[PBT_N_SCALARS];
  if (v->scalars) {
    for (int i = 0; i < PBT_N_SCALARS; ++i) sc[i] = (float)v->scalars[i];
    CU(p, cudaMemcpyAsync(p->scalars + (size_t)member * PBT_N_SCALARS, sc, sizeof(sc), cudaMemcpyHostToDevice, p->stream));
  }
  double hd[PBT_MAX_NH] = {0};
  float hf[PBT_MAX_NH] = {0};
  if (v->hparams) {
    for (int k = 0; k < p->nh; ++k) { hd[k] = v->hparams[k]; hf[k] = (float)v->hparams[k]; }
    if (p->toy) CU(p, cudaMemcpyAsync((double*)p->H + (size_t)member * PBT_MAX_NH, hd, sizeof(hd), cudaMemcpyHostToDevice, p->stream));
    else CU(p, cudaMemcpyAsync((float*)p->H + (size_t)member * PBT_MAX_NH, hf, sizeof(hf), cudaMemcpyHostToDevice, p->stream));
  }
  double fd = 0;
  float ff = 0;
  if (v->fitness) {
    fd = *v->fitness; ff = (float)fd;
    if (p->toy) CU(p, cudaMemcpyAsync((double*)p->fitness + member, &fd, 8, cudaMemcpyHostToDevice, p->stream));
    else CU(p, cudaMemcpyAsync((float*)p->fitness + member, &ff, 4, cudaMemcpyHostToDevice, p->stream));
  }
  long long st = 0, rd = 0;
  if (v->step) { st = *v->step; CU(p, cudaMemcpyAsync(p->tm + member, &st, 8, cudaMemcpyHostToDevice, p->stream)); }
  if (v->round) { rd = *v->round; CU(p, cudaMemcpyAsync(&p->counters->round, &rd, 8, cudaMemcpyHostToDevice, p->stream)); }
  CU(p, cudaStreamSynchronize(p->stream));  // host staging above lives on this frame
  return PBT_OK;
}

int pbt_get_fitness(pbt_t* p, double* out) {
  if (!p || !out) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (p->toy) {
    CU(p, cudaMemcpyAsync(out, p->fitness, (size_t)p->N * 8, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
  } else {
    std::vector<float> f(p->N);
    CU(p, cudaMemcpyAsync(f.data(), p->fitness, (size_t)p->N * 4, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
    for (int i = 0; i < p->N; ++i) out[i] = f[i];
  }
  return check_device_status(p);
}

int pbt_set_fitness(pbt_t* p, const double* in) {
  if (!p || !in) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (p->toy) {
    CU(p, cudaMemcpyAsync(p->fitness, in, (size_t)p->N * 8, cudaMemcpyHostToDevice, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
  } else {
    std::vector<float> f(p->N);
    for (int i = 0; i < p->N; ++i) f[i] = (float)in[i];
    CU(p, cudaMemcpyAsync(p->fitness, f.data(), (size_t)p->N * 4, cudaMemcpyHostToDevice, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
  }
  return PBT_OK;
}

int pbt_get_history(pbt_t* p, double* hist, int32_t* count) {
  if (!p) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  const size_t n = (size_t)p->N * PBT_HISTORY;
  std::vector<int32_t> c(p->N);
  CU(p, cudaMemcpyAsync(c.data(), p->hist_n, (size_t)p->N * 4, cudaMemcpyDeviceToHost, p->stream));
  std::vector<double> hd(n);
  std::vector<float> hf(n);
  if (p->toy) CU(p, cudaMemcpyAsync(hd.data(), p->hist, n * 8, cudaMemcpyDeviceToHost, p->stream));
  else CU(p, cudaMemcpyAsync(hf.data(), p->hist, n * 4, cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  for (int m = 0; m < p->N; ++m) {
    if (count) count[m] = c[m];
    if (hist)
      for (int k = 0; k < PBT_HISTORY; ++k) {
        const size_t i = (size_t)m * PBT_HISTORY + k;
        hist[i] = k < c[m] ? (p->toy ? hd[i] : (double)hf[i]) : 0.0;
      }
  }
  return PBT_OK;
}

int pbt_set_history(pbt_t* p, const double* hist, const int32_t* count) {
  if (!p || !hist || !count) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  for (int m = 0; m < p->N; ++m)
    if (count[m] < 0 || count[m] > PBT_HISTORY) return fail(p, PBT_ERR_INVALID_ARG, "history count out of range");
  const size_t n = (size_t)p->N * PBT_HISTORY;
  std::vector<float> hf(n);
  for (size_t i = 0; i < n; ++i) hf[i] = (float)hist[i];
  if (p->toy) CU(p, cudaMemcpyAsync(p->hist, hist, n * 8, cudaMemcpyHostToDevice, p->stream));
  else CU(p, cudaMemcpyAsync(p->hist, hf.data(), n * 4, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaMemcpyAsync(p->hist_n, count, (size_t)p->N * 4, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  return PBT_OK;
}

int pbt_get_hparams(pbt_t* p, double* out) {
  if (!p || !out) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  const size_t n = (size_t)p->N * PBT_MAX_NH;
  if (p->toy) {
    std::vector<double> hbuf(n);
    CU(p, cudaMemcpyAsync(hbuf.data(), p->H, n * 8, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
    for (int m = 0; m < p->N; ++m) for (int k = 0; k < p->nh; ++k) out[(size_t)m * p->nh + k] = hbuf[(size_t)m * PBT_MAX_NH + k];
  } else {
    std::vector<float> hbuf(n);
    CU(p, cudaMemcpyAsync(hbuf.data(), p->H, n * 4, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
    for (int m = 0; m < p->N; ++m) for (int k = 0; k < p->nh; ++k) out[(size_t)m * p->nh + k] = hbuf[(size_t)m * PBT_MAX_NH + k];
  }
  return PBT_OK;
}

int pbt_set_hparams(pbt_t* p, const double* in) {
  if (!p || !in) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  const size_t n = (size_t)p->N * PBT_MAX_NH;
  std::vector<double> hd(n, 0.0);
  std::vector<float> hf(n, 0.f);
  for (int m = 0; m < p->N; ++m)
    for (int k = 0; k < p->nh; ++k) {
      hd[(size_t)m * PBT_MAX_NH + k] = in[(size_t)m * p->nh + k];
      hf[(size_t)m * PBT_MAX_NH + k] = (float)in[(size_t)m * p->nh + k];
    }
  if (p->toy) CU(p, cudaMemcpyAsync(p->H, hd.data(), n * 8, cudaMemcpyHostToDevice, p->stream));
  else CU(p, cudaMemcpyAsync(p->H, hf.data(), n * 4, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  return PBT_OK;
}

int pbt_get_copy_map(pbt_t* p, int32_t* out) {
  if (!p || !out) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  CU(p, cudaMemcpyAsync(out, p->src, (size_t)p->N * 4, cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  return PBT_OK;
}

int pbt_get_best(pbt_t* p, int32_t* member) {
  if (!p || !member) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  std::vector<double> f(p->N);
  int rc = pbt_get_fitness(p, f.data());
  if (rc) return rc;
  int best = 0;
  double bf = f[0] != f[0] ? -INFINITY : f[0];
  for (int i = 1; i < p->N; ++i) {
    const double v = f[i] != f[i] ? -INFINITY : f[i];
    if (v > bf) { bf = v; best = i; }
  }
  *member = best;
  return PBT_OK;
}

int pbt_get_last_loss(pbt_t* p, double* out) {
  if (!p || !out) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  std::vector<float> f((size_t)p->N * 2);
  CU(p, cudaMemcpyAsync(f.data(), p->last_loss, f.size() * 4, cudaMemcpyDeviceToHost, p->stream));
  CU(p, cudaStreamSynchronize(p->stream));
  for (size_t i = 0; i < f.size(); ++i) out[i] = f[i];
  return PBT_OK;
}

int pbt_set_batch(pbt_t* p, const void* x, const void* y) {
  if (!p || !x || !y) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (p->toy || p->gan) return fail(p, PBT_ERR_UNSUPPORTED, "caller-supplied batches are for MLP populations");
  const pbt_spec& s = p->spec;
  const size_t xb = (size_t)p->N * s.batch * p->st[0].L[0].in * p->esz;
  CU(p, cudaMemcpyAsync(p->act[0][0], x, xb, cudaMemcpyDeviceToDevice, p->stream));
  const size_t trb = target_row_bytes(p) * s.batch;
  const size_t tsz = s.loss == PBT_LOSS_CE_SOFT ? p->esz : 4;
  CU(p, cudaMemcpy2DAsync(p->ybatch, p->ybatch_stride * tsz, y, trb, trb, p->N, cudaMemcpyDeviceToDevice, p->stream));
  CU(p, cudaMemcpyAsync(&p->counters->use_supplied_batch, &kOne, 4, cudaMemcpyHostToDevice, p->stream));
  p->supplied_next = true;
  return PBT_OK;
}

int pbt_step_host(pbt_t* p, const void* x_host, const void* y_host, double* loss_out_host) {
  if (!p || !x_host || !y_host) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (p->toy || p->gan) return fail(p, PBT_ERR_UNSUPPORTED, "host-fed steps are for MLP populations");
  p->launches = 0;
  set_serial_launches(p->spec.programmatic_launches == 0);
  const pbt_spec& s = p->spec;
  const size_t xb = (size_t)p->N * s.batch * p->st[0].L[0].in * p->esz;
  CU(p, cudaMemcpyAsync(p->act[0][0], x_host, xb, cudaMemcpyHostToDevice, p->stream));
  const size_t trb = target_row_bytes(p) * s.batch;
  const size_t tsz = s.loss == PBT_LOSS_CE_SOFT ? p->esz : 4;
  CU(p, cudaMemcpy2DAsync(p->ybatch, p->ybatch_stride * tsz, y_host, trb, trb, p->N, cudaMemcpyHostToDevice, p->stream));
  CU(p, cudaMemcpyAsync(&p->counters->use_supplied_batch, &kOne, 4, cudaMemcpyHostToDevice, p->stream));
  p->supplied_next = true;
  int rc = one_step(p);
  if (rc) return rc;
  if (loss_out_host) {
    float* tmp = p->host_loss.data();
    CU(p, cudaMemcpyAsync(tmp, p->last_loss, (size_t)p->N * 2 * 4, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
    for (int i = 0; i < p->N * 2; ++i) loss_out_host[i] = tmp[i];
  }
  return PBT_OK;
}

int pbt_prefetch_host_batch(pbt_t* p, const void* x_host, const void* y_host) {
  if (!p || !x_host || !y_host) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  if (p->toy || p->gan) return fail(p, PBT_ERR_UNSUPPORTED, "host-fed steps are for MLP populations");
  if (!p->copy_stream) {
    CU(p, cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking));
    CU(p, cudaEventCreateWithFlags(&p->ev_copied, cudaEventDisableTiming));
    CU(p, cudaEventCreateWithFlags(&p->ev_release, cudaEventDisableTiming));
  }
  if (p->prefetched) return fail(p, PBT_ERR_STATE, "the previously prefetched batch has not been consumed yet");
  // The spare buffers were the current ones until the latest swap; everything that used them (earlier prefetched
  // steps, but also pbt_step / pbt_set_batch / pbt_step_host calls made in between) was enqueued before that swap,
  // where ev_release was recorded.  The step enqueued after the swap may still be running: it uses the other pair.
  if (p->pf_steps >= 1) CU(p, cudaStreamWaitEvent(p->copy_stream, p->ev_release, 0));
  const pbt_spec& s = p->spec;
  const size_t xb = (size_t)p->N * s.batch * p->st[0].L[0].in * p->esz;
  CU(p, cudaMemcpyAsync(p->act0_alt, x_host, xb, cudaMemcpyHostToDevice, p->copy_stream));
  const size_t trb = target_row_bytes(p) * s.batch;
  const size_t tsz = s.loss == PBT_LOSS_CE_SOFT ? p->esz : 4;
  CU(p, cudaMemcpy2DAsync(p->ybatch_alt, p->ybatch_stride * tsz, y_host, trb, trb, p->N, cudaMemcpyHostToDevice, p->copy_stream));
  CU(p, cudaEventRecord(p->ev_copied, p->copy_stream));
  p->prefetched = true;
  return PBT_OK;
}

int pbt_step_prefetched(pbt_t* p, double* loss_out_host) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  set_serial_launches(p->spec.programmatic_launches == 0);
  if (!p->prefetched) return fail(p, PBT_ERR_STATE, "no batch has been prefetched");
  p->launches = 0;
  p->prefetched = false;
  CU(p, cudaStreamWaitEvent(p->stream, p->ev_copied, 0));
  // every launch that reads or writes the buffers that become spare now is already in the stream: the next upload
  // into them waits for this point, not for the step enqueued below
  CU(p, cudaEventRecord(p->ev_release, p->stream));
  // the uploaded buffers become the current ones; a captured step graph holds the old addresses
  std::swap(p->act[0][0], p->act0_alt);
  std::swap(p->ybatch, p->ybatch_alt);
  if (p->step_graph) { cudaGraphExecDestroy(p->step_graph); p->step_graph = nullptr; }
  CU(p, cudaMemcpyAsync(&p->counters->use_supplied_batch, &kOne, 4, cudaMemcpyHostToDevice, p->stream));
  p->supplied_next = true;
  int rc = one_step(p);
  if (rc) return rc;
  p->pf_steps++;
  if (loss_out_host) {
    float* tmp = p->host_loss.data();
    CU(p, cudaMemcpyAsync(tmp, p->last_loss, (size_t)p->N * 2 * 4, cudaMemcpyDeviceToHost, p->stream));
    CU(p, cudaStreamSynchronize(p->stream));
    for (int i = 0; i < p->N * 2; ++i) loss_out_host[i] = tmp[i];
  }
  return PBT_OK;
}

int pbt_grouped_gemm(const pbt_gemm_desc* d, void* stream) {
  if (!d || !d->A || !d->B || !d->C) return fail(nullptr, PBT_ERR_INVALID_ARG, "NULL argument");
  if (d->M < 1 || d->N < 1 || d->K < 0 || d->batch < 1) return fail(nullptr, PBT_ERR_INVALID_ARG, "bad GEMM shape");
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.M = d->M; g.N = d->N; g.K = d->K; g.batch = d->batch;
  g.in_dtype = d->in_bf16 ? kBF16 : kF32; g.out_dtype = d->out_bf16 ? kBF16 : kF32;
  g.A = d->A; g.lda = d->lda; g.strideA = d->strideA; g.a_mn = d->a_mn;
  g.B = d->B; g.ldb = d->ldb; g.strideB = d->strideB; g.b_mn = d->b_mn;
  g.C = d->C; g.ldc = d->ldc; g.strideC = d->strideC;
  g.bias = d->bias; g.strideBias = d->strideBias; g.relu = d->relu;
  g.mask = d->mask; g.ldmask = d->ldmask; g.strideMask = d->strideMask;
  const bool tc = gemm_tc_supported(g), pair = gemm_tc_pair_supported(g);
  cudaError_t e;
  if (d->engine == 3 || (d->engine == 0 && pair && gemm_tc_pair_preferred(g) && d->status_device)) {
    if (!pair) return fail(nullptr, PBT_ERR_UNSUPPORTED, "shape / alignment does not qualify for the CTA-pair tensor-core kernel");
    if (!d->status_device) return fail(nullptr, PBT_ERR_INVALID_ARG, "status_device is required by the tensor-core kernels");
    e = launch_gemm_tc_pair(g, (Counters*)d->status_device, (cudaStream_t)stream);
  } else if (d->engine == 2 || (d->engine == 0 && tc && d->status_device)) {
    if (!tc) return fail(nullptr, PBT_ERR_UNSUPPORTED, "shape / alignment does not qualify for the tensor-core kernel");
    if (!d->status_device) return fail(nullptr, PBT_ERR_INVALID_ARG, "status_device is required by the tensor-core kernel");
    e = launch_gemm_tc(g, (Counters*)d->status_device, (cudaStream_t)stream);
  } else {
    e = launch_gemm_simt(g, (cudaStream_t)stream);
  }
  if (e != cudaSuccess) return fail(nullptr, PBT_ERR_CUDA, "grouped GEMM launch: %s", cudaGetErrorString(e));
  return PBT_OK;
}

int pbt_selftest_bounded_wait(void* status_device, int polls, void* stream) {
  if (!status_device) return fail(nullptr, PBT_ERR_INVALID_ARG, "status_device is NULL");
  if (polls < 1 || polls > 100000) return fail(nullptr, PBT_ERR_INVALID_ARG, "polls must lie in [1, 100000]");
  cudaError_t e = launch_selftest_bounded_wait((Counters*)status_device, (uint32_t)polls, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(nullptr, PBT_ERR_CUDA, "self-test launch: %s", cudaGetErrorString(e));
  return PBT_OK;
}

int pbt_get_launch_count(const pbt_t* p, int64_t* count) {
  if (!p || !count) return fail(nullptr, PBT_ERR_INVALID_ARG, "NULL argument");
  *count = p->launches;
  return PBT_OK;
}

int pbt_profile_begin(pbt_t* p) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  for (auto& r : p->prof) { p->event_pool.push_back(r.a); p->event_pool.push_back(r.b); }
  p->prof.clear();
  for (int i = 0; i < kNumClasses; ++i) { p->prof_ms[i] = 0; p->prof_n[i] = 0; }
  p->profiling = true;
  return PBT_OK;
}

int pbt_profile_end(pbt_t* p) {
  if (!p) return fail(nullptr, PBT_ERR_INVALID_ARG, "handle is NULL");
  p->profiling = false;
  CU(p, cudaStreamSynchronize(p->stream));
  for (auto& r : p->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) { p->prof_ms[r.cls] += ms; p->prof_n[r.cls] += 1; }
    p->event_pool.push_back(r.a);
    p->event_pool.push_back(r.b);
  }
  p->prof.clear();
  return PBT_OK;
}

int pbt_profile_get(pbt_t* p, const char* kernel_class, double* ms_total, int64_t* launches) {
  if (!p || !kernel_class) return fail(p, PBT_ERR_INVALID_ARG, "NULL argument");
  for (int i = 0; i < kNumClasses; ++i)
    if (strcmp(kernel_class, kClassNames[i]) == 0) {
      if (ms_total) *ms_total = p->prof_ms[i];
      if (launches) *launches = p->prof_n[i];
      return PBT_OK;
    }
  return fail(p, PBT_ERR_INVALID_ARG, "unknown kernel class '%s'", kernel_class);
}

}  // extern "C"
