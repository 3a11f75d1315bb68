// C ABI, plan (shape grouping, refresh schedule), workspace layout and the
// per-step launch sequence.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "launch.cuh"

using namespace prm;

struct prm_ctx {
  int n_mats = 0;
  std::vector<int64_t> shapes;   // 2*n_mats
  int K = 1;
  float beta = 0.95f;
  int nesterov = 0;
  float lr = 0.f, wd = 0.f;
  float gamma = 0.15f, eps_row = 1e-8f, eps_ns = 1e-7f;
  int scale_mode = 1;
  int io_fp32 = 0;
  int check_mode = 0;
  size_t ns_cap = (size_t)8 << 30;
  float gamma_ns = 1.f;   // multiplier on the NS5 branch (ablation: "scalar-controlled" uses gamma)
  int no_refresh = 0;     // ablation: RowNorm at every step
  int gram_span = 2;      // NS5 schedule of the tensor-core path (PRM_OPT_NS_GRAM_SPAN)
  int split_input = 0;    // NS5 input as two bf16 planes (PRM_OPT_NS_SPLIT_INPUT)
  int wide_kernel = 0;    // row step of wide groups (PRM_OPT_WIDE_KERNEL): 0 persistent kernel where it applies, 1 one row per CTA
  int tall_kernel = 0;    // row step of tall groups (PRM_OPT_TALL_KERNEL): 0 auto, 1 two passes, 2 streaming where possible

  std::vector<Group> groups;
  std::vector<int> group_of_mat, order_in_group, slot_of_mat;   // slot = index in pointer tables

  // workspace layout (byte offsets)
  size_t off_status = 0, off_tables = 0, off_pmaps = 0, off_rmaps = 0, off_fro = 0, off_alpha = 0, off_ns = 0, total_bytes = 0;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  std::vector<void*> host_tables;   // 3*n_mats, grouped order: params | grads | momentum
  std::vector<unsigned char> host_pmaps;   // n_mats tensor maps of 128 bytes over the parameters (table order)
  std::vector<unsigned char> host_rmaps;   // streaming row step: 3 maps (gradient, momentum, parameters) per matrix
  bool tables_uploaded = false;

  TcContext* tc = nullptr;
  std::string err;
  int64_t launches = 0;

  // optional per-class device timing (prm_profile)
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_ev;     // begin/end pairs
  std::vector<int> prof_cls;            // class of pair i
  std::vector<int64_t> prof_launches;   // kernel launches inside pair i
  size_t prof_used = 0;
  int64_t prof_dropped = 0;

  // prm_step_h2d: gradients travel on a copy stream, one event per shape group,
  // so the copy of group g+1 overlaps the kernels of group g (host resources,
  // created on first use)
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t copy_begin = nullptr;
  std::vector<cudaEvent_t> copy_done;   // per group
};

namespace {
constexpr size_t kProfPairs = 8192;

struct ProfScope {
  prm_ctx* c;
  cudaStream_t stream;
  long idx = -1;
  int64_t launches0 = 0;
  ProfScope(prm_ctx* ctx, int cls, cudaStream_t st) : c(ctx), stream(st) {
    if (!c->prof_on) return;
    if (c->prof_used >= kProfPairs) { c->prof_dropped++; return; }
    idx = (long)c->prof_used++;
    c->prof_cls[idx] = cls;
    launches0 = c->launches;
    cudaEventRecord(c->prof_ev[2 * idx], stream);
  }
  ~ProfScope() {
    if (idx < 0) return;
    cudaEventRecord(c->prof_ev[2 * idx + 1], stream);
    c->prof_launches[idx] = c->launches - launches0;
  }
};
}  // namespace

static std::string g_create_err;

static int fail(prm_ctx* ctx, int code, const std::string& msg) {
  if (ctx) ctx->err = msg; else g_create_err = msg;
  return code;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static float shape_scale(int mode, int64_t rows, int64_t cols) {
  // s(W) of Eq. finite_ns5: depends on the stored shape only.
  if (mode == 0) return 1.f;
  if (mode == 1) return (float)sqrt(std::max(1.0, (double)rows / (double)cols));
  return (float)(0.2 * sqrt((double)std::max(rows, cols)));
}

static void compute_layout(prm_ctx* c) {
  size_t off = 0;
  c->off_status = off; off += 256;
  c->off_tables = off; off = align_up(off + (size_t)3 * c->n_mats * sizeof(void*), 256);
  c->off_pmaps = off;  off = align_up(off + (size_t)128 * c->n_mats, 256);
  c->off_rmaps = off;  off = align_up(off + (size_t)384 * c->n_mats, 256);
  size_t fro_max = 0, ns_max = 0;
  int batch_max = 1;
  for (Group& g : c->groups) {
    if (g.tall) {
      const size_t nblk = (size_t)((g.rows + kTallRows - 1) / kTallRows);
      // column partial sums of the two-pass kernels, or the streaming kernel's ring of per-wave sums
      g.tall_scratch_off = off;
      off = align_up(off + std::max((size_t)g.count * nblk * g.cols * 4, tall_stream_partial_bytes()), 256);
      g.tall_nu_off = off;      off = align_up(off + (size_t)g.count * g.cols * 4, 256);
      g.tall_sync_off = off;    off = align_up(off + tall_stream_sync_ints(g.cols, g.count) * sizeof(int), 256);
    }
    g.ns_fp32 = (c->check_mode || g.r < kTinyRows || (c->split_input && split_takes_fp32(g.r))) ? 1 : 0;
    const size_t e = g.ns_fp32 ? 4 : 2;
    g.split = (c->split_input && !g.ns_fp32) ? 1 : 0;
    const Ns5Schedule sched = ns5_schedule(g.r, g.c, c->gram_span, g.ns_fp32 != 0, g.split != 0);
    g.gram_iters = sched.gram_iters;
    g.last_gram_rec = sched.last_gram_rec;
    // X ping-pong (the first buffer twice as large where X_0 is a pair of planes), A, B (+ two
    // more r x r matrices for the Gram-space iterations)
    const size_t per_mat = e * (size_t)((g.split ? 3 : 2) * g.rp * g.cp + (g.gram_iters ? 4 : 2) * g.rp * g.rp);
    int nb = (int)std::min<size_t>((size_t)g.count, std::max<size_t>(1, c->ns_cap / per_mat));
    // equal sub-batches: 42 matrices with room for 18 run as 14+14+14, not 18+18+6
    const int chunks = (g.count + nb - 1) / nb;
    nb = (g.count + chunks - 1) / chunks;
    g.ns_batch = nb;

    ns_max = std::max(ns_max, per_mat * nb);
    // one partial per CTA of the pre-pass: 64 x 64 tiles (tall), 4 rows x 2048 columns (wide), or
    // one per CTA of the persistent kernel (at most 256)
    fro_max = std::max(fro_max, (size_t)nb * std::max({(size_t)((g.rp / 64) * (g.cp / 64)),
                                                       (size_t)((g.rp / 4) * ((g.cp + 2047) / 2048)), (size_t)256}));
    batch_max = std::max(batch_max, nb);
  }
  c->off_fro = off;   off = align_up(off + fro_max * 4, 256);
  c->off_alpha = off; off = align_up(off + (size_t)batch_max * 4, 256);
  c->off_ns = off;    off += ns_max;
  c->total_bytes = off;
}

extern "C" int prm_create(prm_ctx** out, const int64_t* shapes, int n_mats, int K, float beta,
                          int nesterov, float lr, float wd) {
  if (!out) return fail(nullptr, PRM_ERR_ARG, "prm_create: out is NULL");
  *out = nullptr;
  if (!shapes || n_mats < 1) return fail(nullptr, PRM_ERR_ARG, "prm_create: empty shape list");
  if (K < 1) return fail(nullptr, PRM_ERR_ARG, "prm_create: K must be >= 1");
  if (!(beta >= 0.f && beta < 1.f)) return fail(nullptr, PRM_ERR_ARG, "prm_create: beta must be in [0,1)");
  for (int i = 0; i < n_mats; ++i) {
    const int64_t r = shapes[2 * i], cdim = shapes[2 * i + 1];
    if (r < 1 || cdim < 1 || r > 0x7fffffffLL || cdim > 0x7fffffffLL)
      return fail(nullptr, PRM_ERR_SHAPE, "prm_create: dimension out of range");
    if (round_up(std::min(r, cdim), kPad) > 65536 || round_up(std::max(r, cdim), kPad) > (1 << 22))
      return fail(nullptr, PRM_ERR_SHAPE, "prm_create: min(rows,cols) > 65536 or max > 4194304 unsupported");
  }
  prm_ctx* c = new (std::nothrow) prm_ctx();
  if (!c) return fail(nullptr, PRM_ERR_ARG, "prm_create: out of host memory");
  c->n_mats = n_mats;
  c->shapes.assign(shapes, shapes + 2 * n_mats);
  c->K = K; c->beta = beta; c->nesterov = nesterov ? 1 : 0; c->lr = lr; c->wd = wd;
  // Grouping: exact (rows, cols); ids by first appearance; caller order inside.
  c->group_of_mat.resize(n_mats);
  c->order_in_group.resize(n_mats);
  for (int i = 0; i < n_mats; ++i) {
    const int64_t r = shapes[2 * i], cdim = shapes[2 * i + 1];
    int gi = -1;
    for (size_t k = 0; k < c->groups.size(); ++k)
      if (c->groups[k].rows == r && c->groups[k].cols == cdim) { gi = (int)k; break; }
    if (gi < 0) {
      Group g;
      g.rows = r; g.cols = cdim; g.tall = r > cdim;
      g.r = std::min(r, cdim); g.c = std::max(r, cdim);
      g.rp = round_up(g.r, kPad); g.cp = round_up(g.c, kPad);
      c->groups.push_back(g);
      gi = (int)c->groups.size() - 1;
    }
    c->group_of_mat[i] = gi;
    c->order_in_group[i] = c->groups[gi].count++;
  }
  int first = 0;
  for (Group& g : c->groups) { g.first = first; first += g.count; }
  c->slot_of_mat.resize(n_mats);
  for (int i = 0; i < n_mats; ++i)
    c->slot_of_mat[i] = c->groups[c->group_of_mat[i]].first + c->order_in_group[i];
  c->host_tables.assign((size_t)3 * n_mats, nullptr);
  c->host_pmaps.assign((size_t)128 * n_mats, 0);
  c->host_rmaps.assign((size_t)384 * n_mats, 0);
  compute_layout(c);
  *out = c;
  return PRM_OK;
}

extern "C" int prm_set_option(prm_ctx* c, int key, double v) {
  if (!c) return PRM_ERR_ARG;
  const bool attached = c->ws != nullptr;
  switch (key) {
    case PRM_OPT_GAMMA: if (!(v > 0)) return fail(c, PRM_ERR_ARG, "gamma must be > 0"); c->gamma = (float)v; return PRM_OK;
    case PRM_OPT_EPS_ROW: if (v < 0) return fail(c, PRM_ERR_ARG, "eps_row must be >= 0"); c->eps_row = (float)v; return PRM_OK;
    case PRM_OPT_EPS_NS: if (v < 0) return fail(c, PRM_ERR_ARG, "eps_ns must be >= 0"); c->eps_ns = (float)v; return PRM_OK;
    case PRM_OPT_SCALE_MODE:
      if (v != 0 && v != 1 && v != 2) return fail(c, PRM_ERR_ARG, "scale mode must be 0, 1 or 2");
      c->scale_mode = (int)v; return PRM_OK;
    case PRM_OPT_LR: c->lr = (float)v; return PRM_OK;
    case PRM_OPT_WD: c->wd = (float)v; return PRM_OK;
    case PRM_OPT_GAMMA_NS: if (!(v > 0)) return fail(c, PRM_ERR_ARG, "gamma_ns must be > 0"); c->gamma_ns = (float)v; return PRM_OK;
    case PRM_OPT_NO_REFRESH:
      if (v != 0 && v != 1) return fail(c, PRM_ERR_ARG, "value must be 0 or 1");
      c->no_refresh = (int)v; return PRM_OK;
    case PRM_OPT_WIDE_KERNEL:
      if (v != 0 && v != 1) return fail(c, PRM_ERR_ARG, "value must be 0 or 1");
      c->wide_kernel = (int)v; return PRM_OK;
    case PRM_OPT_TALL_KERNEL:
      if (attached) return fail(c, PRM_ERR_STATE, "option must be set before prm_set_workspace");
      if (v != 0 && v != 1 && v != 2) return fail(c, PRM_ERR_ARG, "value must be 0, 1 or 2");
      c->tall_kernel = (int)v; return PRM_OK;
    case PRM_OPT_NS_SPLIT_INPUT:
      if (attached) return fail(c, PRM_ERR_STATE, "option must be set before prm_set_workspace");
      if (v != 0 && v != 1) return fail(c, PRM_ERR_ARG, "value must be 0 or 1");
      c->split_input = (int)v;
      compute_layout(c);
      return PRM_OK;
    case PRM_OPT_IO_DTYPE:
    case PRM_OPT_CHECK_MODE:
    case PRM_OPT_NS_GRAM_SPAN:
    case PRM_OPT_NS_WORKSPACE_BYTES:
      if (attached) return fail(c, PRM_ERR_STATE, "option must be set before prm_set_workspace");
      if (key == PRM_OPT_NS_WORKSPACE_BYTES) {
        if (v < 0) return fail(c, PRM_ERR_ARG, "workspace cap must be >= 0");
        c->ns_cap = (size_t)v;
      } else {
        if (key == PRM_OPT_NS_GRAM_SPAN) {
          if (v != 0 && v != 1 && v != 2) return fail(c, PRM_ERR_ARG, "value must be 0, 1 or 2");
          c->gram_span = (int)v;
        } else {
          if (v != 0 && v != 1) return fail(c, PRM_ERR_ARG, "value must be 0 or 1");
          (key == PRM_OPT_IO_DTYPE ? c->io_fp32 : c->check_mode) = (int)v;
        }
      }
      compute_layout(c);
      return PRM_OK;
    default: return fail(c, PRM_ERR_ARG, "unknown option key");
  }
}

extern "C" size_t prm_workspace_bytes(const prm_ctx* c) { return c ? c->total_bytes : 0; }

extern "C" int prm_set_workspace(prm_ctx* c, void* dev_ptr, size_t bytes) {
  if (!c) return PRM_ERR_ARG;
  if (!dev_ptr) return fail(c, PRM_ERR_ARG, "prm_set_workspace: NULL pointer");
  if (((uintptr_t)dev_ptr & 255) != 0) return fail(c, PRM_ERR_ALIGN, "prm_set_workspace: pointer not 256-byte aligned");
  if (bytes < c->total_bytes) return fail(c, PRM_ERR_WORKSPACE, "prm_set_workspace: workspace too small");
  cudaError_t e = cudaMemset(dev_ptr, 0, 256);
  if (e != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("prm_set_workspace: ") + cudaGetErrorString(e));
  c->ws = (char*)dev_ptr;
  c->ws_bytes = bytes;
  c->tables_uploaded = false;
  if (!c->tc) {
    // The tensor-core products need this context; the streaming row step only uses it where it
    // exists (its tensor maps), so the fp32 check mode works without one.
    std::string err;
    c->tc = tc_create(&err);
    if (!c->tc && !c->check_mode) { c->ws = nullptr; return fail(c, PRM_ERR_CUDA, "prm_set_workspace: " + err); }
  }
  for (Group& g : c->groups) {
    g.stream = TallStreamPlan();
    // The streaming kernel is opt-in: it moves 14 instead of 20 bytes per element, but it is
    // bound by instruction issue and loses to the two passes at the reduced SM clock that
    // follows a power-capped refresh (see rowstep_stream.cu).
    if (!g.tall || !c->tc || c->tall_kernel != 2) continue;
    const TallStreamPlan p = tall_stream_plan(g.rows, g.cols, c->io_fp32, tc_sm_count(c->tc));
    if (p.ok) g.stream = p;
  }
  return PRM_OK;
}

extern "C" int prm_plan(const prm_ctx* c, int64_t step_idx, int* is_refresh, int* n_groups,
                        int* group_of_mat, int* order_in_group) {
  if (!c || step_idx < 0) return PRM_ERR_ARG;
  if (is_refresh) *is_refresh = ((step_idx % c->K) == 0 && !c->no_refresh) ? 1 : 0;
  if (n_groups) *n_groups = (int)c->groups.size();
  if (group_of_mat) memcpy(group_of_mat, c->group_of_mat.data(), sizeof(int) * c->n_mats);
  if (order_in_group) memcpy(order_in_group, c->order_in_group.data(), sizeof(int) * c->n_mats);
  return PRM_OK;
}

extern "C" int prm_group_info(const prm_ctx* c, int group, int64_t* rows, int64_t* cols, int* count,
                              int* ns_batch, int* gram_iters, double* ns5_flop) {
  if (!c || group < 0 || group >= (int)c->groups.size()) return PRM_ERR_ARG;
  const Group& g = c->groups[group];
  if (rows) *rows = g.rows;
  if (cols) *cols = g.cols;
  if (count) *count = g.count;
  if (ns_batch) *ns_batch = g.ns_batch;
  if (gram_iters) *gram_iters = g.gram_iters;
  if (ns5_flop) *ns5_flop = ns5_schedule(g.r, g.c, c->gram_span, g.ns_fp32 != 0, g.split != 0).flop;
  return PRM_OK;
}

// Where the last NS5 iteration puts its result: straight into the parameters
// (Eq. periodic-direction with rho_t = 1), or, with no NsFinal, into the
// workspace as X_5.
struct NsFinal {
  PtrTables tables;
  int first;          // table index of the sub-batch's first matrix
  float decay, lr_s;
};

// The NS5 products of one sub-batch of nb matrices of group g whose oriented
// input U already sits in the first X buffer of the NS5 region, alpha computed.
// *x_out receives the X buffer that holds X_5 when fin is null.
// split: X_0 was written as a pair of bf16 planes per matrix (Group::split, Gram-space order
// only); the first X buffer is then twice as large and is reused as an ordinary X buffer
// once X_3 exists.
static cudaError_t ns5_products(prm_ctx* c, const Group& g, int nb, const NsFinal* fin, const char** x_out,
                                cudaStream_t stream, bool split = false) {
  const size_t e = g.ns_fp32 ? 4 : 2;
  const int64_t rc = g.rp * g.cp, rr = g.rp * g.rp;
  float* alpha = (float*)(c->ws + c->off_alpha);
  int* status = (int*)(c->ws + c->off_status);
  char* base = c->ws + c->off_ns;
  const int x0_planes = g.split ? 2 : 1;           // the layout always leaves room for the pair
  if (split && (!g.split || !g.gram_iters || g.ns_fp32)) return cudaErrorInvalidValue;
  char* X[2] = {base, base + (size_t)x0_planes * e * rc * nb};
  char* R[4];                                      // r x r matrices (lower blocks)
  for (int k = 0; k < 4; ++k) R[k] = base + (size_t)(x0_planes + 1) * e * rc * nb + (size_t)k * e * rr * nb;
  char* A = R[0];
  char* B = R[1];
  cudaError_t ce;
  auto gemm = [&](const GemmProblem& pb, const Epilogue& ep, int cls) -> cudaError_t {
    ProfScope ps(c, cls, stream);
    return g.ns_fp32 ? launch_gemm_simt(pb, ep, stream, &c->launches)
                     : launch_gemm_tc(c->tc, pb, ep, status, stream, &c->launches);
  };
  int cur = 0, it0 = 0;
  ce = cudaSuccess;
  if (g.gram_iters) {
    // The first three iterations without touching X (tensor-core path).  With
    // P_k = aI + B_k, B_k = bA_k + cA_k^2, the recurrence reads X_{k+1} = P_k X_k
    // and A_{k+1} = X_{k+1} X_{k+1}^T = P_k A_k P_k, all polynomials in A_0 and
    // therefore symmetric and commuting.  So A_1, A_2 follow from r x r products,
    // and X_3 = (P_2 P_1 P_0) X_0 = a^3 X_0 + Q X_0 needs one r x c product, where
    // Q (the product without its a^3 I term, which stays an fp32 coefficient) is
    // accumulated beside.  In exact arithmetic this is the printed recurrence;
    // the last two iterations, whose rounding decides the error, run as printed.
    auto sym = [&](const char* Pm, const char* Qm, float k_acc, const char* aux, float k_aux, const char* aux2,
                   float k_aux2, char* dst, int cls) -> cudaError_t {
      GemmProblem pb;
      pb.P = Pm; pb.Q = Qm; pb.Mp = g.rp; pb.Np = g.rp; pb.Kp = g.rp;
      pb.bs_P = rr; pb.bs_Q = rr; pb.batch = nb; pb.symmetric = 1; pb.sym_ops = 3;
      Epilogue ep;
      ep.k_acc = k_acc; ep.k_aux = k_aux; ep.aux = aux; ep.ld_aux = g.rp; ep.bs_aux = rr;
      if (aux2) { ep.aux2 = aux2; ep.k_aux2 = k_aux2; ep.ld_aux2 = g.rp; ep.bs_aux2 = rr; }
      ep.dst = dst; ep.ld_dst = g.rp; ep.bs_dst = rr;
      return gemm(pb, ep, cls);
    };
    auto poly = [&](const char* Am, char* Bm) { return sym(Am, Am, kNsC, Am, kNsB, nullptr, 0.f, Bm, PRM_PROF_POLY); };
    const float a = kNsA;
    GemmProblem pa;
    pa.P = X[0]; pa.Q = X[0]; pa.Mp = g.rp; pa.Np = g.rp; pa.Kp = g.cp;
    pa.bs_P = rc; pa.bs_Q = rc; pa.batch = nb; pa.symmetric = 1;
    if (split) { pa.split = 1; pa.bs_P = pa.bs_Q = 2 * rc; }
    Epilogue ea;
    ea.dst = R[0]; ea.ld_dst = g.rp; ea.bs_dst = rr; ea.alpha = alpha; ea.alpha_pow = 2;
    ce = gemm(pa, ea, PRM_PROF_GRAM);                                                          // A_0
    if (ce == cudaSuccess) ce = poly(R[0], R[1]);                                              // B_0
    if (ce == cudaSuccess) ce = sym(R[0], R[1], 1.f, R[0], a, nullptr, 0.f, R[2], PRM_PROF_GRAMSPACE);   // Z = A_0 P_0
    if (ce == cudaSuccess) ce = sym(R[2], R[1], 1.f, R[2], a, nullptr, 0.f, R[0], PRM_PROF_GRAMSPACE);   // A_1 = Z P_0
    if (ce == cudaSuccess) ce = poly(R[0], R[3]);                                              // B_1
    if (ce == cudaSuccess)                                                                     // Q = P_1 P_0 - a^2 I
      ce = sym(R[3], R[1], 1.f, R[1], a, R[3], a, R[2], PRM_PROF_GRAMSPACE);
    if (ce == cudaSuccess) ce = sym(R[0], R[3], 1.f, R[0], a, nullptr, 0.f, R[1], PRM_PROF_GRAMSPACE);   // Z = A_1 P_1
    if (ce == cudaSuccess) ce = sym(R[1], R[3], 1.f, R[1], a, nullptr, 0.f, R[0], PRM_PROF_GRAMSPACE);   // A_2 = Z P_1
    if (ce == cudaSuccess) ce = poly(R[0], R[3]);                                              // B_2
    if (ce == cudaSuccess)                                                                     // Q = P_2 P_1 P_0 - a^3 I
      ce = sym(R[3], R[2], 1.f, R[2], a, R[3], a * a, R[1], PRM_PROF_GRAMSPACE);
    if (ce == cudaSuccess) {                                                                   // X_3 = alpha (a^3 X_0 + Q X_0)
      GemmProblem pu;
      pu.P = R[1]; pu.Q = X[0]; pu.q_mn = 1; pu.sym_ops = 1; pu.Mp = g.rp; pu.Np = g.cp; pu.Kp = g.rp;
      pu.bs_P = rr; pu.bs_Q = rc; pu.batch = nb; pu.symmetric = 0;
      Epilogue eu;
      eu.k_acc = 1.f; eu.k_aux = a * a * a; eu.aux = X[0]; eu.ld_aux = g.cp; eu.bs_aux = rc;
      if (split) { pu.split = 1; pu.bs_Q = 2 * rc; eu.bs_aux = 2 * rc; }
      eu.alpha = alpha; eu.alpha_pow = 1;
      eu.dst = X[1]; eu.ld_dst = g.cp; eu.bs_dst = rc;
      ce = gemm(pu, eu, PRM_PROF_UPDATE);
    }
    cur = 1;
    it0 = kGramIters;
  }
  for (int it = it0; it < kNsIters && ce == cudaSuccess; ++it) {
    // A = X X^T (times alpha^2 in the first iteration), unless the previous iteration already
    // produced it from its own Gram matrix
    if (!(g.last_gram_rec && it == kNsIters - 1)) {
      GemmProblem pa;
      pa.P = X[cur]; pa.Q = X[cur]; pa.Mp = g.rp; pa.Np = g.rp; pa.Kp = g.cp;
      pa.bs_P = rc; pa.bs_Q = rc; pa.batch = nb; pa.symmetric = 1;
      Epilogue ea;
      ea.dst = A; ea.ld_dst = g.rp; ea.bs_dst = rr;   // blocks on and below the diagonal only
      if (it == 0) { ea.alpha = alpha; ea.alpha_pow = 2; }
      if ((ce = gemm(pa, ea, PRM_PROF_GRAM)) != cudaSuccess) break;
    }
    // B = b A + c A^2
    GemmProblem pp;
    pp.P = A; pp.Q = A; pp.Mp = g.rp; pp.Np = g.rp; pp.Kp = g.rp;
    pp.bs_P = rr; pp.bs_Q = rr; pp.batch = nb; pp.symmetric = 1; pp.sym_ops = 3;
    Epilogue eb;
    eb.k_acc = kNsC; eb.k_aux = kNsB; eb.aux = A; eb.ld_aux = g.rp; eb.bs_aux = rr;
    eb.dst = B; eb.ld_dst = g.rp; eb.bs_dst = rr;
    if ((ce = gemm(pp, eb, PRM_PROF_POLY)) != cudaSuccess) break;
    if (g.last_gram_rec && it == kNsIters - 2) {
      // A_4 = (aI + B_3) A_3 (aI + B_3) from r x r products: Z = aA_3 + A_3 B_3, then A_4 = aZ + Z B_3.
      // X_4 is still formed below with B_3; only the Gram matrix of the last iteration is not
      // recomputed from the rounded X_4.
      auto step = [&](const char* Pm, char* dst) -> cudaError_t {
        GemmProblem pb;
        pb.P = Pm; pb.Q = B; pb.Mp = g.rp; pb.Np = g.rp; pb.Kp = g.rp;
        pb.bs_P = rr; pb.bs_Q = rr; pb.batch = nb; pb.symmetric = 1; pb.sym_ops = 3;
        Epilogue ep;
        ep.k_acc = 1.f; ep.k_aux = kNsA; ep.aux = Pm; ep.ld_aux = g.rp; ep.bs_aux = rr;
        ep.dst = dst; ep.ld_dst = g.rp; ep.bs_dst = rr;
        return gemm(pb, ep, PRM_PROF_GRAMSPACE);
      };
      if ((ce = step(A, R[2])) != cudaSuccess) break;
      if ((ce = step(R[2], A)) != cudaSuccess) break;       // A_3 is no longer needed: A now holds A_4
    }
    // X <- a X + B X (times alpha in the first iteration); last iteration
    // goes straight into the parameters.
    GemmProblem pu;
    // (B X)[i,j] = sum_k B[i,k] X[k,j]: X itself is the second operand, read with j contiguous.
    pu.P = B; pu.Q = X[cur]; pu.q_mn = 1; pu.sym_ops = 1; pu.Mp = g.rp; pu.Np = g.cp; pu.Kp = g.rp;
    pu.bs_P = rr; pu.bs_Q = rc; pu.batch = nb; pu.symmetric = 0;
    Epilogue eu;
    eu.k_acc = 1.f; eu.k_aux = kNsA; eu.aux = X[cur]; eu.ld_aux = g.cp; eu.bs_aux = rc;
    if (it == 0) { eu.alpha = alpha; eu.alpha_pow = 1; }
    if (it + 1 < kNsIters) {
      eu.dst = X[cur ^ 1]; eu.ld_dst = g.cp; eu.bs_dst = rc;
    } else if (!fin) {
      eu.dst = X[cur ^ 1]; eu.ld_dst = g.cp; eu.bs_dst = rc;     // X_5 stays in the workspace
    } else {
      eu.kind = 1; eu.tables = fin->tables; eu.first = fin->first;
      eu.rows = (int)g.rows; eu.cols = (int)g.cols; eu.tall = g.tall ? 1 : 0;
      eu.io_fp32 = c->io_fp32; eu.decay = fin->decay; eu.lr_s = fin->lr_s;
      // bf16 parameters with 16-byte aligned rows are updated through TMA-staged tiles.
      if (!g.ns_fp32 && !c->io_fp32 && g.cols % 8 == 0) eu.param_maps = c->ws + c->off_pmaps;
    }
    if ((ce = gemm(pu, eu, it + 1 < kNsIters ? PRM_PROF_UPDATE : PRM_PROF_UPDATE_FINAL)) != cudaSuccess) break;
    cur ^= 1;
  }
  if (x_out) *x_out = X[cur];
  return ce;
}

static int refresh_group(prm_ctx* c, const Group& g, const PtrTables& t, StepScalars s,
                         cudaStream_t stream) {
  float* fro = (float*)(c->ws + c->off_fro);
  float* alpha = (float*)(c->ws + c->off_alpha);
  for (int done = 0; done < g.count; done += g.ns_batch) {
    const int nb = std::min(g.ns_batch, g.count - done);
    const int first = g.first + done;
    cudaError_t ce;
    {
      ProfScope ps(c, PRM_PROF_PREPASS, stream);
      const int n_sm = tc_sm_count(c->tc);
      if (c->wide_kernel != 1 && n_sm > 0 && prepass_stream_takes(g, c->io_fp32, g.ns_fp32)) {
        ce = launch_ns_prepass_stream(t, g, first, nb, s, g.split, c->ws + c->off_ns, fro, n_sm,
                                      (int*)(c->ws + c->off_status), stream);
        if (ce == cudaSuccess) {
          launch_ns_alpha(fro, prepass_stream_parts(n_sm, g.rp, nb), s.eps_ns, alpha, nb, stream);
          ce = cudaGetLastError();
        }
        c->launches += 2;
      } else {
        ce = launch_ns_prepass(t, g, first, nb, s, c->io_fp32, g.ns_fp32, g.split, c->ws + c->off_ns, fro, alpha,
                               stream, &c->launches);
      }
    }
    if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("pre-pass: ") + cudaGetErrorString(ce));
    NsFinal fin{t, first, s.decay, s.lr_s * c->gamma_ns};
    ce = ns5_products(c, g, nb, &fin, nullptr, stream, g.split != 0);
    if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("NS5 product: ") + cudaGetErrorString(ce));
  }
  return PRM_OK;
}

// Refresh of a bucket of matrices whose rows sit in one segment per rank
// (Algorithm 2 lines 4-6 for one bucket, on one rank).
extern "C" int prm_refresh_segments(prm_ctx* c, const int* mats, int n, const void* const* segments,
                                    int64_t segment_elems, const int64_t* offsets, int world, int rank,
                                    void* const* param_shards, void* cuda_stream) {
  if (!c) return PRM_ERR_ARG;
  if (!c->ws) return fail(c, PRM_ERR_WORKSPACE, "prm_refresh_segments: no workspace attached");
  if (n < 0 || (n > 0 && (!mats || !offsets || !param_shards || !segments)))
    return fail(c, PRM_ERR_ARG, "prm_refresh_segments: NULL argument");
  if (world < 1 || rank < 0 || rank >= world) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: bad world or rank");
  if (world > kMaxWorld) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: more than 64 ranks");
  if (segment_elems < 0) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: negative segment size");
  SegmentPtrs segs = {};
  bool vec_ok = true;
  for (int q = 0; q < world && n > 0; ++q) {
    if (!segments[q]) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: NULL segment pointer");
    if (((uintptr_t)segments[q] & 1) != 0) return fail(c, PRM_ERR_ALIGN, "prm_refresh_segments: segment not 2-byte aligned");
    vec_ok = vec_ok && ((uintptr_t)segments[q] & 15) == 0;
    segs.seg[q] = segments[q];
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  for (int k = 0; k < n; ++k) {
    if (mats[k] < 0 || mats[k] >= c->n_mats) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: matrix index out of range");
    const Group& g = c->groups[c->group_of_mat[mats[k]]];
    const int64_t chunk = shard_chunk(g.rows, world);
    if (offsets[k] < 0 || offsets[k] + chunk * g.cols > segment_elems)
      return fail(c, PRM_ERR_SHAPE, "prm_refresh_segments: a matrix does not fit its segment");
    int64_t start, count;
    shard_rows(g.rows, world, rank, &start, &count);
    if (count > 0) {
      if (!param_shards[k]) return fail(c, PRM_ERR_ARG, "prm_refresh_segments: NULL parameter shard");
      if (((uintptr_t)param_shards[k] & (c->io_fp32 ? 3 : 1)) != 0)
        return fail(c, PRM_ERR_ALIGN, "prm_refresh_segments: parameter shard not aligned to its element size");
    }
  }
  float* fro = (float*)(c->ws + c->off_fro);
  float* alpha = (float*)(c->ws + c->off_alpha);
  std::vector<int64_t> offs;
  std::vector<void*> shards;
  for (size_t gi = 0; gi < c->groups.size(); ++gi) {
    const Group& g = c->groups[gi];
    const size_t e = g.ns_fp32 ? 4 : 2;
    offs.clear();
    shards.clear();
    for (int k = 0; k < n; ++k)
      if (c->group_of_mat[mats[k]] == (int)gi) { offs.push_back(offsets[k]); shards.push_back(param_shards[k]); }
    if (offs.empty()) continue;
    int64_t row_start, rows_local;
    shard_rows(g.rows, world, rank, &row_start, &rows_local);
    const float decay = 1.f - c->lr * c->wd;
    const float lr_s = c->lr * shape_scale(c->scale_mode, g.rows, g.cols) * c->gamma_ns;
    const int total = (int)offs.size();
    for (int done = 0; done < total; done += g.ns_batch) {
      const int nb = std::min(g.ns_batch, total - done);
      cudaError_t ce;
      {
        ProfScope ps(c, PRM_PROF_PREPASS, stream);
        ce = launch_ns_gather_prepass(segs, vec_ok, shard_chunk(g.rows, world), offs.data() + done, g, nb,
                                      c->eps_ns, g.ns_fp32, c->ws + c->off_ns, fro, alpha, stream, &c->launches);
      }
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("gathered pre-pass: ") + cudaGetErrorString(ce));
      const char* X5 = nullptr;
      ce = ns5_products(c, g, nb, nullptr, &X5, stream);
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("NS5 product: ") + cudaGetErrorString(ce));
      {
        ProfScope ps(c, PRM_PROF_UPDATE_FINAL, stream);
        ce = launch_ns_slice_update(X5, g.ns_fp32, g, nb, shards.data() + done, row_start, rows_local, c->io_fp32,
                                    decay, lr_s, stream, &c->launches);
      }
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("slice update: ") + cudaGetErrorString(ce));
    }
  }
  return PRM_OK;
}

// The same with the segments laid out one after the other in one buffer, as an
// all-gather delivers them.
extern "C" int prm_refresh_gathered(prm_ctx* c, const int* mats, int n, const void* gathered,
                                    int64_t segment_elems, const int64_t* offsets, int world, int rank,
                                    void* const* param_shards, void* cuda_stream) {
  if (!c) return PRM_ERR_ARG;
  if (world < 1 || world > kMaxWorld) return fail(c, PRM_ERR_ARG, "prm_refresh_gathered: bad world (1..64)");
  if (n > 0 && !gathered) return fail(c, PRM_ERR_ARG, "prm_refresh_gathered: NULL argument");
  if (segment_elems < 0) return fail(c, PRM_ERR_ARG, "prm_refresh_gathered: negative segment size");
  if (((uintptr_t)gathered & 15) != 0) return fail(c, PRM_ERR_ALIGN, "prm_refresh_gathered: buffer not 16-byte aligned");
  const void* segs[kMaxWorld];
  for (int q = 0; q < world; ++q) segs[q] = (const char*)gathered + (size_t)q * (size_t)segment_elems * 2;
  return prm_refresh_segments(c, mats, n, segs, segment_elems, offsets, world, rank, param_shards, cuda_stream);
}

static int step_impl(prm_ctx* c, void* const* params, void* const* grads_dev,
                     const void* const* grads_host, float* const* momentum, int64_t step_idx,
                     cudaStream_t stream) {
  if (!c) return PRM_ERR_ARG;
  if (!params || !grads_dev || !momentum) return fail(c, PRM_ERR_ARG, "prm_step: NULL pointer array");
  if (step_idx < 0) return fail(c, PRM_ERR_ARG, "prm_step: negative step index");
  if (!c->ws) return fail(c, PRM_ERR_WORKSPACE, "prm_step: no workspace attached");
  bool changed = !c->tables_uploaded;
  const int n = c->n_mats;
  for (int i = 0; i < n; ++i) {
    if (!params[i] || !grads_dev[i] || !momentum[i]) return fail(c, PRM_ERR_ARG, "prm_step: NULL matrix pointer");
    if ((((uintptr_t)params[i] | (uintptr_t)grads_dev[i] | (uintptr_t)momentum[i]) & 15) != 0)
      return fail(c, PRM_ERR_ALIGN, "prm_step: matrix pointer not 16-byte aligned");
    const int slot = c->slot_of_mat[i];
    void* want[3] = {params[i], grads_dev[i], (void*)momentum[i]};
    for (int k = 0; k < 3; ++k) {
      if (c->host_tables[(size_t)k * n + slot] != want[k]) { c->host_tables[(size_t)k * n + slot] = want[k]; changed = true; }
    }
  }
  cudaError_t ce;
  if (changed) {
    // Pageable source: the runtime stages the bytes before returning.
    ce = cudaMemcpyAsync(c->ws + c->off_tables, c->host_tables.data(), (size_t)3 * n * sizeof(void*),
                         cudaMemcpyHostToDevice, stream);
    if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("pointer tables: ") + cudaGetErrorString(ce));
    if (!c->check_mode && !c->io_fp32) {
      for (int i = 0; i < n; ++i) {
        const Group& g = c->groups[c->group_of_mat[i]];
        if (g.cols % 8 != 0 || g.ns_fp32) continue;
        if (!tc_encode_param_map(c->tc, params[i], g.rows, g.cols, g.tall ? 1 : 0,
                                 c->host_pmaps.data() + (size_t)128 * c->slot_of_mat[i]))
          return fail(c, PRM_ERR_CUDA, "cannot encode a tensor map over a parameter matrix");
      }
      ce = cudaMemcpyAsync(c->ws + c->off_pmaps, c->host_pmaps.data(), (size_t)128 * n, cudaMemcpyHostToDevice, stream);
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("parameter tensor maps: ") + cudaGetErrorString(ce));
    }
    bool any_stream = false;
    for (int i = 0; i < n; ++i) {
      const Group& g = c->groups[c->group_of_mat[i]];
      if (!g.stream.ok) continue;
      any_stream = true;
      unsigned char* dst = c->host_rmaps.data() + (size_t)384 * c->slot_of_mat[i];
      const int pw = tall_stream_panel();
      if (!tc_encode_tile_map(c->tc, grads_dev[i], g.rows, g.cols, 2, pw, g.stream.R, dst) ||
          !tc_encode_tile_map(c->tc, momentum[i], g.rows, g.cols, 4, pw, g.stream.R, dst + 128) ||
          !tc_encode_tile_map(c->tc, params[i], g.rows, g.cols, 2, pw, g.stream.R, dst + 256))
        return fail(c, PRM_ERR_CUDA, "cannot encode the tensor maps of the streaming row step");
    }
    if (any_stream) {
      ce = cudaMemcpyAsync(c->ws + c->off_rmaps, c->host_rmaps.data(), (size_t)384 * n, cudaMemcpyHostToDevice, stream);
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("row-step tensor maps: ") + cudaGetErrorString(ce));
    }
    c->tables_uploaded = true;
  }
  if (grads_host) {
    const size_t esz = c->io_fp32 ? 4 : 2;
    for (int i = 0; i < n; ++i)
      if (!grads_host[i]) return fail(c, PRM_ERR_ARG, "prm_step_h2d: NULL host gradient pointer");
    if (!c->copy_stream) {
      ce = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
      if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&c->copy_begin, cudaEventDisableTiming);
      c->copy_done.assign(c->groups.size(), nullptr);
      for (size_t k = 0; k < c->groups.size() && ce == cudaSuccess; ++k)
        ce = cudaEventCreateWithFlags(&c->copy_done[k], cudaEventDisableTiming);
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("copy stream: ") + cudaGetErrorString(ce));
    }
    // The copies may not overtake work already queued on the caller's stream
    // (the previous step still reads the gradient buffers).
    ce = cudaEventRecord(c->copy_begin, stream);
    if (ce == cudaSuccess) ce = cudaStreamWaitEvent(c->copy_stream, c->copy_begin, 0);
    for (size_t k = 0; k < c->groups.size() && ce == cudaSuccess; ++k) {
      for (int i = 0; i < n && ce == cudaSuccess; ++i) {
        if (c->group_of_mat[i] != (int)k) continue;
        ce = cudaMemcpyAsync(grads_dev[i], grads_host[i], esz * (size_t)c->shapes[2 * i] * (size_t)c->shapes[2 * i + 1],
                             cudaMemcpyHostToDevice, c->copy_stream);
      }
      if (ce == cudaSuccess) ce = cudaEventRecord(c->copy_done[k], c->copy_stream);
    }
    if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("gradient copy: ") + cudaGetErrorString(ce));
  }
  PtrTables t;
  void** tb = (void**)(c->ws + c->off_tables);
  t.params = tb;
  t.grads = (const void**)(tb + n);
  t.momentum = (float**)(tb + 2 * n);
  const bool refresh = (step_idx % c->K) == 0 && !c->no_refresh;
  for (size_t gi = 0; gi < c->groups.size(); ++gi) {
    const Group& g = c->groups[gi];
    if (grads_host) {
      ce = cudaStreamWaitEvent(stream, c->copy_done[gi], 0);   // this group's gradients have landed
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("gradient copy: ") + cudaGetErrorString(ce));
    }
    StepScalars s;
    s.beta = c->beta; s.omb = 1.f - c->beta; s.nesterov = c->nesterov;
    s.decay = 1.f - c->lr * c->wd;
    s.lr_s = c->lr * shape_scale(c->scale_mode, g.rows, g.cols);
    s.gamma = c->gamma; s.eps_row = c->eps_row; s.eps_ns = c->eps_ns;
    if (refresh) {
      int rc = refresh_group(c, g, t, s, stream);
      if (rc != PRM_OK) return rc;
    } else {
      ProfScope ps(c, g.tall ? PRM_PROF_ROW_TALL : PRM_PROF_ROW_WIDE, stream);
      if (g.tall && g.stream.ok)
        ce = launch_rowstep_tall_stream(t, g, s, g.stream, c->ws + c->off_rmaps + (size_t)384 * g.first,
                                        (float*)(c->ws + g.tall_scratch_off), (float*)(c->ws + g.tall_nu_off),
                                        (int*)(c->ws + g.tall_sync_off), (int*)(c->ws + c->off_status),
                                        tc_sm_count(c->tc), stream, &c->launches);
      else if (!g.tall && c->wide_kernel != 1 && tc_sm_count(c->tc) > 0 && wide_stream_takes(g, c->io_fp32))
        ce = launch_rowstep_wide_stream(t, g, s, tc_sm_count(c->tc), (int*)(c->ws + c->off_status), stream,
                                        &c->launches);
      else
        ce = launch_rowstep(t, g, s, c->io_fp32, (float*)(c->ws + g.tall_scratch_off),
                            (float*)(c->ws + g.tall_nu_off), stream, &c->launches);
      if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("row step: ") + cudaGetErrorString(ce));
    }
  }
  return PRM_OK;
}

extern "C" int prm_step(prm_ctx* c, void* const* params, const void* const* grads,
                        float* const* momentum, int64_t step_idx, void* cuda_stream) {
  return step_impl(c, params, (void* const*)grads, nullptr, momentum, step_idx, (cudaStream_t)cuda_stream);
}

extern "C" int prm_step_h2d(prm_ctx* c, void* const* params, void* const* grads_dev,
                            const void* const* grads_host, float* const* momentum,
                            int64_t step_idx, void* cuda_stream) {
  if (c && !grads_host) return fail(c, PRM_ERR_ARG, "prm_step_h2d: NULL host gradient array");
  return step_impl(c, params, grads_dev, grads_host, momentum, step_idx, (cudaStream_t)cuda_stream);
}

extern "C" int prm_status(prm_ctx* c) {
  if (!c) return PRM_ERR_ARG;
  if (!c->ws) return fail(c, PRM_ERR_WORKSPACE, "prm_status: no workspace attached");
  cudaError_t ce = cudaDeviceSynchronize();
  int word = 0;
  if (ce == cudaSuccess) ce = cudaMemcpy(&word, c->ws + c->off_status, sizeof(int), cudaMemcpyDeviceToHost);
  if (ce == cudaSuccess && word != 0) ce = cudaMemset(c->ws + c->off_status, 0, sizeof(int));
  if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("prm_status: ") + cudaGetErrorString(ce));
  if (word & kStatusTimeout) return fail(c, PRM_ERR_DEVICE_TIMEOUT, "a device-side wait gave up");
  return PRM_OK;
}

extern "C" int prm_profile(prm_ctx* c, int enable) {
  if (!c) return PRM_ERR_ARG;
  if (enable && c->prof_ev.empty()) {
    c->prof_ev.resize(2 * kProfPairs);
    for (size_t i = 0; i < c->prof_ev.size(); ++i) {
      cudaError_t ce = cudaEventCreate(&c->prof_ev[i]);
      if (ce != cudaSuccess) {
        for (size_t k = 0; k < i; ++k) cudaEventDestroy(c->prof_ev[k]);
        c->prof_ev.clear();
        return fail(c, PRM_ERR_CUDA, std::string("prm_profile: ") + cudaGetErrorString(ce));
      }
    }
    c->prof_cls.assign(kProfPairs, 0);
    c->prof_launches.assign(kProfPairs, 0);
  }
  c->prof_on = enable != 0;
  c->prof_used = 0;
  c->prof_dropped = 0;
  return PRM_OK;
}

extern "C" int prm_profile_read(prm_ctx* c, double* ms, int64_t* launches, int n_classes) {
  if (!c || !ms || !launches || n_classes < 1) return PRM_ERR_ARG;
  for (int k = 0; k < n_classes; ++k) { ms[k] = 0.0; launches[k] = 0; }
  for (size_t i = 0; i < c->prof_used; ++i) {
    cudaError_t ce = cudaEventSynchronize(c->prof_ev[2 * i + 1]);
    float t = 0.f;
    if (ce == cudaSuccess) ce = cudaEventElapsedTime(&t, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]);
    if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("prm_profile_read: ") + cudaGetErrorString(ce));
    const int cls = c->prof_cls[i];
    if (cls < n_classes) { ms[cls] += t; launches[cls] += c->prof_launches[i]; }
  }
  const bool dropped = c->prof_dropped != 0;
  c->prof_used = 0;
  c->prof_dropped = 0;
  return dropped ? fail(c, PRM_ERR_STATE, "prm_profile_read: event pool overflowed, totals incomplete") : PRM_OK;
}

extern "C" int prm_selftest_timeout(prm_ctx* c, double limit_ms, void* cuda_stream) {
  if (!c) return PRM_ERR_ARG;
  if (!c->ws) return fail(c, PRM_ERR_WORKSPACE, "prm_selftest_timeout: no workspace attached");
  if (!(limit_ms > 0) || limit_ms > 1000.0) return fail(c, PRM_ERR_ARG, "prm_selftest_timeout: limit must be in (0, 1000] ms");
  cudaError_t ce = launch_wait_probe((int*)(c->ws + c->off_status), (uint64_t)(limit_ms * 1e6), nullptr,
                                     (cudaStream_t)cuda_stream);
  c->launches += 1;
  if (ce != cudaSuccess) return fail(c, PRM_ERR_CUDA, std::string("prm_selftest_timeout: ") + cudaGetErrorString(ce));
  return PRM_OK;
}

extern "C" double prm_shape_scale(int mode, int64_t rows, int64_t cols) {
  if (mode < 0 || mode > 2 || rows < 1 || cols < 1) return 0.0;
  return (double)shape_scale(mode, rows, cols);
}

extern "C" const char* prm_last_error(const prm_ctx* c) { return c ? c->err.c_str() : g_create_err.c_str(); }

extern "C" int64_t prm_launch_count(const prm_ctx* c) { return c ? c->launches : 0; }

extern "C" int prm_destroy(prm_ctx* c) {
  if (!c) return PRM_ERR_ARG;
  if (c->tc) tc_destroy(c->tc);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  for (cudaEvent_t e : c->copy_done) if (e) cudaEventDestroy(e);
  if (c->copy_begin) cudaEventDestroy(c->copy_begin);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  delete c;
  return PRM_OK;
}
