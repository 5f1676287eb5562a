// Host side of the spectral-correction library: the C ABI, argument checks, workspace layout and the
// order in which the kernels of one anchor arrival / one optimizer step are queued.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "sc_internal.cuh"

using namespace sc;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int round_up_int(int x, int a) { return (x + a - 1) / a * a; }

// Bump allocator over the workspace; with base == nullptr it only measures.
struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(char* b) : base(b) {}
  template <typename T>
  T* take(size_t count) {
    off = align_up(off);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

struct Dims {
  int rp, rk, l, lp, q;
};

bool derive_dims(int rank, const sc_hparams* hp, Dims* d) {
  if (rank < 0 || rank > kMaxRank) return false;
  int l = hp->sketch_width > 0 ? hp->sketch_width : rank;
  if (l < rank || l > kMaxRank) return false;
  if (hp->power_iters < 0 || hp->power_iters > 16) return false;
  if (hp->warm_power_iters < 0 || hp->warm_power_iters > 16) return false;
  d->rp = rank > 0 ? round_up_int(rank, 16) : 0;
  d->rk = round_up_int(d->rp, 64);
  d->l = l;
  d->lp = rank > 0 ? round_up_int(l, 32) : 0;   // whole 32-column swizzle atoms for the tf32 operands
  d->q = hp->power_iters;
  return true;
}

bool valid_hparams(const sc_hparams* hp) {
  if (!hp) return false;
  if (!(hp->alpha >= 0.f && hp->alpha <= 1.f)) return false;
  if (!(hp->tau_p >= 0.f)) return false;
  if (!(hp->beta_anc >= 0.f && hp->beta_anc < 1.f)) return false;
  if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f)) return false;
  if (!(hp->eps >= 0.f) || !isfinite(hp->lr) || !(hp->weight_decay >= 0.f)) return false;
  if (hp->optimizer != SC_OPT_ADAMW && hp->optimizer != SC_OPT_ADEMAMIX) return false;
  if (hp->optimizer == SC_OPT_ADEMAMIX &&
      (!(hp->beta3 >= 0.f && hp->beta3 < 1.f) || !(hp->mix_alpha >= 0.f) || !isfinite(hp->mix_alpha)))
    return false;
  if (hp->full_spectrum != 0 && hp->full_spectrum != 1) return false;
  if (hp->full_spectrum) {
    if (!(hp->tau_p > 0.f) || hp->grad_dtype != SC_DTYPE_BF16 || hp->optimizer != SC_OPT_ADAMW || hp->max_grad_norm > 0.f)
      return false;
    if (hp->fs_sqrt_iters < 1 || hp->fs_sqrt_iters > 200 || hp->fs_inv_iters < 1 || hp->fs_inv_iters > 200) return false;
  }
  return true;
}

// The full-spectrum variant has no rank and runs its contractions on 256 x 256 tensor-core tiles.
sc_status check_full_spectrum(const sc_shape* shapes, int n_mats, int rank) {
  if (rank != 0) return SC_ERR_INVALID_ARG;
  for (int i = 0; i < n_mats; ++i) {
    if (shapes[i].rows < 256 || shapes[i].cols < 256 || (shapes[i].rows % 8) || (shapes[i].cols % 8)) return SC_ERR_SHAPE;
    if (shapes[i].rows > 8192 || shapes[i].cols > 8192) return SC_ERR_TOO_LARGE;
  }
  return SC_OK;
}

struct ClassKey {
  int64_t m, n;
};

// Groups matrices by shape, in order of first appearance.
void build_classes(const sc_shape* shapes, int n_mats, std::vector<ShapeClass>& classes, std::vector<int>& class_of,
                   std::vector<int>& inst_of) {
  class_of.assign(n_mats, -1);
  inst_of.assign(n_mats, -1);
  for (int i = 0; i < n_mats; ++i) {
    int c = -1;
    for (size_t k = 0; k < classes.size(); ++k)
      if (classes[k].m == shapes[i].rows && classes[k].n == shapes[i].cols) { c = (int)k; break; }
    if (c < 0) {
      classes.emplace_back();
      c = (int)classes.size() - 1;
      classes[c].m = shapes[i].rows;
      classes[c].n = shapes[i].cols;
    }
    class_of[i] = c;
    inst_of[i] = (int)classes[c].mats.size();
    classes[c].mats.push_back(i);
  }
}

int choose_ksplit(const ShapeClass& c) {
  const int64_t tiles = (c.m + 127) / 128 * (int64_t)c.mats.size();
  int ks = 1;   // every K slice keeps >= 1024 columns, so no slice is ever empty
  while (ks < 8 && tiles * ks < 148 * 2 && c.n / (ks * 2) >= 1024) ks *= 2;
  return ks;
}

// Lays the whole workspace out. With p->ws == nullptr nothing is dereferenced: it only measures.
size_t layout(sc_plan* p, bool assign) {
  Carver cv(assign ? p->ws : nullptr);
  const int n_mats = p->n_mats, rp = p->rp, rk = p->rk, lp = p->lp;
  MatDev* tab = cv.take<MatDev>(n_mats);
  float* clip = cv.take<float>(1);
  unsigned* status = cv.take<unsigned>(1);
  unsigned* work = cv.take<unsigned>(1);
  float* stats = cv.take<float>((size_t)n_mats * kStatsFloats);
  if (assign) { p->dev_tab = tab; p->clip_dev = clip; p->status_dev = status; p->work_dev = work; p->stats_dev = stats; }
  for (auto& c : p->classes) {
    int* a = cv.take<int>(c.mats.size());
    int* b = cv.take<int>(c.mats.size());
    int* b2 = cv.take<int>(c.mats.size());
    if (assign) c.idx_dyn2 = b2;
    float* om = cv.take<float>((size_t)lp * c.n);
    float* omr = c.tensor ? cv.take<float>((size_t)lp * c.n) : nullptr;
    if (assign) c.omega = omr;
    void* tm = c.tensor ? (void*)cv.take<char>(tc_tmaps_bytes((int)c.mats.size())) : nullptr;
    if (assign) { c.idx_all = a; c.idx_dyn = b; c.omega_t = om; c.tmaps = tm; }
  }
  // persistent + per-step scratch, per matrix
  for (int i = 0; i < n_mats; ++i) {
    const size_t m = (size_t)p->shapes[i].rows, n = (size_t)p->shapes[i].cols;
    const ShapeClass& c = p->classes[p->class_of[i]];
    MatDev md;
    memset(&md, 0, sizeof(md));
    md.m = (int)m; md.n = (int)n;
    md.Manc = cv.take<float>(m * n);
    md.U = cv.take<float>(m * rp);
    md.V = cv.take<float>(n * rp);
    md.sv = cv.take<float>(rp);
    md.d = cv.take<float>(rp);
    md.X = cv.take<float>((size_t)rp * rp);
    md.Xs = cv.take<float>((size_t)rp * rp);
    md.T = cv.take<float>((size_t)c.ksplit * m * rp);
    md.Ct = cv.take<float>(n * rp);
    md.xpart = cv.take<float>((size_t)c.split_m * rp * rp);
    md.sqpart = cv.take<float>(kSqnormBlocks);
    if (c.tensor) {
      md.Uhi = cv.take<bf16>(m * rk); md.Ulo = cv.take<bf16>(m * rk);
      md.Vthi = cv.take<bf16>(n * rp); md.Vtlo = cv.take<bf16>(n * rp);
      md.Cthi = cv.take<bf16>(n * rk); md.Ctlo = cv.take<bf16>(n * rk);
    }
    md.stats = assign ? p->stats_dev + (size_t)i * kStatsFloats : nullptr;
    md.omega_t = c.omega_t;
    md.omega = c.omega;
    md.inst = p->inst_of[i];
    if (assign) p->host_tab[i] = md;
  }
  // anchor-update scratch, per matrix: the basis build runs phase by phase over all shape classes, so every
  // matrix needs its own Y / Z panels and l x l factors at the same time
  for (int i = 0; i < n_mats; ++i) {
    const size_t m = (size_t)p->shapes[i].rows, n = (size_t)p->shapes[i].cols;
    float* Y = cv.take<float>(m * lp); float* Y2 = cv.take<float>(m * lp);
    float* Z = cv.take<float>(n * lp); float* Z2 = cv.take<float>(n * lp);
    float* gram = cv.take<float>((size_t)lp * lp); float* rmat = cv.take<float>((size_t)lp * lp);
    const ShapeClass& cls = p->classes[p->class_of[i]];
    float* gpart = cv.take<float>((size_t)std::max(cls.split_m, cls.split_n) * lp * lp);
    const int ssp = std::max(cls.sweep_split_n, cls.sweep_split_t);
    float* spart = ssp > 1 ? cv.take<float>((size_t)ssp * std::max(m, n) * lp) : nullptr;
    float* rmat2 = cv.take<float>((size_t)lp * lp); float* rinv = cv.take<float>((size_t)lp * lp);
    float* racc = cv.take<float>((size_t)lp * lp); float* jk = cv.take<float>((size_t)lp * lp);
    float* jv = cv.take<float>((size_t)lp * lp);
    float* ub = cv.take<float>((size_t)lp * rp); float* wb = cv.take<float>((size_t)lp * rp);
    if (assign) {
      MatDev& md = p->host_tab[i];
      md.Y = Y; md.Y2 = Y2; md.Z = Z; md.Z2 = Z2; md.gram = gram; md.gpart = gpart; md.spart = spart; md.rmat = rmat; md.rmat2 = rmat2;
      md.rinv = rinv; md.racc = racc; md.jk = jk; md.jv = jv; md.ub = ub; md.wb = wb;
    }
  }
  int* glob = cv.take<int>(n_mats);
  int* glob2 = cv.take<int>(n_mats);
  if (assign) { p->idx_glob = glob; p->idx_glob2 = glob2; }
  return align_up(cv.off);
}

void fill_plan_basics(sc_plan* p, const sc_shape* shapes, int n_mats, int rank, const sc_hparams* hp, const Dims& d) {
  p->n_mats = n_mats; p->rank = rank; p->rp = d.rp; p->rk = d.rk; p->l = d.l; p->lp = d.lp; p->q = d.q;
  p->hp = *hp;
  p->shapes.assign(shapes, shapes + n_mats);
  build_classes(shapes, n_mats, p->classes, p->class_of, p->inst_of);
  for (auto& c : p->classes) {
    c.tensor = hp->engine == SC_ENGINE_AUTO && hp->grad_dtype == SC_DTYPE_BF16 && rank > 0 &&
               tc_shape_supported(c.m, c.n, d.rp);
    c.ksplit = c.tensor ? choose_ksplit(c) : 1;
    if (c.tensor) {
      // sweeps: one block per 128 output rows and matrix; split K when that leaves most SMs idle (slices >= 1024 long)
      auto sweep_split = [&](int64_t rows_out, int64_t kdim) {
        const int64_t tiles = (rows_out + 127) / 128 * (int64_t)c.mats.size();
        int s = 1;
        while (s < 8 && tiles * s < 148 && kdim / (s * 2) >= 1024) s *= 2;
        return s;
      };
      c.sweep_split_n = sweep_split(c.m, c.n);
      c.sweep_split_t = sweep_split(c.n, c.m);
    }
    c.split_m = atb_splits((int)c.m, (int)c.mats.size());
    c.split_n = atb_splits((int)c.n, (int)c.mats.size());
    p->tensor_any = p->tensor_any || c.tensor;
  }
}

sc_status check_shapes(const sc_shape* shapes, int n_mats, int rank) {
  if (!shapes || n_mats <= 0 || n_mats > (1 << 20)) return SC_ERR_INVALID_ARG;
  for (int i = 0; i < n_mats; ++i) {
    if (shapes[i].rows <= 0 || shapes[i].cols <= 0) return SC_ERR_SHAPE;
    if (shapes[i].rows > (1 << 24) || shapes[i].cols > (1 << 24)) return SC_ERR_TOO_LARGE;
    if (rank > shapes[i].rows || rank > shapes[i].cols) return SC_ERR_SHAPE;
  }
  return SC_OK;
}

GemmArgs gemm(sc_plan* p, const int* idx, int offA, int offB, int offC, int M, int N, int K, int lda, int ldb, int ldc,
              int tA, int tB, int a_bf16 = 0) {
  GemmArgs a{};
  a.tab = p->dev_tab; a.idx = idx; a.offA = offA; a.offB = offB; a.offC = offC;
  a.M = M; a.N = N; a.K = K; a.lda = lda; a.ldb = ldb; a.ldc = ldc; a.transA = tA; a.transB = tB;
  a.a_bf16 = a_bf16; a.alpha = 1.f;
  return a;
}

#define OFF(f) ((int)offsetof(MatDev, f))

enum { PROF_EMA = 0, PROF_PASS, PROF_SMALL, PROF_PROJECT, PROF_FILTER, PROF_UPDATE };

// Brackets the launches queued during its lifetime with a pair of events (only when profiling is on).
struct ProfScope {
  sc_plan* p;
  size_t k;
  bool live;
  ProfScope(sc_plan* plan, int cat) : p(plan), k(0), live(plan->prof_on) {
    if (!live) return;
    k = p->prof_used++;
    while (p->prof_events.size() < 2 * (k + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { live = false; --p->prof_used; return; }
      p->prof_events.push_back(e);
    }
    if (p->prof_cats.size() <= k) p->prof_cats.resize(k + 1);
    p->prof_cats[k] = cat;
    cudaEventRecord(p->prof_events[2 * k], p->stream);
  }
  ~ProfScope() {
    if (live) cudaEventRecord(p->prof_events[2 * k + 1], p->stream);
  }
};

// One class's share of an anchor arrival: the matrices that received a gradient.
struct ActiveClass {
  ShapeClass* c;
  const int* idx;
  int cnt;
};

// Q <- orth(Y) by Cholesky QR over all active classes; Y (rows x lp) is overwritten, tmp is scratch of the same
// size. rounds = 2 (Cholesky QR twice) gives a basis orthonormal to working precision; rounds = 1 is enough for
// an intermediate basis of the subspace iteration, whose only job is to keep the next sweep well conditioned
// (the spanned subspace is the same either way); with one round the result is left in tmp.
// The tall products run per class; the l x l factorisations of every class go out in one launch.
// keepR: leave the two factors in rmat / rmat2 and their product in racc.
void cholqr(sc_plan* p, const std::vector<ActiveClass>& act, const int* idx_all, int n_all, int offY, int offTmp,
            bool left, bool keepR, int rounds) {
  const int lp = p->lp;
  cudaStream_t s = p->stream;
  ProfScope ps(p, PROF_SMALL);
  for (int round = 0; round < rounds; ++round) {
    const int src = round == 0 ? offY : offTmp, dst = round == 0 ? offTmp : offY;
    for (const auto& a : act) {
      const int rows = (int)(left ? a.c->m : a.c->n), slices = left ? a.c->split_m : a.c->split_n;
      if (a.c->tensor) {     // Gram matrix on the tensor cores: the panel is read once, row-slice partials, fixed-order sum
        tc_launch_gram(p, *a.c, a.idx, a.cnt, src, rows, slices);
        launch_sum_slices(p->dev_tab, a.idx, a.cnt, OFF(gpart), OFF(gram), lp * lp, slices, s);
      } else {
        launch_atb(p->dev_tab, a.idx, a.cnt, src, src, OFF(gpart), OFF(gram), rows, lp, lp, lp, lp, slices, s);
      }
    }
    launch_chol(p->dev_tab, idx_all, n_all, lp, round == 0 ? OFF(rmat) : OFF(rmat2), s);
    for (const auto& a : act)
      launch_gemm(gemm(p, a.idx, src, OFF(rinv), dst, (int)(left ? a.c->m : a.c->n), lp, lp, lp, lp, lp, 0, 0), a.cnt, s);
  }
  if (keepR && rounds == 2)
    launch_gemm(gemm(p, idx_all, OFF(rmat2), OFF(rmat), OFF(racc), lp, lp, lp, lp, lp, lp, 0, 0), n_all, s);
}

// Rebuild d (Eq. 2) and the bf16 operand copies of one matrix list after its U, s, V changed.
void refresh_operands(sc_plan* p, const ShapeClass& c, const int* idx, int cnt) {
  if (c.tensor) launch_split_basis(p->dev_tab, idx, cnt, (int)c.m, (int)c.n, p->rp, p->rk, p->stream);
}

sc_status check_ptr_array(const void* const* arr, int n, bool allow_null_entries) {
  if (!arr) return SC_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!arr[i]) { if (allow_null_entries) continue; return SC_ERR_INVALID_ARG; }
    if (reinterpret_cast<uintptr_t>(arr[i]) & 15u) return SC_ERR_ALIGNMENT;
  }
  return SC_OK;
}

}  // namespace

namespace sc {

std::atomic<long long> g_kernel_launches{0};

sc_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? SC_OK : SC_ERR_CUDA; }

// Copies the host mirror of the table to the device if it changed since the last upload. The copy goes
// through a ring of pinned buffers so that a later call never overwrites bytes an earlier, still queued
// copy has yet to read.
sc_status upload_table(sc_plan* p) {
  const size_t bytes = (size_t)p->n_mats * sizeof(MatDev);
  if (!p->table_dirty && p->last_uploaded.size() == p->host_tab.size() &&
      memcmp(p->last_uploaded.data(), p->host_tab.data(), bytes) == 0)
    return SC_OK;
  const int slot = p->staging_next;
  p->staging_next = (slot + 1) % kStagingSlots;
  if (cudaEventSynchronize(p->staging_ev[slot]) != cudaSuccess) return SC_ERR_CUDA;
  char* buf = p->staging + (size_t)slot * p->staging_bytes;
  memcpy(buf, p->host_tab.data(), bytes);
  if (cudaMemcpyAsync(p->dev_tab, buf, bytes, cudaMemcpyHostToDevice, p->stream) != cudaSuccess) return SC_ERR_CUDA;
  if (cudaEventRecord(p->staging_ev[slot], p->stream) != cudaSuccess) return SC_ERR_CUDA;
  p->last_uploaded = p->host_tab;
  p->table_dirty = false;
  return SC_OK;
}

}  // namespace sc

// ============================================================================================ ABI

extern "C" {

sc_status sc_hparams_default(sc_hparams* hp) {
  if (!hp) return SC_ERR_INVALID_ARG;
  memset(hp, 0, sizeof(*hp));
  hp->alpha = 0.3f; hp->tau_p = 1e-3f; hp->beta_anc = 0.9f;
  hp->lr = 2e-5f; hp->beta1 = 0.9f; hp->beta2 = 0.999f; hp->eps = 1e-8f; hp->weight_decay = 0.f;
  hp->max_grad_norm = 0.f; hp->grads_prescaled = 1; hp->grad_dtype = SC_DTYPE_BF16;
  hp->sketch_width = 0; hp->power_iters = 1; hp->engine = SC_ENGINE_AUTO; hp->collect_stats = 0; hp->seed = 0;
  hp->warm_start = 0; hp->warm_power_iters = 0;
  hp->optimizer = SC_OPT_ADAMW; hp->beta3 = 0.9999f; hp->mix_alpha = 5.f;
  hp->full_spectrum = 0; hp->fs_sqrt_iters = 24; hp->fs_inv_iters = 12;
  return SC_OK;
}

size_t sc_plan_workspace_bytes(const sc_shape* shapes, int n_mats, int rank, const sc_hparams* hp) {
  Dims d;
  if (!valid_hparams(hp) || check_shapes(shapes, n_mats, rank) != SC_OK || !derive_dims(rank, hp, &d)) return 0;
  if (hp->full_spectrum && check_full_spectrum(shapes, n_mats, rank) != SC_OK) return 0;
  sc_plan tmp;
  fill_plan_basics(&tmp, shapes, n_mats, rank, hp, d);
  tmp.ws = nullptr;
  return layout(&tmp, false) + (hp->full_spectrum ? fs_layout(&tmp, nullptr) : 0);
}

sc_status sc_plan_create(sc_plan** out, const sc_shape* shapes, int n_mats, int rank, float keep_ratio,
                         const sc_hparams* hp, void* workspace, size_t workspace_bytes, void* stream) {
  if (!out) return SC_ERR_INVALID_ARG;
  *out = nullptr;
  if (!valid_hparams(hp)) return SC_ERR_INVALID_ARG;
  if (!(keep_ratio > 0.f && keep_ratio <= 1.f)) return SC_ERR_INVALID_ARG;
  if (hp->grad_dtype != SC_DTYPE_BF16 && hp->grad_dtype != SC_DTYPE_FP32) return SC_ERR_DTYPE;
  if (hp->engine != SC_ENGINE_AUTO && hp->engine != SC_ENGINE_SIMT) return SC_ERR_INVALID_ARG;
  sc_status st = check_shapes(shapes, n_mats, rank);
  if (st != SC_OK) return st;
  Dims d;
  if (!derive_dims(rank, hp, &d)) return SC_ERR_INVALID_ARG;
  if (hp->full_spectrum && (st = check_full_spectrum(shapes, n_mats, rank)) != SC_OK) return st;
  if (!workspace) return SC_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) return SC_ERR_ALIGNMENT;

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SC_ERR_CUDA;
  if (prop.major != 10) return SC_ERR_UNSUPPORTED_ARCH;
  const int n_sm = prop.multiProcessorCount;

  sc_plan* p = new (std::nothrow) sc_plan();
  if (!p) return SC_ERR_INVALID_ARG;
  fill_plan_basics(p, shapes, n_mats, rank, hp, d);
  p->keep = keep_ratio;
  p->n_sm = n_sm;
  p->no_tmem_u = getenv("SC_NO_TMEM_U") != nullptr;
  p->no_pair_project = getenv("SC_NO_PAIR_PROJECT") != nullptr;
  p->no_fused_filter = getenv("SC_NO_FUSED_FILTER") != nullptr;
  p->ut_tiles = getenv("SC_UT_TILES") ? atoi(getenv("SC_UT_TILES")) : 0;
  if (p->ut_tiles < 0 || p->ut_tiles > 64) p->ut_tiles = 0;
  p->stream = reinterpret_cast<cudaStream_t>(stream);
  p->ws = nullptr;
  p->full = hp->full_spectrum != 0;
  const size_t need_base = layout(p, false);
  const size_t need = need_base + (p->full ? fs_layout(p, nullptr) : 0);
  if (workspace_bytes < need) { delete p; return SC_ERR_WORKSPACE; }
  p->ws = static_cast<char*>(workspace);
  p->ws_bytes = need;
  p->host_tab.resize(n_mats);
  p->has_basis.assign(n_mats, 0);
  p->dbg_out.assign(n_mats, nullptr);
  layout(p, true);
  if (p->full) fs_layout(p, p->ws + need_base);
  for (auto& c : p->classes)
    for (int id : c.mats) { p->host_tab[id].omega_t = c.omega_t; p->host_tab[id].omega = c.omega; }

  if (p->tensor_any && tc_init() != SC_OK) { delete p; return SC_ERR_CUDA; }

  cudaStream_t s = p->stream;
  bool ok = cudaMemsetAsync(p->ws, 0, need, s) == cudaSuccess;
  p->staging_bytes = align_up((size_t)n_mats * sizeof(MatDev));
  ok = ok && cudaHostAlloc(reinterpret_cast<void**>(&p->staging), p->staging_bytes * kStagingSlots,
                           cudaHostAllocDefault) == cudaSuccess;
  for (int i = 0; ok && i < kStagingSlots; ++i)
    ok = cudaEventCreateWithFlags(&p->staging_ev[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&p->copy_gate, cudaEventDisableTiming) == cudaSuccess;
  p->overlap_classes = getenv("SC_NO_OVERLAP") == nullptr;
  p->class_streams.assign(p->classes.size(), nullptr);
  p->join_evs.assign(p->classes.size(), nullptr);
  ok = ok && cudaEventCreateWithFlags(&p->fork_ev, cudaEventDisableTiming) == cudaSuccess;
  for (size_t k = 0; ok && k < p->classes.size(); ++k)
    ok = cudaStreamCreateWithFlags(&p->class_streams[k], cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&p->join_evs[k], cudaEventDisableTiming) == cudaSuccess;
  p->copy_done.resize(p->classes.size(), nullptr);
  for (size_t k = 0; ok && k < p->classes.size(); ++k)
    ok = cudaEventCreateWithFlags(&p->copy_done[k], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { sc_plan_destroy(p); return SC_ERR_CUDA; }
  const float one = 1.f;
  ok = cudaMemcpyAsync(p->clip_dev, &one, sizeof(float), cudaMemcpyHostToDevice, s) == cudaSuccess;
  for (auto& c : p->classes) {
    ok = ok && cudaMemcpyAsync(c.idx_all, c.mats.data(), c.mats.size() * sizeof(int), cudaMemcpyHostToDevice, s) ==
                   cudaSuccess;
    if (p->lp > 0) launch_sketch(c.omega_t, p->lp, p->l, c.n, p->hp.seed, s);
    if (p->lp > 0 && c.omega) launch_sketch_padded(c.omega, c.n, p->lp, p->l, p->hp.seed, s);
    if (c.tensor && ok) ok = tc_encode_class(p, c, true, false) == SC_OK;
  }
  p->table_dirty = true;
  ok = ok && upload_table(p) == SC_OK;
  // The small host-to-device copies above read host memory that lives only in this call.
  ok = ok && cudaStreamSynchronize(s) == cudaSuccess && cudaGetLastError() == cudaSuccess;
  if (!ok) { sc_plan_destroy(p); return SC_ERR_CUDA; }
  *out = p;
  return SC_OK;
}

sc_status sc_plan_destroy(sc_plan* p) {
  if (!p) return SC_ERR_INVALID_ARG;
  cudaStreamSynchronize(p->stream);
  for (int i = 0; i < kStagingSlots; ++i)
    if (p->staging_ev[i]) cudaEventDestroy(p->staging_ev[i]);
  for (cudaEvent_t e : p->prof_events) cudaEventDestroy(e);
  for (cudaEvent_t e : p->copy_done)
    if (e) cudaEventDestroy(e);
  if (p->copy_gate) cudaEventDestroy(p->copy_gate);
  if (p->fork_ev) cudaEventDestroy(p->fork_ev);
  for (cudaEvent_t e : p->join_evs)
    if (e) cudaEventDestroy(e);
  for (cudaStream_t cs : p->class_streams)
    if (cs) { cudaStreamSynchronize(cs); cudaStreamDestroy(cs); }
  if (p->copy_stream) { cudaStreamSynchronize(p->copy_stream); cudaStreamDestroy(p->copy_stream); }
  if (p->staging) cudaFreeHost(p->staging);
  delete p;
  return SC_OK;
}

// Anchor arrival. Dense form: anchor_grads[i] is G_anc (grad_dtype). Factored form (q_factors != nullptr):
// anchor_grads[i] is P (rows x rho fp32), q_factors[i] is Q (cols x rho fp32) and G_anc = P Q^T is never formed.
static sc_status anchor_impl(sc_plan* p, const void* const* anchor_grads, const void* const* q_factors, int rho,
                             int64_t step_tag) {
  if (!p) return SC_ERR_INVALID_ARG;
  sc_status st = check_ptr_array(anchor_grads, p->n_mats, true);
  if (st != SC_OK) return st;
  if (q_factors) {
    if (rho < 1 || rho > 1024) return SC_ERR_INVALID_ARG;
    if ((st = check_ptr_array(q_factors, p->n_mats, true)) != SC_OK) return st;
    for (int i = 0; i < p->n_mats; ++i)
      if ((anchor_grads[i] == nullptr) != (q_factors[i] == nullptr)) return SC_ERR_INVALID_ARG;
  }
  if (step_tag < p->last_tag) return SC_ERR_STALE_TAG;
  cudaStream_t s = p->stream;
  const int lp = p->lp, rp = p->rp;
  const int g_bf16 = p->hp.grad_dtype == SC_DTYPE_BF16;
  for (int i = 0; i < p->n_mats; ++i) {
    p->host_tab[i].Ganc = anchor_grads[i];
    p->host_tab[i].Qanc = q_factors ? q_factors[i] : nullptr;
  }
  if ((st = upload_table(p)) != SC_OK) return st;
  // The matrices that received a gradient, class by class, in two groups: cold starts (range finder from the
  // sketch) and warm starts (from the previous right basis), each with one flat list for the class-independent kernels.
  // dense bf16 anchors on tensor-core classes: Eq. 1 rides on the first sweep of the range finder
  const bool fuse_ema = !q_factors && g_bf16 && p->rank > 0;
  std::vector<ActiveClass> act[2];
  std::vector<int> flat[2];
  for (auto& c : p->classes) {
    std::vector<int> ids[2];
    for (int id : c.mats)
      if (anchor_grads[id]) ids[(p->hp.warm_start && p->has_basis[id] && p->rank > 0) ? 1 : 0].push_back(id);
    for (int w = 0; w < 2; ++w) {
      if (ids[w].empty()) continue;
      const int* idx = c.idx_all;
      if (ids[w].size() != c.mats.size()) {
        int* dyn = w ? c.idx_dyn2 : c.idx_dyn;
        // pageable source: the runtime has taken its copy of the list when this returns
        if (cudaMemcpyAsync(dyn, ids[w].data(), ids[w].size() * sizeof(int), cudaMemcpyHostToDevice, s) != cudaSuccess)
          return SC_ERR_CUDA;
        idx = dyn;
      }
      act[w].push_back(ActiveClass{&c, idx, (int)ids[w].size()});
      flat[w].insert(flat[w].end(), ids[w].begin(), ids[w].end());
      if (fuse_ema && c.tensor && (st = tc_encode_anchor(p, c, ids[w])) != SC_OK) return st;
    }
  }
  if (flat[0].empty() && flat[1].empty()) { p->last_tag = step_tag; return SC_OK; }
  for (int w = 0; w < 2; ++w)
    if (!flat[w].empty() &&
        cudaMemcpyAsync(w ? p->idx_glob2 : p->idx_glob, flat[w].data(), flat[w].size() * sizeof(int),
                        cudaMemcpyHostToDevice, s) != cudaSuccess)
      return SC_ERR_CUDA;
  {
    ProfScope ps(p, PROF_EMA);
    for (int w = 0; w < 2; ++w)
      for (const auto& a : act[w]) {
        if (fuse_ema && a.c->tensor) continue;      // done inside the first sweep below
        if (!q_factors) {
          launch_ema(p->dev_tab, a.idx, a.cnt, a.c->m * a.c->n, g_bf16, p->hp.beta_anc, s);           // Eq. 1
        } else {
          // Eq. 1 with G_anc = P Q^T: M <- beta M + (1 - beta) P Q^T, tile by tile
          const int m = (int)a.c->m, n = (int)a.c->n;
          GemmArgs ga = gemm(p, a.idx, OFF(Ganc), OFF(Qanc), OFF(Manc), m, n, rho, rho, rho, n, 0, 1);
          ga.alpha = 1.f - p->hp.beta_anc;
          ga.beta_c = p->hp.beta_anc;
          launch_gemm(ga, a.cnt, s);
        }
      }
  }
  if (p->full) {      // no basis: the two soft projectors of every arrived matrix, by matrix products only
    ProfScope ps(p, PROF_SMALL);
    for (int w = 0; w < 2; ++w)
      for (int id : flat[w])
        if ((st = fs_refresh(p, id)) != SC_OK) return st;
  }
  // The basis build of one group of matrices (ac: their classes; glob / n_all: the flat list for the kernels that take
  // all classes in one launch). Everything is queued on p->stream as it is at the time of the call.
  auto run_chain = [&](const std::vector<ActiveClass>& ac, const int* glob, int n_all, int w) {
    const int q = w ? p->hp.warm_power_iters : p->q;
    // one sweep over the momentum: transposed ? Z <- M^T B : Y <- M B
    bool first_sweep = true;
    auto pass = [&](int offB, bool transposed) {
      ProfScope ps(p, PROF_PASS);
      for (const auto& a : ac) {
        const int m = (int)a.c->m, n = (int)a.c->n;
        if (a.c->tensor && first_sweep && fuse_ema) { tc_launch_ema_pass(p, *a.c, a.idx, a.cnt, offB); continue; }
        if (a.c->tensor) { tc_launch_pass(p, *a.c, a.idx, a.cnt, transposed, offB); continue; }
        const int tB = offB == OFF(omega_t);
        if (!transposed)
          launch_gemm(gemm(p, a.idx, OFF(Manc), offB, OFF(Y), m, lp, n, n, tB ? n : lp, lp, 0, tB), a.cnt, p->stream);
        else
          launch_gemm(gemm(p, a.idx, OFF(Manc), offB, OFF(Z), n, lp, m, n, lp, lp, 1, 0), a.cnt, p->stream);
      }
      first_sweep = false;
    };
    // range finder: Y = M S with S the sketch (cold) or [previous V | sketch columns] (warm); Q = orth(Y)
    if (w) {
      {
        ProfScope ps(p, PROF_SMALL);
        for (const auto& a : ac)
          launch_warm_start(p->dev_tab, a.idx, a.cnt, (int)a.c->n, lp, p->l, rp, p->rank, p->hp.seed, p->stream);
      }
      pass(OFF(Z2), false);
    } else {
      pass(OFF(omega_t), false);
    }
    int curY = OFF(Y);
    if (q == 0) cholqr(p, ac, glob, n_all, OFF(Y), OFF(Y2), true, false, 2);
    else { cholqr(p, ac, glob, n_all, OFF(Y), OFF(Y2), true, false, 1); curY = OFF(Y2); }   // intermediate basis
    for (int it = 0; it < q; ++it) {
      pass(curY, true);                                                            // Z = M^T Q
      cholqr(p, ac, glob, n_all, OFF(Z), OFF(Z2), false, false, 1);
      pass(OFF(Z2), false);                                                        // Y = M Z
      if (it == q - 1) { cholqr(p, ac, glob, n_all, OFF(Y), OFF(Y2), true, false, 2); curY = OFF(Y); }
      else { cholqr(p, ac, glob, n_all, OFF(Y), OFF(Y2), true, false, 1); curY = OFF(Y2); }
    }
    // B^T = M^T Q = Qb R ; SVD of the small factor ; U = Q Ub, V = Qb Wb
    pass(OFF(Y), true);
    cholqr(p, ac, glob, n_all, OFF(Z), OFF(Z2), false, true, 2);
    {
      ProfScope ps(p, PROF_SMALL);
      launch_jacobi(p->dev_tab, glob, n_all, lp, rp, p->rank, p->hp.tau_p, p->stream);                 // + Eq. 2
      for (const auto& a : ac) {
        const int m = (int)a.c->m, n = (int)a.c->n;
        launch_gemm(gemm(p, a.idx, OFF(Y), OFF(ub), OFF(U), m, rp, lp, lp, rp, rp, 0, 0), a.cnt, p->stream);
        launch_gemm(gemm(p, a.idx, OFF(Z), OFF(wb), OFF(V), n, rp, lp, lp, rp, rp, 0, 0), a.cnt, p->stream);
        refresh_operands(p, *a.c, a.idx, a.cnt);
      }
    }
  };
  const size_t n_chains = act[0].size() + act[1].size();
  if (p->rank > 0 && p->overlap_classes && n_chains > 1) {
    // The chains of different shape classes are independent (every matrix has its own panels and factors), so each
    // class runs on a stream of its own: the short, latency-bound factorisation kernels of one class then run beside
    // the HBM-bound sweeps of another instead of leaving the chip idle between them.
    cudaStream_t main_stream = p->stream;
    if (cudaEventRecord(p->fork_ev, main_stream) != cudaSuccess) return SC_ERR_CUDA;
    for (int w = 0; w < 2; ++w)
      for (const auto& a : act[w]) {
        const size_t ci = (size_t)(a.c - p->classes.data());
        cudaStream_t cs = p->class_streams[ci];
        if (cudaStreamWaitEvent(cs, p->fork_ev, 0) != cudaSuccess) return SC_ERR_CUDA;
        p->stream = cs;
        run_chain(std::vector<ActiveClass>{a}, a.idx, a.cnt, w);
        p->stream = main_stream;
        if (cudaEventRecord(p->join_evs[ci], cs) != cudaSuccess || cudaStreamWaitEvent(main_stream, p->join_evs[ci], 0) != cudaSuccess)
          return SC_ERR_CUDA;
      }
  } else {
    for (int w = 0; w < 2 && p->rank > 0; ++w)
      if (!flat[w].empty()) run_chain(act[w], w ? p->idx_glob2 : p->idx_glob, (int)flat[w].size(), w);
  }
  for (int w = 0; w < 2; ++w)
    for (int id : flat[w]) p->has_basis[id] = 1;
  p->last_tag = step_tag;
  return cuda_ok(cudaGetLastError());
}

sc_status sc_anchor_update(sc_plan* p, const void* const* anchor_grads, int64_t step_tag) {
  return anchor_impl(p, anchor_grads, nullptr, 0, step_tag);
}

sc_status sc_anchor_update_factored(sc_plan* p, const void* const* P_factors, const void* const* Q_factors, int rho,
                                    int64_t step_tag) {
  if (!Q_factors) return SC_ERR_INVALID_ARG;
  return anchor_impl(p, P_factors, Q_factors, rho, step_tag);
}

// One optimizer step. With host_grads != nullptr the masked gradients are first copied from host memory into
// masked_grads (device staging) on the plan's copy stream, one shape class ahead of the kernels that read them.
static sc_status step_impl(sc_plan* p, const void* const* masked_grads, void* const* params,
                           const sc_opt_state* state, int64_t step, const void* const* host_grads) {
  if (!p || !state || step < 1) return SC_ERR_INVALID_ARG;
  sc_status st;
  if ((st = check_ptr_array(masked_grads, p->n_mats, false)) != SC_OK) return st;
  if ((st = check_ptr_array(reinterpret_cast<const void* const*>(params), p->n_mats, false)) != SC_OK) return st;
  if ((st = check_ptr_array(reinterpret_cast<const void* const*>(state->exp_avg), p->n_mats, false)) != SC_OK) return st;
  if ((st = check_ptr_array(reinterpret_cast<const void* const*>(state->exp_avg_sq), p->n_mats, false)) != SC_OK) return st;
  if (state->params_bf16 &&
      (st = check_ptr_array(reinterpret_cast<const void* const*>(state->params_bf16), p->n_mats, true)) != SC_OK)
    return st;
  const bool mix = p->hp.optimizer == SC_OPT_ADEMAMIX;
  if (mix && (st = check_ptr_array(reinterpret_cast<const void* const*>(state->exp_avg_slow), p->n_mats, false)) != SC_OK)
    return st;
  cudaStream_t s = p->stream;
  const sc_hparams& hp = p->hp;
  const int rp = p->rp;
  const int g_bf16 = hp.grad_dtype == SC_DTYPE_BF16;
  bool g_changed = false;
  for (int i = 0; i < p->n_mats; ++i) {
    MatDev& md = p->host_tab[i];
    const MatDev before = md;
    md.G = masked_grads[i];
    md.W = static_cast<float*>(params[i]);
    md.m1 = static_cast<float*>(state->exp_avg[i]);
    md.m2 = static_cast<float*>(state->exp_avg_sq[i]);
    md.Wb = state->params_bf16 ? static_cast<bf16*>(state->params_bf16[i]) : nullptr;
    md.ms = mix ? static_cast<float*>(state->exp_avg_slow[i]) : nullptr;
    g_changed = g_changed || before.G != md.G || before.W != md.W || before.m1 != md.m1 || before.m2 != md.m2 ||
                before.Wb != md.Wb || before.ms != md.ms;
    md.gproj_dbg = static_cast<float*>(p->dbg_out[i]);
  }
  if ((st = upload_table(p)) != SC_OK) return st;
  if (g_changed)
    for (auto& c : p->classes)
      if (c.tensor && (st = tc_encode_class(p, c, false, true)) != SC_OK) return st;

  const float scale = hp.grads_prescaled ? 1.f : 1.f / p->keep;
  const double bc1 = 1.0 - pow((double)hp.beta1, (double)step), bc2 = 1.0 - pow((double)hp.beta2, (double)step);
  StepScalars sc{};
  sc.alpha_s = hp.alpha * scale;
  sc.beta1 = hp.beta1; sc.beta2 = hp.beta2; sc.one_m_beta1 = 1.f - hp.beta1; sc.one_m_beta2 = 1.f - hp.beta2;
  sc.step_size = (float)((double)hp.lr / bc1);
  sc.inv_sqrt_bc2 = (float)(1.0 / sqrt(bc2));
  sc.eps = hp.eps;
  sc.decay = 1.f - hp.lr * hp.weight_decay;
  sc.mix = mix ? 1 : 0;
  sc.beta3 = hp.beta3; sc.one_m_beta3 = 1.f - hp.beta3;
  sc.lr_mix = hp.lr * hp.mix_alpha;
  const bool clip_on = hp.max_grad_norm > 0.f;
  const bool want_norm = clip_on || hp.collect_stats;

  if (host_grads) {
    // queue every host-to-device copy now, class by class; the kernels of a class wait only for its own event
    const size_t esz = g_bf16 ? 2 : 4;
    if (cudaEventRecord(p->copy_gate, s) != cudaSuccess || cudaStreamWaitEvent(p->copy_stream, p->copy_gate, 0) != cudaSuccess)
      return SC_ERR_CUDA;   // earlier work on the plan's stream may still be reading the staging buffers
    for (size_t k = 0; k < p->classes.size(); ++k) {
      for (int id : p->classes[k].mats) {
        const size_t bytes = (size_t)p->shapes[id].rows * p->shapes[id].cols * esz;
        if (cudaMemcpyAsync(const_cast<void*>(masked_grads[id]), host_grads[id], bytes, cudaMemcpyHostToDevice,
                            p->copy_stream) != cudaSuccess)
          return SC_ERR_CUDA;
      }
      if (cudaEventRecord(p->copy_done[k], p->copy_stream) != cudaSuccess) return SC_ERR_CUDA;
    }
  }
  if (p->full) {
    if (host_grads)
      for (size_t k = 0; k < p->classes.size(); ++k)
        if (cudaStreamWaitEvent(s, p->copy_done[k], 0) != cudaSuccess) return SC_ERR_CUDA;
    bool any = false;
    for (int i = 0; i < p->n_mats; ++i) {
      { ProfScope ps(p, PROF_PROJECT); if ((st = fs_step_filter(p, i, (1.f - hp.alpha) * scale)) != SC_OK) return st; }
      { ProfScope ps(p, PROF_UPDATE);  if ((st = fs_step_update(p, i, sc)) != SC_OK) return st; }
      any = any || p->has_basis[i];
    }
    if (cudaGetLastError() != cudaSuccess) return SC_ERR_CUDA;
    return any ? SC_OK : SC_WARN_NO_ANCHOR;
  }
  auto project = [&](ShapeClass& c) -> sc_status {
    const int cnt = (int)c.mats.size(), m = (int)c.m, n = (int)c.n;
    const int* idx = c.idx_all;
    if (host_grads && cudaStreamWaitEvent(s, p->copy_done[&c - p->classes.data()], 0) != cudaSuccess) return SC_ERR_CUDA;
    if (rp > 0) {
      ProfScope ps(p, PROF_PROJECT);
      if (c.tensor) {
        sc_status e = tc_launch_project(p, c, idx, cnt);                     // T = G V, as c.ksplit partials over K
        if (e != SC_OK) return e;
      } else {
        launch_gemm(gemm(p, idx, OFF(G), OFF(V), OFF(T), m, rp, n, n, rp, rp, 0, 0, g_bf16), cnt, s);
      }
    }
    ProfScope ps(p, PROF_FILTER);
    // X = U^T T as row-slice partials, added up in slice order: by a launch of its own, or inside xs_kernel when one
    // block per matrix can do it
    // few matrices: the filter and C^T in one launch (every block re-forms Xs, which only pays while there are few
    // blocks); many matrices: the batched launches, whose launch latency is shared by the whole class
    const bool one_launch = filter_ct_supported(rp) && (int64_t)cnt * ((n + 63) / 64) <= 1024 && !p->no_fused_filter;
    const bool sum_in_xs = !one_launch && (size_t)c.split_m * rp * rp <= (size_t)(1 << 16);
    if (rp > 0 && c.tensor) {
      // plans with few matrices split K in the projection: add those partials of T up first (in place, slice 0)
      launch_reduce_partials(p->dev_tab, idx, cnt, (int64_t)m * rp, c.ksplit, s);
      sc_status e = tc_launch_xpart(p, c, idx, cnt, c.split_m);        // tensor cores, T read once
      if (e != SC_OK) return e;
      if (!sum_in_xs) launch_sum_slices(p->dev_tab, idx, cnt, OFF(xpart), OFF(X), rp * rp, c.split_m, s);
    } else if (rp > 0) {
      launch_atb(p->dev_tab, idx, cnt, OFF(U), OFF(T), OFF(xpart), OFF(X), m, rp, rp, rp, rp, c.split_m, s, c.ksplit,
                 !sum_in_xs);
    }
    if (want_norm) launch_sqnorm(p->dev_tab, idx, cnt, (int64_t)m * n, g_bf16, s);
    if (one_launch) {
      launch_filter_ct(p->dev_tab, idx, cnt, rp, p->rank, n, p->rk, scale, hp.alpha, p->status_dev, s);   // D X D, C^T = V Xs^T
    } else {
      launch_xs(p->dev_tab, idx, cnt, rp, p->rank, (rp > 0 && sum_in_xs) ? c.split_m : 0, scale, hp.alpha, p->status_dev, s);   // D X D
      if (rp > 0) {
        GemmArgs ga = gemm(p, idx, OFF(V), OFF(Xs), OFF(Ct), n, rp, rp, rp, rp, rp, 0, 1);             // C^T = V Xs^T
        if (c.tensor) { ga.offHi = OFF(Cthi); ga.offLo = OFF(Ctlo); ga.ld_split = p->rk; ga.split_only = 1; }
        launch_gemm(ga, cnt, s);
      }
    }
    return SC_OK;
  };
  auto update = [&](ShapeClass& c) -> sc_status {
    const int cnt = (int)c.mats.size(), m = (int)c.m, n = (int)c.n;
    ProfScope ps(p, PROF_UPDATE);
    if (c.tensor) return tc_launch_epilogue(p, c, c.idx_all, cnt, sc);
    launch_epilogue_simt(p->dev_tab, c.idx_all, cnt, m, n, rp, g_bf16, sc, p->clip_dev, s);
    return SC_OK;
  };

  // Device gradients, several shape classes: the projections and the short filter chains of the classes are independent,
  // so each class runs them on its own stream (forked from and joined to the plan's stream, as in the anchor update)
  // and one class's latency-bound chain runs beside another's projection; the updates follow on the plan's stream.
  // Host gradients keep the class-by-class order, in which a class's update overlaps the next class's copy.
  const bool fork = p->overlap_classes && !host_grads && p->classes.size() > 1 && rp > 0;
  if (fork) {
    cudaStream_t main_stream = p->stream;
    if (cudaEventRecord(p->fork_ev, main_stream) != cudaSuccess) return SC_ERR_CUDA;
    for (size_t ci = 0; ci < p->classes.size(); ++ci) {
      cudaStream_t cs = p->class_streams[ci];
      if (cudaStreamWaitEvent(cs, p->fork_ev, 0) != cudaSuccess) return SC_ERR_CUDA;
      p->stream = cs; s = cs;
      st = project(p->classes[ci]);
      p->stream = main_stream; s = main_stream;
      if (st != SC_OK) return st;
      if (cudaEventRecord(p->join_evs[ci], cs) != cudaSuccess || cudaStreamWaitEvent(main_stream, p->join_evs[ci], 0) != cudaSuccess)
        return SC_ERR_CUDA;
    }
    if (clip_on) launch_clip(p->dev_tab, p->n_mats, hp.max_grad_norm, p->clip_dev, s);
    for (auto& c : p->classes) if ((st = update(c)) != SC_OK) return st;
  } else if (clip_on) {
    for (auto& c : p->classes) if ((st = project(c)) != SC_OK) return st;
    launch_clip(p->dev_tab, p->n_mats, hp.max_grad_norm, p->clip_dev, s);
    for (auto& c : p->classes) if ((st = update(c)) != SC_OK) return st;
  } else {
    for (auto& c : p->classes) {
      if ((st = project(c)) != SC_OK) return st;
      if ((st = update(c)) != SC_OK) return st;
    }
  }
  if (cudaGetLastError() != cudaSuccess) return SC_ERR_CUDA;
  bool any = false;
  for (char h : p->has_basis) any = any || h;
  return (p->rank > 0 && !any) ? SC_WARN_NO_ANCHOR : SC_OK;
}

sc_status sc_correct_and_step(sc_plan* p, const void* const* masked_grads, void* const* params,
                              const sc_opt_state* state, int64_t step) {
  return step_impl(p, masked_grads, params, state, step, nullptr);
}

sc_status sc_correct_and_step_host(sc_plan* p, const void* const* host_grads, void* const* grad_staging,
                                   void* const* params, const sc_opt_state* state, int64_t step,
                                   sc_mat_stats* stats_out, float* clip_out) {
  if (!p || !host_grads || !grad_staging) return SC_ERR_INVALID_ARG;
  for (int i = 0; i < p->n_mats; ++i)
    if (!host_grads[i]) return SC_ERR_INVALID_ARG;
  sc_status st = step_impl(p, reinterpret_cast<const void* const*>(grad_staging), params, state, step, host_grads);
  if (st != SC_OK && st != SC_WARN_NO_ANCHOR) return st;
  if (stats_out) {
    const sc_status s2 = sc_get_stats(p, stats_out, clip_out);   // device-to-host read; waits for the step
    if (s2 != SC_OK) return s2;
  } else if (cudaStreamSynchronize(p->stream) != cudaSuccess) {
    return SC_ERR_CUDA;
  }
  return st;
}

// -------------------------------------------------------------------------------------- inspection

static sc_status check_mat(sc_plan* p, int mat) {
  if (!p || mat < 0 || mat >= p->n_mats) return SC_ERR_INVALID_ARG;
  return SC_OK;
}

sc_status sc_export_basis(sc_plan* p, int mat, void* U_dev, void* s_dev, void* V_dev) {
  sc_status st = check_mat(p, mat);
  if (st != SC_OK) return st;
  const MatDev& md = p->host_tab[mat];
  const int r = p->rank, rp = p->rp;
  if (r == 0) return SC_OK;
  if (U_dev) launch_unpad_copy(static_cast<float*>(U_dev), r, md.U, rp, md.m, r, p->stream);
  if (V_dev) launch_unpad_copy(static_cast<float*>(V_dev), r, md.V, rp, md.n, r, p->stream);
  if (s_dev && cudaMemcpyAsync(s_dev, md.sv, r * sizeof(float), cudaMemcpyDeviceToDevice, p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  return cuda_ok(cudaGetLastError());
}

sc_status sc_import_basis(sc_plan* p, int mat, const void* U_dev, const void* s_dev, const void* V_dev) {
  sc_status st = check_mat(p, mat);
  if (st != SC_OK) return st;
  if (!U_dev || !s_dev || !V_dev) return SC_ERR_INVALID_ARG;
  const MatDev& md = p->host_tab[mat];
  const int r = p->rank, rp = p->rp;
  if (r == 0) return SC_OK;
  cudaStream_t s = p->stream;
  if ((st = upload_table(p)) != SC_OK) return st;
  launch_pad_copy(md.U, rp, static_cast<const float*>(U_dev), r, md.m, r, rp, s);
  launch_pad_copy(md.V, rp, static_cast<const float*>(V_dev), r, md.n, r, rp, s);
  launch_pad_copy(md.sv, rp, static_cast<const float*>(s_dev), r, 1, r, rp, s);
  ShapeClass& c = p->classes[p->class_of[mat]];
  const int* idx = c.idx_all + p->inst_of[mat];
  launch_filter_weights(p->dev_tab, idx, 1, rp, r, p->hp.tau_p, s);
  refresh_operands(p, c, idx, 1);
  p->has_basis[mat] = 1;
  return cuda_ok(cudaGetLastError());
}

sc_status sc_export_projection(sc_plan* p, int mat, void* T_dev, void* X_dev) {
  sc_status st = check_mat(p, mat);
  if (st != SC_OK) return st;
  const MatDev& md = p->host_tab[mat];
  const int r = p->rank, rp = p->rp;
  if (r == 0) return SC_OK;
  if (T_dev) {
    // the step has already added the K-slice partials of the tensor-core projection into slice 0
    launch_unpad_copy(static_cast<float*>(T_dev), r, md.T, rp, md.m, r, p->stream);
  }
  if (X_dev) launch_unpad_copy(static_cast<float*>(X_dev), r, md.X, rp, r, r, p->stream);
  return cuda_ok(cudaGetLastError());
}

sc_status sc_export_anchor_momentum(sc_plan* p, int mat, void* M_dev) {
  sc_status st = check_mat(p, mat);
  if (st != SC_OK) return st;
  if (!M_dev) return SC_ERR_INVALID_ARG;
  const MatDev& md = p->host_tab[mat];
  return cuda_ok(cudaMemcpyAsync(M_dev, md.Manc, (size_t)md.m * md.n * sizeof(float), cudaMemcpyDeviceToDevice,
                                 p->stream));
}

sc_status sc_import_anchor_momentum(sc_plan* p, int mat, const void* M_dev) {
  sc_status st = check_mat(p, mat);
  if (st != SC_OK) return st;
  if (!M_dev) return SC_ERR_INVALID_ARG;
  const MatDev& md = p->host_tab[mat];
  return cuda_ok(cudaMemcpyAsync(md.Manc, M_dev, (size_t)md.m * md.n * sizeof(float), cudaMemcpyDeviceToDevice,
                                 p->stream));
}

sc_status sc_export_sketch(sc_plan* p, int64_t rows, int width, void* Omega_dev) {
  if (!p || !Omega_dev || rows <= 0 || width <= 0 || width > 1024) return SC_ERR_INVALID_ARG;
  launch_sketch_rowmajor(static_cast<float*>(Omega_dev), rows, width, p->hp.seed, p->stream);
  return cuda_ok(cudaGetLastError());
}

sc_status sc_set_debug_gproj_out(sc_plan* p, void* const* gproj_out) {
  if (!p) return SC_ERR_INVALID_ARG;
  for (int i = 0; i < p->n_mats; ++i) p->dbg_out[i] = gproj_out ? gproj_out[i] : nullptr;
  return SC_OK;
}

sc_status sc_get_stats(sc_plan* p, sc_mat_stats* stats, float* clip) {
  if (!p || !stats) return SC_ERR_INVALID_ARG;
  std::vector<float> h((size_t)p->n_mats * kStatsFloats);
  if (cudaMemcpyAsync(h.data(), p->stats_dev, h.size() * sizeof(float), cudaMemcpyDeviceToHost, p->stream) !=
      cudaSuccess)
    return SC_ERR_CUDA;
  float c = 1.f;
  if (cudaMemcpyAsync(&c, p->clip_dev, sizeof(float), cudaMemcpyDeviceToHost, p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess) return SC_ERR_CUDA;
  for (int i = 0; i < p->n_mats; ++i) {
    const float* f = &h[(size_t)i * kStatsFloats];
    stats[i].g_sqnorm = f[0]; stats[i].x_sqnorm = f[1]; stats[i].gproj_sqnorm = f[2]; stats[i].r_eff = f[3];
  }
  if (clip) *clip = c;
  return SC_OK;
}

sc_status sc_get_device_status(sc_plan* p) {
  if (!p) return SC_ERR_INVALID_ARG;
  unsigned w = 0;
  if (cudaMemcpyAsync(&w, p->status_dev, sizeof(w), cudaMemcpyDeviceToHost, p->stream) != cudaSuccess ||
      cudaStreamSynchronize(p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  // one condition is reported per call and only its bit is cleared, so a second latched condition is reported by
  // the next call (the bits live in the low byte of the word, which is what the one-byte memset rewrites)
  const unsigned reported = (w & kDevTimeout) ? kDevTimeout : (w & kDevNonfinite);
  if (reported && cudaMemsetAsync(p->status_dev, (int)(w & ~reported & 0xFFu), 1, p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  if (reported == kDevTimeout) return SC_ERR_TIMEOUT;
  if (reported == kDevNonfinite) return SC_ERR_NONFINITE;
  return SC_OK;
}

sc_status sc_get_anchor_info(sc_plan* p, int64_t* last_tag, int* n_with_basis) {
  if (!p) return SC_ERR_INVALID_ARG;
  if (last_tag) *last_tag = p->last_tag;
  if (n_with_basis) {
    int k = 0;
    for (char h : p->has_basis) k += h ? 1 : 0;
    *n_with_basis = k;
  }
  return SC_OK;
}

// ---- checkpoint / resume: anchor momentum and cached basis of every matrix as one host blob --------------
namespace {
struct StateHeader {
  uint32_t magic, version;
  int32_t n_mats, rank, rp, pad;
  int64_t last_tag;
};
constexpr uint32_t kStateMagic = 0x53435354u;   // "SCST"
constexpr uint32_t kStateVersion = 2u;          // 2: the blob lists every matrix's rows and cols after the flags

size_t state_shape_bytes(const sc_plan* p) { return align_up((size_t)p->n_mats * sizeof(sc_shape), 16); }

size_t state_bytes(const sc_plan* p) {
  size_t b = sizeof(StateHeader) + align_up((size_t)p->n_mats, 16) + state_shape_bytes(p);
  for (int i = 0; i < p->n_mats; ++i) {
    const size_t m = (size_t)p->shapes[i].rows, n = (size_t)p->shapes[i].cols;
    b += (m * n + (m + n + 2) * (size_t)p->rp) * sizeof(float);
  }
  return b;
}
}  // namespace

size_t sc_state_bytes(const sc_plan* p) { return p ? state_bytes(p) : 0; }

sc_status sc_state_export(sc_plan* p, void* host_buf, size_t bytes) {
  if (!p || !host_buf) return SC_ERR_INVALID_ARG;
  if (bytes < state_bytes(p)) return SC_ERR_WORKSPACE;
  char* out = static_cast<char*>(host_buf);
  StateHeader h{kStateMagic, kStateVersion, p->n_mats, p->rank, p->rp, 0, p->last_tag};
  memcpy(out, &h, sizeof(h));
  char* flags = out + sizeof(h);
  memset(flags, 0, align_up((size_t)p->n_mats, 16));
  for (int i = 0; i < p->n_mats; ++i) flags[i] = p->has_basis[i];
  char* shp = flags + align_up((size_t)p->n_mats, 16);
  memset(shp, 0, state_shape_bytes(p));
  memcpy(shp, p->shapes.data(), (size_t)p->n_mats * sizeof(sc_shape));
  char* cur = shp + state_shape_bytes(p);
  auto pull = [&](const float* src, size_t count) {
    const bool ok = count == 0 ||
                    cudaMemcpyAsync(cur, src, count * sizeof(float), cudaMemcpyDeviceToHost, p->stream) == cudaSuccess;
    cur += count * sizeof(float);
    return ok;
  };
  for (int i = 0; i < p->n_mats; ++i) {
    const MatDev& md = p->host_tab[i];
    const size_t m = (size_t)md.m, n = (size_t)md.n, rp = (size_t)p->rp;
    if (!pull(md.Manc, m * n) || !pull(md.U, m * rp) || !pull(md.V, n * rp) || !pull(md.sv, rp) || !pull(md.d, rp))
      return SC_ERR_CUDA;
  }
  return cuda_ok(cudaStreamSynchronize(p->stream));
}

sc_status sc_state_import(sc_plan* p, const void* host_buf, size_t bytes) {
  if (!p || !host_buf) return SC_ERR_INVALID_ARG;
  if (bytes < state_bytes(p)) return SC_ERR_WORKSPACE;
  const char* in = static_cast<const char*>(host_buf);
  StateHeader h;
  memcpy(&h, in, sizeof(h));
  if (h.magic != kStateMagic || h.version != kStateVersion) return SC_ERR_INVALID_ARG;
  if (h.n_mats != p->n_mats || h.rank != p->rank || h.rp != p->rp) return SC_ERR_SHAPE;
  const char* flags = in + sizeof(h);
  const char* shp = flags + align_up((size_t)p->n_mats, 16);
  for (int i = 0; i < p->n_mats; ++i) {      // same shapes in the same order, or the arrays would land in the wrong matrices
    sc_shape sh;
    memcpy(&sh, shp + (size_t)i * sizeof(sc_shape), sizeof(sh));
    if (sh.rows != p->shapes[i].rows || sh.cols != p->shapes[i].cols) return SC_ERR_SHAPE;
  }
  sc_status st = upload_table(p);
  if (st != SC_OK) return st;
  const char* cur = shp + state_shape_bytes(p);
  auto push = [&](float* dst, size_t count) {
    const bool ok = count == 0 ||
                    cudaMemcpyAsync(dst, cur, count * sizeof(float), cudaMemcpyHostToDevice, p->stream) == cudaSuccess;
    cur += count * sizeof(float);
    return ok;
  };
  for (int i = 0; i < p->n_mats; ++i) {
    const MatDev& md = p->host_tab[i];
    const size_t m = (size_t)md.m, n = (size_t)md.n, rp = (size_t)p->rp;
    if (!push(md.Manc, m * n) || !push(md.U, m * rp) || !push(md.V, n * rp) || !push(md.sv, rp) || !push(md.d, rp))
      return SC_ERR_CUDA;
  }
  // Eq. 2 from the imported singular values and THIS plan's tau_p (the blob's d belongs to the exporting plan)
  for (auto& c : p->classes) {
    if (p->rp > 0) launch_filter_weights(p->dev_tab, c.idx_all, (int)c.mats.size(), p->rp, p->rank, p->hp.tau_p, p->stream);
    refresh_operands(p, c, c.idx_all, (int)c.mats.size());
  }
  // the copies above read caller memory: finish them before returning
  if (cudaStreamSynchronize(p->stream) != cudaSuccess) return SC_ERR_CUDA;
  for (int i = 0; i < p->n_mats; ++i) p->has_basis[i] = flags[i];
  if (p->full)       // the soft projectors are not part of the blob: rebuild them from the imported momentum
    for (int i = 0; i < p->n_mats; ++i)
      if (p->has_basis[i] && (st = fs_refresh(p, i)) != SC_OK) return st;
  p->last_tag = h.last_tag;
  return cuda_ok(cudaGetLastError());
}

sc_status sc_debug_wait_probe(sc_plan* p, int max_polls) {
  if (!p || max_polls < 1 || max_polls > (1 << 20)) return SC_ERR_INVALID_ARG;
  return tc_launch_wait_probe(p, max_polls);
}

sc_status sc_set_profiling(sc_plan* p, int on) {
  if (!p) return SC_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(p->stream) != cudaSuccess) return SC_ERR_CUDA;
  p->prof_on = on != 0;
  p->prof_used = 0;
  return SC_OK;
}

sc_status sc_get_profile(sc_plan* p, sc_profile* out) {
  if (!p || !out) return SC_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  if (cudaStreamSynchronize(p->stream) != cudaSuccess) return SC_ERR_CUDA;
  for (size_t k = 0; k < p->prof_used; ++k) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p->prof_events[2 * k], p->prof_events[2 * k + 1]) != cudaSuccess) return SC_ERR_CUDA;
    const int cat = p->prof_cats[k];
    if (cat >= 0 && cat < SC_PROFILE_CATEGORIES) { out->ms[cat] += ms; out->spans[cat] += 1; }
  }
  p->prof_used = 0;
  return SC_OK;
}

int64_t sc_kernel_launch_count(void) { return (int64_t)g_kernel_launches.load(); }

int sc_plan_uses_tensor_cores(const sc_plan* p) { return p && (p->tensor_any || p->full) ? 1 : 0; }

const char* sc_status_string(sc_status s) {
  switch (s) {
    case SC_OK: return "ok";
    case SC_WARN_NO_ANCHOR: return "no anchor gradient has arrived yet (empty basis)";
    case SC_ERR_INVALID_ARG: return "invalid argument";
    case SC_ERR_SHAPE: return "invalid shape or rank larger than a matrix dimension";
    case SC_ERR_DTYPE: return "unsupported dtype";
    case SC_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
    case SC_ERR_WORKSPACE: return "workspace too small";
    case SC_ERR_STALE_TAG: return "anchor step tag older than the last accepted one";
    case SC_ERR_CUDA: return "CUDA error";
    case SC_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    case SC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case SC_ERR_NONFINITE: return "non-finite value encountered";
    case SC_ERR_TOO_LARGE: return "dimension too large";
  }
  return "unknown status";
}

int sc_version(void) { return 100; }

}  // extern "C"
