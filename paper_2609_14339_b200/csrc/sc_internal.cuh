// Internal declarations shared by the translation units of the spectral-correction library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "spectral_correction.h"

namespace sc {

typedef __nv_bfloat16 bf16;

constexpr int kMaxRank = 256;
constexpr int kStatsFloats = 8;        // per-matrix statistics slot
constexpr int kSqnormBlocks = 128;     // partial sums of ||G||^2 per matrix (fixed-order reduction)
constexpr int kAtbMaxSplits = 64;      // row slices of the A^T B kernel (fixed-order two-stage reduction)
constexpr int kStagingSlots = 4;       // ring of pinned upload buffers for the per-call pointer table

// Device status word bits (latched, read by sc_get_device_status).
constexpr unsigned kDevTimeout = 1u;
constexpr unsigned kDevNonfinite = 2u;

// One record per weight matrix, resident in device memory (the "table"). The first block of fields is
// fixed at plan creation (addresses inside the workspace); the second block is rewritten by every call.
struct MatDev {
  // cached basis and anchor momentum (persistent)
  float* Manc;   // m x n       anchor momentum, Eq. 1
  float* U;      // m x rp      left basis, fp32, columns >= rank are zero
  float* V;      // n x rp      right basis
  float* sv;     // rp          singular values
  float* d;      // rp          filter weights, Eq. 2
  bf16* Uhi;     // m x rk      bf16 split of U  (U ~= Uhi + Ulo), K-major MMA operand, rk = rp rounded up to 64
  bf16* Ulo;
  bf16* Vthi;    // rp x n      bf16 split of V^T, K-major MMA operand
  bf16* Vtlo;
  // per-step scratch (slot shared by matrices of different shape classes)
  float* T;      // ksplit x m x rp   T = G V (partials)
  float* X;      // rp x rp     X = U^T G V (unscaled)
  float* Xs;     // rp x rp     (1-alpha) * scale * D X D
  float* Ct;     // n x rp      C^T = V Xs^T, fp32
  bf16* Cthi;    // n x rk      bf16 split of C^T
  bf16* Ctlo;
  float* xpart;  // split_m x rp x rp   row-slice partials of X
  float* sqpart; // kSqnormBlocks partial sums of ||G||^2
  float* stats;  // kStatsFloats
  // anchor-update scratch
  float* Y;      // m x lp
  float* Y2;     // m x lp
  float* Z;      // n x lp
  float* Z2;     // n x lp
  float* gram;   // lp x lp
  float* spart;  // sweep_split x max(m, n) x lp   K-slice partials of a sweep (plans with few matrices only)
  float* gpart;  // kAtbMaxSplits x lp x lp   row-slice partials of the Gram matrix
  float* rmat;   // lp x lp   Cholesky factor (upper), first pass
  float* rmat2;  // lp x lp   second pass
  float* rinv;   // lp x lp   inverse of the factor
  float* racc;   // lp x lp   rmat2 * rmat
  float* jk;     // lp x lp   Jacobi work: columns being orthogonalised
  float* jv;     // lp x lp   accumulated rotations
  float* ub;     // lp x rp   left singular vectors of the small factor (selected, sorted)
  float* wb;     // lp x rp   right singular vectors
  const float* omega_t;  // lp x n  Rademacher sketch, transposed (shared by a shape class)
  const float* omega;    // n x lp  the same sketch, row-major (tensor-core classes only)
  // per call
  const void* G;      // masked gradient
  const void* Ganc;   // anchor gradient (dense), or its left factor P (rows x rho fp32)
  const void* Qanc;   // right factor Q (cols x rho fp32) of a factored anchor gradient, else null
  float* W;           // fp32 master weights
  float* m1;          // AdamW first moment
  float* m2;          // AdamW second moment
  bf16* Wb;           // optional bf16 weight copy
  float* ms;          // slow EMA of the dual-EMA optimizer (null for AdamW)
  float* gproj_dbg;   // optional G_proj output
  int m, n;
  int inst;           // index of this matrix inside its shape class (selects its tensor maps)
  int pad1;
};

// All matrices of one shape; kernels are launched once per class with blockIdx.z = instance.
struct ShapeClass {
  int64_t m = 0, n = 0;
  std::vector<int> mats;   // matrix ids, in plan order
  float* omega_t = nullptr;
  float* omega = nullptr;
  int* idx_all = nullptr;  // device: mats[]
  int* idx_dyn = nullptr;  // device: subset list written per call (anchor arrivals, cold starts)
  int* idx_dyn2 = nullptr; // device: subset list written per call (anchor arrivals, warm starts)
  bool tensor = false;     // served by the tcgen05 kernels
  int ksplit = 1;
  int sweep_split_n = 1, sweep_split_t = 1;   // K slices of the plain / transposed sweeps over the momentum
  int split_m = 1, split_n = 1;   // row slices of A^T B products over m / n rows (fixed at plan creation)
  void* tmaps = nullptr;   // device: per-instance tensor maps (tensor engine only)
};

struct StepScalars {       // scalars of one step, passed by value to kernels
  float alpha_s;           // alpha * scale
  float beta1, beta2, one_m_beta1, one_m_beta2;
  float step_size;         // lr / (1 - beta1^t)
  float inv_sqrt_bc2;      // 1 / sqrt(1 - beta2^t)
  float eps;
  float decay;             // 1 - lr * weight_decay
  // dual-EMA optimizer only (mix != 0): W <- W decay - (step_size m1 + lr_mix m_slow) / den
  float beta3, one_m_beta3;
  float lr_mix;            // lr * mix_alpha (the slow EMA is not bias-corrected)
  int mix;
};

// Full-spectrum variant (no rank cut): per-matrix soft projectors and the scratch one matrix needs at a time.
struct FsMat {
  bf16 *PUhi, *PUlo;   // m x m, P_U = U diag(d) U^T as a bf16 hi/lo pair
  bf16 *PVhi, *PVlo;   // n x n
};
struct FsState {
  std::vector<FsMat> mats;
  double* work[5] = {};     // k x k fp64 each, k = the largest dimension of any matrix
  double* part = nullptr;   // partial sums of the norms
  double* scal = nullptr;   // [0] ||Gram||_F, [1] ||Y||_F
  bf16* T1hi = nullptr;     // (G^T P_U) as hi/lo, n x m
  bf16* T1lo = nullptr;
  float* F = nullptr;       // (1 - alpha) scale * P_U G P_V, m x n
};

}  // namespace sc

struct sc_plan {
  int n_mats = 0, rank = 0, rp = 0, rk = 0, l = 0, lp = 0, q = 0;   // rk: row stride of the bf16 K-operand copies
  float keep = 1.f;
  sc_hparams hp{};
  cudaStream_t stream = nullptr;
  std::vector<sc_shape> shapes;
  std::vector<sc::ShapeClass> classes;
  std::vector<int> class_of;       // matrix -> class
  std::vector<int> inst_of;        // matrix -> instance index inside its class
  std::vector<sc::MatDev> host_tab;   // host mirror of the device table
  std::vector<sc::MatDev> last_uploaded;
  sc::MatDev* dev_tab = nullptr;
  int* idx_glob = nullptr;            // device: flat list of the matrices an anchor call touches (cold starts)
  int* idx_glob2 = nullptr;           // the same for warm starts
  char* staging = nullptr;            // pinned, kStagingSlots * staging_bytes
  size_t staging_bytes = 0;
  cudaEvent_t staging_ev[sc::kStagingSlots]{};
  int staging_next = 0;
  float* clip_dev = nullptr;          // clip factor applied to G_proj
  unsigned* status_dev = nullptr;     // latched device status bits
  unsigned* work_dev = nullptr;       // work-item counter of the streaming update kernel (zeroed before each launch)
  float* stats_dev = nullptr;         // n_mats * kStatsFloats
  char* ws = nullptr;
  size_t ws_bytes = 0;
  int64_t last_tag = -1;
  std::vector<char> has_basis;
  std::vector<void*> dbg_out;
  bool table_dirty = true;
  bool tensor_any = false;
  bool full = false;                  // full-spectrum soft filter (no rank cut)
  bool no_tmem_u = false;             // test hook (environment SC_NO_TMEM_U): ranks above 64 re-fetch U per tile instead
  bool no_fused_filter = false;       // test hook (environment SC_NO_FUSED_FILTER): filter and C^T as separate launches
  bool no_pair_project = false;       // test hook (environment SC_NO_PAIR_PROJECT): one block per 128-row tile instead
  int ut_tiles = 0;                   // test hook (environment SC_UT_TILES): tiles per item with U in tensor memory
  sc::FsState fs;
  int n_sm = 0;                       // SM count of the plan's device
  // anchor refresh: the basis builds of different shape classes run on streams of their own (fork / join on `stream`)
  bool overlap_classes = true;        // test hook (environment SC_NO_OVERLAP): queue everything on `stream` instead
  std::vector<cudaStream_t> class_streams;
  cudaEvent_t fork_ev = nullptr;
  std::vector<cudaEvent_t> join_evs;
  // host-gradient path: copies run on their own stream, one event per shape class
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t copy_gate = nullptr;
  std::vector<cudaEvent_t> copy_done;
  // optional per-category device timing (cudaEvent pairs around groups of launches)
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_events;
  std::vector<int> prof_cats;         // category of span k; its events are prof_events[2k], [2k+1]
  size_t prof_used = 0;               // spans recorded since the last read-out
};

namespace sc {

// ---- host helpers (sc_plan.cu) -------------------------------------------------------------------------
extern std::atomic<long long> g_kernel_launches;   // kernels this library has launched in this process (all plans)
sc_status upload_table(sc_plan* p);
sc_status cuda_ok(cudaError_t e);

// ---- CUDA-core kernels (sc_simt.cu) ----------------------------------------------------------------------
struct GemmArgs {
  const MatDev* tab;
  const int* idx;
  int offA, offB, offC;    // byte offsets of the pointer fields inside MatDev
  int M, N, K;
  int lda, ldb, ldc;
  int transA, transB;
  int a_bf16;              // A holds bf16 (gradients) instead of fp32
  float alpha;
  float beta_c;            // C = alpha * acc + beta_c * C_old (0: plain store)
  int offHi, offLo, ld_split;   // when offHi != 0: also write the result as a bf16 hi/lo pair with this row stride
  int split_only;               // with offHi: the fp32 result itself is not wanted (tsgemm_kernel only)
};
void launch_gemm(const GemmArgs& a, int count, cudaStream_t s);
int atb_splits(int rows, int count);
void launch_sum_slices(const MatDev* tab, const int* idx, int count, int offPart, int offOut, int numel, int nsplit,
                       cudaStream_t s);
void launch_atb(const MatDev* tab, const int* idx, int count, int offA, int offB, int offPart, int offOut, int rows,
                int ca, int cb, int lda, int ldb, int nsplit, cudaStream_t s, int b_slices = 1, bool sum_here = true);
void launch_epilogue_simt(const MatDev* tab, const int* idx, int count, int m, int n, int rp, int g_bf16,
                          const StepScalars& sc, const float* clip, cudaStream_t s);
void launch_ema(const MatDev* tab, const int* idx, int count, int64_t numel, int g_bf16, float beta, cudaStream_t s);
void launch_sketch(float* omega_t, int lp, int l, int64_t n, uint64_t seed, cudaStream_t s);
void launch_sketch_rowmajor(float* omega, int64_t rows, int width, uint64_t seed, cudaStream_t s);
void launch_warm_start(const MatDev* tab, const int* idx, int count, int n, int lp, int l, int rp, int rank,
                       uint64_t seed, cudaStream_t s);
void launch_sketch_padded(float* omega, int64_t rows, int lp, int l, uint64_t seed, cudaStream_t s);
void launch_chol(const MatDev* tab, const int* idx, int count, int lp, int offR, cudaStream_t s);
void launch_jacobi(const MatDev* tab, const int* idx, int count, int lp, int rp, int rank, float tau_p, cudaStream_t s);
void launch_filter_weights(const MatDev* tab, const int* idx, int count, int rp, int rank, float tau_p, cudaStream_t s);
void launch_split_basis(const MatDev* tab, const int* idx, int count, int m, int n, int rp, int rk, cudaStream_t s);
void launch_sqnorm(const MatDev* tab, const int* idx, int count, int64_t numel, int g_bf16, cudaStream_t s);
void launch_xs(const MatDev* tab, const int* idx, int count, int rp, int rank, int x_slices, float scale, float alpha,
               unsigned* status, cudaStream_t s);
void launch_clip(const MatDev* tab, int n_mats, float max_norm, float* clip, cudaStream_t s);
void launch_pad_copy(float* dst, int ldd, const float* src, int lds, int rows, int cols, int cols_dst, cudaStream_t s);
void launch_unpad_copy(float* dst, int ldd, const float* src, int lds, int rows, int cols, cudaStream_t s);
bool filter_ct_supported(int rp);
void launch_filter_ct(const MatDev* tab, const int* idx, int count, int rp, int rank, int n, int rk, float scale,
                      float alpha, unsigned* status, cudaStream_t s);
void launch_reduce_partials(const MatDev* tab, const int* idx, int count, int64_t numel, int ksplit, cudaStream_t s);

// ---- tensor-core kernels (sc_tc.cu) -----------------------------------------------------------------------
bool tc_shape_supported(int64_t m, int64_t n, int rp);
size_t tc_tmaps_bytes(int count);
sc_status tc_init();   // resolves the driver entry point for tensor-map encoding
sc_status tc_encode_class(sc_plan* p, ShapeClass& c, bool static_part, bool per_call_part);
sc_status tc_launch_project(sc_plan* p, ShapeClass& c, const int* idx, int count);   // T = G V
sc_status tc_launch_epilogue(sc_plan* p, ShapeClass& c, const int* idx, int count, const StepScalars& sc);   // AdamW or dual EMA (sc.mix)
sc_status tc_launch_wait_probe(sc_plan* p, int max_polls);
sc_status tc_encode_anchor(sc_plan* p, ShapeClass& c, const std::vector<int>& ids);
sc_status tc_launch_ema_pass(sc_plan* p, ShapeClass& c, const int* idx, int count, int b_field_off);
sc_status tc_launch_gram(sc_plan* p, ShapeClass& c, const int* idx, int count, int panel_field_off, int rows, int slices);
sc_status tc_launch_xpart(sc_plan* p, ShapeClass& c, const int* idx, int count, int slices);
sc_status tc_launch_pass(sc_plan* p, ShapeClass& c, const int* idx, int count, bool transposed, int b_field_off);

// ---- full-spectrum soft filter (sc_fullspec.cu) and the general A^T B tensor-core GEMM (sc_wgrad.cu) ------------
size_t fs_layout(sc_plan* p, char* base);       // base == nullptr: only measures
sc_status fs_refresh(sc_plan* p, int mat);
sc_status fs_step_filter(sc_plan* p, int mat, float filt_scale);
sc_status fs_step_update(sc_plan* p, int mat, const StepScalars& sc);
sc_status launch_tn_gemm(const void* const* A_segs, const void* const* B_segs, int nseg, int64_t K, int64_t M, int64_t N,
                         void* out, void* out_lo, int out_mode, float scale, float diag, unsigned* status,
                         cudaStream_t s);

}  // namespace sc
