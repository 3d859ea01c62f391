// Host layer of the LoRDO hot path: context, workspace carving, launch plans, the C ABI.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include <cuda.h>

#include "lordo_kernels.h"

using namespace lordo;

namespace {

constexpr int kMaxK = 64;

enum StepType { ST_GEMM = 0, ST_CHOL = 1, ST_RANDOM = 2, ST_COPY = 3, ST_SKETCH = 4, ST_CONVERT = 5, ST_NORM = 6, ST_EIG = 7 };
enum Phase { PH_SUBSPACE = 0, PH_ROTATE = 1, PH_COMMIT = 2 };

// One launch of the refresh / init / inner-step plans. The entries it works on are a contiguous
// range [first, first + count) of the table of its type (GEMM problems, Cholesky problems, ...).
struct PlanStep {
  int type = ST_GEMM, phase = PH_SUBSPACE;
  int atrans = 0, dual = 0, a_square = 0;  // gemm
  int r_max = 0;                           // chol
  int p0 = 0;                              // random: 1 = initial projection (draw index 0), 0 = sketch (index = refresh count)
  long long first = 0, tiles = 0;          // tiles: gemm tiles or 256-thread blocks
  int count = 0;
};

// Collects, slot by slot, the entries of many matrices that run the same sequence of steps, so
// that each step of the sequence becomes one launch over all of them.
struct SlotBuilder {
  struct Slot {
    PlanStep st;
    std::vector<GemmProblem> g;
    std::vector<CholProblem> ch;
    std::vector<RandProblem> rn;
    std::vector<CopyProblem> cp;
    std::vector<SkProblem> sk;
    std::vector<ConvProblem> cv;
    std::vector<NormProblem> nm;
    std::vector<EigProblem> eg;
  };
  std::vector<Slot> slots;
  size_t cur = 0;
  void rewind() { cur = 0; }
  Slot& next(int type, int phase, int atrans = 0, int dual = 0, int a_square = 0, int p0 = 0) {
    if (cur == slots.size()) {
      Slot sl;
      sl.st.type = type; sl.st.phase = phase; sl.st.atrans = atrans; sl.st.dual = dual; sl.st.a_square = a_square; sl.st.p0 = p0;
      slots.push_back(sl);
    }
    return slots[cur++];
  }
};

// Bump allocator over the workspace; with base == nullptr it only measures.
struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(void* b) : base(reinterpret_cast<char*>(b)) {}
  template <class T>
  T* take(size_t count) {
    off = (off + 255) & ~size_t(255);
    T* p = reinterpret_cast<T*>(base + off);  // base may be null: only offsets matter then
    off += count * sizeof(T);
    return p;
  }
};

}  // namespace

struct lordo_ctx {
  lordo_config cfg;
  std::vector<lordo_mat> mats;
  std::vector<MatDev> h_mats;
  int n_mats = 0, K = 0;

  // device workspace pieces
  MatDev* d_mats = nullptr;
  long long *d_chunk_start = nullptr, *d_mom_start = nullptr, *d_wblk_start = nullptr, *d_sblk_start = nullptr;
  const void** d_Gtab = nullptr;
  double *d_partial = nullptr, *d_sumsq = nullptr;
  float* d_coef = nullptr;
  unsigned* d_status = nullptr;
  GemmProblem* d_probs = nullptr;
  CholProblem* d_chols = nullptr;
  RandProblem* d_rands = nullptr;
  CopyProblem* d_copies = nullptr;
  SkProblem* d_sks = nullptr;
  ConvProblem* d_convs = nullptr;
  NormProblem* d_norms = nullptr;
  EigProblem* d_eigs = nullptr;
  float* d_scratch = nullptr;
  long long total_chunks = 0, total_mom_tiles = 0, total_wblks = 0, total_sblks = 0;

  // tensor-core path of the inner step (check_mode == 0 and every r <= 256)
  bool tc = false;
  TcProblem* d_tc_probs = nullptr;
  // the update kernel runs once per side present: its table lists the problems stored as they are
  // projected first, then the ones stored transposed (matrices projected from the right)
  TcProblem* d_tc_apply = nullptr;
  std::vector<TcProblem> h_tc_apply;
  int tc_n_left = 0;
  long long tc_strips_left = 0;
  TcPrep* d_tc_prep = nullptr;
  long long* d_prep_start = nullptr;
  char* d_tc_bf16 = nullptr;  // all bf16 operand copies, zeroed once by lordo_init
  size_t tc_bf16_bytes = 0;
  long long tc_strips = 0, tc_strips_p = 0, prep_blocks = 0;
  int tc_rn_max = 0, tc_rk_max = 0;
  // TMA-fed kernels (bf16 storage): tensor maps per matrix, gradient maps re-encoded per pointer change
  bool tma = false;
  int sm_count = 0;
  TmaMatMaps* d_maps = nullptr;
  TmaGradMaps* d_gmaps = nullptr;
  TmaGradMaps* h_gmaps = nullptr;  // pinned, two slots of n_mats entries
  std::vector<TcProblem> h_tc;
  std::vector<TcPrep> h_prep;
  std::vector<long long> h_prep_start;

  // host plans
  std::vector<GemmProblem> h_probs;
  std::vector<CholProblem> h_chols;
  std::vector<RandProblem> h_rands;
  std::vector<CopyProblem> h_copies;
  std::vector<SkProblem> h_sks;
  std::vector<DiagProblem> h_diag;  // one per rotation matrix, ordered by matrix then batch entry
  DiagProblem* d_diag = nullptr;
  std::vector<ConvProblem> h_convs;
  std::vector<NormProblem> h_norms;
  std::vector<EigProblem> h_eigs;
  struct SketchBufs {
    __nv_bfloat16 *om16 = nullptr, *pn16 = nullptr, *zq16 = nullptr;
    // hi|lo planes of the tensor-core QR and rotation (null when those run in fp32)
    __nv_bfloat16 *x16 = nullptr, *rinv16 = nullptr, *phl = nullptr, *rt16 = nullptr, *sq16 = nullptr, *uh16 = nullptr, *wr16 = nullptr;
  };
  std::vector<SketchBufs> h_skbufs;  // per matrix: bf16 right-hand sides of the sketch products (refresh scratch)
  std::vector<PlanStep> inner_proj, inner_apply;  // one launch per side present
  std::vector<PlanStep> refresh_steps, init_steps;
  std::vector<PlanStep> tb_steps;  // Delta rebuilt from the time buffers (lordo_outer_step with time_buffer)

  // pinned host staging
  const void** h_Gtab = nullptr;  // pinned, two slots of n_mats entries
  unsigned* h_status = nullptr;   // pinned
  std::vector<const void*> last_G;
  cudaEvent_t g_slot_ev[2] = {nullptr, nullptr};  // behind the last copy out of each staging slot
  bool g_slot_used[2] = {false, false};
  int g_slot = 0;

  // counters and call-order state
  int64_t steps = 0, refreshes = 0, outers = 0, launches = 0;
  int steps_in_round = 0;
  bool after_outer = false;
  bool rot_valid = false;       // the rotation matrices in the workspace were written by a refresh of this context
  bool p_copies_stale = false;  // the caller may have restored P: the bf16 operand copies are remade before the next use
  std::string err;

  // optional per-kernel-class timing (lordo_profile_enable)
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;
  struct Span { int cls; cudaEvent_t a, b; };
  std::vector<Span> spans;
};

namespace {

typedef CUresult (*tmap_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

tmap_encode_fn tmap_encoder() {
  static tmap_encode_fn fn = []() -> tmap_encode_fn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return reinterpret_cast<tmap_encode_fn>(p);
  }();
  return fn;
}

// bf16 tensor [d2][d1][d0] (d0 contiguous), box b0 x b1 x 1, written into 128 bytes at `out`.
bool encode_map3(unsigned char* out, const void* base, long long d0, long long d1, long long d2, int b0, int b1, bool swizzle) {
  tmap_encode_fn fn = tmap_encoder();
  if (!fn) return false;
  alignas(64) CUtensorMap tm;
  const cuuint64_t dims[3] = {(cuuint64_t)d0, (cuuint64_t)d1, (cuuint64_t)d2};
  const cuuint64_t strides[2] = {(cuuint64_t)d0 * 2, (cuuint64_t)d0 * (cuuint64_t)d1 * 2};
  const cuuint32_t box[3] = {(cuuint32_t)b0, (cuuint32_t)b1, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  std::memcpy(out, &tm, 128);
  return true;
}

int fail(lordo_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate_config(const lordo_config* cfg, std::string& why) {
  if (!cfg || !cfg->mats) { why = "null config or matrix list"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->n_mats < 1 || cfg->K < 1 || cfg->K > kMaxK || cfg->H < 1) { why = "n_mats, K (1..64) or H out of range"; return LORDO_ERR_INVALID_ARG; }
  auto dt_ok = [](int d) { return d == LORDO_F32 || d == LORDO_BF16; };
  if (!dt_ok(cfg->w_dtype) || !dt_ok(cfg->g_dtype) || !dt_ok(cfg->e_dtype)) { why = "unknown dtype"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->variant != LORDO_GLOBAL && cfg->variant != LORDO_LOCAL) { why = "unknown variant"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->outer != LORDO_OUTER_AVG && cfg->outer != LORDO_OUTER_NESTEROV) { why = "unknown outer optimizer"; return LORDO_ERR_INVALID_ARG; }
  if (!(cfg->beta2 >= 0.f && cfg->beta2 < 1.f) || !(cfg->eps >= 0.f)) { why = "beta2 or eps out of range"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->power_iters < 0 || cfg->power_iters > 8) { why = "power_iters out of range (0..8)"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->clip_scope != 0 && cfg->clip_scope != 1) { why = "clip_scope must be 0 or 1"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->time_buffer != 0 && cfg->time_buffer != 1) { why = "time_buffer must be 0 or 1"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->oversample < 0 || cfg->oversample % 8 != 0) { why = "oversample must be a non-negative multiple of 8"; return LORDO_ERR_INVALID_ARG; }
  if (cfg->oversample > 0 && cfg->warm_start) { why = "oversample needs a fresh sketch: warm_start must be 0"; return LORDO_ERR_UNSUPPORTED; }
  for (int i = 0; i < cfg->n_mats; ++i) {
    const lordo_mat& a = cfg->mats[i];
    if (a.m < 1 || a.n < 1 || a.r < 1) { why = "non-positive shape"; return LORDO_ERR_SHAPE; }
    if (a.n % 8 != 0 || a.r % 8 != 0) { why = "n and r must be multiples of 8"; return LORDO_ERR_ALIGN; }
    if (a.side != 0 && a.side != 1) { why = "side must be 0 (left) or 1 (right)"; return LORDO_ERR_INVALID_ARG; }
    if (a.side == 1 && a.m % 8 != 0) { why = "m must be a multiple of 8 for a matrix projected from the right"; return LORDO_ERR_ALIGN; }
    if (a.side == 1 && (cfg->time_buffer || cfg->oversample > 0)) { why = "projection from the right is not available with time_buffer or oversample"; return LORDO_ERR_UNSUPPORTED; }
    if (a.r > a.m || a.r > a.n) { why = "r must not exceed min(m, n)"; return LORDO_ERR_SHAPE; }
    if (cfg->oversample > 0 && (a.r + cfg->oversample > a.m || a.r + cfg->oversample > a.n || a.r + cfg->oversample > 600)) {
      why = "r + oversample must not exceed min(m, n) nor 600";
      return LORDO_ERR_SHAPE;
    }
    if (a.r > 4096) { why = "r above 4096 is not supported"; return LORDO_ERR_UNSUPPORTED; }
  }
  return LORDO_OK;
}

Operand plain(const void* p0, long long ld, int dt0 = LORDO_F32) {
  Operand o;
  std::memset(&o, 0, sizeof(o));
  o.p0 = p0; o.ld = ld; o.dt0 = dt0; o.dt1 = LORDO_F32; o.kind = OP_PLAIN;
  return o;
}

void prefix_arrays(const lordo_config& cfg, std::vector<long long>& chunk_start, std::vector<long long>& mom_start,
                   std::vector<long long>& wblk, std::vector<long long>& sblk) {
  const int n_mats = cfg.n_mats, K = cfg.K;
  chunk_start.assign(n_mats + 1, 0); mom_start.assign(n_mats + 1, 0); wblk.assign(n_mats + 1, 0); sblk.assign(n_mats + 1, 0);
  for (int i = 0; i < n_mats; ++i) {
    const lordo_mat& a = cfg.mats[i];
    const long long elems = a.m * a.n;
    chunk_start[i + 1] = chunk_start[i] + (long long)K * ((elems + kSqChunk - 1) / kSqChunk);
    const long long ln = a.side ? a.m : a.n;  // columns of the low-rank arrays
    mom_start[i + 1] = mom_start[i] + (long long)K * ((ln + 127) / 128);
    wblk[i + 1] = wblk[i] + (elems + 1023) / 1024;
    sblk[i + 1] = sblk[i] + ((long long)a.r * ln + 1023) / 1024;
  }
}

// Builds everything that lives in the workspace. With ws == nullptr only the size is computed.
size_t build(lordo_ctx* c, const lordo_buffers* buf, void* ws) {
  const lordo_config& cfg = c->cfg;
  const int n_mats = cfg.n_mats, K = cfg.K;
  const bool real = ws != nullptr && buf != nullptr;
  const bool local = cfg.variant == LORDO_LOCAL;
  const bool warm = cfg.warm_start != 0;  // start the subspace iteration from the previous P instead of a random sketch
  const int q = (warm && cfg.power_iters < 1) ? 1 : cfg.power_iters;
  Carver cv(ws);

  c->d_mats = cv.take<MatDev>(n_mats);
  c->d_chunk_start = cv.take<long long>(n_mats + 1);
  c->d_mom_start = cv.take<long long>(n_mats + 1);
  c->d_wblk_start = cv.take<long long>(n_mats + 1);
  c->d_sblk_start = cv.take<long long>(n_mats + 1);
  c->d_Gtab = cv.take<const void*>(n_mats);
  c->d_status = cv.take<unsigned>(64);
  c->d_sumsq = cv.take<double>((size_t)n_mats * K);
  c->d_coef = cv.take<float>((size_t)n_mats * K);

  std::vector<long long> chunk_start, mom_start, wblk, sblk;
  prefix_arrays(cfg, chunk_start, mom_start, wblk, sblk);
  // Refresh scratch: matrices are processed in groups whose scratch fits kRefreshScratchFloats;
  // every step of the refresh is one launch over a whole group.
  constexpr size_t kRefreshScratchFloats = size_t(1) << 33;  // 32 GiB: fewer, fuller launches (a launch of the factorisation kernel takes as long for 64 matrices as for 148)
  std::vector<size_t> mat_scratch(n_mats);
  std::vector<int> group_of(n_mats);
  size_t scratch_floats = 0;
  {
    size_t acc = 0;
    int grp = 0;
    for (int i = 0; i < n_mats; ++i) {
      const lordo_mat& a = cfg.mats[i];
      const long long maxd = a.m > a.n ? a.m : a.n;
      const size_t pm = a.side ? a.n : a.m, ln = a.side ? a.m : a.n;  // rows of P, columns of the low-rank arrays
      const size_t nb = local ? K : 1;
      const size_t rs = (size_t)a.r + cfg.oversample;  // columns of the sketch and of everything up to the truncation
      size_t per = ln * rs + 2 * pm * rs + (size_t)maxd * rs + ((q > 0 || cfg.oversample > 0) ? 2 * ln * rs : 0) + 4 * rs * rs;
      if (cfg.oversample > 0) per += 3 * rs * rs + rs * a.r;  // eigen-solver work and the truncating projector
      // bf16 right-hand sides of the tensor-core sketch products (Omega, P', Z), counted in floats
      per += (ln * a.r + (q > 0 ? pm * a.r + ln * a.r : 0)) / 2 + 64;
      size_t states16 = 0;
      if (cfg.check_mode == 0 && cfg.w_dtype == LORDO_BF16) {
        // bf16 planes of the tensor-core QR and rotation: X and R^-1 in three planes, P, Rot^T, its square
        // (per batch entry) and the two moment operands of every worker in two
        per += 3 * (size_t)maxd * a.r / 2 + pm * a.r + 7 * (size_t)a.r * a.r / 2 + 128;
        states16 = 2 * (size_t)K * a.r * ln + 64;
      }
      mat_scratch[i] = nb * per + states16;
      if (acc > 0 && acc + mat_scratch[i] > kRefreshScratchFloats) { ++grp; acc = 0; }
      group_of[i] = grp;
      acc += mat_scratch[i];
      if (acc > scratch_floats) scratch_floats = acc;
    }
  }
  c->total_chunks = chunk_start[n_mats];
  c->total_mom_tiles = mom_start[n_mats];
  c->total_wblks = wblk[n_mats];
  c->total_sblks = sblk[n_mats];
  c->d_partial = cv.take<double>((size_t)c->total_chunks);

  c->h_mats.assign(n_mats, MatDev());
  for (int i = 0; i < n_mats; ++i) {
    const lordo_mat& a = cfg.mats[i];
    MatDev& md = c->h_mats[i];
    md.m = a.m; md.n = a.n; md.r = a.r; md.side = a.side; md.Delta16 = nullptr;
    md.pm = a.side ? a.n : a.m; md.ln = a.side ? a.m : a.n;
    md.ghat = cv.take<float>((size_t)K * a.r * md.ln);
    md.util = cv.take<float>((size_t)K * a.r * md.ln);
    md.dcol = cv.take<float>((size_t)K * md.ln);
    md.T = cfg.time_buffer ? cv.take<float>((size_t)K * a.r * md.ln) : nullptr;
    md.p_stride = local ? md.pm * a.r : 0;
    if (real) {
      md.W = buf->W[i]; md.E = buf->E ? buf->E[i] : nullptr; md.P = buf->P[i]; md.u = buf->u[i]; md.v = buf->v[i];
      md.X0 = buf->X0[i]; md.B = buf->B ? buf->B[i] : nullptr; md.Delta = buf->Delta[i];
    }
  }
  c->d_scratch = cv.take<float>(scratch_floats);

  // ---------------- tensor-core operand copies and problem table ----------------
  c->tc = cfg.check_mode == 0 && cfg.g_dtype == cfg.w_dtype && (!cfg.error_feedback || cfg.e_dtype == cfg.w_dtype);
  for (int i = 0; i < n_mats; ++i)  // ranks above 512 (above 256 with fp32 storage) run on the fp32 path
    if (cfg.mats[i].r > (cfg.w_dtype == LORDO_BF16 ? 512 : 256) || (cfg.mats[i].side && cfg.w_dtype != LORDO_BF16)) c->tc = false;
  c->h_tc.clear(); c->h_prep.clear(); c->h_prep_start.assign(1, 0);
  c->tc_strips = 0; c->tc_strips_p = 0; c->tc_rn_max = 0; c->tc_rk_max = 0;
  if (c->tc) {
    auto up = [](long long x, long long q) { return (x + q - 1) / q * q; };
    (void)cv.take<char>(0);
    const size_t bf16_begin = cv.off;
    for (int i = 0; i < n_mats; ++i) {
      const MatDev& md = c->h_mats[i];
      const int r_k = (int)up(md.r, 64), r_n = (int)up(md.r, 16), m_k = (int)up(md.pm, 64);
      const int copies = local ? K : 1;
      __nv_bfloat16* P16 = cv.take<__nv_bfloat16>((size_t)copies * m_k * r_k);
      __nv_bfloat16* PT16 = cv.take<__nv_bfloat16>((size_t)copies * r_n * m_k);
      const size_t n_pad = (size_t)up(md.ln, 128);  // whole strips: the TMA-fed kernels store these per strip
      __nv_bfloat16* gT16 = cv.take<__nv_bfloat16>((size_t)K * n_pad * r_k);
      __nv_bfloat16* uT16 = cv.take<__nv_bfloat16>((size_t)K * n_pad * r_k);
      const int nsplit = (cfg.w_dtype == LORDO_BF16 && r_n > 256) ? 2 : 1;  // TMA-fed projection: one strip per half of the rank
      float* dcol2 = nsplit == 2 ? cv.take<float>((size_t)K * md.ln) : nullptr;
      if (r_n > c->tc_rn_max) c->tc_rn_max = r_n;
      if (r_k > c->tc_rk_max) c->tc_rk_max = r_k;
      for (int k = 0; k < copies; ++k) {
        TcPrep pp;
        std::memset(&pp, 0, sizeof(pp));
        pp.P = md.P ? md.P + (long long)k * md.pm * md.r : nullptr;
        pp.P16 = P16 + (size_t)k * m_k * r_k; pp.PT16 = PT16 + (size_t)k * r_n * m_k;
        pp.m = md.pm; pp.r = md.r; pp.r_k = r_k; pp.m_k = m_k;
        c->h_prep.push_back(pp);
        c->h_prep_start.push_back(c->h_prep_start.back() + ((md.pm + 63) / 64) * ((md.r + 63) / 64));  // 64 x 64 tiles
      }
      for (int k = 0; k < K; ++k) {
        const long long wo = (long long)k * md.m * md.n, so = (long long)k * md.r * md.ln;
        const int pk = local ? k : 0;
        TcProblem tp;
        std::memset(&tp, 0, sizeof(tp));
        tp.strip_start = c->tc_strips;
        tp.m = (int)md.pm; tp.n = (int)md.ln; tp.tr = md.side; tp.r = md.r; tp.r_k = r_k; tp.r_n = r_n; tp.m_k = m_k;
        tp.PT16 = PT16 + (size_t)pk * r_n * m_k; tp.P16 = P16 + (size_t)pk * m_k * r_k;
        tp.gT16 = gT16 + (size_t)k * n_pad * r_k; tp.uT16 = uT16 + (size_t)k * n_pad * r_k;
        tp.u = md.u ? md.u + so : nullptr; tp.v = md.v ? md.v + so : nullptr;
        tp.dcol = md.dcol + (long long)k * md.ln;
        tp.tb = md.T ? md.T + so : nullptr;
        if (real) {
          tp.W = cfg.w_dtype == LORDO_F32 ? (void*)((float*)md.W + wo) : (void*)((unsigned short*)md.W + wo);
          tp.E = md.E ? (cfg.e_dtype == LORDO_F32 ? (void*)((float*)md.E + wo) : (void*)((unsigned short*)md.E + wo)) : nullptr;
        }
        tp.G_ind = c->d_Gtab + i; tp.G_off = wo;
        tp.cptr = c->d_coef + (size_t)i * K + k;
        tp.mat = i; tp.replica = k; tp.pcopy = pk;
        tp.strip_start_p = c->tc_strips_p; tp.nsplit = nsplit; tp.dcol2 = dcol2 ? dcol2 + (long long)k * md.ln : nullptr;
        c->h_tc.push_back(tp);
        c->tc_strips += (md.ln + 127) / 128;
        c->tc_strips_p += (long long)nsplit * ((md.ln + 255) / 256);  // the projection runs as CTA pairs: two strips each
      }
    }
    c->d_tc_bf16 = ws ? reinterpret_cast<char*>(ws) + bf16_begin : nullptr;
    c->tc_bf16_bytes = cv.off - bf16_begin;
    c->prep_blocks = c->h_prep_start.back();
    c->d_tc_probs = cv.take<TcProblem>(c->h_tc.size());
    c->d_tc_apply = cv.take<TcProblem>(c->h_tc.size());
    c->h_tc_apply.clear();
    c->tc_n_left = 0; c->tc_strips_left = 0;
    {
      long long strips = 0;
      for (int side = 0; side < 2; ++side) {
        for (const TcProblem& tp : c->h_tc) {
          if (tp.tr != side) continue;
          TcProblem q2 = tp;
          q2.strip_start = strips;
          strips += (tp.n + 127) / 128;
          c->h_tc_apply.push_back(q2);
        }
        if (side == 0) { c->tc_n_left = (int)c->h_tc_apply.size(); c->tc_strips_left = strips; }
      }
    }
    c->d_tc_prep = cv.take<TcPrep>(c->h_prep.size());
    c->d_prep_start = cv.take<long long>(c->h_prep_start.size());
    c->tma = cfg.w_dtype == LORDO_BF16;
    c->d_maps = cv.take<TmaMatMaps>(n_mats);
    c->d_gmaps = cv.take<TmaGradMaps>(n_mats);
    if (c->tma && !local)
      for (int i = 0; i < n_mats; ++i) c->h_mats[i].Delta16 = cv.take<__nv_bfloat16>((size_t)c->h_mats[i].m * c->h_mats[i].n);
  }

  // ---------------- launch plans ----------------
  std::vector<GemmProblem>& P = c->h_probs;
  P.clear(); c->h_chols.clear(); c->h_rands.clear(); c->h_copies.clear(); c->h_sks.clear(); c->h_convs.clear(); c->h_norms.clear(); c->h_eigs.clear(); c->h_diag.clear();
  c->h_skbufs.assign(n_mats, lordo_ctx::SketchBufs());
  const bool tc_sketch = c->tc && c->tma && cfg.oversample == 0;  // products of the refresh on tensor cores
  auto gemm_prob = [&](int M, int N, int Kd, const Operand& A, const Operand& B, const Operand* B2, const Epilogue& ep) {
    GemmProblem g;
    std::memset(&g, 0, sizeof(g));
    g.M = M; g.N = N; g.Kd = Kd;
    g.tiles_n = (N + 63) / 64;
    g.A = A; g.B = B;
    if (B2) g.B2 = *B2; else g.B2 = B;
    g.epi = ep;
    return g;
  };
  auto store_epi = [](float* C, long long ldc) {
    Epilogue e;
    std::memset(&e, 0, sizeof(e));
    e.kind = EPI_STORE; e.C = C; e.ldc = ldc;
    return e;
  };
  // Turns the slots of a builder into launches, appending their entries to the tables.
  auto flatten = [&](SlotBuilder& sb, std::vector<PlanStep>& out) {
    for (SlotBuilder::Slot& sl : sb.slots) {
      PlanStep st = sl.st;
      if (st.type == ST_GEMM) {
        st.first = (long long)P.size(); st.count = (int)sl.g.size(); st.tiles = 0;
        for (GemmProblem& g : sl.g) {
          g.tile_start = st.tiles;
          st.tiles += (long long)((g.M + 63) / 64) * g.tiles_n;
          P.push_back(g);
        }
      } else if (st.type == ST_CHOL) {
        st.first = (long long)c->h_chols.size(); st.count = (int)sl.ch.size(); st.r_max = 0;
        for (const CholProblem& x : sl.ch) { if (x.r > st.r_max) st.r_max = x.r; c->h_chols.push_back(x); }
      } else if (st.type == ST_RANDOM) {
        st.first = (long long)c->h_rands.size(); st.count = (int)sl.rn.size(); st.tiles = 0;
        for (RandProblem& x : sl.rn) { x.blk_start = st.tiles; st.tiles += (x.count + 2047) / 2048; c->h_rands.push_back(x); }  // 8 per thread
      } else if (st.type == ST_SKETCH) {
        st.first = (long long)c->h_sks.size(); st.count = (int)sl.sk.size(); st.tiles = 0;
        // the kernel runs as CTA pairs: tiles of 256 rows, 128 per CTA
        for (SkProblem& x : sl.sk) { x.tile_start = st.tiles; st.tiles += (x.M + 255) / 256; c->h_sks.push_back(x); }
      } else if (st.type == ST_CONVERT) {
        st.first = (long long)c->h_convs.size(); st.count = (int)sl.cv.size(); st.tiles = 0;
        for (ConvProblem& x : sl.cv) { x.blk_start = st.tiles; st.tiles += (x.count + 1023) / 1024; c->h_convs.push_back(x); }
      } else if (st.type == ST_EIG) {
        st.first = (long long)c->h_eigs.size(); st.count = (int)sl.eg.size(); st.r_max = 0;
        for (const EigProblem& x : sl.eg) { if (x.w > st.r_max) st.r_max = x.w; c->h_eigs.push_back(x); }
      } else if (st.type == ST_NORM) {
        st.first = (long long)c->h_norms.size(); st.count = (int)sl.nm.size(); st.tiles = 0;
        for (NormProblem& x : sl.nm) { x.blk_start = st.tiles; st.tiles += (x.r + 31) / 32; c->h_norms.push_back(x); }
      } else {
        st.first = (long long)c->h_copies.size(); st.count = (int)sl.cp.size(); st.tiles = 0;
        for (CopyProblem& x : sl.cp) { x.blk_start = st.tiles; st.tiles += (x.chunks + 1023) / 1024; c->h_copies.push_back(x); }
      }
      out.push_back(st);
    }
  };
  auto add_copy = [](SlotBuilder& sb, int phase, void* dst, const void* src, size_t bytes) {
    CopyProblem cp;
    cp.dst = dst; cp.src = src; cp.chunks = (long long)(bytes / 16); cp.blk_start = 0;
    sb.next(ST_COPY, phase).cp.push_back(cp);
  };

  // inner step: g = P^T (c G + E)   and   E' = A - P g ; W' = W - lr (...)
  c->inner_proj.clear();
  c->inner_apply.clear();
  for (int side = 0; side < 2; ++side) {
    SlotBuilder sb;
    for (int i = 0; i < n_mats; ++i) {
      const MatDev& md = c->h_mats[i];
      if (md.side != side) continue;
      for (int k = 0; k < K; ++k) {
        sb.rewind();
        const long long wo = (long long)k * md.m * md.n, so = (long long)k * md.r * md.ln;
        Operand Pk = plain(md.P ? md.P + k * md.p_stride : nullptr, md.r);
        Operand S = plain(nullptr, md.n, cfg.g_dtype);  // c G + E, stored [m][n]
        S.p0_ind = c->d_Gtab + i; S.p0_off = wo;
        S.s0_ptr = c->d_coef + (size_t)i * K + k;
        if (cfg.error_feedback && real) {
          S.p1 = cfg.e_dtype == LORDO_F32 ? (const void*)((const float*)md.E + wo) : (const void*)((const unsigned short*)md.E + wo);
          S.dt1 = cfg.e_dtype;
        }
        if (!side) {  // g [r][n] = P^T (c G + E)
          sb.next(ST_GEMM, 0, 1, 0, 0).g.push_back(gemm_prob(md.r, (int)md.n, (int)md.m, Pk, S, nullptr, store_epi(md.ghat + so, md.n)));
        } else {      // (c G + E) P is [m][r]; kept as its transpose [r][m]
          Epilogue et = store_epi(md.ghat + so, md.m);
          et.trans = 1;
          sb.next(ST_GEMM, 0, 0, 0, 0).g.push_back(gemm_prob((int)md.m, md.r, (int)md.n, S, Pk, nullptr, et));
        }
        Operand B1 = plain(md.ghat + so, md.ln);
        Operand B2 = plain(md.util + so, md.ln);
        Epilogue e;
        std::memset(&e, 0, sizeof(e));
        e.kind = EPI_APPLY;
        e.W = !real ? nullptr : cfg.w_dtype == LORDO_F32 ? (void*)((float*)md.W + wo) : (void*)((unsigned short*)md.W + wo);
        e.E = md.E ? (cfg.e_dtype == LORDO_F32 ? (void*)((float*)md.E + wo) : (void*)((unsigned short*)md.E + wo)) : nullptr;
        e.G_ind = c->d_Gtab + i; e.G_off = wo;
        e.dcol = md.dcol + (long long)k * md.ln;
        e.cptr = c->d_coef + (size_t)i * K + k;
        e.trans = side; e.ldt = md.n;  // side 1: the product P g' is [n][m], element (row, col) is W[col][row]
        sb.next(ST_GEMM, 0, 0, 1, 0).g.push_back(gemm_prob((int)md.pm, (int)md.ln, md.r, Pk, B1, &B2, e));
      }
    }
    std::vector<PlanStep> two;
    flatten(sb, two);
    if (two.size() == 2) { c->inner_proj.push_back(two[0]); c->inner_apply.push_back(two[1]); }
  }

  // CholeskyQR2 of X (rows x r, batch of nb with stride sx) into O, through T.
  auto cholqr2 = [&](SlotBuilder& sb, int phase, float* X, long long sx, float* T, long long st, float* O, long long so,
                     long long rows, int r, int nb, float* gram, float* lw, float* rinv) {
    float* src = X; long long ss = sx;
    for (int pass = 0; pass < 2; ++pass) {
      float* dst = pass == 0 ? T : O;
      const long long sd = pass == 0 ? st : so;
      SlotBuilder::Slot& g = sb.next(ST_GEMM, phase, 1, 0, 0);
      for (int b = 0; b < nb; ++b) {
        Operand A = plain(src + b * ss, r), B = plain(src + b * ss, r);
        g.g.push_back(gemm_prob(r, r, (int)rows, A, B, nullptr, store_epi(gram + (long long)b * r * r, r)));
      }
      SlotBuilder::Slot& ch = sb.next(ST_CHOL, phase);
      for (int b = 0; b < nb; ++b) {
        CholProblem cp;
        cp.gram = gram + (long long)b * r * r; cp.lwork = lw + (long long)b * r * r; cp.rinv = rinv + (long long)b * r * r; cp.r = r; cp.pad = 0;
        ch.ch.push_back(cp);
      }
      SlotBuilder::Slot& ap = sb.next(ST_GEMM, phase, 0, 0, 0);
      for (int b = 0; b < nb; ++b) {
        Operand A = plain(src + b * ss, r), B = plain(rinv + (long long)b * r * r, r);
        ap.g.push_back(gemm_prob((int)rows, r, r, A, B, nullptr, store_epi(dst + b * sd, r)));
      }
      src = dst; ss = sd;
    }
  };

  c->refresh_steps.clear();
  c->init_steps.clear();
  const int n_groups = n_mats ? group_of[n_mats - 1] + 1 : 0;
  for (int grp = 0; grp < n_groups; ++grp) {
    // one sequence of launches per side: a launch has one operand-major setting for all its problems
    SlotBuilder Rs[2], Is[2];
    size_t goff = 0;
    for (int i = 0; i < n_mats; ++i) {
      if (group_of[i] != grp) continue;
      const MatDev& md = c->h_mats[i];
      SlotBuilder &R = Rs[md.side], &I = Is[md.side];
      R.rewind(); I.rewind();
      // the problem as the refresh sees it: P is m x r, the low-rank arrays have n columns, the signal is
      // m x n. For a matrix projected from the right that is the transpose of what is stored (sd = 1).
      const long long m = md.pm, n = md.ln;
      const int sd = md.side;
      const int r = md.r;
      const int nb = local ? K : 1;
      const long long maxd = m > n ? m : n;
      // scratch carve of this matrix inside its group (batch-strided arrays)
      float* s = c->d_scratch + goff;
      goff += mat_scratch[i];
      const bool rr = cfg.oversample > 0;  // oversampled sketch, Rayleigh-Ritz truncation back to r columns
      const int rs = r + cfg.oversample;   // equals r on the tensor-core path
      float* Om = s; s += (size_t)nb * n * rs;
      float* Ya = s; s += (size_t)nb * m * rs;
      float* Pn = s; s += (size_t)nb * m * rs;
      float* Yb = s; s += (size_t)nb * maxd * rs;
      float *Za = nullptr, *Zq = nullptr;
      if (q > 0 || rr) { Za = s; s += (size_t)nb * n * rs; Zq = s; s += (size_t)nb * n * rs; }
      float* gram = s; s += (size_t)nb * rs * rs;
      float* lw = s; s += (size_t)nb * rs * rs;
      float* rinv = s; s += (size_t)nb * rs * rs;
      float* rot = s; s += (size_t)nb * rs * rs;
      float *eigw = nullptr, *mr = nullptr;
      if (rr) { eigw = s; s += (size_t)nb * 3 * rs * rs; mr = s; s += (size_t)nb * rs * r; }
      __nv_bfloat16* om16 = reinterpret_cast<__nv_bfloat16*>(s); s += ((size_t)nb * n * r) / 2 + 16;
      __nv_bfloat16 *pn16 = nullptr, *zq16 = nullptr;
      if (q > 0) {
        pn16 = reinterpret_cast<__nv_bfloat16*>(s); s += ((size_t)nb * m * r) / 2 + 16;
        zq16 = reinterpret_cast<__nv_bfloat16*>(s); s += ((size_t)nb * n * r) / 2 + 16;
      }
      c->h_skbufs[i].om16 = om16; c->h_skbufs[i].pn16 = pn16; c->h_skbufs[i].zq16 = zq16;
      // tensor-core QR and rotation: bf16 planes, plane p of batch entry b at index p * nb + b
      __nv_bfloat16 *x16 = nullptr, *rinv16 = nullptr, *phl = nullptr, *rt16 = nullptr, *sq16 = nullptr, *uh16 = nullptr, *wr16 = nullptr;
      if (tc_sketch) {
        auto take16 = [&](size_t floats) { __nv_bfloat16* p16 = reinterpret_cast<__nv_bfloat16*>(s); s += floats + 16; return p16; };
        x16 = take16(3 * (size_t)nb * maxd * r / 2);
        phl = take16((size_t)nb * m * r);
        rinv16 = take16(3 * (size_t)nb * r * r / 2);
        rt16 = take16((size_t)nb * r * r);
        sq16 = take16((size_t)nb * r * r);
        uh16 = take16((size_t)K * r * n);
        wr16 = take16((size_t)K * r * n);
        lordo_ctx::SketchBufs& kb = c->h_skbufs[i];
        kb.x16 = x16; kb.rinv16 = rinv16; kb.phl = phl; kb.rt16 = rt16; kb.sq16 = sq16; kb.uh16 = uh16; kb.wr16 = wr16;
      }
      TmaMatMaps* mmi = c->d_maps + i;
      auto conv = [&](SlotBuilder& sb, int phase, const ConvProblem& cp) { sb.next(ST_CONVERT, phase).cv.push_back(cp); };
      auto conv_split = [&](SlotBuilder& sb, int phase, const float* src, long long sstride, __nv_bfloat16* planes, long long elems, int np) {
        SlotBuilder::Slot& sl = sb.next(ST_CONVERT, phase);
        for (int b = 0; b < nb; ++b) {
          ConvProblem cp;
          std::memset(&cp, 0, sizeof(cp));
          cp.mode = CONV_SPLIT; cp.src = src ? src + b * sstride : nullptr; cp.count = elems;
          cp.dst = planes + (long long)b * elems; cp.plane = (long long)nb * elems; cp.planes = np;
          sl.cv.push_back(cp);
        }
      };
      // C = A B as the sum of the products of np-plane split operands; planes as above. a_mn: A stored [Kd][M].
      auto sk_split = [&](SlotBuilder::Slot& sl, int a_mn, const unsigned char* map_a, int a_b, int a_nb, const unsigned char* map_b, int b_b, int b_nb,
                          long long Mo, long long Kd, float* C, long long ldc, int c_trans, int np) {
        SkProblem sp;
        std::memset(&sp, 0, sizeof(sp));
        sp.M = (int)Mo; sp.Kd = (int)Kd; sp.r = r; sp.r_n = (r + 15) / 16 * 16;
        sp.a_mn = a_mn; sp.a_c2 = a_b; sp.a_pl = a_nb; sp.b_c2 = b_b; sp.b_pl = b_nb;
        sp.split = np; sp.c_trans = c_trans;
        sp.map_a = map_a; sp.map_b = map_b; sp.C = C; sp.ldc = ldc;
        sl.sk.push_back(sp);
      };
      // CholeskyQR2 with the Gram matrices and the products with R^-1 on tensor cores, operands in three
      // planes: the Gram matrix then carries fp32's rounding noise, which the breakdown threshold of the
      // Cholesky step assumes
      // `last` = false: the result only serves as the right-hand side of the next product of the subspace
      // iteration. Such a basis has to span the same subspace and be well conditioned, no more: one pass
      // instead of two, which leaves it orthonormal to cond(X)^2 * 1e-7. Both products keep their three
      // planes: with fewer, the rounding of X (relative 2^-9 or 2^-17) times cond(X) would enter the
      // weak directions of the span (measured: angles of 0.03..0.1 rad with one plane on a sketch of
      // condition 1e3).
      auto cholqr2_tc = [&](SlotBuilder& sb, int phase, float* X, long long sx, float* T, long long st, float* O, long long so, long long rows,
                            bool last) {
        const bool by_m = rows == m;
        const unsigned char* x_sw = by_m ? mmi->xm_sw : mmi->xn_sw;
        const unsigned char* x_kb = by_m ? mmi->xm_kb : mmi->xn_kb;
        float* src = X; long long ss = sx;
        for (int pass = last ? 0 : 1; pass < 2; ++pass) {
          float* dst = pass == 0 ? T : O;
          const long long sd = pass == 0 ? st : so;
          conv_split(sb, phase, src, ss, x16, rows * r, 3);
          SlotBuilder::Slot& g = sb.next(ST_SKETCH, phase);
          for (int b = 0; b < nb; ++b) sk_split(g, 1, x_sw, b, nb, x_sw, b, nb, r, rows, gram + (long long)b * r * r, r, 0, 3);
          SlotBuilder::Slot& ch = sb.next(ST_CHOL, phase);
          for (int b = 0; b < nb; ++b) {
            CholProblem cp;
            cp.gram = gram + (long long)b * r * r; cp.lwork = lw + (long long)b * r * r; cp.rinv = rinv + (long long)b * r * r; cp.r = r; cp.pad = 0;
            ch.ch.push_back(cp);
          }
          conv_split(sb, phase, rinv, (long long)r * r, rinv16, (long long)r * r, 3);
          SlotBuilder::Slot& ap = sb.next(ST_SKETCH, phase);
          for (int b = 0; b < nb; ++b) sk_split(ap, 0, x_kb, b, nb, mmi->rinv_sw, b, nb, rows, r, dst + b * sd, r, 0, 3);
          src = dst; ss = sd;
        }
        if (!last) return;
        SlotBuilder::Slot& nr = sb.next(ST_NORM, phase);  // the columns of Q back to unit length
        for (int b = 0; b < nb; ++b) {
          NormProblem np;
          np.X = O + b * so; np.blk_start = 0; np.rows = (int)rows; np.r = r;
          nr.nm.push_back(np);
        }
      };
      auto qr2 = [&](SlotBuilder& sb, int phase, float* X, long long sx, float* T, long long st, float* O, long long so, long long rows, int w,
                     bool last = true) {
        if (tc_sketch) cholqr2_tc(sb, phase, X, sx, T, st, O, so, rows, last);
        else cholqr2(sb, phase, X, sx, T, st, O, so, rows, w, nb, gram, lw, rinv);
      };
      // S * B on tensor cores: a_mn = 0 -> S rows are the output rows (Y = S B), 1 -> S^T B
      auto sketch = [&](SlotBuilder& sb, int a_mn, unsigned char* map_b, float* C, long long cstride, long long Mo, long long Kd) {
        SlotBuilder::Slot& sl = sb.next(ST_SKETCH, PH_SUBSPACE);
        for (int b = 0; b < nb; ++b) {
          SkProblem sp;
          std::memset(&sp, 0, sizeof(sp));
          sp.M = (int)Mo; sp.Kd = (int)Kd; sp.r = r; sp.r_n = (r + 15) / 16 * 16;
          const int st_mn = a_mn ^ sd;  // how the stored signal lies with respect to this product
          sp.a_mn = st_mn; sp.a_c2 = local ? b : 0; sp.b_c2 = b;
          TmaMatMaps* mm = c->d_maps + i;
          TmaGradMaps* gm = c->d_gmaps + i;
          if (local) {
            sp.map_a = st_mn ? gm->g_sw : gm->g_kb;
            if (cfg.error_feedback) { sp.map_e = st_mn ? mm->e_sw : mm->e_kb; sp.cptr = c->d_coef + (size_t)i * K + b; }
          } else {
            sp.map_a = st_mn ? mm->d_sw : mm->d_kb;
          }
          sp.map_b = map_b;
          sp.C = C + (long long)b * cstride; sp.ldc = r;
          sl.sk.push_back(sp);
        }
      };
      auto convert = [&](SlotBuilder& sb, const float* src, __nv_bfloat16* dst, size_t count) {
        ConvProblem cp;
        std::memset(&cp, 0, sizeof(cp));
        cp.mode = CONV_BF16; cp.src = src; cp.dst = dst; cp.count = (long long)count;
        sb.next(ST_CONVERT, PH_SUBSPACE).cv.push_back(cp);
      };

      auto signal = [&](int b) {  // S of problem b: Delta (Global) or c_k G_k + E_k (Local), as stored: [md.m][md.n]
        if (!local) return plain(md.Delta, md.n);
        Operand A = plain(nullptr, md.n, cfg.g_dtype);
        A.p0_ind = c->d_Gtab + i; A.p0_off = (long long)b * m * n;
        A.s0_ptr = c->d_coef + (size_t)i * K + b;
        if (cfg.error_feedback && real) {
          A.p1 = cfg.e_dtype == LORDO_F32 ? (const void*)((const float*)md.E + (long long)b * m * n)
                                          : (const void*)((const unsigned short*)md.E + (long long)b * m * n);
          A.dt1 = cfg.e_dtype;
        }
        return A;
      };
      if (warm) {  // block power iteration warm-started from the current basis
        if (tc_sketch && !local) convert(R, md.Delta, md.Delta16, (size_t)m * n);
        add_copy(R, PH_SUBSPACE, Pn, md.P, (size_t)nb * m * r * sizeof(float));
      } else {
        {
          SlotBuilder::Slot& f = R.next(ST_RANDOM, PH_SUBSPACE);
          for (int b = 0; b < nb; ++b) {
            RandProblem rp;
            rp.out = tc_sketch ? nullptr : Om + (long long)b * n * rs;
            rp.out16 = tc_sketch ? om16 + (long long)b * n * r : nullptr;
            rp.count = n * rs; rp.blk_start = 0; rp.purpose = 2; rp.mat = i; rp.replica = local ? b : 0; rp.pad = 0;
            f.rn.push_back(rp);
          }
        }
        if (tc_sketch) {  // Y = S Omega
          if (!local) convert(R, md.Delta, md.Delta16, (size_t)m * n);  // bf16 copy of the Global signal
          sketch(R, 0, (c->d_maps + i)->om16, Ya, m * r, m, n);
        } else {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, sd, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob((int)m, rs, (int)n, signal(b), plain(Om + (long long)b * n * rs, rs), nullptr, store_epi(Ya + (long long)b * m * rs, rs)));
        }
        qr2(R, PH_SUBSPACE, Ya, m * rs, Yb, maxd * rs, Pn, m * rs, m, rs, q == 0 || rr);
      }
      for (int it = 0; it < q; ++it) {
        if (tc_sketch) {  // Z = S^T P'
          convert(R, Pn, pn16, (size_t)nb * m * r);
          sketch(R, 1, (c->d_maps + i)->pn16, Za, n * r, n, m);
        } else {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, 1 - sd, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob((int)n, rs, (int)m, signal(b), plain(Pn + (long long)b * m * rs, rs), nullptr, store_epi(Za + (long long)b * n * rs, rs)));
        }
        qr2(R, PH_SUBSPACE, Za, n * rs, Yb, maxd * rs, Zq, n * rs, n, rs, rr);
        if (tc_sketch) {  // Y = S Z
          convert(R, Zq, zq16, (size_t)nb * n * r);
          sketch(R, 0, (c->d_maps + i)->zq16, Ya, m * r, m, n);
        } else {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, sd, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob((int)m, rs, (int)n, signal(b), plain(Zq + (long long)b * n * rs, rs), nullptr, store_epi(Ya + (long long)b * m * rs, rs)));
        }
        qr2(R, PH_SUBSPACE, Ya, m * rs, Yb, maxd * rs, Pn, m * rs, m, rs, it == q - 1 || rr);
      }
      if (rr) {
        // Rayleigh-Ritz truncation of the (r + p)-column basis Q (in Pn): Z = S^T Q, C = Z^T Z, the
        // projector onto the r leading eigenvectors of C, P' = qr(Q M[:, :r])
        {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, 1, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob((int)n, rs, (int)m, signal(b), plain(Pn + (long long)b * m * rs, rs), nullptr, store_epi(Za + (long long)b * n * rs, rs)));
        }
        {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, 1, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob(rs, rs, (int)n, plain(Za + (long long)b * n * rs, rs), plain(Za + (long long)b * n * rs, rs), nullptr, store_epi(gram + (long long)b * rs * rs, rs)));
        }
        {
          SlotBuilder::Slot& e = R.next(ST_EIG, PH_SUBSPACE);
          for (int b = 0; b < nb; ++b) {
            EigProblem ep;
            ep.C = gram + (long long)b * rs * rs; ep.work = eigw + (long long)b * 3 * rs * rs; ep.Mr = mr + (long long)b * rs * r; ep.w = rs; ep.r = r;
            e.eg.push_back(ep);
          }
        }
        {
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, 0, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob((int)m, r, rs, plain(Pn + (long long)b * m * rs, rs), plain(mr + (long long)b * rs * r, r), nullptr, store_epi(Ya + (long long)b * m * r, r)));
        }
        qr2(R, PH_SUBSPACE, Ya, m * r, Yb, maxd * r, Pn, m * r, m, r);
      }
      for (int b = 0; b < nb; ++b) {
        DiagProblem dp;
        dp.rot = rot + (long long)b * r * r; dp.r = r; dp.pad = 0;
        c->h_diag.push_back(dp);
      }
      if (tc_sketch) {
        // Rot = P'^T P and the rotated moments on tensor cores, operands in two planes (16 bits each)
        conv_split(R, PH_SUBSPACE, Pn, m * r, x16, m * r, 2);
        conv_split(R, PH_SUBSPACE, md.P, md.p_stride, phl, m * r, 2);
        {
          SlotBuilder::Slot& g = R.next(ST_SKETCH, PH_SUBSPACE);
          for (int b = 0; b < nb; ++b) sk_split(g, 1, mmi->xm_sw, b, nb, mmi->phl_sw, b, nb, r, m, rot + (long long)b * r * r, r, 0, 2);
        }
        {  // Rot^T and its element-wise square as right-hand sides
          SlotBuilder::Slot& sl = R.next(ST_CONVERT, PH_ROTATE);
          for (int b = 0; b < nb; ++b) {
            ConvProblem cp;
            std::memset(&cp, 0, sizeof(cp));
            cp.mode = CONV_ROT_T; cp.src = rot + (long long)b * r * r; cp.count = (long long)r * r; cp.ld = r;
            cp.dst = rt16 + (long long)b * r * r; cp.dst2 = sq16 + (long long)b * r * r; cp.plane = (long long)nb * r * r; cp.planes = 2;
            sl.cv.push_back(cp);
          }
        }
        {  // u^ and v^ - u^ u^ of all workers as hi|lo planes [2K][r][n]
          ConvProblem cp;
          std::memset(&cp, 0, sizeof(cp));
          cp.mode = CONV_STATES; cp.src = md.u; cp.src2 = md.v; cp.count = (long long)K * r * n;
          cp.dst = uh16; cp.dst2 = wr16; cp.plane = (long long)K * r * n; cp.planes = 2;
          conv(R, PH_ROTATE, cp);
        }
        {  // (Rot u^)^T = u^^T Rot^T, stored back as [r][n] into the transient g^ area; same for the second moment
          SlotBuilder::Slot& g1 = R.next(ST_SKETCH, PH_ROTATE);
          for (int k = 0; k < K; ++k)
            sk_split(g1, 1, mmi->uh_sw, k, K, mmi->rt_sw, local ? k : 0, nb, n, r, md.ghat + (long long)k * r * n, n, 1, 2);
          SlotBuilder::Slot& g2 = R.next(ST_SKETCH, PH_ROTATE);
          for (int k = 0; k < K; ++k)
            sk_split(g2, 1, mmi->wr_sw, k, K, mmi->sq_sw, local ? k : 0, nb, n, r, md.util + (long long)k * r * n, n, 1, 2);
        }
        {  // u = bc1 (Rot u^), v = bc2 |Rot^2 (v^ - u^ u^) + (Rot u^)^2|
          ConvProblem cp;
          std::memset(&cp, 0, sizeof(cp));
          cp.mode = CONV_COMBINE; cp.src = md.ghat; cp.src2 = md.util; cp.outf = md.u; cp.outf2 = md.v; cp.count = (long long)K * r * n;
          conv(R, PH_ROTATE, cp);
        }
      } else {
        {  // Rot = P'^T P (always formed: it also carries the MSSV diagnostic)
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_SUBSPACE, 1, 0, 0);
          for (int b = 0; b < nb; ++b) g.g.push_back(gemm_prob(r, r, (int)m, plain(Pn + (long long)b * m * r, r), plain(md.P ? md.P + b * md.p_stride : nullptr, r), nullptr, store_epi(rot + (long long)b * r * r, r)));
        }
        {  // u', v' (into the transient g^ / U~ areas), then back
          SlotBuilder::Slot& g = R.next(ST_GEMM, PH_ROTATE, 0, 1, 1);
          for (int k = 0; k < K; ++k) {
            const long long so = (long long)k * r * n;
            Operand A = plain(rot + (long long)(local ? k : 0) * r * r, r);
            Operand B = plain(md.u ? md.u + so : nullptr, n); B.kind = OP_UHAT;
            Operand B2 = plain(md.u ? md.u + so : nullptr, n); B2.kind = OP_VRES; B2.p1 = md.v ? md.v + so : nullptr;
            Epilogue e;
            std::memset(&e, 0, sizeof(e));
            e.kind = EPI_ROTATE; e.u_out = md.ghat + so; e.v_out = md.util + so;
            g.g.push_back(gemm_prob(r, (int)n, r, A, B, &B2, e));
          }
          add_copy(R, PH_ROTATE, md.u, md.ghat, (size_t)K * r * n * sizeof(float));
          add_copy(R, PH_ROTATE, md.v, md.util, (size_t)K * r * n * sizeof(float));
        }
      }
      add_copy(R, PH_COMMIT, md.P, Pn, (size_t)nb * m * r * sizeof(float));
      if (!local) {  // P_0 = orthonormalised random m x r matrix
        RandProblem rp;
        rp.out = Ya; rp.out16 = nullptr; rp.count = m * r; rp.blk_start = 0; rp.purpose = 1; rp.mat = i; rp.replica = 0; rp.pad = 0;
        I.next(ST_RANDOM, PH_SUBSPACE, 0, 0, 0, 1).rn.push_back(rp);
        cholqr2(I, PH_SUBSPACE, Ya, m * r, Yb, maxd * r, md.P, m * r, m, r, 1, gram, lw, rinv);
      }
    }
    for (int sd = 0; sd < 2; ++sd) {
      flatten(Rs[sd], c->refresh_steps);
      flatten(Is[sd], c->init_steps);
    }
  }
  // Up-link time buffer: Delta = P T_mean (Global, after the buffers were averaged) or the sum over
  // the workers of P_k T_k (Local; the outer kernel divides by K), one grouped GEMM per term.
  c->tb_steps.clear();
  if (cfg.time_buffer) {
    SlotBuilder TB;
    for (int i = 0; i < n_mats; ++i) {
      TB.rewind();
      const MatDev& md = c->h_mats[i];
      const int terms = local ? K : 1;
      for (int k = 0; k < terms; ++k) {
        Epilogue e = store_epi(md.Delta, md.n);
        e.pad = k > 0;  // accumulate
        TB.next(ST_GEMM, 0, 0, 0, 0).g.push_back(gemm_prob((int)md.m, (int)md.n, md.r, plain(md.P ? md.P + (long long)k * md.p_stride : nullptr, md.r),
                                                            plain(md.T + (long long)k * md.r * md.n, md.n), nullptr, e));
      }
    }
    flatten(TB, c->tb_steps);
  }
  c->d_probs = cv.take<GemmProblem>(P.size());
  c->d_chols = cv.take<CholProblem>(c->h_chols.size() + 1);
  c->d_rands = cv.take<RandProblem>(c->h_rands.size() + 1);
  c->d_copies = cv.take<CopyProblem>(c->h_copies.size() + 1);
  c->d_sks = cv.take<SkProblem>(c->h_sks.size() + 1);
  c->d_convs = cv.take<ConvProblem>(c->h_convs.size() + 1);
  c->d_norms = cv.take<NormProblem>(c->h_norms.size() + 1);
  c->d_eigs = cv.take<EigProblem>(c->h_eigs.size() + 1);
  c->d_diag = cv.take<DiagProblem>(c->h_diag.size() + 1);

  c->last_G.assign(n_mats, nullptr);
  return (cv.off + 255) & ~size_t(255);
}

#define CUDA_OK(c, call)                                                                          \
  do {                                                                                            \
    cudaError_t e_ = (call);                                                                      \
    if (e_ != cudaSuccess) return fail(c, LORDO_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
  } while (0)

int check_launch(lordo_ctx* c, const char* what) {
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) return fail(c, LORDO_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
  return LORDO_OK;
}

// Kernel classes reported by lordo_profile_read.
enum ProfClass { PC_CLIP = 0, PC_PROJECT = 1, PC_MOMENTS = 2, PC_APPLY = 3, PC_OUTER_STATES = 4, PC_OUTER_WEIGHTS = 5, PC_REFRESH = 6 };

cudaEvent_t take_event(lordo_ctx* c) {
  if (!c->ev_pool.empty()) { cudaEvent_t e = c->ev_pool.back(); c->ev_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct ProfScope {
  lordo_ctx* c; cudaStream_t st; int cls; cudaEvent_t a = nullptr;
  ProfScope(lordo_ctx* c_, cudaStream_t st_, int cls_) : c(c_), st(st_), cls(cls_) {
    if (c->profiling) { a = take_event(c); cudaEventRecord(a, st); }
  }
  ~ProfScope() {
    if (a) { cudaEvent_t b = take_event(c); cudaEventRecord(b, st); c->spans.push_back({cls, a, b}); }
  }
};

GemmScalars base_scalars(const lordo_ctx* c) {
  GemmScalars s;
  std::memset(&s, 0, sizeof(s));
  s.w_dt = c->cfg.w_dtype; s.e_dt = c->cfg.e_dtype; s.g_dt = c->cfg.g_dtype;
  s.ef = c->cfg.error_feedback;
  s.inv_bc1 = s.inv_bc2 = s.bc1 = s.bc2 = 1.f;
  return s;
}

int run_plan_step(lordo_ctx* c, const PlanStep& s, GemmScalars sc, cudaStream_t st) {
  if (s.count == 0) return LORDO_OK;
  switch (s.type) {
    case ST_GEMM:
      sc.a_square = s.a_square;
      launch_gemm(c->d_probs + s.first, s.count, s.tiles, s.atrans, s.dual, c->cfg.check_mode != 0, sc, st);
      c->launches += 1;
      return check_launch(c, "gemm");
    case ST_CHOL:
      launch_chol_inverse(c->d_chols + s.first, s.count, s.r_max, c->d_status, st);
      c->launches += 1;
      return check_launch(c, "chol_inverse");
    case ST_RANDOM:
      launch_fill_random_grouped(c->d_rands + s.first, s.count, s.tiles, c->cfg.seed, s.p0 ? 0 : c->refreshes, st);
      c->launches += 1;
      return check_launch(c, "fill_random");
    case ST_SKETCH:
      launch_sketch_tma(c->d_sks + s.first, s.count, s.tiles, c->sm_count, c->tc_rn_max > 256, c->d_status, st);
      c->launches += 1;
      return check_launch(c, "sketch");
    case ST_CONVERT:
      launch_convert_grouped(c->d_convs + s.first, s.count, s.tiles, sc, st);
      c->launches += 1;
      return check_launch(c, "convert");
    case ST_EIG:
      launch_jacobi_projector(c->d_eigs + s.first, s.count, s.r_max, st);
      c->launches += 1;
      return check_launch(c, "jacobi_projector");
    case ST_NORM:
      launch_colnorm_grouped(c->d_norms + s.first, s.count, s.tiles, st);
      c->launches += 1;
      return check_launch(c, "colnorm");
    case ST_COPY:
      launch_copy_grouped(c->d_copies + s.first, s.count, s.tiles, st);
      c->launches += 1;
      return check_launch(c, "copy");
  }
  return LORDO_OK;
}

// Makes the device copy of the gradient pointer table (and of the gradients' tensor maps) current.
// The pinned staging tables have two slots, each with an event recorded behind its last copy, so a
// change of pointers waits at most for the copy made two changes ago, never for the whole stream.
// Nothing of the context is updated until every tensor map has been encoded: a failed call leaves
// the previous tables in force and is not mistaken for "same pointers" on a retry.
int set_gradients(lordo_ctx* c, const void* const* G, cudaStream_t st) {
  bool same = true;
  for (int i = 0; i < c->n_mats; ++i) {
    if (!G[i]) return fail(c, LORDO_ERR_INVALID_ARG, "null gradient pointer");
    if (!aligned16(G[i])) return fail(c, LORDO_ERR_ALIGN, "gradient pointer not 16-byte aligned");
    if (G[i] != c->last_G[i]) same = false;
  }
  if (same) return LORDO_OK;
  const int slot = c->g_slot ^ 1;
  if (c->g_slot_used[slot]) CUDA_OK(c, cudaEventSynchronize(c->g_slot_ev[slot]));
  const void** tab = c->h_Gtab + (size_t)slot * c->n_mats;
  TmaGradMaps* gm = c->tma ? c->h_gmaps + (size_t)slot * c->n_mats : nullptr;
  if (c->tma) {
    for (int i = 0; i < c->n_mats; ++i) {
      const lordo_mat& a = c->mats[i];
      if (!encode_map3(gm[i].g_sw, G[i], a.n, a.m, c->K, 64, 64, true) || !encode_map3(gm[i].g_kb, G[i], a.n, a.m, c->K, 64, 128, true))
        return fail(c, LORDO_ERR_CUDA, "tensor map encoding failed for a gradient");
    }
  }
  for (int i = 0; i < c->n_mats; ++i) tab[i] = G[i];
  cudaError_t e = cudaMemcpyAsync(c->d_Gtab, tab, sizeof(void*) * c->n_mats, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && c->tma) e = cudaMemcpyAsync(c->d_gmaps, gm, sizeof(TmaGradMaps) * c->n_mats, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaEventRecord(c->g_slot_ev[slot], st);
  if (e != cudaSuccess) {
    // the device tables may be half written: force the next call to write them again
    c->last_G.assign(c->n_mats, nullptr);
    return fail(c, LORDO_ERR_CUDA, std::string("gradient tables: ") + cudaGetErrorString(e));
  }
  c->g_slot = slot;
  c->g_slot_used[slot] = true;
  for (int i = 0; i < c->n_mats; ++i) c->last_G[i] = G[i];
  return LORDO_OK;
}

int run_clip(lordo_ctx* c, cudaStream_t st) {
  if (!(c->cfg.clip_rho > 0.f)) return LORDO_OK;  // coefficients stay at 1
  launch_sumsq_partial(c->d_mats, c->d_Gtab, c->d_chunk_start, c->n_mats, c->K, c->cfg.g_dtype, c->d_partial, c->total_chunks, st);
  launch_clip_finalize(c->d_mats, c->d_chunk_start, c->n_mats, c->K, c->d_partial, c->cfg.clip_rho, c->cfg.clip_scope, c->d_coef,
                       c->d_sumsq, c->d_status, st);
  c->launches += 3;
  return check_launch(c, "clip");
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

const char* lordo_status_string(int s) {
  switch (s) {
    case LORDO_OK: return "ok";
    case LORDO_ERR_INVALID_ARG: return "invalid argument";
    case LORDO_ERR_SHAPE: return "bad shape";
    case LORDO_ERR_ALIGN: return "bad alignment";
    case LORDO_ERR_STATE: return "call out of order";
    case LORDO_ERR_NOMEM: return "workspace too small or host allocation failed";
    case LORDO_ERR_CUDA: return "CUDA error";
    case LORDO_ERR_NUMERIC: return "numerical flag set on the device";
    case LORDO_ERR_UNSUPPORTED: return "unsupported configuration";
  }
  return "unknown status";
}

int lordo_query_workspace(const lordo_config* cfg, size_t* bytes) {
  std::string why;
  int rc = validate_config(cfg, why);
  if (rc != LORDO_OK) return rc;
  if (!bytes) return LORDO_ERR_INVALID_ARG;
  lordo_ctx tmp;
  tmp.cfg = *cfg;
  tmp.n_mats = cfg->n_mats; tmp.K = cfg->K;
  *bytes = build(&tmp, nullptr, nullptr);
  return LORDO_OK;
}

int lordo_init(const lordo_config* cfg, const lordo_buffers* buf, void* workspace, size_t workspace_bytes, void* stream,
               lordo_ctx** out) {
  std::string why;
  int rc = validate_config(cfg, why);
  if (rc != LORDO_OK) return rc;
  if (!buf || !workspace || !out) return LORDO_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LORDO_ERR_ALIGN;
  if (!buf->W || !buf->P || !buf->u || !buf->v || !buf->X0 || !buf->Delta) return LORDO_ERR_INVALID_ARG;
  if (cfg->error_feedback && !buf->E) return LORDO_ERR_INVALID_ARG;
  if (cfg->outer == LORDO_OUTER_NESTEROV && !buf->B) return LORDO_ERR_INVALID_ARG;
  for (int i = 0; i < cfg->n_mats; ++i) {
    const void* ptrs[8] = {buf->W[i], cfg->error_feedback ? buf->E[i] : (void*)16, buf->P[i], buf->u[i], buf->v[i], buf->X0[i],
                           cfg->outer == LORDO_OUTER_NESTEROV ? (void*)buf->B[i] : (void*)16, buf->Delta[i]};
    for (const void* p : ptrs) {
      if (!p) return LORDO_ERR_INVALID_ARG;
      if (!aligned16(p)) return LORDO_ERR_ALIGN;
    }
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  lordo_ctx* c = new (std::nothrow) lordo_ctx;
  if (!c) return LORDO_ERR_NOMEM;
  c->cfg = *cfg;
  c->mats.assign(cfg->mats, cfg->mats + cfg->n_mats);
  c->cfg.mats = c->mats.data();
  c->n_mats = cfg->n_mats; c->K = cfg->K;
  const size_t need = build(c, buf, workspace);
  if (need > workspace_bytes) { delete c; return LORDO_ERR_NOMEM; }

  auto bail = [&](int code) { lordo_destroy(c); return code; };
  if (cudaHostAlloc((void**)&c->h_Gtab, 2 * sizeof(void*) * c->n_mats, cudaHostAllocDefault) != cudaSuccess) return bail(LORDO_ERR_NOMEM);
  for (int sl = 0; sl < 2; ++sl)
    if (cudaEventCreateWithFlags(&c->g_slot_ev[sl], cudaEventDisableTiming) != cudaSuccess) return bail(LORDO_ERR_CUDA);
  if (cudaHostAlloc((void**)&c->h_status, 256, cudaHostAllocDefault) != cudaSuccess) return bail(LORDO_ERR_NOMEM);

  std::vector<long long> cs, ms, wb, sb;
  prefix_arrays(c->cfg, cs, ms, wb, sb);
  const int nm = c->n_mats;
#define INIT_CUDA(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return bail(LORDO_ERR_CUDA); } } while (0)
  INIT_CUDA(cudaMemcpyAsync(c->d_mats, c->h_mats.data(), sizeof(MatDev) * nm, cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->d_chunk_start, cs.data(), 8 * (nm + 1), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->d_mom_start, ms.data(), 8 * (nm + 1), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->d_wblk_start, wb.data(), 8 * (nm + 1), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->d_sblk_start, sb.data(), 8 * (nm + 1), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemcpyAsync(c->d_probs, c->h_probs.data(), sizeof(GemmProblem) * c->h_probs.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_chols.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_chols, c->h_chols.data(), sizeof(CholProblem) * c->h_chols.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_rands.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_rands, c->h_rands.data(), sizeof(RandProblem) * c->h_rands.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_copies.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_copies, c->h_copies.data(), sizeof(CopyProblem) * c->h_copies.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_sks.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_sks, c->h_sks.data(), sizeof(SkProblem) * c->h_sks.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_diag.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_diag, c->h_diag.data(), sizeof(DiagProblem) * c->h_diag.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_convs.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_convs, c->h_convs.data(), sizeof(ConvProblem) * c->h_convs.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_norms.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_norms, c->h_norms.data(), sizeof(NormProblem) * c->h_norms.size(), cudaMemcpyHostToDevice, st));
  if (!c->h_eigs.empty()) INIT_CUDA(cudaMemcpyAsync(c->d_eigs, c->h_eigs.data(), sizeof(EigProblem) * c->h_eigs.size(), cudaMemcpyHostToDevice, st));
  INIT_CUDA(cudaMemsetAsync(c->d_status, 0, 256, st));
  if (c->tc) {
    if (!c->tma) INIT_CUDA(tc_configure(c->tc_rn_max, c->tc_rk_max));  // register-staged kernels (fp32 storage)
    INIT_CUDA(cudaMemsetAsync(c->d_tc_bf16, 0, c->tc_bf16_bytes, st));
    INIT_CUDA(cudaMemcpyAsync(c->d_tc_probs, c->h_tc.data(), sizeof(TcProblem) * c->h_tc.size(), cudaMemcpyHostToDevice, st));
    INIT_CUDA(cudaMemcpyAsync(c->d_tc_apply, c->h_tc_apply.data(), sizeof(TcProblem) * c->h_tc_apply.size(), cudaMemcpyHostToDevice, st));
    INIT_CUDA(cudaMemcpyAsync(c->d_tc_prep, c->h_prep.data(), sizeof(TcPrep) * c->h_prep.size(), cudaMemcpyHostToDevice, st));
    INIT_CUDA(cudaMemcpyAsync(c->d_prep_start, c->h_prep_start.data(), 8 * c->h_prep_start.size(), cudaMemcpyHostToDevice, st));
    if (c->tma) {
      int dev = 0;
      INIT_CUDA(cudaGetDevice(&dev));
      INIT_CUDA(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
      if (c->sm_count < 2) return bail(LORDO_ERR_UNSUPPORTED);  // the projection and the refresh products run as CTA pairs
      std::vector<TmaMatMaps> hm(nm);
      bool good = tmap_encoder() != nullptr;
      const bool loc = c->cfg.variant == LORDO_LOCAL;
      for (int i = 0; i < nm && good; ++i) {
        const MatDev& md = c->h_mats[i];
        const TcProblem& tp = c->h_tc[(size_t)i * c->K];  // worker 0 of matrix i: base pointers of the copies
        const int copies = loc ? c->K : 1;
        std::memset(&hm[i], 0, sizeof(TmaMatMaps));
        if (md.E) {
          good = good && encode_map3(hm[i].e_sw, md.E, md.n, md.m, c->K, 64, 64, true);
          good = good && encode_map3(hm[i].e_st, md.E, md.n, md.m, c->K, 64, 16, true);
        }
        good = good && encode_map3(hm[i].w_sw, md.W, md.n, md.m, c->K, 64, 64, true);
        good = good && encode_map3(hm[i].w_st, md.W, md.n, md.m, c->K, 64, 16, true);
        if (md.side) {  // tiles of 128 stored rows x 64 stored columns, handed back 32 rows at a time
          good = good && encode_map3(hm[i].w_kb, md.W, md.n, md.m, c->K, 64, 128, true);
          good = good && encode_map3(hm[i].w_st32, md.W, md.n, md.m, c->K, 64, 32, true);
          if (md.E) good = good && encode_map3(hm[i].e_st32, md.E, md.n, md.m, c->K, 64, 32, true);
        }
        good = good && encode_map3(hm[i].pt, tp.PT16, tp.m_k, tp.r_n, copies, 64, tp.r_n <= 256 ? tp.r_n / 2 : 128, true);  // a CTA's half of an MMA's rows
        good = good && encode_map3(hm[i].p16, tp.P16, tp.r_k, tp.m_k, copies, 64, 64, true);
        // refresh: signal as rows (64 k x 128 rows) and right-hand sides [batch][Kd][r]
        const int nbatch = loc ? c->K : 1;
        if (md.E) good = good && encode_map3(hm[i].e_kb, md.E, md.n, md.m, c->K, 64, 128, true);
        if (md.Delta16) {
          good = good && encode_map3(hm[i].d_kb, md.Delta16, md.n, md.m, 1, 64, 128, true);
          good = good && encode_map3(hm[i].d_sw, md.Delta16, md.n, md.m, 1, 64, 64, true);
        }
        const lordo_ctx::SketchBufs& sb = c->h_skbufs[i];
        good = good && encode_map3(hm[i].om16, sb.om16, md.r, md.ln, nbatch, 64, 64, true);
        if (sb.pn16) good = good && encode_map3(hm[i].pn16, sb.pn16, md.r, md.pm, nbatch, 64, 64, true);
        if (sb.zq16) good = good && encode_map3(hm[i].zq16, sb.zq16, md.r, md.ln, nbatch, 64, 64, true);
        if (sb.x16) {  // hi|lo planes of the tensor-core QR and rotation
          good = good && encode_map3(hm[i].xm_sw, sb.x16, md.r, md.pm, 3 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].xm_kb, sb.x16, md.r, md.pm, 3 * nbatch, 64, 128, true);
          good = good && encode_map3(hm[i].xn_sw, sb.x16, md.r, md.ln, 3 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].xn_kb, sb.x16, md.r, md.ln, 3 * nbatch, 64, 128, true);
          good = good && encode_map3(hm[i].rinv_sw, sb.rinv16, md.r, md.r, 3 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].phl_sw, sb.phl, md.r, md.pm, 2 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].rt_sw, sb.rt16, md.r, md.r, 2 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].sq_sw, sb.sq16, md.r, md.r, 2 * nbatch, 64, 64, true);
          good = good && encode_map3(hm[i].uh_sw, sb.uh16, md.ln, md.r, 2 * c->K, 64, 64, true);
          good = good && encode_map3(hm[i].wr_sw, sb.wr16, md.ln, md.r, 2 * c->K, 64, 64, true);
        }
      }
      if (good) {
        INIT_CUDA(cudaMemcpyAsync(c->d_maps, hm.data(), sizeof(TmaMatMaps) * nm, cudaMemcpyHostToDevice, st));
        INIT_CUDA(cudaStreamSynchronize(st));
        INIT_CUDA(tma_configure());
        if (cudaHostAlloc((void**)&c->h_gmaps, 2 * sizeof(TmaGradMaps) * nm, cudaHostAllocDefault) != cudaSuccess) return bail(LORDO_ERR_NOMEM);
      } else {
        return bail(LORDO_ERR_CUDA);  // tensor maps could not be encoded (driver without cuTensorMapEncodeTiled?)
      }
    }
  }
  INIT_CUDA(cudaMemsetAsync(c->d_Gtab, 0, sizeof(void*) * nm, st));
  INIT_CUDA(cudaStreamSynchronize(st));  // the host vectors above may now be reused

  // Require block: replicas and anchor from W[0]; zero states; clip coefficients 1; P_0
  launch_init_weights(c->d_mats, c->d_wblk_start, nm, c->total_wblks, c->K, c->cfg.w_dtype, st);
  launch_fill_float(c->d_coef, (long long)nm * c->K, 1.f, st);
  c->launches += 2;
  for (int i = 0; i < nm; ++i) {
    const MatDev& md = c->h_mats[i];
    const size_t wn = (size_t)md.m * md.n, sn = (size_t)c->K * md.r * md.ln;
    if (md.E) INIT_CUDA(cudaMemsetAsync(md.E, 0, (size_t)c->K * wn * (c->cfg.e_dtype == LORDO_F32 ? 4 : 2), st));
    INIT_CUDA(cudaMemsetAsync(md.u, 0, sn * 4, st));
    INIT_CUDA(cudaMemsetAsync(md.v, 0, sn * 4, st));
    if (md.T) INIT_CUDA(cudaMemsetAsync(md.T, 0, sn * 4, st));
    if (md.B) INIT_CUDA(cudaMemsetAsync(md.B, 0, wn * 4, st));
    INIT_CUDA(cudaMemsetAsync(md.Delta, 0, wn * 4, st));
    if (c->cfg.variant == LORDO_LOCAL) {
      launch_identity_projection(md.P, md.pm, md.r, c->K, st);
      c->launches += 1;
    }
  }
  GemmScalars sc = base_scalars(c);
  for (const PlanStep& s : c->init_steps) {
    rc = run_plan_step(c, s, sc, st);
    if (rc != LORDO_OK) return bail(rc);
  }
  if (c->tc) {
    launch_prep_projection(c->d_tc_prep, c->d_prep_start, (int)c->h_prep.size(), c->prep_blocks, st);
    c->launches += 1;
  }
  INIT_CUDA(cudaStreamSynchronize(st));
  if (cudaGetLastError() != cudaSuccess) return bail(LORDO_ERR_CUDA);
#undef INIT_CUDA
  *out = c;
  return LORDO_OK;
}

int lordo_inner_step(lordo_ctx* c, const void* const* G, float lr, float beta1, float omega, int form, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  if (!G) return fail(c, LORDO_ERR_INVALID_ARG, "G is null");
  if (form != LORDO_QHM_NONE && form != LORDO_QHM_LOW && form != LORDO_QHM_FULL) return fail(c, LORDO_ERR_INVALID_ARG, "unknown QHM form");
  if (c->cfg.time_buffer && form == LORDO_QHM_FULL)
    return fail(c, LORDO_ERR_UNSUPPORTED, "time_buffer: the full-rank QHM update has no low-rank factorisation");
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(omega >= 0.f && omega <= 1.f)) return fail(c, LORDO_ERR_INVALID_ARG, "beta1 or omega out of range");
  if (c->steps_in_round >= c->cfg.H) return fail(c, LORDO_ERR_STATE, "H inner steps done: lordo_outer_step is due");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int rc = set_gradients(c, G, st);
  if (rc != LORDO_OK) return rc;
  {
    ProfScope ps(c, st, PC_CLIP);
    rc = run_clip(c, st);
  }
  if (rc != LORDO_OK) return rc;

  const int64_t s = c->steps + 1;
  const double bc1 = 1.0 - std::pow((double)beta1, (double)s), bc2 = 1.0 - std::pow((double)c->cfg.beta2, (double)s);
  GemmScalars gs = base_scalars(c);
  gs.lr = lr; gs.omega = omega; gs.form = form;
  gs.inv_bc1 = (float)(1.0 / bc1); gs.inv_bc2 = (float)(1.0 / bc2); gs.bc1 = (float)bc1; gs.bc2 = (float)bc2;
  StepScalars ss;
  ss.lr = lr; ss.beta1 = beta1; ss.beta2 = c->cfg.beta2; ss.omega = omega; ss.eps = c->cfg.eps;
  ss.inv_bc1 = gs.inv_bc1; ss.inv_bc2 = gs.inv_bc2; ss.form = form; ss.ef = c->cfg.error_feedback; ss.K = c->K;

  if (c->tc) {
    ss.lr = lr;
    if (c->p_copies_stale) {
      launch_prep_projection(c->d_tc_prep, c->d_prep_start, (int)c->h_prep.size(), c->prep_blocks, st);
      c->launches += 1;
      c->p_copies_stale = false;
    }
    if (c->tma) {
      const int big = c->tc_rn_max > 256;
      {
        ProfScope ps(c, st, PC_PROJECT);  // includes the moment update (fused epilogue)
        launch_project_tma(c->d_tc_probs, (int)c->h_tc.size(), c->tc_strips_p, c->d_maps, c->d_gmaps, ss, c->sm_count, c->d_status, st);
      }
      {
        ProfScope ps(c, st, PC_APPLY);
        const int n_all = (int)c->h_tc_apply.size();
        for (int side = 0; side < 2; ++side) {  // problems stored as projected, then the ones stored transposed
          const TcProblem* pb = c->d_tc_apply + (side ? c->tc_n_left : 0);
          const int np = side ? n_all - c->tc_n_left : c->tc_n_left;
          const long long s0 = side ? c->tc_strips_left : 0, s1 = side ? c->tc_strips : c->tc_strips_left;
          if (np == 0) continue;
          if (!big) {
            launch_apply_tma(pb, np, s0, s1, c->d_maps, c->d_gmaps, ss, c->sm_count, 0, side, c->d_status, st);
            c->launches += 1;
          } else {  // 256 < r <= 512: the error-feedback sweep, then the model-update sweep
            if (c->cfg.error_feedback) {
              launch_apply_tma(pb, np, s0, s1, c->d_maps, c->d_gmaps, ss, c->sm_count, 1, side, c->d_status, st);
              c->launches += 1;
            }
            launch_apply_tma(pb, np, s0, s1, c->d_maps, c->d_gmaps, ss, c->sm_count, 2, side, c->d_status, st);
            c->launches += 1;
          }
        }
      }
      c->launches -= 1;  // the common tail below counts one update launch
    } else {
    {
      ProfScope ps(c, st, PC_PROJECT);  // includes the moment update (fused epilogue)
      launch_project_tc(c->d_tc_probs, (int)c->h_tc.size(), c->tc_strips, c->tc_rn_max, ss, c->cfg.w_dtype == LORDO_BF16,
                        c->d_status, st);
    }
    {
      ProfScope ps(c, st, PC_APPLY);
      launch_apply_tc(c->d_tc_probs, (int)c->h_tc.size(), c->tc_strips, c->tc_rk_max, ss, c->cfg.w_dtype == LORDO_BF16,
                      c->d_status, st);
    }
    }
    c->launches += 2;
    rc = check_launch(c, "tensor-core inner step");
    if (rc != LORDO_OK) return rc;
    c->steps = s;
    c->steps_in_round += 1;
    c->after_outer = false;
    return LORDO_OK;
  }
  {
    ProfScope ps(c, st, PC_PROJECT);
    for (const PlanStep& s : c->inner_proj) {
      rc = run_plan_step(c, s, gs, st);
      if (rc != LORDO_OK) break;
    }
  }
  if (rc != LORDO_OK) return rc;
  {
    ProfScope ps(c, st, PC_MOMENTS);
    launch_moments(c->d_mats, c->d_mom_start, c->n_mats, c->total_mom_tiles, ss, st);
  }
  c->launches += 1;
  rc = check_launch(c, "moments");
  if (rc != LORDO_OK) return rc;
  {
    ProfScope ps(c, st, PC_APPLY);
    for (const PlanStep& s : c->inner_apply) {
      rc = run_plan_step(c, s, gs, st);
      if (rc != LORDO_OK) break;
    }
  }
  if (rc != LORDO_OK) return rc;
  c->steps = s;
  c->steps_in_round += 1;
  c->after_outer = false;
  return LORDO_OK;
}

int lordo_inner_step_host(lordo_ctx* c, const void* const* G_host, void* const* G_stage, float lr, float beta1, float omega,
                          int form, float* clip_out_host, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  if (!G_host || !G_stage) return fail(c, LORDO_ERR_INVALID_ARG, "null gradient table");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t esz = c->cfg.g_dtype == LORDO_F32 ? 4 : 2;
  for (int i = 0; i < c->n_mats; ++i) {
    if (!G_host[i] || !G_stage[i]) return fail(c, LORDO_ERR_INVALID_ARG, "null gradient pointer");
    const size_t bytes = (size_t)c->K * c->mats[i].m * c->mats[i].n * esz;
    CUDA_OK(c, cudaMemcpyAsync(G_stage[i], G_host[i], bytes, cudaMemcpyHostToDevice, st));
  }
  int rc = lordo_inner_step(c, (const void* const*)G_stage, lr, beta1, omega, form, stream);
  if (rc != LORDO_OK) return rc;
  if (clip_out_host) CUDA_OK(c, cudaMemcpyAsync(clip_out_host, c->d_coef, sizeof(float) * c->K, cudaMemcpyDeviceToHost, st));
  CUDA_OK(c, cudaStreamSynchronize(st));
  return LORDO_OK;
}

int lordo_outer_step(lordo_ctx* c, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  if (c->steps_in_round != c->cfg.H) return fail(c, LORDO_ERR_STATE, "lordo_outer_step needs exactly H inner steps since the last one");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const bool tb = c->cfg.time_buffer != 0, local = c->cfg.variant == LORDO_LOCAL;
  const int which = (c->cfg.sync_u ? 1 : 0) | (c->cfg.sync_v ? 2 : 0) | ((tb && !local) ? 4 : 0);
  if (which) {
    ProfScope ps(c, st, PC_OUTER_STATES);
    launch_outer_states(c->d_mats, c->d_sblk_start, c->n_mats, c->total_sblks, c->K, which, st);
    c->launches += 1;
  }
  int rc;
  {
    ProfScope ps(c, st, PC_OUTER_WEIGHTS);
    if (tb) {  // Delta from the low-rank accumulators instead of the weight replicas
      const GemmScalars gs = base_scalars(c);
      for (const PlanStep& s : c->tb_steps) {
        rc = run_plan_step(c, s, gs, st);
        if (rc != LORDO_OK) return rc;
      }
    }
    launch_outer_weights(c->d_mats, c->d_wblk_start, c->n_mats, c->total_wblks, c->K, c->cfg.w_dtype, c->cfg.outer, c->cfg.outer_lr,
                         c->cfg.outer_momentum, tb ? (local ? 1.f / (float)c->K : 1.f) : 0.f, st);
  }
  c->launches += 1;
  rc = check_launch(c, "outer");
  if (rc != LORDO_OK) return rc;
  if (tb)
    for (int i = 0; i < c->n_mats; ++i)
      CUDA_OK(c, cudaMemsetAsync(c->h_mats[i].T, 0, sizeof(float) * (size_t)c->K * c->h_mats[i].r * c->h_mats[i].ln, st));
  c->steps_in_round = 0;
  c->outers += 1;
  c->after_outer = true;
  return LORDO_OK;
}

int lordo_sync_states(lordo_ctx* c, int sync_u, int sync_v, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  const int which = (sync_u ? 1 : 0) | (sync_v ? 2 : 0);
  if (!which) return LORDO_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  {
    ProfScope ps(c, st, PC_OUTER_STATES);
    launch_outer_states(c->d_mats, c->d_sblk_start, c->n_mats, c->total_sblks, c->K, which, st);
  }
  c->launches += 1;
  return check_launch(c, "sync_states");
}

int lordo_refresh_subspace(lordo_ctx* c, const void* const* G, float beta1, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  const bool local = c->cfg.variant == LORDO_LOCAL;
  if (!(beta1 >= 0.f && beta1 < 1.f)) return fail(c, LORDO_ERR_INVALID_ARG, "beta1 out of range");
  if (local && !G) return fail(c, LORDO_ERR_INVALID_ARG, "Local refresh needs the gradients of the coming step");
  if (!local && G) return fail(c, LORDO_ERR_INVALID_ARG, "Global refresh takes its signal from Delta: G must be NULL");
  if (local && c->steps_in_round != 0) return fail(c, LORDO_ERR_STATE, "Local refresh only before the first inner step of a round");
  if (!local && !c->after_outer) return fail(c, LORDO_ERR_STATE, "Global refresh only directly after lordo_outer_step");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int rc;
  if (local) {
    rc = set_gradients(c, G, st);
    if (rc != LORDO_OK) return rc;
    rc = run_clip(c, st);
    if (rc != LORDO_OK) return rc;
  }
  GemmScalars gs = base_scalars(c);
  const bool rotate = c->steps > 0;
  if (rotate) {
    const double bc1 = 1.0 - std::pow((double)beta1, (double)c->steps), bc2 = 1.0 - std::pow((double)c->cfg.beta2, (double)c->steps);
    gs.inv_bc1 = (float)(1.0 / bc1); gs.inv_bc2 = (float)(1.0 / bc2); gs.bc1 = (float)bc1; gs.bc2 = (float)bc2;
  }
  {
    ProfScope ps(c, st, PC_REFRESH);
    for (const PlanStep& s : c->refresh_steps) {
      if (s.phase == PH_ROTATE && !rotate) continue;
      rc = run_plan_step(c, s, gs, st);
      if (rc != LORDO_OK) return rc;
    }
    if (c->tc) {  // bf16 operand copies of the new P
      launch_prep_projection(c->d_tc_prep, c->d_prep_start, (int)c->h_prep.size(), c->prep_blocks, st);
      c->launches += 1;
      rc = check_launch(c, "prep_projection");
      if (rc != LORDO_OK) return rc;
    }
  }
  c->refreshes += 1;
  c->after_outer = false;
  c->rot_valid = true;
  return LORDO_OK;
}

int lordo_poll_status(lordo_ctx* c, void* stream, uint32_t* flags) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  CUDA_OK(c, cudaMemcpyAsync(c->h_status, c->d_status, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
  CUDA_OK(c, cudaStreamSynchronize(st));
  CUDA_OK(c, cudaGetLastError());
  if (flags) *flags = *c->h_status;
  if (*c->h_status) return fail(c, LORDO_ERR_NUMERIC, "device flag word is non-zero");
  return LORDO_OK;
}

int lordo_diagnostics(lordo_ctx* c, float* mssv_dev, float* e_norm_dev, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  if (!mssv_dev && !e_norm_dev) return fail(c, LORDO_ERR_INVALID_ARG, "nothing requested");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (mssv_dev) {
    if (!c->rot_valid) return fail(c, LORDO_ERR_STATE, "no refresh has run on this context yet: there is no rotation matrix");
    launch_mssv(c->d_diag, (int)c->h_diag.size(), mssv_dev, st);
    c->launches += 1;
  }
  if (e_norm_dev) {
    if (!c->cfg.error_feedback) return fail(c, LORDO_ERR_STATE, "error feedback is off: there is no error buffer");
    launch_error_norms(c->d_mats, c->n_mats, c->K, c->cfg.e_dtype, e_norm_dev, st);
    c->launches += 1;
  }
  return check_launch(c, "diagnostics");
}

int lordo_selftest_wait_timeout(lordo_ctx* c, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  launch_selftest_wait(c->d_status, reinterpret_cast<cudaStream_t>(stream));
  c->launches += 1;
  return check_launch(c, "selftest_wait");
}

int lordo_clear_status(lordo_ctx* c, void* stream) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  CUDA_OK(c, cudaMemsetAsync(c->d_status, 0, sizeof(unsigned), reinterpret_cast<cudaStream_t>(stream)));
  return LORDO_OK;
}

int lordo_get_counters(const lordo_ctx* c, int64_t out[4]) {
  if (!c || !out) return LORDO_ERR_INVALID_ARG;
  out[0] = c->steps; out[1] = c->refreshes; out[2] = c->outers; out[3] = c->steps_in_round;
  return LORDO_OK;
}

int lordo_set_counters(lordo_ctx* c, const int64_t in[4]) {
  if (!c || !in) return LORDO_ERR_INVALID_ARG;
  if (in[0] < 0 || in[1] < 0 || in[2] < 0 || in[3] < 0 || in[3] > c->cfg.H) return fail(c, LORDO_ERR_INVALID_ARG, "counter out of range");
  if (c->cfg.time_buffer && in[3] != 0)
    return fail(c, LORDO_ERR_UNSUPPORTED, "time_buffer: the accumulators live in the workspace, so a checkpoint can only be restored at a round boundary");
  c->steps = in[0]; c->refreshes = in[1]; c->outers = in[2]; c->steps_in_round = (int)in[3];
  // Global rule: a checkpoint taken between lordo_outer_step and lordo_refresh_subspace still owes its
  // refresh; the counters show it (a round boundary with one refresh fewer than synchronisations)
  c->after_outer = c->cfg.variant == LORDO_GLOBAL && in[3] == 0 && in[2] > 0 && in[1] < in[2];
  c->rot_valid = false;  // the rotation matrices are workspace state and were not restored
  c->p_copies_stale = true;  // a restored checkpoint brings its own P
  return LORDO_OK;
}

int lordo_clip_coefficients(const lordo_ctx* c, const float** device_ptr) {
  if (!c || !device_ptr) return LORDO_ERR_INVALID_ARG;
  *device_ptr = c->d_coef;
  return LORDO_OK;
}

int64_t lordo_launch_count(const lordo_ctx* c) { return c ? c->launches : -1; }

int lordo_profile_enable(lordo_ctx* c, int on) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  c->profiling = on != 0;
  return LORDO_OK;
}

int lordo_profile_read(lordo_ctx* c, void* stream, float ms_out[8]) {
  if (!c || !ms_out) return LORDO_ERR_INVALID_ARG;
  CUDA_OK(c, cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)));
  for (int i = 0; i < 8; ++i) ms_out[i] = 0.f;
  for (const lordo_ctx::Span& sp : c->spans) {
    float ms = 0.f;
    CUDA_OK(c, cudaEventElapsedTime(&ms, sp.a, sp.b));
    ms_out[sp.cls] += ms;
    c->ev_pool.push_back(sp.a);
    c->ev_pool.push_back(sp.b);
  }
  c->spans.clear();
  return LORDO_OK;
}

const char* lordo_last_error(const lordo_ctx* c) { return c ? c->err.c_str() : "null context"; }

int lordo_destroy(lordo_ctx* c) {
  if (!c) return LORDO_ERR_INVALID_ARG;
  if (c->h_Gtab) cudaFreeHost(c->h_Gtab);
  if (c->h_status) cudaFreeHost(c->h_status);
  if (c->h_gmaps) cudaFreeHost(c->h_gmaps);
  for (int sl = 0; sl < 2; ++sl)
    if (c->g_slot_ev[sl]) cudaEventDestroy(c->g_slot_ev[sl]);
  for (const lordo_ctx::Span& sp : c->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  delete c;
  return LORDO_OK;
}

int lordo_fill_random(uint64_t seed, int32_t purpose, int32_t mat, int64_t index, int32_t replica, int64_t rows, int64_t cols,
                      float* out_dev, void* stream) {
  if (!out_dev || rows < 1 || cols < 1) return LORDO_ERR_INVALID_ARG;
  RandomKeys keys;
  keys.key[0] = stream_key(seed, purpose, mat, index, replica);
  launch_fill_random(out_dev, rows * cols, rows * cols, keys, 1, reinterpret_cast<cudaStream_t>(stream));
  return cudaPeekAtLastError() == cudaSuccess ? LORDO_OK : LORDO_ERR_CUDA;
}

}  // extern "C"
