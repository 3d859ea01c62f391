// TMA-fed, persistent tensor-core kernels of the inner step for bf16 storage of G, E and W.
//
//   project_tma_kernel  The streamed operand never passes through registers as single elements:
//                       TMA brings 64-row tiles of G, E (and of P^T) into 128B-swizzled shared
//                       memory, four warps turn the G tile into c*G + E in place (16-byte vector
//                       operations, layout-agnostic), and the tile is consumed as an MN-major
//                       operand by tcgen05.mma. Two accumulator buffers in tensor memory let the
//                       moment-update epilogue of one strip run under the main loop of the next
//                       (ranks above 256 as two half-rank strips, see the kernel). Runs as CTA
//                       pairs (clusters of two, tcgen05 cta_group::2): one strip per CTA, each CTA
//                       holding half of the rows of the P^T tile.
//   apply_tma_kernel    The strip's two low-rank operands (g^T, U~^T) live in tensor memory as the
//                       A operands; rows of P and the tiles of G, E, W arrive by TMA; the epilogue
//                       works on the swizzled tiles in shared memory (four neighbouring columns per
//                       thread, 8-byte accesses) and the updated E and W tiles leave by TMA stores.
//
// One CTA per SM; a CTA (the update kernel) or a CTA pair (the projection) walks the list of 128-column
// strips, or of pairs of strips, with the stride of the grid. Every role walks the same list, so stage
// and phase counters stay in step without further communication.
#include "lordo_kernels.h"
#include "lordo_umma.cuh"

namespace lordo {

using namespace umma;

namespace {

constexpr int kStrip = 128;

__device__ __forceinline__ int find_problem(const TcProblem* __restrict__ probs, int nprobs, long long strip) {
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].strip_start <= strip) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// the projection numbers its strips on its own: a problem with 256 < r <= 512 has two per 128 columns
__device__ __forceinline__ int find_problem_p(const TcProblem* __restrict__ probs, int nprobs, long long strip) {
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].strip_start_p <= strip) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ float bf_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf_hi(uint32_t x) { return __uint_as_float(x & 0xFFFF0000u); }

// ---- projection ---------------------------------------------------------------------------------
constexpr int kPStages = 4;
constexpr uint32_t kPStageBytes = 49152;  // G 16 KB | E 16 KB | this CTA's rows of the P^T tile, up to 16 KB
constexpr int kPXformWarps = 4, kPEpiWarps = 8;
constexpr int kPThreads = (2 + kPXformWarps + kPEpiWarps) * 32;  // 448

// ---- update -------------------------------------------------------------------------------------
constexpr int kARows = 64;                // rows of W per step = MMA N
constexpr int kAInStages = 3;             // G | E | W tiles, 16 KB each
constexpr uint32_t kAInStageBytes = 49152;
constexpr int kAPStages = 2;              // rows of P, up to 32 KB
constexpr uint32_t kAPStageBytes = 32768;
constexpr int kAEpiWarps = 16;
constexpr int kAThreads = (3 + kAEpiWarps) * 32;  // 608: TMA inputs, MMA, 16 epilogue warps, TMA rows of P

}  // namespace

// =================================================================================================
// 256 < r <= 512: the accumulator of a whole strip would fill all 512 columns of tensor memory and leave
// no second buffer, so such a problem is dealt out as two strips per 128 columns, one per half of the
// rank (rows [0, 256) and [256, r) of P^T, of the moments and of the low-rank operands). The two halves
// are neighbours in the strip list, hence run on neighbouring CTAs at the same time, and the second
// read of the G and E tiles is served by L2. Each half is then the r <= 256 pipeline: four stages, two
// accumulator buffers, the moment epilogue of one strip under the main loop of the next.
//
// The kernel runs as CTA pairs (clusters of two, tcgen05 cta_group::2): a pair works on two neighbouring
// strips of a problem (and the same half of the rank), one per CTA, and every MMA spans both (M = 256),
// so each CTA fetches and keeps only half of the rows of the P^T tile. Each CTA's loads complete on
// its own barrier; its transform warps pass the stage on to the MMA thread of the pair's first CTA.
// strip_start_p and total_pairs count such pairs; a problem with an odd number of strips ends in a
// pair whose second CTA reads zeros and stores nothing.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPThreads, 1)
    project_tma_kernel(const TcProblem* __restrict__ probs, int nprobs, long long total_pairs, const TmaMatMaps* __restrict__ maps,
                       const TmaGradMaps* __restrict__ gmaps, StepScalars sc, unsigned* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int ST = kPStages;
  constexpr uint32_t SB = kPStageBytes;
  // xform_bar and acc_empty are waited on by the MMA thread of the pair's first CTA only and fed by the
  // warps of both CTAs; empty_bar and acc_full are signalled in both CTAs by that thread's commits
  __shared__ uint64_t full_bar[kPStages], xform_bar[kPStages], empty_bar[kPStages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ float dsum_s[kStrip];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool ef = sc.ef != 0;
  const uint32_t rank = cluster_rank();
  const long long pair_first = blockIdx.x >> 1, pair_step = gridDim.x >> 1;

  if (tid == 0) {
    for (int s = 0; s < ST; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&xform_bar[s], 2 * kPXformWarps); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * kPEpiWarps); }
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc_pair(&tmem_slot, 512);
  tc_fence_before_sync();
  cluster_sync();  // both CTAs' barriers exist before either reaches into the other
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  // pair lp of a problem -> this CTA's 128 columns and its half of the rank (split problems: the two
  // halves of a column pair are neighbouring pairs)
#define LORDO_PAIR_COORDS(pr, pp)                                                              \
  const int lp = (int)((pp) - (pr)->strip_start_p);                                            \
  const int cs = 2 * ((pr)->nsplit == 2 ? lp >> 1 : lp) + (int)rank;                          \
  const int r_lo = (pr)->nsplit == 2 ? (lp & 1) * 256 : 0;

  if (warp == 0) {
    // ---------------- TMA producer ------------------------------------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (long long strip = pair_first; strip < total_pairs && ok; strip += pair_step) {
        const TcProblem* __restrict__ pr = probs + find_problem_p(probs, nprobs, strip);
        LORDO_PAIR_COORDS(pr, strip)
        const int n0 = cs * kStrip;
        const TmaMatMaps* mm = maps + pr->mat;
        const TmaGradMaps* gm = gmaps + pr->mat;
        const int nkb = pr->m_k / 64, rep = pr->replica, pc = pr->pcopy;
        const int pt_rows = pr->r_n <= 256 ? pr->r_n / 2 : 128;  // rows of one P^T box: a CTA's half of an MMA's N
        const int n_h = pr->r_n - r_lo < 256 ? pr->r_n - r_lo : 256;
        const int pt_row0 = r_lo + (int)rank * (n_h / 2);
        const uint32_t tx = 16384u + (ef ? 16384u : 0u) + (uint32_t)pt_rows * 128u;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % ST;
          ok = mbar_wait(&empty_bar[s], ((it / ST) & 1u) ^ 1u, status);
          if (!ok) break;
          unsigned char* base = smem + s * SB;
          mbar_expect_tx(&full_bar[s], tx);
          if (pr->tr) {  // stored transposed: the strip's 128 elements are stored rows, the k-block 64 stored columns
            tma_load_3d(base, gm->g_kb, kb * 64, n0, rep, &full_bar[s]);
            if (ef) tma_load_3d(base + 16384, mm->e_kb, kb * 64, n0, rep, &full_bar[s]);
          } else {
            tma_load_3d(base, gm->g_sw, n0, kb * 64, rep, &full_bar[s]);
            tma_load_3d(base + 8192, gm->g_sw, n0 + 64, kb * 64, rep, &full_bar[s]);
            if (ef) {
              tma_load_3d(base + 16384, mm->e_sw, n0, kb * 64, rep, &full_bar[s]);
              tma_load_3d(base + 24576, mm->e_sw, n0 + 64, kb * 64, rep, &full_bar[s]);
            }
          }
          tma_load_3d(base + 32768, mm->pt, kb * 64, pt_row0, pc, &full_bar[s]);  // rows past r_n arrive as zeros
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue ---------------------------------------------------------------
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, si = 0;
      bool ok = true;
      // the barriers the commits arrive on, in this CTA and in the other (8 bytes apart within an array)
      const uint32_t eb0 = cluster_addr(&empty_bar[0], 0), eb1 = cluster_addr(&empty_bar[0], 1);
      const uint32_t af0 = cluster_addr(&acc_full[0], 0), af1 = cluster_addr(&acc_full[0], 1);
      for (long long strip = pair_first; strip < total_pairs && ok; strip += pair_step, ++si) {
        const TcProblem* __restrict__ pr = probs + find_problem_p(probs, nprobs, strip);
        const int r_lo = pr->nsplit == 2 ? ((int)(strip - pr->strip_start_p) & 1) * 256 : 0;
        const int nkb = pr->m_k / 64;
        const uint32_t n_h = (uint32_t)(pr->r_n - r_lo < 256 ? pr->r_n - r_lo : 256);
        const bool tr = pr->tr != 0;  // the tile then lies as [128 strip elements][64 k]: a K-major operand
        const uint32_t idesc = idesc_bf16_f32(256, n_h) | (tr ? 0u : kIdescAMajorMN);
        const uint32_t buf = si & 1u;
        ok = mbar_wait(&acc_empty[buf], ((si >> 1) & 1u) ^ 1u, status);
        if (!ok) break;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % ST;
          ok = mbar_wait(&xform_bar[s], (it / ST) & 1u, status);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t sA = smem_u32(smem + s * SB), sB = sA + 32768;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16)
            mma_bf16_pair(tmem + buf * 256, tr ? smem_desc_k128(sA + k16 * 32) : smem_desc_mn128(sA + k16 * 2048), smem_desc_k128(sB + k16 * 32),
                          idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
          mma_commit_pair(eb0 + 8u * s); mma_commit_pair(eb1 + 8u * s);
        }
        if (ok) { mma_commit_pair(af0 + 8u * buf); mma_commit_pair(af1 + 8u * buf); }
      }
    }
  } else if (warp < 2 + kPXformWarps) {
    // ---------------- transform: G tile <- c*G + E, in place ------------------------------------
    const int xt = tid - 64;
    uint32_t it = 0;
    bool ok = true;
    const uint32_t xf = cluster_addr(&xform_bar[0], 0);
    for (long long strip = pair_first; strip < total_pairs && ok; strip += pair_step) {
      const TcProblem* __restrict__ pr = probs + find_problem_p(probs, nprobs, strip);
      const int nkb = pr->m_k / 64;
      const float c = *pr->cptr;
      for (int kb = 0; kb < nkb; ++kb, ++it) {
        const int s = it % ST;
        ok = mbar_wait(&full_bar[s], (it / ST) & 1u, status);
        if (!ok) break;
        uint4* G = reinterpret_cast<uint4*>(smem + s * SB);
        const uint4* E = G + 1024;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int idx = xt + i * 128;
          const uint4 g = G[idx];
          uint4 e = make_uint4(0u, 0u, 0u, 0u);
          if (ef) e = E[idx];
          uint4 a;
          a.x = pack2_bf16(fmaf(c, bf_lo(g.x), bf_lo(e.x)), fmaf(c, bf_hi(g.x), bf_hi(e.x)));
          a.y = pack2_bf16(fmaf(c, bf_lo(g.y), bf_lo(e.y)), fmaf(c, bf_hi(g.y), bf_hi(e.y)));
          a.z = pack2_bf16(fmaf(c, bf_lo(g.z), bf_lo(e.z)), fmaf(c, bf_hi(g.z), bf_hi(e.z)));
          a.w = pack2_bf16(fmaf(c, bf_lo(g.w), bf_lo(e.w)), fmaf(c, bf_hi(g.w), bf_hi(e.w)));
          G[idx] = a;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(xf + 8u * s);  // this CTA's half of the stage is ready for the pair's MMAs
      }
    }
  } else {
    // ---------------- epilogue: moments on this thread's column, out of tensor memory -----------
    const int q = warp & 3, half = (warp - (2 + kPXformWarps)) >> 2;
    const float b1 = sc.beta1, b2 = sc.beta2, w = sc.omega;
    const bool low = sc.form == LORDO_QHM_LOW;
    uint32_t si = 0;
    bool ok = true;
    const uint32_t ae = cluster_addr(&acc_empty[0], 0);
    for (long long strip = pair_first; strip < total_pairs && ok; strip += pair_step, ++si) {
      const TcProblem* __restrict__ pr = probs + find_problem_p(probs, nprobs, strip);
      LORDO_PAIR_COORDS(pr, strip)
      const int n = pr->n, r = pr->r, r_k = pr->r_k;
      const int rn_h = pr->r_n - r_lo < 256 ? pr->r_n - r_lo : 256;  // rank rows of this strip, padded to 16
      const long long n0 = (long long)cs * kStrip;
      const long long ecol = n0 + q * 32 + lane;
      const bool e_ok = ecol < n;
      const long long ecolc = e_ok ? ecol : (long long)n - 1;
      float* __restrict__ up_ = pr->u;
      float* __restrict__ vp_ = pr->v;
      float* __restrict__ tb_ = pr->tb;
      // this column's 16-byte pieces inside the strip's block [r_k/8][128][8], from k-chunk r_lo/8 on
      const size_t lr_off = (size_t)cs * (size_t)r_k * 128 + (size_t)r_lo * 128 + (size_t)(q * 32 + lane) * 8;
      __nv_bfloat16* __restrict__ gT = pr->gT16 + lr_off;
      __nv_bfloat16* __restrict__ uT = pr->uT16 + lr_off;
      const uint32_t buf = si & 1u;
      ok = mbar_wait<64>(&acc_full[buf], (si >> 1) & 1u, status);
      if (!ok) break;
      tc_fence_after_sync();
      float dsum = 0.f;
      for (int ch = half; ch < rn_h / 16; ch += 2) {
        float u[16], v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const size_t idx = (size_t)(unsigned)min(r_lo + ch * 16 + i, r - 1) * (size_t)n + (size_t)ecolc;
          u[i] = up_[idx];
          v[i] = vp_[idx];
        }
        float g[16];
        tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + buf * 256 + (uint32_t)(ch * 16), g);
        uint32_t gp[8], upk[8];
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          float o[2];
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const int row = r_lo + ch * 16 + i + t;
            const float gg = g[i + t];
            const float un = b1 * u[i + t] + (1.f - b1) * gg;
            const float vn = b2 * v[i + t] + (1.f - b2) * gg * gg;
            const float uh = un * sc.inv_bc1;
            const float D = sqrtf(vn * sc.inv_bc2) + sc.eps;
            o[t] = low ? (w * uh + (1.f - w) * gg) / D : uh / D;
            if (e_ok && row < r) {
              const size_t idx = (size_t)(unsigned)row * (size_t)n + (size_t)ecol;
              up_[idx] = un;
              vp_[idx] = vn;
              if (tb_) tb_[idx] += sc.lr * o[t];
              dsum += D;
            } else {
              o[t] = 0.f;
            }
          }
          gp[i >> 1] = pack2_bf16(g[i], g[i + 1]);
          upk[i >> 1] = pack2_bf16(o[0], o[1]);
        }
        if (e_ok) {
          uint4* gd = reinterpret_cast<uint4*>(gT + (size_t)ch * 2048);  // k-chunks 2ch and 2ch+1, 128 pieces apart
          uint4* ud = reinterpret_cast<uint4*>(uT + (size_t)ch * 2048);
          gd[0] = make_uint4(gp[0], gp[1], gp[2], gp[3]); gd[128] = make_uint4(gp[4], gp[5], gp[6], gp[7]);
          ud[0] = make_uint4(upk[0], upk[1], upk[2], upk[3]); ud[128] = make_uint4(upk[4], upk[5], upk[6], upk[7]);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(ae + 8u * buf);
      if (sc.form == LORDO_QHM_FULL) {  // mu(D): mean over the rank axis, one value per column (a split problem: this half's share)
        if (half == 1) dsum_s[q * 32 + lane] = dsum;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (half == 0 && e_ok) (r_lo ? pr->dcol2 : pr->dcol)[ecol] = (dsum + dsum_s[q * 32 + lane]) / (float)r;
        asm volatile("bar.sync 1, 256;" ::: "memory");
      }
    }
  }
#undef LORDO_PAIR_COORDS
  tc_fence_before_sync();
  __syncwarp();
  cluster_sync();  // neither CTA leaves while the other may still signal one of its barriers
  if (warp == 1) tmem_free_pair(tmem, 512);
}

// =================================================================================================
// MODE 0: r <= 256, both products in one sweep. For 256 < r <= 512 one low-rank operand alone fills
// 256 columns of tensor memory, so the update is two sweeps of the same kernel: MODE 1 does the
// error-feedback line (operand g^T, tiles G and E), MODE 2 the model update (operand U~^T, tiles G, W).
// TR: the problems of this launch are matrices projected from the right, whose W, G, E are stored
// transposed with respect to the problem: a strip is 128 stored rows, a step 64 stored columns, and the
// accumulator tile (lane = strip element, column = step element) already lies the way the tiles are
// stored, so a thread works on 16 neighbouring stored columns of its own row.
template <int MODE, bool TR>
__global__ void __launch_bounds__(kAThreads, 1) apply_tma_kernel(const TcProblem* __restrict__ probs, int nprobs, long long strip_begin,
                                                                 long long strip_end, const TmaMatMaps* __restrict__ maps,
                                                                 const TmaGradMaps* __restrict__ gmaps, StepScalars sc,
                                                                 unsigned* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr uint32_t PSB = MODE ? 65536u : kAPStageBytes;  // one stage of rows of P
  constexpr int INST = kAInStages;
  constexpr bool DO_E = MODE != 2, DO_W = MODE != 1;
  constexpr uint32_t A2COL = MODE ? 0u : 128u;             // first column of the U~^T operand
  // a stage holds the tiles the mode works on: G | E | W (MODE 0), G | E (MODE 1), G | W (MODE 2)
  constexpr uint32_t ISB = MODE ? 32768u : kAInStageBytes;
  constexpr uint32_t EOFF = 16384u, WOFF = MODE == 2 ? 16384u : 32768u;
  unsigned char* sP = smem;                      // kAPStages stages of rows of P
  unsigned char* sIn = smem + kAPStages * PSB;   // INST stages of tiles
  __shared__ uint64_t p_full[kAPStages], p_empty[kAPStages], in_full[kAInStages], in_free[kAInStages], acc_full[2], acc_empty[2], x_ready;
  __shared__ uint32_t tmem_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool ef = sc.ef != 0;

  if (tid == 0) {
    for (int s = 0; s < kAPStages; ++s) { mbar_init(&p_full[s], 1); mbar_init(&p_empty[s], 1); }
    for (int s = 0; s < INST; ++s) { mbar_init(&in_full[s], 1); mbar_init(&in_free[s], 4); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], kAEpiWarps * 32); }
    mbar_init(&x_ready, kAEpiWarps * 32);
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(&tmem_slot, 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  // tensor memory: columns [0,256) the low-rank operands, two bf16 per column (MODE 0: g^T then U~^T,
  // 128 columns each); [256,512) two buffers of two accumulators

  if (warp == 0) {
    // ---------------- TMA producer: tiles of G, E, W ---------------------------------------------
    if (lane == 0) {
      uint32_t jt = 0;
      bool ok = true;
      for (long long strip = strip_begin + blockIdx.x; strip < strip_end && ok; strip += gridDim.x) {
        const TcProblem* __restrict__ pr = probs + find_problem(probs, nprobs, strip);
        const int n0 = (int)(strip - pr->strip_start) * kStrip;
        const TmaMatMaps* mm = maps + pr->mat;
        const TmaGradMaps* gm = gmaps + pr->mat;
        const int rep = pr->replica;
        const int nsteps = (pr->m + kARows - 1) / kARows;
        for (int t = 0; t < nsteps; ++t, ++jt) {
          const int is = jt % INST;
          ok = mbar_wait(&in_free[is], ((jt / INST) & 1u) ^ 1u, status);
          if (!ok) break;
          unsigned char* base = sIn + is * ISB;
          const bool ld_e = DO_E && ef;
          mbar_expect_tx(&in_full[is], 16384u + (ld_e ? 16384u : 0u) + (DO_W ? 16384u : 0u));
          if (TR) {  // one box of 128 stored rows x 64 stored columns per tile
            tma_load_3d(base, gm->g_kb, t * kARows, n0, rep, &in_full[is]);
            if (ld_e) tma_load_3d(base + EOFF, mm->e_kb, t * kARows, n0, rep, &in_full[is]);
            if (DO_W) tma_load_3d(base + WOFF, mm->w_kb, t * kARows, n0, rep, &in_full[is]);
          } else {
            for (int hh = 0; hh < 2; ++hh) {  // two 64-column halves per tile, 8 KB each
              tma_load_3d(base + hh * 8192, gm->g_sw, n0 + hh * 64, t * kARows, rep, &in_full[is]);
              if (ld_e) tma_load_3d(base + EOFF + hh * 8192, mm->e_sw, n0 + hh * 64, t * kARows, rep, &in_full[is]);
              if (DO_W) tma_load_3d(base + WOFF + hh * 8192, mm->w_sw, n0 + hh * 64, t * kARows, rep, &in_full[is]);
            }
          }
        }
      }
    }
  } else if (warp == 2 + kAEpiWarps) {
    // ---------------- TMA producer: rows of P ---------------------------------------------------
    if (lane == 0) {
      uint32_t jt = 0;
      bool ok = true;
      for (long long strip = strip_begin + blockIdx.x; strip < strip_end && ok; strip += gridDim.x) {
        const TcProblem* __restrict__ pr = probs + find_problem(probs, nprobs, strip);
        const TmaMatMaps* mm = maps + pr->mat;
        const int nkb = pr->r_k / 64, pc = pr->pcopy;
        const int nsteps = (pr->m + kARows - 1) / kARows;
        for (int t = 0; t < nsteps; ++t, ++jt) {
          const int ps = jt % kAPStages;
          ok = mbar_wait(&p_empty[ps], ((jt / kAPStages) & 1u) ^ 1u, status);
          if (!ok) break;
          mbar_expect_tx(&p_full[ps], (uint32_t)nkb * 8192u);
          for (int kb = 0; kb < nkb; ++kb) tma_load_3d(sP + ps * PSB + kb * 8192, mm->p16, kb * 64, t * kARows, pc, &p_full[ps]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue: A operands from tensor memory ----------------------------------
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, kARows);
      uint32_t jt = 0, si = 0;
      bool ok = true;
      for (long long strip = strip_begin + blockIdx.x; strip < strip_end && ok; strip += gridDim.x, ++si) {
        const TcProblem* __restrict__ pr = probs + find_problem(probs, nprobs, strip);
        const int nkb = pr->r_k / 64;
        const int nsteps = (pr->m + kARows - 1) / kARows;
        ok = mbar_wait(&x_ready, si & 1u, status);
        if (!ok) break;
        for (int t = 0; t < nsteps; ++t, ++jt) {
          const int ps = jt % kAPStages;
          const uint32_t b = jt & 1u;
          ok = mbar_wait(&p_full[ps], (jt / kAPStages) & 1u, status);
          if (ok) ok = mbar_wait(&acc_empty[b], ((jt >> 1) & 1u) ^ 1u, status);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t pbase = smem_u32(sP + ps * PSB);
          const uint32_t d1 = tmem + 256 + b * 128, d2 = d1 + 64;
          for (int kb = 0; kb < nkb; ++kb) {
#pragma unroll
            for (int k16 = 0; k16 < 4; ++k16) {
              const uint32_t acc = (kb > 0 || k16 > 0) ? 1u : 0u;
              const uint64_t bd = smem_desc_k128(pbase + kb * 8192 + k16 * 32);
              const uint32_t acol = (uint32_t)(kb * 4 + k16) * 8;
              if (DO_E) mma_bf16_ts(d1, tmem + acol, bd, idesc, acc);
              if (DO_W) mma_bf16_ts(d2, tmem + A2COL + acol, bd, idesc, acc);
            }
          }
          mma_commit(&p_empty[ps]);
          mma_commit(&acc_full[b]);
        }
      }
    }
  } else {
    // ---------------- epilogue: 4 columns x 4 rows per thread and step ---------------------------
    // Lane l = 8a + b of a warp's lane quarter holds strip column 32q + 4b + a, so that the two
    // 16-lane accumulator loads hand thread t the four neighbouring columns 4(t/4)..+3 of rows
    // 2(t%4), +1, +8, +9 of its row group: 8-byte accesses to the swizzled tiles, free of conflicts.
    const int ew = warp - 2;
    const int q = warp & 3, grp = ew >> 2;  // lane quarter (fixed by the hardware), row group 0..3
    const int colq = TR ? q * 32 + lane : q * 32 + 4 * (lane & 7) + (lane >> 3);  // strip element this lane's operands belong to
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const int tb = lane >> 2, tr = lane & 3;
    const int ecol0 = q * 32 + 4 * tb;  // first of this thread's four epilogue columns
    // byte offsets inside a 16 KB tile (two halves of 64 rows x 128 bytes, 128-byte swizzle)
    uint32_t toff[4];
#pragma unroll
    for (int ri = 0; ri < 4; ++ri) {
      const int rho = grp * 16 + (ri >> 1) * 8 + 2 * tr + (ri & 1);
      const int chunk = 4 * (q & 1) + (tb >> 1);
      toff[ri] = (uint32_t)((q >> 1) * 8192 + rho * 128 + ((chunk ^ (rho & 7)) << 4) + 8 * (tb & 1));
    }
    const float lr = sc.lr, om = sc.omega;
    const bool full = sc.form == LORDO_QHM_FULL;
    const float a2w = full ? om : 1.f;
    uint32_t jt = 0, si = 0;
    bool ok = true;
    for (long long strip = strip_begin + blockIdx.x; strip < strip_end && ok; strip += gridDim.x, ++si) {
      const TcProblem* __restrict__ pr = probs + find_problem(probs, nprobs, strip);
      const int n = pr->n, r_k = pr->r_k;
      const int n0 = (int)(strip - pr->strip_start) * kStrip;
      const TmaMatMaps* mm = maps + pr->mat;
      const int rep = pr->replica;
      const int nsteps = (pr->m + kARows - 1) / kARows;
      const long long col = (long long)n0 + colq;
      const float c = *pr->cptr;
      float cd[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        // TR: one strip element per thread (its own row); else the four columns of the thread's epilogue block
        const long long ec = TR ? col : (long long)n0 + ecol0 + j;
        const long long ecc = ec < n ? ec : (long long)n - 1;
        cd[j] = full ? (1.f - om) * c / (pr->dcol[ecc] + (pr->dcol2 ? pr->dcol2[ecc] : 0.f)) : 0.f;
      }
      // this thread's quarter of its column's low-rank operands -> tensor memory (r_k/8 columns each)
      {
        const int per = r_k / 8;  // 32-bit columns of one operand handled by this row group
        // strip block [r_k/8][128][8]: this row group's k-chunks, this lane's column; a warp reads 512
        // contiguous bytes per instruction
        const size_t lr_off = (size_t)(strip - pr->strip_start) * (size_t)r_k * 128 + (size_t)grp * (r_k / 32) * 1024 + (size_t)colq * 8;
        const uint4* __restrict__ g16 = reinterpret_cast<const uint4*>(pr->gT16 + lr_off);
        const uint4* __restrict__ u16 = reinterpret_cast<const uint4*>(pr->uT16 + lr_off);
        const bool live = col < n;
        for (int c0 = 0; c0 < per; c0 += 8) {
          if (DO_E) {
            uint4 glo = g16[(c0 >> 2) * 128], ghi = g16[(c0 >> 2) * 128 + 128];
            if (!live) glo = ghi = make_uint4(0u, 0u, 0u, 0u);
            tmem_st8(tmem + lane_base + (uint32_t)(grp * per + c0), glo, ghi);
          }
          if (DO_W) {
            uint4 ulo = u16[(c0 >> 2) * 128], uhi = u16[(c0 >> 2) * 128 + 128];
            if (!live) ulo = uhi = make_uint4(0u, 0u, 0u, 0u);
            tmem_st8(tmem + lane_base + A2COL + (uint32_t)(grp * per + c0), ulo, uhi);
          }
        }
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(&x_ready);
      }
      for (int t = 0; t < nsteps; ++t, ++jt) {
        const int is = jt % INST;
        const uint32_t b = jt & 1u;
        unsigned char* base = sIn + is * ISB;
        ok = mbar_wait<32>(&in_full[is], (jt / INST) & 1u, status);
        if (ok) ok = mbar_wait<32>(&acc_full[b], (jt >> 1) & 1u, status);
        if (!ok) break;
        tc_fence_after_sync();
        if constexpr (TR) {
          // this thread: stored row 32q + lane of the strip, stored columns 16 grp .. +15 of the step
          const int row = q * 32 + lane;
          const uint32_t o0 = swz_chunk(row, 2 * grp), o1 = swz_chunk(row, 2 * grp + 1);
          float a1[16], a2[16];
          const uint32_t taddr = tmem + lane_base + 256 + b * 128 + (uint32_t)(grp * 16);
          if (DO_E && DO_W) tmem_ld16x2(taddr, taddr + 64, a1, a2);
          else if (DO_E) tmem_ld16(taddr, a1);
          else tmem_ld16(taddr + 64, a2);
          tc_fence_before_sync();
          mbar_arrive(&acc_empty[b]);
          const uint4 gq[2] = {*reinterpret_cast<const uint4*>(base + o0), *reinterpret_cast<const uint4*>(base + o1)};
          const float cdv = cd[0];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t off = h ? o1 : o0;
            const uint32_t gw[4] = {gq[h].x, gq[h].y, gq[h].z, gq[h].w};
            if (DO_E && ef) {
              const uint4 eq = *reinterpret_cast<const uint4*>(base + EOFF + off);
              const uint32_t ew4[4] = {eq.x, eq.y, eq.z, eq.w};
              uint32_t o[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                o[j] = pack2_bf16((c * bf_lo(gw[j]) + bf_lo(ew4[j])) - a1[8 * h + 2 * j], (c * bf_hi(gw[j]) + bf_hi(ew4[j])) - a1[8 * h + 2 * j + 1]);
              *reinterpret_cast<uint4*>(base + EOFF + off) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            if (DO_W) {
              const uint4 wq = *reinterpret_cast<const uint4*>(base + WOFF + off);
              const uint32_t ww[4] = {wq.x, wq.y, wq.z, wq.w};
              uint32_t o[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                o[j] = pack2_bf16(bf_lo(ww[j]) - lr * (cdv * bf_lo(gw[j]) + a2w * a2[8 * h + 2 * j]),
                                  bf_hi(ww[j]) - lr * (cdv * bf_hi(gw[j]) + a2w * a2[8 * h + 2 * j + 1]));
              *reinterpret_cast<uint4*>(base + WOFF + off) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
          // the four warps that share 32 stored rows hand them to the TMA engine on their own
          fence_async_smem();
          asm volatile("bar.sync %0, 128;" ::"r"(2 + q) : "memory");
          if (grp == 0 && lane == 0) {
            if (n0 + q * 32 < n) {
              if (DO_E && ef) tma_store_3d(mm->e_st32, t * kARows, n0 + q * 32, rep, base + EOFF + q * 4096);
              if (DO_W) tma_store_3d(mm->w_st32, t * kARows, n0 + q * 32, rep, base + WOFF + q * 4096);
            }
            tma_store_commit();
            tma_store_wait_read();
            mbar_arrive(&in_free[is]);
          }
        } else {
          const uint32_t taddr = tmem + lane_base + 256 + b * 128 + (uint32_t)(grp * 16);
          // both accumulators come out of tensor memory together and the buffer goes back to the MMA
          // warp before any arithmetic. a?[h][4k + 2jj + p]: column 2h + jj, row 8k + 2(t%4) + p.
          float a1[2][8], a2[2][8];
  #pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (DO_E) tmem_ld_16x256b_x2(taddr + ((uint32_t)(h * 16) << 16), a1[h]);       // (P g)^T
            if (DO_W) tmem_ld_16x256b_x2(taddr + 64 + ((uint32_t)(h * 16) << 16), a2[h]);  // (P U~)^T
          }
          tmem_ld_wait();
  #pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (DO_E) tmem_ld_pin8(a1[h]);
            if (DO_W) tmem_ld_pin8(a2[h]);
          }
          tc_fence_before_sync();
          mbar_arrive(&acc_empty[b]);
          uint2 gv[4], ev[4], wv[4];
  #pragma unroll
          for (int ri = 0; ri < 4; ++ri) {
            gv[ri] = *reinterpret_cast<const uint2*>(base + toff[ri]);
            if (DO_E && ef) ev[ri] = *reinterpret_cast<const uint2*>(base + EOFF + toff[ri]);
            if (DO_W) wv[ri] = *reinterpret_cast<const uint2*>(base + WOFF + toff[ri]);
          }
  #pragma unroll
          for (int ri = 0; ri < 4; ++ri) {
            const int k = ri >> 1, p = ri & 1;
            const float g0 = bf_lo(gv[ri].x), g1 = bf_hi(gv[ri].x), g2 = bf_lo(gv[ri].y), g3 = bf_hi(gv[ri].y);
            if (DO_E && ef) {
              const float e0 = (c * g0 + bf_lo(ev[ri].x)) - a1[0][4 * k + p];
              const float e1 = (c * g1 + bf_hi(ev[ri].x)) - a1[0][4 * k + 2 + p];
              const float e2 = (c * g2 + bf_lo(ev[ri].y)) - a1[1][4 * k + p];
              const float e3 = (c * g3 + bf_hi(ev[ri].y)) - a1[1][4 * k + 2 + p];
              *reinterpret_cast<uint2*>(base + EOFF + toff[ri]) = make_uint2(pack2_bf16(e0, e1), pack2_bf16(e2, e3));
            }
            if (DO_W) {
              const float w0 = bf_lo(wv[ri].x) - lr * (cd[0] * g0 + a2w * a2[0][4 * k + p]);
              const float w1 = bf_hi(wv[ri].x) - lr * (cd[1] * g1 + a2w * a2[0][4 * k + 2 + p]);
              const float w2 = bf_lo(wv[ri].y) - lr * (cd[2] * g2 + a2w * a2[1][4 * k + p]);
              const float w3 = bf_hi(wv[ri].y) - lr * (cd[3] * g3 + a2w * a2[1][4 * k + 2 + p]);
              *reinterpret_cast<uint2*>(base + WOFF + toff[ri]) = make_uint2(pack2_bf16(w0, w1), pack2_bf16(w2, w3));
            }
          }
          // the four warps of a row group hand their 16 rows to the TMA engine on their own
          fence_async_smem();
          asm volatile("bar.sync %0, 128;" ::"r"(2 + grp) : "memory");
          if ((ew & 3) == 0 && lane == 0) {
            unsigned char* sb = base + grp * 2048;
            const int row = t * kARows + grp * 16;
            for (int hh = 0; hh < 2; ++hh) {
              if (n0 + hh * 64 >= n) break;
              if (DO_E && ef) tma_store_3d(mm->e_st, n0 + hh * 64, row, rep, sb + EOFF + hh * 8192);
              if (DO_W) tma_store_3d(mm->w_st, n0 + hh * 64, row, rep, sb + WOFF + hh * 8192);
            }
            tma_store_commit();
            tma_store_wait_read();
            mbar_arrive(&in_free[is]);
          }
        }
      }
    }
    if ((TR ? grp == 0 : (ew & 3) == 0) && lane == 0) tma_store_wait_all();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_free(tmem, 512);
}

// =================================================================================================
cudaError_t sketch_configure();

// How many CTA pairs of `kernel` the device holds at once. A persistent kernel that launched more would
// still be correct (no pair waits for another pair), but the pairs that start late would double its time.
template <typename Kernel>
static cudaError_t max_resident_pairs(Kernel kernel, int threads, size_t smem, int* pairs) {
  cudaLaunchConfig_t lc = {};
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeClusterDimension;
  at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
  lc.gridDim = dim3(2048, 1, 1); lc.blockDim = dim3((unsigned)threads, 1, 1); lc.dynamicSmemBytes = smem;
  lc.attrs = &at; lc.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(pairs, kernel, &lc);
}
static int g_project_pairs = 0, g_sketch_pairs = 0;  // set by tma_configure, per process (one device model per process)

cudaError_t tma_configure() {
  cudaError_t e = sketch_configure();
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(project_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kPStages * kPStageBytes + 1024));
  if (e != cudaSuccess) return e;
  e = max_resident_pairs(project_tma_kernel, kPThreads, kPStages * kPStageBytes + 1024, &g_project_pairs);
  if (e != cudaSuccess) return e;
  const int smem = (int)(kAPStages * 65536 + kAInStages * 32768 + 1024);  // the largest of the three modes
  e = cudaFuncSetAttribute(apply_tma_kernel<0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(apply_tma_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(apply_tma_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(apply_tma_kernel<0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(apply_tma_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(apply_tma_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

void launch_project_tma(const TcProblem* probs, int nprobs, long long total_pairs, const TmaMatMaps* maps, const TmaGradMaps* gmaps,
                        const StepScalars& sc, int grid, unsigned* status, cudaStream_t st) {
  if (total_pairs <= 0 || grid < 2) return;
  long long pairs = grid / 2;
  if (g_project_pairs > 0 && pairs > g_project_pairs) pairs = g_project_pairs;
  const unsigned g = 2u * (unsigned)(total_pairs < pairs ? total_pairs : pairs);
  project_tma_kernel<<<g, kPThreads, kPStages * kPStageBytes + 1024, st>>>(probs, nprobs, total_pairs, maps, gmaps, sc, status);
}
void launch_apply_tma(const TcProblem* probs, int nprobs, long long strip_begin, long long strip_end, const TmaMatMaps* maps,
                      const TmaGradMaps* gmaps, const StepScalars& sc, int grid, int mode, int tr, unsigned* status, cudaStream_t st) {
  const long long total = strip_end - strip_begin;
  if (total <= 0) return;
  const unsigned g = (unsigned)(total < grid ? total : grid);
  const size_t small = kAPStages * kAPStageBytes + kAInStages * kAInStageBytes + 1024, large = kAPStages * 65536 + kAInStages * 32768 + 1024;
#define LORDO_APPLY(M, T, SM) apply_tma_kernel<M, T><<<g, kAThreads, SM, st>>>(probs, nprobs, strip_begin, strip_end, maps, gmaps, sc, status)
  if (!tr) {
    if (mode == 0) LORDO_APPLY(0, false, small);
    else if (mode == 1) LORDO_APPLY(1, false, large);
    else LORDO_APPLY(2, false, large);
  } else {
    if (mode == 0) LORDO_APPLY(0, true, small);
    else if (mode == 1) LORDO_APPLY(1, true, large);
    else LORDO_APPLY(2, true, large);
  }
#undef LORDO_APPLY
}

}  // namespace lordo

// =================================================================================================
// Sketch products of the refresh: C = S * B (fp32 out), S streamed by TMA. Same pipeline as the
// projection: TMA -> (optional c*G + E in place) -> tcgen05.mma -> epilogue out of tensor memory,
// two accumulator buffers.
//
// The kernel runs as CTA pairs (clusters of two, tcgen05 cta_group::2): a pair works on 256 rows of
// S, 128 per CTA, and every MMA spans both CTAs (M = 256), so each CTA fetches and keeps only half of
// the columns of B. With both operands in shared memory an MMA of one CTA reads 4 KB of A and 8 KB of B
// per 16-deep step at r = 256, more than the shared memory can feed at the tensor cores' rate; the
// pair halves B's share and its L2 traffic, and the freed shared memory holds one more stage. Each
// CTA's loads complete on its own barrier; its transform warps (which form c*G + E where asked) pass
// the stage on to the MMA thread of the pair's first CTA. The table counts tiles in pairs; a problem
// with an odd number of 128-row tiles ends in a pair whose second CTA reads zeros and stores nothing.
// =================================================================================================
namespace lordo {
using namespace umma;
namespace {
constexpr int kSMaxStages = 4;
constexpr uint32_t kSSmemBytes = 196608 + 1024;  // 4 stages of A 16 KB | E 16 KB | B 16 KB, or 3 with 32 KB of B
constexpr int kSThreads = (2 + 4 + 4) * 32;  // TMA, MMA, 4 transform warps, 4 epilogue warps
constexpr uint32_t kIdescBMajorMN = 1u << 16;
__device__ __forceinline__ int sk_passes(int split) { return split == 3 ? 6 : (split == 2 ? 3 : 1); }

__device__ __forceinline__ int find_sk(const SkProblem* __restrict__ probs, int nprobs, long long tile) {
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].tile_start <= tile) lo = mid; else hi = mid - 1;
  }
  return lo;
}
}  // namespace

template <bool BIG>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kSThreads, 1)
    sketch_tma_kernel(const SkProblem* __restrict__ probs, int nprobs, long long total_tiles, unsigned* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int ST = BIG ? 3 : 4;
  constexpr uint32_t SB = BIG ? 65536u : 49152u;  // A 16 KB | E 16 KB | this CTA's columns of B: up to 2 (+ 2) boxes of 8 KB
  static_assert(ST * SB + 1024 <= kSSmemBytes, "stages do not fit the shared memory asked for");
  // xform_bar and acc_empty are waited on by the MMA thread of the pair's first CTA only and fed by the
  // warps of both CTAs; empty_bar and acc_full are signalled in both CTAs by that thread's commits
  __shared__ uint64_t full_bar[kSMaxStages], xform_bar[kSMaxStages], empty_bar[kSMaxStages], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_slot;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();
  const long long tile_first = blockIdx.x >> 1, tile_step = gridDim.x >> 1;  // tiles of 256 rows, one per pair

  if (tid == 0) {
    for (int s = 0; s < ST; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&xform_bar[s], 8); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc_pair(&tmem_slot, 512);
  tc_fence_before_sync();
  cluster_sync();  // both CTAs' barriers exist before either reaches into the other
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (long long tile = tile_first; tile < total_tiles && ok; tile += tile_step) {
        const SkProblem* __restrict__ pr = probs + find_sk(probs, nprobs, tile);
        const int m0 = (2 * (int)(tile - pr->tile_start) + (int)rank) * 128;
        const int nkb1 = (pr->Kd + 63) / 64;
        // this CTA's columns of B: half of the first 256 (one MMA) and half of the rest (a second MMA)
        const int n_lo = pr->r_n < 256 ? pr->r_n : 256, n_hi = pr->r_n - n_lo;
        const int c_lo = (int)rank * (n_lo / 2), c_hi = 256 + (int)rank * (n_hi / 2);
        const int nbox_lo = (n_lo / 2 + 63) / 64, nbox_hi = (n_hi / 2 + 63) / 64;
        const int nkb = nkb1 * sk_passes(pr->split);
        const bool has_e = pr->map_e != nullptr;
        const uint32_t tx = 16384u + (has_e ? 16384u : 0u) + (uint32_t)(nbox_lo + nbox_hi) * 8192u;
        for (int j = 0; j < nkb; ++j, ++it) {
          const int seg = j / nkb1, kb = j - seg * nkb1;  // plane pairs (0,0) (0,1) (1,0) (1,1) (0,2) (2,0)
          const int a_c2 = pr->a_c2 + ((0x201100 >> (4 * seg)) & 3) * pr->a_pl, b_c2 = pr->b_c2 + ((0x021010 >> (4 * seg)) & 3) * pr->b_pl;
          const int s = it % ST;
          ok = mbar_wait(&empty_bar[s], ((it / ST) & 1u) ^ 1u, status);
          if (!ok) break;
          unsigned char* base = smem + s * SB;
          mbar_expect_tx(&full_bar[s], tx);
          if (pr->a_mn) {  // S stored [Kd][M]: two boxes of 64 k-rows x 64 columns
            tma_load_3d(base, pr->map_a, m0, kb * 64, a_c2, &full_bar[s]);
            tma_load_3d(base + 8192, pr->map_a, m0 + 64, kb * 64, a_c2, &full_bar[s]);
            if (has_e) {
              tma_load_3d(base + 16384, pr->map_e, m0, kb * 64, a_c2, &full_bar[s]);
              tma_load_3d(base + 24576, pr->map_e, m0 + 64, kb * 64, a_c2, &full_bar[s]);
            }
          } else {         // S stored [M][Kd]: one box of 128 rows x 64 k
            tma_load_3d(base, pr->map_a, kb * 64, m0, a_c2, &full_bar[s]);
            if (has_e) tma_load_3d(base + 16384, pr->map_e, kb * 64, m0, a_c2, &full_bar[s]);
          }
          for (int x = 0; x < nbox_lo; ++x) tma_load_3d(base + 32768 + x * 8192, pr->map_b, c_lo + x * 64, kb * 64, b_c2, &full_bar[s]);
          for (int x = 0; x < nbox_hi; ++x) tma_load_3d(base + 49152 + x * 8192, pr->map_b, c_hi + x * 64, kb * 64, b_c2, &full_bar[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, si = 0;
      bool ok = true;
      // the barriers the commits arrive on, in this CTA and in the other (8 bytes apart within an array)
      const uint32_t eb0 = cluster_addr(&empty_bar[0], 0), eb1 = cluster_addr(&empty_bar[0], 1);
      const uint32_t af0 = cluster_addr(&acc_full[0], 0), af1 = cluster_addr(&acc_full[0], 1);
      for (long long tile = tile_first; tile < total_tiles && ok; tile += tile_step, ++si) {
        const SkProblem* __restrict__ pr = probs + find_sk(probs, nprobs, tile);
        const int nkb = ((pr->Kd + 63) / 64) * sk_passes(pr->split);
        const bool a_mn = pr->a_mn != 0;
        const uint32_t n_lo = pr->r_n < 256 ? (uint32_t)pr->r_n : 256u, n_hi = (uint32_t)pr->r_n - n_lo;
        const uint32_t majors = kIdescBMajorMN | (a_mn ? kIdescAMajorMN : 0u);
        const uint32_t idesc = idesc_bf16_f32(256, n_lo) | majors, idesc_hi = idesc_bf16_f32(256, n_hi ? n_hi : 16u) | majors;
        const uint32_t buf = BIG ? 0u : (si & 1u);
        ok = mbar_wait(&acc_empty[buf], ((BIG ? si : (si >> 1)) & 1u) ^ 1u, status);
        if (!ok) break;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % ST;
          ok = mbar_wait(&xform_bar[s], (it / ST) & 1u, status);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t sA = smem_u32(smem + s * SB), sB = sA + 32768;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16) {
            const uint64_t ad = a_mn ? smem_desc_mn128(sA + k16 * 2048) : smem_desc_k128(sA + k16 * 32);
            mma_bf16_pair(tmem + buf * 256, ad, smem_desc_mn128(sB + k16 * 2048), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
            if (BIG && n_hi) mma_bf16_pair(tmem + 256, ad, smem_desc_mn128(sB + 2 * 8192 + k16 * 2048), idesc_hi, (kb > 0 || k16 > 0) ? 1u : 0u);
          }
          mma_commit_pair(eb0 + 8u * s); mma_commit_pair(eb1 + 8u * s);
        }
        if (ok) { mma_commit_pair(af0 + 8u * buf); mma_commit_pair(af1 + 8u * buf); }
      }
    }
  } else if (warp < 6) {
    const int xt = tid - 64;
    uint32_t it = 0;
    bool ok = true;
    const uint32_t xf = cluster_addr(&xform_bar[0], 0);
    for (long long tile = tile_first; tile < total_tiles && ok; tile += tile_step) {
      const SkProblem* __restrict__ pr = probs + find_sk(probs, nprobs, tile);
      const int nkb = ((pr->Kd + 63) / 64) * sk_passes(pr->split);
      const bool has_e = pr->map_e != nullptr;
      const float c = pr->cptr ? *pr->cptr : 1.f;
      for (int kb = 0; kb < nkb; ++kb, ++it) {
        const int s = it % ST;
        ok = mbar_wait(&full_bar[s], (it / ST) & 1u, status);
        if (!ok) break;
        if (has_e) {
          uint4* G = reinterpret_cast<uint4*>(smem + s * SB);
          const uint4* E = G + 1024;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int idx = xt + i * 128;
            const uint4 g = G[idx], e = E[idx];
            uint4 a;
            a.x = pack2_bf16(fmaf(c, bf_lo(g.x), bf_lo(e.x)), fmaf(c, bf_hi(g.x), bf_hi(e.x)));
            a.y = pack2_bf16(fmaf(c, bf_lo(g.y), bf_lo(e.y)), fmaf(c, bf_hi(g.y), bf_hi(e.y)));
            a.z = pack2_bf16(fmaf(c, bf_lo(g.z), bf_lo(e.z)), fmaf(c, bf_hi(g.z), bf_hi(e.z)));
            a.w = pack2_bf16(fmaf(c, bf_lo(g.w), bf_lo(e.w)), fmaf(c, bf_hi(g.w), bf_hi(e.w)));
            G[idx] = a;
          }
          fence_async_smem();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(xf + 8u * s);  // this CTA's half of the stage is ready for the pair's MMAs
      }
    }
  } else {
    // epilogue: lane = row of the tile, r_n fp32 columns out of tensor memory
    const int q = warp & 3;
    uint32_t si = 0;
    bool ok = true;
    const uint32_t ae = cluster_addr(&acc_empty[0], 0);
    for (long long tile = tile_first; tile < total_tiles && ok; tile += tile_step, ++si) {
      const SkProblem* __restrict__ pr = probs + find_sk(probs, nprobs, tile);
      const long long row = (2 * (tile - pr->tile_start) + rank) * 128 + q * 32 + lane;
      const bool row_ok = row < pr->M;
      float* __restrict__ crow = pr->C + (row_ok ? row : 0) * pr->ldc;
      const int r = pr->r, r_n = pr->r_n;
      const uint32_t buf = BIG ? 0u : (si & 1u);
      ok = mbar_wait<64>(&acc_full[buf], (BIG ? si : (si >> 1)) & 1u, status);
      if (!ok) break;
      tc_fence_after_sync();
      for (int ch = 0; ch < r_n / 16; ++ch) {
        float v[16];
        tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + buf * 256 + (uint32_t)(ch * 16), v);
        if (row_ok && !pr->c_trans) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            if (ch * 16 + j < r) *reinterpret_cast<float4*>(crow + ch * 16 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        } else if (row_ok) {  // transposed: the warp's lanes write 32 neighbouring floats of each output row
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (ch * 16 + j < r) pr->C[(long long)(ch * 16 + j) * pr->ldc + row] = v[j];
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(ae + 8u * buf);
    }
  }
  tc_fence_before_sync();
  __syncwarp();
  cluster_sync();  // neither CTA leaves while the other may still signal one of its barriers
  if (warp == 1) tmem_free_pair(tmem, 512);
}

cudaError_t sketch_configure() {
  cudaError_t e = cudaFuncSetAttribute(sketch_tma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(sketch_tma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSSmemBytes);
  if (e != cudaSuccess) return e;
  return max_resident_pairs(sketch_tma_kernel<true>, kSThreads, kSSmemBytes, &g_sketch_pairs);
}
// total_tiles counts tiles of 256 rows (tile_start in `probs` does too); a CTA pair per SM pair.
void launch_sketch_tma(const SkProblem* probs, int nprobs, long long total_tiles, int grid, int big, unsigned* status, cudaStream_t st) {
  if (total_tiles <= 0 || grid < 2) return;
  long long pairs = grid / 2;
  if (g_sketch_pairs > 0 && pairs > g_sketch_pairs) pairs = g_sketch_pairs;
  const unsigned g = 2u * (unsigned)(total_tiles < pairs ? total_tiles : pairs);
  if (big) sketch_tma_kernel<true><<<g, kSThreads, kSSmemBytes, st>>>(probs, nprobs, total_tiles, status);
  else sketch_tma_kernel<false><<<g, kSThreads, kSSmemBytes, st>>>(probs, nprobs, total_tiles, status);
}

}  // namespace lordo

// =================================================================================================
// Self-test of the bounded wait: one thread waits on an mbarrier phase that nothing completes. The
// wait must give up after its limit, set LORDO_FLAG_DEVICE_TIMEOUT in *status and let the kernel end.
// =================================================================================================
namespace lordo {
__global__ void selftest_wait_kernel(unsigned* __restrict__ status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    umma::mbar_init(&bar, 1);
    umma::mbar_init_fence();
    (void)umma::mbar_wait(&bar, 0u, status);
  }
}
void launch_selftest_wait(unsigned* status, cudaStream_t st) { selftest_wait_kernel<<<1, 32, 0, st>>>(status); }
}  // namespace lordo
