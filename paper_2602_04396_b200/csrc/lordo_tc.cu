// Tensor-core (tcgen05 + tensor memory) kernels of the inner step, "fast mode":
//
//   project_tc_kernel  g^T = (cG+E)^T P  for one 128-column strip of one (matrix, worker), swept
//                      down the m rows; the low-rank moment update (Algorithm 1: u, v lines and the
//                      bracket of the update cases) runs in its epilogue straight out of tensor
//                      memory, so the low-rank gradient never goes to global memory in fp32.
//   apply_tc_kernel    (P g)^T and (P U~)^T for the same strip with the two low-rank operands
//                      resident in shared memory, swept down the m rows in steps of 64; its
//                      epilogue is the error-feedback line and the model update of Algorithm 1.
//
// Orientation: the strip's columns (n) are the 128 lanes of tensor memory, so every epilogue
// thread owns one column and a warp touches 32 consecutive columns of a row of G, E, W, u or v.
// bf16 operands, fp32 accumulation. Operand tiles are written to shared memory by the kernels
// themselves (the streamed operand has to be formed as c*G + E and transposed anyway).
#include "lordo_kernels.h"
#include "lordo_umma.cuh"

namespace lordo {

using namespace umma;

namespace {

constexpr int kStrip = 128;        // columns per strip = MMA M
constexpr int kProjThreads = 288;  // 8 producer/epilogue warps + 1 MMA warp
constexpr int kApplyEpiWarps = 16, kApplyProdWarps = 4;
constexpr int kApplyThreads = (kApplyEpiWarps + kApplyProdWarps + 1) * 32;
constexpr int kApplyRows = 64;     // rows of W per sweep step = MMA N

__device__ __forceinline__ int find_problem(const TcProblem* __restrict__ probs, int nprobs, long long strip) {
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].strip_start <= strip) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// two adjacent elements (row, col), (row, col+1) as floats
__device__ __forceinline__ float2 load_pair(const void* base, int dt, long long idx) {
  if (dt == LORDO_F32) return *reinterpret_cast<const float2*>(reinterpret_cast<const float*>(base) + idx);
  const uint32_t raw = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const unsigned short*>(base) + idx);
  return make_float2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xFFFF0000u));
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// P (fp32 [m][r]) -> P16 [m_r][r_k] and PT16 [r_n][m_k] in bf16; the pads stay zero.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) prep_projection_kernel(const TcPrep* __restrict__ items, const long long* __restrict__ blk_start,
                                                              int nitems) {
  const long long blk = blockIdx.x;
  const int i = find_segment(blk_start, nitems, blk);
  const TcPrep it = items[i];
  const long long e = (blk - blk_start[i]) * 256 + threadIdx.x;
  if (e >= it.m * it.r) return;
  const long long row = e / it.r;
  const int col = (int)(e - row * it.r);
  const __nv_bfloat16 h = __float2bfloat16_rn(it.P[e]);
  it.P16[row * it.r_k + col] = h;
  it.PT16[(long long)col * it.m_k + row] = h;
}

// ---------------------------------------------------------------------------------------------
// project + moments
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kProjThreads, 2) project_tc_kernel(const TcProblem* __restrict__ probs, int nprobs, StepScalars sc,
                                                                  int g_dt, int e_dt, unsigned* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[2], empty_bar[2], done_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ float dsum_s[kStrip];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long strip = blockIdx.x;
  const TcProblem& pr = probs[find_problem(probs, nprobs, strip)];
  const int m = pr.m, n = pr.n, r = pr.r, r_n = pr.r_n;
  const long long n0 = (strip - pr.strip_start) * kStrip;
  const int nkb = pr.m_k / 64;
  const uint32_t a_bytes = kStrip * 128, b_bytes = (uint32_t)r_n * 128, stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023u);
  const uint32_t ncols = tmem_cols_pow2((uint32_t)r_n);

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(&full_bar[s], 256); mbar_init(&empty_bar[s], 1); }
    mbar_init(&done_bar, 1);
    mbar_init_fence();
  }
  if (warp == 8) tmem_alloc(&tmem_slot, ncols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  if (warp < 8) {
    // ---------------- producers: form (cG+E)^T tiles and copy P^T tiles -----------------------
    const int cp = tid & 63, kg = tid >> 6;  // column pair 0..63, k-group of 16 rows 0..3
    const long long col = n0 + 2 * cp;
    const bool col_ok = col < n;
    const void* G = *pr.G_ind;
    const float c = *pr.cptr;
    const bool have_e = sc.ef != 0;
    bool ok = true;
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb & 1, use = kb >> 1;
      float2 a[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const long long row = (long long)kb * 64 + kg * 16 + j;
        float2 x = make_float2(0.f, 0.f);
        if (col_ok && row < m) {
          const long long idx = row * n + col;
          const float2 g = load_pair(G, g_dt, pr.G_off + idx);
          x = make_float2(c * g.x, c * g.y);
          if (have_e) {
            const float2 e = load_pair(pr.E, e_dt, idx);
            x.x += e.x; x.y += e.y;
          }
        }
        a[j] = x;
      }
      uint4 pt[8];
      const int pt_chunks = r_n * 8;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int idx = tid + t * 256;
        if (idx < pt_chunks) pt[t] = *reinterpret_cast<const uint4*>(pr.PT16 + (long long)(idx >> 3) * pr.m_k + kb * 64 + (idx & 7) * 8);
      }
      ok = mbar_wait(&empty_bar[s], (uint32_t)((use & 1) ^ 1), status);
      if (!ok) break;
      unsigned char* sA = smem + s * stage_bytes;
      unsigned char* sB = sA + a_bytes;
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        uint4 lo, hi;
        lo.x = pack2_bf16(a[8 * q + 0].x, a[8 * q + 1].x); lo.y = pack2_bf16(a[8 * q + 2].x, a[8 * q + 3].x);
        lo.z = pack2_bf16(a[8 * q + 4].x, a[8 * q + 5].x); lo.w = pack2_bf16(a[8 * q + 6].x, a[8 * q + 7].x);
        hi.x = pack2_bf16(a[8 * q + 0].y, a[8 * q + 1].y); hi.y = pack2_bf16(a[8 * q + 2].y, a[8 * q + 3].y);
        hi.z = pack2_bf16(a[8 * q + 4].y, a[8 * q + 5].y); hi.w = pack2_bf16(a[8 * q + 6].y, a[8 * q + 7].y);
        *reinterpret_cast<uint4*>(sA + swz_chunk(2 * cp, kg * 2 + q)) = lo;
        *reinterpret_cast<uint4*>(sA + swz_chunk(2 * cp + 1, kg * 2 + q)) = hi;
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int idx = tid + t * 256;
        if (idx < pt_chunks) *reinterpret_cast<uint4*>(sB + swz_chunk(idx >> 3, idx & 7)) = pt[t];
      }
      if (r_n > 256) {  // rows 256.. of the P^T tile (r up to 512)
        for (int idx = 2048 + tid; idx < pt_chunks; idx += 256) {
          const uint4 v = *reinterpret_cast<const uint4*>(pr.PT16 + (long long)(idx >> 3) * pr.m_k + kb * 64 + (idx & 7) * 8);
          *reinterpret_cast<uint4*>(sB + swz_chunk(idx >> 3, idx & 7)) = v;
        }
      }
      fence_async_smem();
      mbar_arrive(&full_bar[s]);
    }

    // ---------------- epilogue: moments on this thread's column ------------------------------
    if (ok) ok = mbar_wait(&done_bar, 0u, status);
    tc_fence_after_sync();
    const int q = warp & 3, half = warp >> 2;
    const long long ecol = n0 + q * 32 + lane;
    const bool e_ok = ok && ecol < n;
    const float b1 = sc.beta1, b2 = sc.beta2, w = sc.omega;
    float dsum = 0.f;
    for (int ch = half; ch < r_n / 16; ch += 2) {
      float g[16];
      tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 16), g);
      float u[16], v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int row = ch * 16 + i;
        const bool live = e_ok && row < r;
        const long long idx = (long long)row * n + ecol;
        u[i] = live ? pr.u[idx] : 0.f;
        v[i] = live ? pr.v[idx] : 0.f;
      }
      uint32_t gp[8], up[8];
#pragma unroll
      for (int i = 0; i < 16; i += 2) {
        float o[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const int row = ch * 16 + i + t;
          const float gg = g[i + t];
          const float un = b1 * u[i + t] + (1.f - b1) * gg;
          const float vn = b2 * v[i + t] + (1.f - b2) * gg * gg;
          const float uh = un * sc.inv_bc1;
          const float D = sqrtf(vn * sc.inv_bc2) + sc.eps;
          o[t] = (sc.form == LORDO_QHM_LOW) ? (w * uh + (1.f - w) * gg) / D : uh / D;
          if (e_ok && row < r) {
            const long long idx = (long long)row * n + ecol;
            pr.u[idx] = un;
            pr.v[idx] = vn;
            dsum += D;
          } else {
            o[t] = 0.f;
          }
        }
        gp[i >> 1] = pack2_bf16(g[i], g[i + 1]);
        up[i >> 1] = pack2_bf16(o[0], o[1]);
      }
      if (e_ok) {
        uint4* gd = reinterpret_cast<uint4*>(pr.gT16 + ecol * pr.r_k + ch * 16);
        uint4* ud = reinterpret_cast<uint4*>(pr.uT16 + ecol * pr.r_k + ch * 16);
        gd[0] = make_uint4(gp[0], gp[1], gp[2], gp[3]); gd[1] = make_uint4(gp[4], gp[5], gp[6], gp[7]);
        ud[0] = make_uint4(up[0], up[1], up[2], up[3]); ud[1] = make_uint4(up[4], up[5], up[6], up[7]);
      }
    }
    if (sc.form == LORDO_QHM_FULL) {  // mu(D): mean over the rank axis, one value per column
      if (half == 1) dsum_s[q * 32 + lane] = dsum;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (half == 0 && e_ok) pr.dcol[ecol] = (dsum + dsum_s[q * 32 + lane]) / (float)r;
    }
  } else if (lane == 0) {
    // ---------------- MMA issue ---------------------------------------------------------------
    const uint32_t n_lo = r_n > 256 ? 256u : (uint32_t)r_n, n_hi = r_n > 256 ? (uint32_t)(r_n - 256) : 0u;
    const uint32_t idesc_lo = idesc_bf16_f32(128, n_lo), idesc_hi = idesc_bf16_f32(128, n_hi);
    bool ok = true;
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb & 1, use = kb >> 1;
      ok = mbar_wait(&full_bar[s], (uint32_t)(use & 1), status);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t sA = smem_u32(smem + s * stage_bytes), sB = sA + a_bytes;
#pragma unroll
      for (int k16 = 0; k16 < 4; ++k16) {
        const uint32_t acc = (kb > 0 || k16 > 0) ? 1u : 0u;
        mma_bf16(tmem, smem_desc_k128(sA + k16 * 32), smem_desc_k128(sB + k16 * 32), idesc_lo, acc);
        if (n_hi) mma_bf16(tmem + 256, smem_desc_k128(sA + k16 * 32), smem_desc_k128(sB + 256 * 128 + k16 * 32), idesc_hi, acc);
      }
      mma_commit(&empty_bar[s]);
    }
    mma_commit(&done_bar);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 8) tmem_free(tmem, ncols);
}

// ---------------------------------------------------------------------------------------------
// back-projection + error feedback + model update
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kApplyThreads, 1) apply_tc_kernel(const TcProblem* __restrict__ probs, int nprobs, StepScalars sc,
                                                                    int g_dt, int e_dt, int w_dt, unsigned* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t p_full[2], p_empty[2], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long strip = blockIdx.x;
  const TcProblem& pr = probs[find_problem(probs, nprobs, strip)];
  const int m = pr.m, n = pr.n, r_k = pr.r_k;
  const long long n0 = (strip - pr.strip_start) * kStrip;
  const int nkb = r_k / 64;
  const int nsteps = (m + kApplyRows - 1) / kApplyRows;
  const uint32_t x_bytes = (uint32_t)nkb * kStrip * 128;      // one resident operand (g^T or U~^T)
  const uint32_t p_bytes = (uint32_t)nkb * kApplyRows * 128;  // one ring stage of P rows
  unsigned char* sX1 = smem;
  unsigned char* sX2 = smem + x_bytes;
  unsigned char* sP = smem + 2 * x_bytes;
  constexpr uint32_t kCols = 256;  // 2 buffers x (2 accumulators x 64 rows)

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&p_full[s], kApplyProdWarps * 32); mbar_init(&p_empty[s], 1);
      mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], kApplyEpiWarps * 32);
    }
    mbar_init_fence();
  }
  if (warp == kApplyEpiWarps + kApplyProdWarps) tmem_alloc(&tmem_slot, kCols);

  // resident operands: rows = the strip's columns, k = rank index (zero rows beyond n)
  {
    const int chunks_per_row = r_k / 8;
    const int total = 2 * kStrip * chunks_per_row;
    for (int idx = tid; idx < total; idx += kApplyThreads) {
      const int which = idx >= kStrip * chunks_per_row;
      const int rem = idx - which * kStrip * chunks_per_row;
      const int row = rem / chunks_per_row, ch = rem - row * chunks_per_row;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (n0 + row < n) v = *reinterpret_cast<const uint4*>((which ? pr.uT16 : pr.gT16) + (n0 + row) * r_k + ch * 8);
      *reinterpret_cast<uint4*>((which ? sX2 : sX1) + (ch >> 3) * (kStrip * 128) + swz_chunk(row, ch & 7)) = v;
    }
  }
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  if (warp < kApplyEpiWarps) {
    // ---------------- epilogue: one column per thread, 16 rows per step -----------------------
    const int q = warp & 3, grp = warp >> 2;
    const long long col = n0 + q * 32 + lane;
    const bool col_ok = col < n;
    const void* G = *pr.G_ind;
    const float c = *pr.cptr;
    const float lr = sc.lr, om = sc.omega;
    const bool full = sc.form == LORDO_QHM_FULL, ef = sc.ef != 0;
    const float cd = (full && col_ok) ? (1.f - om) * c / pr.dcol[col] : 0.f;
    bool ok = true;
    for (int t = 0; t < nsteps && ok; ++t) {
      const int b = t & 1;
      const long long row0 = (long long)t * kApplyRows + grp * 16;
      float g[16], e[16], wv[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const bool live = col_ok && row0 + j < m;
        const long long idx = (row0 + j) * n + col;
        g[j] = live ? load1(G, g_dt, pr.G_off + idx) : 0.f;
        e[j] = (live && ef) ? load1(pr.E, e_dt, idx) : 0.f;
        wv[j] = live ? load1(pr.W, w_dt, idx) : 0.f;
      }
      ok = mbar_wait(&acc_full[b], (uint32_t)((t >> 1) & 1), status);
      if (!ok) break;
      tc_fence_after_sync();
      float a1[16], a2[16];
      const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * 128 + grp * 16);
      tmem_ld16(taddr, a1);
      tmem_ld16(taddr + 64, a2);
      tc_fence_before_sync();
      mbar_arrive(&acc_empty[b]);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (col_ok && row0 + j < m) {
          const long long idx = (row0 + j) * n + col;
          const float upd = full ? cd * g[j] + om * a2[j] : a2[j];
          if (ef) store1(pr.E, e_dt, idx, (c * g[j] + e[j]) - a1[j]);
          store1(pr.W, w_dt, idx, wv[j] - lr * upd);
        }
      }
    }
  } else if (warp < kApplyEpiWarps + kApplyProdWarps) {
    // ---------------- producers: rows of P for the next step ----------------------------------
    const int ptid = tid - kApplyEpiWarps * 32;
    const int chunks_per_row = r_k / 8;
    const int total = kApplyRows * chunks_per_row;  // <= 2048 for r_k <= 256
    bool ok = true;
    for (int t = 0; t < nsteps && ok; ++t) {
      const int s = t & 1;
      uint4 v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int idx = ptid + i * (kApplyProdWarps * 32);
        if (idx < total) {
          const int row = idx / chunks_per_row, ch = idx - row * chunks_per_row;
          v[i] = *reinterpret_cast<const uint4*>(pr.P16 + ((long long)t * kApplyRows + row) * r_k + ch * 8);
        }
      }
      ok = mbar_wait(&p_empty[s], (uint32_t)(((t >> 1) & 1) ^ 1), status);
      if (!ok) break;
      unsigned char* dst = sP + s * p_bytes;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int idx = ptid + i * (kApplyProdWarps * 32);
        if (idx < total) {
          const int row = idx / chunks_per_row, ch = idx - row * chunks_per_row;
          *reinterpret_cast<uint4*>(dst + (ch >> 3) * (kApplyRows * 128) + swz_chunk(row, ch & 7)) = v[i];
        }
      }
      fence_async_smem();
      mbar_arrive(&p_full[s]);
    }
  } else if (lane == 0) {
    // ---------------- MMA issue ---------------------------------------------------------------
    const uint32_t idesc = idesc_bf16_f32(128, kApplyRows);
    const uint32_t x1 = smem_u32(sX1), x2 = smem_u32(sX2);
    bool ok = true;
    for (int t = 0; t < nsteps && ok; ++t) {
      const int s = t & 1;
      ok = mbar_wait(&p_full[s], (uint32_t)((t >> 1) & 1), status);
      if (ok) ok = mbar_wait(&acc_empty[s], (uint32_t)(((t >> 1) & 1) ^ 1), status);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t pbase = smem_u32(sP + s * p_bytes);
      for (int kb = 0; kb < nkb; ++kb) {
#pragma unroll
        for (int k16 = 0; k16 < 4; ++k16) {
          const uint32_t acc = (kb > 0 || k16 > 0) ? 1u : 0u;
          const uint64_t bd = smem_desc_k128(pbase + kb * (kApplyRows * 128) + k16 * 32);
          mma_bf16(tmem + s * 128, smem_desc_k128(x1 + kb * (kStrip * 128) + k16 * 32), bd, idesc, acc);
          mma_bf16(tmem + s * 128 + 64, smem_desc_k128(x2 + kb * (kStrip * 128) + k16 * 32), bd, idesc, acc);
        }
      }
      mma_commit(&p_empty[s]);
      mma_commit(&acc_full[s]);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kApplyEpiWarps + kApplyProdWarps) tmem_free(tmem, kCols);
}

// ---------------------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------------------
size_t project_tc_smem(int r_n_max) {
  const size_t stage = (size_t)kStrip * 128 + (((size_t)r_n_max * 128 + 1023) & ~size_t(1023));
  return 2 * stage + 1024;
}
size_t apply_tc_smem(int r_k_max) {
  const size_t nkb = (size_t)r_k_max / 64;
  return 2 * nkb * kStrip * 128 + 2 * nkb * kApplyRows * 128 + 1024;
}

cudaError_t tc_configure(int r_n_max, int r_k_max) {
  cudaError_t e = cudaFuncSetAttribute(project_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)project_tc_smem(r_n_max));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(apply_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_tc_smem(r_k_max));
}

void launch_prep_projection(const TcPrep* items, const long long* blk_start, int nitems, long long total_blocks, cudaStream_t st) {
  prep_projection_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(items, blk_start, nitems);
}
void launch_project_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_n_max, const StepScalars& sc, int g_dt,
                       int e_dt, unsigned* status, cudaStream_t st) {
  project_tc_kernel<<<(unsigned)total_strips, kProjThreads, project_tc_smem(r_n_max), st>>>(probs, nprobs, sc, g_dt, e_dt, status);
}
void launch_apply_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_k_max, const StepScalars& sc, int g_dt,
                     int e_dt, int w_dt, unsigned* status, cudaStream_t st) {
  apply_tc_kernel<<<(unsigned)total_strips, kApplyThreads, apply_tc_smem(r_k_max), st>>>(probs, nprobs, sc, g_dt, e_dt, w_dt, status);
}

}  // namespace lordo
