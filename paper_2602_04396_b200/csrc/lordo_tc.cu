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
constexpr int kApplyEpiWarps = 16, kApplyProdWarps = 2;
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

// Storage type of G, E and W inside the tensor-core kernels: all bf16 or all fp32. Loads are kept
// as raw values in registers (no use before the whole batch has been issued), converted afterwards.
template <bool BF16>
struct Elem;
template <>
struct Elem<true> {
  using one = unsigned short;
  using pair = uint32_t;
  static __device__ __forceinline__ float cvt(one x) { return __uint_as_float(((uint32_t)x) << 16); }
  static __device__ __forceinline__ float2 cvt2(pair x) { return make_float2(__uint_as_float(x << 16), __uint_as_float(x & 0xFFFF0000u)); }
  static __device__ __forceinline__ one pack(float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    return *reinterpret_cast<const unsigned short*>(&h);
  }
};
template <>
struct Elem<false> {
  using one = float;
  using pair = float2;
  static __device__ __forceinline__ float cvt(one x) { return x; }
  static __device__ __forceinline__ float2 cvt2(pair x) { return x; }
  static __device__ __forceinline__ one pack(float v) { return v; }
};

}  // namespace

// ---------------------------------------------------------------------------------------------
// P (fp32 [m][r]) -> P16 [m_r][r_k] and PT16 [r_n][m_k] in bf16; the pads stay zero.
// ---------------------------------------------------------------------------------------------
// One block per 64 x 64 tile of P: rows of P16 and, through a transposed tile in shared memory, rows of
// PT16 are both written as runs of consecutive addresses.
__global__ void __launch_bounds__(256) prep_projection_kernel(const TcPrep* __restrict__ items, const long long* __restrict__ blk_start,
                                                              int nitems) {
  __shared__ __nv_bfloat16 tile[64][66];
  const long long blk = blockIdx.x;
  const int i = find_segment(blk_start, nitems, blk);
  const TcPrep it = items[i];
  const long long local = blk - blk_start[i];
  const int tiles_c = (it.r + 63) / 64;
  const long long row0 = (local / tiles_c) * 64;
  const int col0 = (int)(local % tiles_c) * 64;
  for (int e = threadIdx.x; e < 64 * 64; e += 256) {
    const int rr = e >> 6, cc = e & 63;
    const long long row = row0 + rr;
    const int col = col0 + cc;
    if (row < it.m && col < it.r) {
      const __nv_bfloat16 h = __float2bfloat16_rn(it.P[row * it.r + col]);
      it.P16[row * it.r_k + col] = h;
      tile[rr][cc] = h;
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 64 * 64; e += 256) {
    const int cc = e >> 6, rr = e & 63;
    const long long row = row0 + rr;
    const int col = col0 + cc;
    if (row < it.m && col < it.r) it.PT16[(long long)col * it.m_k + row] = tile[rr][cc];
  }
}

// ---------------------------------------------------------------------------------------------
// project + moments
// ---------------------------------------------------------------------------------------------
template <bool BF16>
__global__ void __launch_bounds__(kProjThreads, 2) project_tc_kernel(const TcProblem* __restrict__ probs, int nprobs, StepScalars sc,
                                                                     unsigned* __restrict__ status) {
  using EL = Elem<BF16>;
  using one_t = typename EL::one;
  using pair_t = typename EL::pair;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[2], empty_bar[2], done_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ float dsum_s[kStrip];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long strip = blockIdx.x;
  const TcProblem* __restrict__ prp = probs + find_problem(probs, nprobs, strip);
  const int m = prp->m, n = prp->n, r = prp->r, r_n = prp->r_n, m_k = prp->m_k, r_k = prp->r_k;
  const long long n0 = (strip - prp->strip_start) * kStrip;
  const int nkb = m_k / 64;
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
    const long long colc = col_ok ? col : (long long)n - 2;  // loads stay in bounds, results are masked
    const one_t* __restrict__ Gp = reinterpret_cast<const one_t*>(*prp->G_ind) + prp->G_off;
    const bool have_e = sc.ef != 0;
    const one_t* __restrict__ Ep = have_e ? reinterpret_cast<const one_t*>(prp->E) : Gp;
    const one_t* __restrict__ Gc = Gp + colc;
    const one_t* __restrict__ Ec = Ep + colc;
    const float c = *prp->cptr;
    const float es = have_e ? 1.f : 0.f;
    const __nv_bfloat16* __restrict__ PT = prp->PT16;
    const int pt_chunks = r_n * 8;
    bool ok = true;
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb & 1, use = kb >> 1;
      pair_t rg[16], re[16];
      const int rbase = kb * 64 + kg * 16;
      if (rbase + 16 <= m) {
        const size_t base = (size_t)rbase * (size_t)n;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          rg[j] = *reinterpret_cast<const pair_t*>(Gc + base + (size_t)(unsigned)(j * n));
          re[j] = *reinterpret_cast<const pair_t*>(Ec + base + (size_t)(unsigned)(j * n));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const size_t off = (size_t)(unsigned)min(rbase + j, m - 1) * (size_t)n;
          rg[j] = *reinterpret_cast<const pair_t*>(Gc + off);
          re[j] = *reinterpret_cast<const pair_t*>(Ec + off);
        }
      }
      uint4 pt[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        int idx = tid + t * 256;
        idx = idx < pt_chunks ? idx : pt_chunks - 1;
        pt[t] = *reinterpret_cast<const uint4*>(PT + (long long)(idx >> 3) * m_k + kb * 64 + (idx & 7) * 8);
      }
      float2 a[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float2 g = EL::cvt2(rg[j]), e = EL::cvt2(re[j]);
        const float live = (col_ok && rbase + j < m) ? 1.f : 0.f;
        a[j] = make_float2(live * (c * g.x + es * e.x), live * (c * g.y + es * e.y));
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
          const uint4 v = *reinterpret_cast<const uint4*>(PT + (long long)(idx >> 3) * m_k + kb * 64 + (idx & 7) * 8);
          *reinterpret_cast<uint4*>(sB + swz_chunk(idx >> 3, idx & 7)) = v;
        }
      }
      fence_async_smem();
      mbar_arrive(&full_bar[s]);
    }

    // ---------------- epilogue: moments on this thread's column ------------------------------
    if (ok) ok = mbar_wait<64>(&done_bar, 0u, status);
    tc_fence_after_sync();
    const int q = warp & 3, half = warp >> 2;
    const long long ecol = n0 + q * 32 + lane;
    const bool e_ok = ok && ecol < n;
    const long long ecolc = ecol < n ? ecol : (long long)n - 1;
    float* __restrict__ up_ = prp->u;
    float* __restrict__ vp_ = prp->v;
    __nv_bfloat16* __restrict__ gT = prp->gT16 + ecolc * r_k;
    __nv_bfloat16* __restrict__ uT = prp->uT16 + ecolc * r_k;
    const float b1 = sc.beta1, b2 = sc.beta2, w = sc.omega;
    const bool low = sc.form == LORDO_QHM_LOW;
    float dsum = 0.f;
    for (int ch = half; ch < r_n / 16; ch += 2) {
      float u[16], v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const size_t idx = (size_t)(unsigned)min(ch * 16 + i, r - 1) * (size_t)n + (size_t)ecolc;
        u[i] = up_[idx];
        v[i] = vp_[idx];
      }
      float g[16];
      tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 16), g);
      uint32_t gp[8], upk[8];
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
          o[t] = low ? (w * uh + (1.f - w) * gg) / D : uh / D;
          if (e_ok && row < r) {
            const size_t idx = (size_t)(unsigned)row * (size_t)n + (size_t)ecol;
            up_[idx] = un;
            vp_[idx] = vn;
            if (prp->tb) prp->tb[idx] += sc.lr * o[t];
            dsum += D;
          } else {
            o[t] = 0.f;
          }
        }
        gp[i >> 1] = pack2_bf16(g[i], g[i + 1]);
        upk[i >> 1] = pack2_bf16(o[0], o[1]);
      }
      if (e_ok) {
        uint4* gd = reinterpret_cast<uint4*>(gT + ch * 16);
        uint4* ud = reinterpret_cast<uint4*>(uT + ch * 16);
        gd[0] = make_uint4(gp[0], gp[1], gp[2], gp[3]); gd[1] = make_uint4(gp[4], gp[5], gp[6], gp[7]);
        ud[0] = make_uint4(upk[0], upk[1], upk[2], upk[3]); ud[1] = make_uint4(upk[4], upk[5], upk[6], upk[7]);
      }
    }
    if (sc.form == LORDO_QHM_FULL) {  // mu(D): mean over the rank axis, one value per column
      if (half == 1) dsum_s[q * 32 + lane] = dsum;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (half == 0 && e_ok) prp->dcol[ecol] = (dsum + dsum_s[q * 32 + lane]) / (float)r;
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
template <bool BF16>
__global__ void __launch_bounds__(kApplyThreads, 1) apply_tc_kernel(const TcProblem* __restrict__ probs, int nprobs, StepScalars sc,
                                                                    unsigned* __restrict__ status) {
  using EL = Elem<BF16>;
  using one_t = typename EL::one;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t p_full[2], p_empty[2], acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long strip = blockIdx.x;
  const TcProblem* __restrict__ prp = probs + find_problem(probs, nprobs, strip);
  const int m = prp->m, n = prp->n, r_k = prp->r_k;
  const long long n0 = (strip - prp->strip_start) * kStrip;
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
    const int per_op = kStrip * chunks_per_row;
    const int total = 2 * per_op;
    const __nv_bfloat16* __restrict__ g16 = prp->gT16;
    const __nv_bfloat16* __restrict__ u16 = prp->uT16;
    for (int base = tid; base < total; base += 4 * kApplyThreads) {
      uint4 v[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        int idx = base + t * kApplyThreads;
        idx = idx < total ? idx : total - 1;
        const int which = idx >= per_op;
        const int rem = idx - which * per_op;
        const int row = rem / chunks_per_row, ch = rem - row * chunks_per_row;
        long long grow = n0 + row;
        grow = grow < n ? grow : (long long)n - 1;
        v[t] = *reinterpret_cast<const uint4*>((which ? u16 : g16) + grow * r_k + ch * 8);
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int idx = base + t * kApplyThreads;
        if (idx < total) {
          const int which = idx >= per_op;
          const int rem = idx - which * per_op;
          const int row = rem / chunks_per_row, ch = rem - row * chunks_per_row;
          const uint4 val = (n0 + row < n) ? v[t] : make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>((which ? sX2 : sX1) + (ch >> 3) * (kStrip * 128) + swz_chunk(row, ch & 7)) = val;
        }
      }
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
    const long long colc = col_ok ? col : (long long)n - 1;
    const one_t* __restrict__ Gp = reinterpret_cast<const one_t*>(*prp->G_ind) + prp->G_off;
    one_t* __restrict__ Wp = reinterpret_cast<one_t*>(prp->W);
    const bool ef = sc.ef != 0;
    one_t* __restrict__ Ep = ef ? reinterpret_cast<one_t*>(prp->E) : Wp;
    const float c = *prp->cptr;
    const float lr = sc.lr, om = sc.omega;
    const bool full = sc.form == LORDO_QHM_FULL;
    const float cd = full ? (1.f - om) * c / prp->dcol[colc] : 0.f;
    const float a2w = full ? om : 1.f;
    const one_t* __restrict__ Gc = Gp + colc;
    one_t* __restrict__ Ec = Ep + colc;
    one_t* __restrict__ Wc = Wp + colc;
    bool ok = true;
    for (int t = 0; t < nsteps && ok; ++t) {
      const int b = t & 1;
      const int row0 = t * kApplyRows + grp * 16;
      const bool whole = row0 + 16 <= m;
      const size_t base = (size_t)(unsigned)min(row0, m - 1) * (size_t)n;
      one_t rg[16], re[16], rw[16];
      if (whole) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const size_t off = base + (size_t)(unsigned)(j * n);
          rg[j] = Gc[off];
          re[j] = Ec[off];
          rw[j] = Wc[off];
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const size_t off = (size_t)(unsigned)min(row0 + j, m - 1) * (size_t)n;
          rg[j] = Gc[off];
          re[j] = Ec[off];
          rw[j] = Wc[off];
        }
      }
      ok = mbar_wait<40>(&acc_full[b], (uint32_t)((t >> 1) & 1), status);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * 128 + grp * 16);
      float acc[16];
      tmem_ld16(taddr, acc);  // (P g)^T
      if (ef && col_ok) {
        if (whole) {
#pragma unroll
          for (int j = 0; j < 16; ++j) Ec[base + (size_t)(unsigned)(j * n)] = EL::pack((c * EL::cvt(rg[j]) + EL::cvt(re[j])) - acc[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (row0 + j < m) Ec[base + (size_t)(unsigned)(j * n)] = EL::pack((c * EL::cvt(rg[j]) + EL::cvt(re[j])) - acc[j]);
        }
      }
      tmem_ld16(taddr + 64, acc);  // (P U~)^T
      tc_fence_before_sync();
      mbar_arrive(&acc_empty[b]);
      if (col_ok) {
        if (whole) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            Wc[base + (size_t)(unsigned)(j * n)] = EL::pack(EL::cvt(rw[j]) - lr * (cd * EL::cvt(rg[j]) + a2w * acc[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (row0 + j < m) Wc[base + (size_t)(unsigned)(j * n)] = EL::pack(EL::cvt(rw[j]) - lr * (cd * EL::cvt(rg[j]) + a2w * acc[j]));
        }
      }
    }
  } else if (warp < kApplyEpiWarps + kApplyProdWarps) {
    // ---------------- producers: rows of P for the next step (asynchronous 16-byte copies) -----
    const int ptid = tid - kApplyEpiWarps * 32;
    const int chunks_per_row = r_k / 8;
    const int total = kApplyRows * chunks_per_row;
    const __nv_bfloat16* __restrict__ P16 = prp->P16;
    bool ok = true;
    for (int t = 0; t < nsteps && ok; ++t) {
      const int s = t & 1;
      ok = mbar_wait(&p_empty[s], (uint32_t)(((t >> 1) & 1) ^ 1), status);
      if (!ok) break;
      const uint32_t dst = smem_u32(sP + s * p_bytes);
      for (int idx = ptid; idx < total; idx += kApplyProdWarps * 32) {
        const int row = idx / chunks_per_row, ch = idx - row * chunks_per_row;
        const __nv_bfloat16* src = P16 + ((long long)t * kApplyRows + row) * r_k + ch * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (ch >> 3) * (kApplyRows * 128) + swz_chunk(row, ch & 7)),
                     "l"(src)
                     : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
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
  cudaError_t e = cudaFuncSetAttribute(project_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)project_tc_smem(r_n_max));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(project_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)project_tc_smem(r_n_max));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(apply_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_tc_smem(r_k_max));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(apply_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_tc_smem(r_k_max));
}

void launch_prep_projection(const TcPrep* items, const long long* blk_start, int nitems, long long total_blocks, cudaStream_t st) {
  prep_projection_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(items, blk_start, nitems);
}
void launch_project_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_n_max, const StepScalars& sc, int bf16,
                       unsigned* status, cudaStream_t st) {
  if (bf16) project_tc_kernel<true><<<(unsigned)total_strips, kProjThreads, project_tc_smem(r_n_max), st>>>(probs, nprobs, sc, status);
  else project_tc_kernel<false><<<(unsigned)total_strips, kProjThreads, project_tc_smem(r_n_max), st>>>(probs, nprobs, sc, status);
}
void launch_apply_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_k_max, const StepScalars& sc, int bf16,
                     unsigned* status, cudaStream_t st) {
  if (bf16) apply_tc_kernel<true><<<(unsigned)total_strips, kApplyThreads, apply_tc_smem(r_k_max), st>>>(probs, nprobs, sc, status);
  else apply_tc_kernel<false><<<(unsigned)total_strips, kApplyThreads, apply_tc_smem(r_k_max), st>>>(probs, nprobs, sc, status);
}

}  // namespace lordo
