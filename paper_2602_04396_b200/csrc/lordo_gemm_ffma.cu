// Grouped fp32 FFMA GEMM with fused operand formation and epilogues: the fp32-accurate ("check
// mode") realisation of every contraction of the path -- P^T(cG+E), P g, P U~, the sketch and
// subspace-iteration products, Gram matrices, R^-1 application, Rot = P'^T P and the rotation of
// the moments. 64 x 64 output tile, 16-deep k-slices, 256 threads, 4 x 4 outputs per thread.
// Products are formed and summed in fp32 inside a k-slice; the slice sums are carried across slices
// in fp64, so a result is accurate to fp32 rounding whatever the contraction length.
#include "lordo_kernels.h"

namespace lordo {

constexpr int BM = 64, BN = 64, BK = 16, PADS = 4;

__device__ __forceinline__ const void* operand_base(const Operand& op) {
  return op.p0_ind ? *op.p0_ind : op.p0;
}

// Four consecutive stored elements (row, col..col+3) of an operand, zero outside (rows, cols).
__device__ __forceinline__ float4 operand_load4(const Operand& op, const void* base, float s0, const GemmScalars& sc, long long row,
                                                long long col, long long rows, long long cols) {
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  if (row >= rows || col >= cols) return o;
  const long long idx = row * op.ld + col;
  if (col + 3 < cols) {
    const float4 a = load4(base, op.dt0, op.p0_off + idx);
    if (op.kind == OP_PLAIN) {
      o = make_float4(s0 * a.x, s0 * a.y, s0 * a.z, s0 * a.w);
      if (op.p1) {
        const float4 b = load4(op.p1, op.dt1, idx);
        o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
      }
    } else if (op.kind == OP_UHAT) {
      o = make_float4(sc.inv_bc1 * a.x, sc.inv_bc1 * a.y, sc.inv_bc1 * a.z, sc.inv_bc1 * a.w);
    } else {
      const float4 b = load4(op.p1, op.dt1, idx);
      const float ux = sc.inv_bc1 * a.x, uy = sc.inv_bc1 * a.y, uz = sc.inv_bc1 * a.z, uw = sc.inv_bc1 * a.w;
      o = make_float4(sc.inv_bc2 * b.x - ux * ux, sc.inv_bc2 * b.y - uy * uy, sc.inv_bc2 * b.z - uz * uz,
                      sc.inv_bc2 * b.w - uw * uw);
    }
    return o;
  }
  float t[4] = {0.f, 0.f, 0.f, 0.f};
  for (int e = 0; e < 4 && col + e < cols; ++e) {
    const float a = load1(base, op.dt0, op.p0_off + idx + e);
    if (op.kind == OP_PLAIN) {
      t[e] = s0 * a + (op.p1 ? load1(op.p1, op.dt1, idx + e) : 0.f);
    } else if (op.kind == OP_UHAT) {
      t[e] = sc.inv_bc1 * a;
    } else {
      const float uh = sc.inv_bc1 * a;
      t[e] = sc.inv_bc2 * load1(op.p1, op.dt1, idx + e) - uh * uh;
    }
  }
  return make_float4(t[0], t[1], t[2], t[3]);
}

// CARRY = 1: slice sums carried across k-slices in fp64 (parity mode). CARRY = 0: plain fp32
// accumulation, half the registers (the fp32 work of the fast mode: QR and moment rotation).
template <int ATRANS, int DUAL, int CARRY>
__global__ void __launch_bounds__(256) gemm_ffma_kernel(const GemmProblem* __restrict__ probs, int nprobs, GemmScalars sc) {
  __shared__ __align__(16) float sA[BK][BM + PADS];
  __shared__ __align__(16) float sB[BK][BN + PADS];
  __shared__ __align__(16) float sB2[DUAL ? BK : 1][BN + PADS];

  // locate the problem of this block
  const long long blk = blockIdx.x;
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].tile_start <= blk) lo = mid; else hi = mid - 1;
  }
  const GemmProblem& pr = probs[lo];
  const long long local = blk - pr.tile_start;
  const int tile_m = (int)(local / pr.tiles_n), tile_n = (int)(local - (long long)tile_m * pr.tiles_n);
  const int M = pr.M, N = pr.N, Kd = pr.Kd;
  const long long m0 = (long long)tile_m * BM, n0 = (long long)tile_n * BN;

  const void* baseA = operand_base(pr.A);
  const void* baseB = operand_base(pr.B);
  const void* baseB2 = DUAL ? operand_base(pr.B2) : nullptr;
  const float sA0 = pr.A.s0_ptr ? *pr.A.s0_ptr : 1.f;
  const float sB0 = pr.B.s0_ptr ? *pr.B.s0_ptr : 1.f;
  float sB20 = 1.f;
  if constexpr (DUAL) sB20 = pr.B2.s0_ptr ? *pr.B2.s0_ptr : 1.f;

  const int t = threadIdx.x;
  const int tx = t & 15, ty = t >> 4;
  // B tile loader: one float4 per thread, row kk = t/16, columns (t%16)*4
  const int bk = t >> 4, bc = (t & 15) * 4;
  // A tile loader. ATRANS: as B (stored [Kd][M]). Otherwise stored [M][Kd]: row t/4, k (t%4)*4.
  const int ar = ATRANS ? (t >> 4) : (t >> 2), ac = ATRANS ? (t & 15) * 4 : (t & 3) * 4;

  float acc[4][4], acc2[DUAL ? 4 : 1][4];
  double tot[CARRY ? 4 : 1][4], tot2[(CARRY && DUAL) ? 4 : 1][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc[i][j] = 0.f;
      if constexpr (CARRY) tot[i][j] = 0.0;
      if constexpr (DUAL) {
        acc2[i][j] = 0.f;
        if constexpr (CARRY) tot2[i][j] = 0.0;
      }
    }

  float4 ra, rb, rb2 = make_float4(0.f, 0.f, 0.f, 0.f);
  auto fetch = [&](int k0) {
    if (ATRANS) ra = operand_load4(pr.A, baseA, sA0, sc, k0 + ar, m0 + ac, Kd, M);
    else ra = operand_load4(pr.A, baseA, sA0, sc, m0 + ar, k0 + ac, M, Kd);
    rb = operand_load4(pr.B, baseB, sB0, sc, k0 + bk, n0 + bc, Kd, N);
    if constexpr (DUAL) rb2 = operand_load4(pr.B2, baseB2, sB20, sc, k0 + bk, n0 + bc, Kd, N);
  };
  auto stash = [&]() {
    if (ATRANS) {
      *reinterpret_cast<float4*>(&sA[ar][ac]) = ra;
    } else {
      sA[ac + 0][ar] = ra.x; sA[ac + 1][ar] = ra.y; sA[ac + 2][ar] = ra.z; sA[ac + 3][ar] = ra.w;
    }
    *reinterpret_cast<float4*>(&sB[bk][bc]) = rb;
    if constexpr (DUAL) *reinterpret_cast<float4*>(&sB2[bk][bc]) = rb2;
  };

  fetch(0);
  for (int k0 = 0; k0 < Kd; k0 += BK) {
    stash();
    __syncthreads();
    if (k0 + BK < Kd) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&sA[kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&sB[kk][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w};
      const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      if constexpr (DUAL) {
        const float4 c4 = *reinterpret_cast<const float4*>(&sB2[kk][tx * 4]);
        const float c[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float a2 = sc.a_square ? a[i] * a[i] : a[i];
#pragma unroll
          for (int j = 0; j < 4; ++j) acc2[i][j] = fmaf(a2, c[j], acc2[i][j]);
        }
      }
    }
    if constexpr (CARRY) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          tot[i][j] += (double)acc[i][j];
          acc[i][j] = 0.f;
          if constexpr (DUAL) { tot2[i][j] += (double)acc2[i][j]; acc2[i][j] = 0.f; }
        }
    }
    __syncthreads();
  }
  if constexpr (CARRY) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[i][j] = (float)tot[i][j];
        if constexpr (DUAL) acc2[i][j] = (float)tot2[i][j];
      }
  }

  // ---- epilogue: each thread owns rows m0+ty*4.., columns n0+tx*4..+3 (N is a multiple of 4)
  const Epilogue& ep = pr.epi;
  const long long col = n0 + tx * 4;
  if (col >= N) return;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long row = m0 + ty * 4 + i;
    if (row >= M) break;
    if (ep.kind == EPI_STORE && ep.trans) {  // C[col][row]
      const float o[4] = {acc[i][0], acc[i][1], acc[i][2], acc[i][3]};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float* cp = ep.C + (col + j) * ep.ldc + row;
        *cp = ep.pad ? *cp + o[j] : o[j];
      }
    } else if (ep.kind == EPI_STORE) {
      float4* cp = reinterpret_cast<float4*>(ep.C + row * ep.ldc + col);
      float4 o = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      if (ep.pad) {  // accumulate into C
        const float4 old = *cp;
        o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
      }
      *cp = o;
    } else if (ep.kind == EPI_APPLY && ep.trans) {
      // the product was formed for the transposed problem: output (row, col) is weight element (col, row),
      // and the full-rank QHM scale belongs to the output column = the weight's row
      if constexpr (DUAL) {
        const float c = *ep.cptr;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const long long idx = (col + j) * ep.ldt + row;
          const float g = load1(*ep.G_ind, sc.g_dt, ep.G_off + idx);
          const float w = load1(ep.W, sc.w_dt, idx);
          float upd = acc2[i][j];
          if (sc.form == LORDO_QHM_FULL) upd = (1.f - sc.omega) * (c * g) / ep.dcol[col + j] + sc.omega * upd;
          if (sc.ef) store1(ep.E, sc.e_dt, idx, (c * g + load1(ep.E, sc.e_dt, idx)) - acc[i][j]);
          store1(ep.W, sc.w_dt, idx, w - sc.lr * upd);
        }
      }
    } else if (ep.kind == EPI_APPLY) {
      if constexpr (DUAL) {
        const long long idx = row * (long long)N + col;
        const float c = *ep.cptr;
        const float4 g = load4(*ep.G_ind, sc.g_dt, ep.G_off + idx);
        const float4 w = load4(ep.W, sc.w_dt, idx);
        float4 upd = make_float4(acc2[i][0], acc2[i][1], acc2[i][2], acc2[i][3]);
        if (sc.form == LORDO_QHM_FULL) {
          const float4 d = *reinterpret_cast<const float4*>(ep.dcol + col);
          const float w1 = 1.f - sc.omega;
          upd.x = w1 * (c * g.x) / d.x + sc.omega * upd.x;
          upd.y = w1 * (c * g.y) / d.y + sc.omega * upd.y;
          upd.z = w1 * (c * g.z) / d.z + sc.omega * upd.z;
          upd.w = w1 * (c * g.w) / d.w + sc.omega * upd.w;
        }
        if (sc.ef) {
          const float4 e = load4(ep.E, sc.e_dt, idx);
          float4 en;
          en.x = (c * g.x + e.x) - acc[i][0];
          en.y = (c * g.y + e.y) - acc[i][1];
          en.z = (c * g.z + e.z) - acc[i][2];
          en.w = (c * g.w + e.w) - acc[i][3];
          store4(ep.E, sc.e_dt, idx, en);
        }
        store4(ep.W, sc.w_dt, idx, make_float4(w.x - sc.lr * upd.x, w.y - sc.lr * upd.y, w.z - sc.lr * upd.z, w.w - sc.lr * upd.w));
      }
    } else {  // EPI_ROTATE: acc = Rot u^, acc2 = (Rot o Rot)(v^ - u^ o u^)
      if constexpr (DUAL) {
        const long long idx = row * (long long)N + col;
        float4 un, vn;
        un.x = sc.bc1 * acc[i][0]; un.y = sc.bc1 * acc[i][1]; un.z = sc.bc1 * acc[i][2]; un.w = sc.bc1 * acc[i][3];
        vn.x = sc.bc2 * fabsf(acc2[i][0] + acc[i][0] * acc[i][0]);
        vn.y = sc.bc2 * fabsf(acc2[i][1] + acc[i][1] * acc[i][1]);
        vn.z = sc.bc2 * fabsf(acc2[i][2] + acc[i][2] * acc[i][2]);
        vn.w = sc.bc2 * fabsf(acc2[i][3] + acc[i][3] * acc[i][3]);
        *reinterpret_cast<float4*>(ep.u_out + idx) = un;
        *reinterpret_cast<float4*>(ep.v_out + idx) = vn;
      }
    }
  }
}

void launch_gemm(const GemmProblem* probs, int nprobs, long long total_tiles, int atrans, int dual, int carry, const GemmScalars& sc,
                 cudaStream_t st) {
  const unsigned grid = (unsigned)total_tiles;
  if (carry) {
    if (atrans && !dual) gemm_ffma_kernel<1, 0, 1><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else if (!atrans && !dual) gemm_ffma_kernel<0, 0, 1><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else if (!atrans && dual) gemm_ffma_kernel<0, 1, 1><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else gemm_ffma_kernel<1, 1, 1><<<grid, 256, 0, st>>>(probs, nprobs, sc);
  } else {
    if (atrans && !dual) gemm_ffma_kernel<1, 0, 0><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else if (!atrans && !dual) gemm_ffma_kernel<0, 0, 0><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else if (!atrans && dual) gemm_ffma_kernel<0, 1, 0><<<grid, 256, 0, st>>>(probs, nprobs, sc);
    else gemm_ffma_kernel<1, 1, 0><<<grid, 256, 0, st>>>(probs, nprobs, sc);
  }
}

// ---------------------------------------------------------------------------------------------
// Cholesky of the Gram matrix + inverse of the triangular factor, one block per problem.
// Blocked left-looking Cholesky with fp64 accumulation, panels of 32 columns: a thread owns a row i
// of L and keeps that row's 32 panel entries in registers; the contribution of the columns before
// the panel is a rank-j0 update in which every value of L loaded from memory meets 32 values of a
// 32 x 32 tile in shared memory, so that the column-by-column part (two barriers per column) is left
// with at most 31 multiply-adds. The factor is kept TRANSPOSED in global memory (Lt[k][i] = L[i][k],
// L2-resident) so that the threads' reads of their own rows are consecutive addresses.
// L^-1 the same way with a thread per column: 32 rows of X at a time, the part below the panel's
// diagonal block as a tile product, the block itself by substitution in registers.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kCB = 32;
}

__global__ void __launch_bounds__(512) chol_inverse_kernel(const CholProblem* __restrict__ probs, unsigned* __restrict__ status) {
  __shared__ double tile[kCB][kCB + 1];  // [panel entry][k within the chunk]
  __shared__ float dblk[kCB][kCB + 1];   // diagonal block of L, row-major
  __shared__ float pivot_s;
  __shared__ float maxdiag_s;
  const CholProblem pb = probs[blockIdx.x];
  const int r = pb.r;
  const float* __restrict__ A = pb.gram;
  float* __restrict__ Lt = pb.lwork;  // distinct buffers; every other view of them below is derived from these
  float* __restrict__ X = pb.rinv;
  const int t = threadIdx.x, nt = blockDim.x;

  if (t == 0) {
    float md = 0.f;
    for (int i = 0; i < r; ++i) md = fmaxf(md, fabsf(A[(long long)i * r + i]));
    maxdiag_s = md;
  }
  __syncthreads();
  // A pivot is the squared distance of column j of the factored matrix from the span of the
  // columns before it. Below kBreakdown times the column's own squared norm that distance is
  // inside the rounding noise of an fp32 Gram matrix: the column is treated as dependent, the
  // flag is raised and the pivot is clamped so that everything stays finite.
  constexpr float kBreakdown = 3e-5f;
  const float abs_floor = maxdiag_s > 0.f ? maxdiag_s * 1e-12f : 1.f;

  for (int j0 = 0; j0 < r; j0 += kCB) {
    const int nbw = r - j0 < kCB ? r - j0 : kCB;
    for (int ib = j0; ib < r; ib += nt) {  // one pass unless r - j0 exceeds the block
      const int i = ib + t;
      const bool live = i < r;
      // s_i[jj] = A[i][j0+jj] - sum_{k<j0} L[i][k] L[j0+jj][k]   (A is symmetric: row j0+jj is read)
      double acc[kCB];
#pragma unroll
      for (int jj = 0; jj < kCB; ++jj) acc[jj] = (live && jj < nbw) ? (double)A[(long long)(j0 + jj) * r + i] : 0.0;
      for (int k0 = 0; k0 < j0; k0 += kCB) {
        __syncthreads();
        for (int e = t; e < kCB * kCB; e += nt) {
          const int jj = e / kCB, kk = e - jj * kCB;
          tile[jj][kk] = jj < nbw ? (double)Lt[(long long)(k0 + kk) * r + j0 + jj] : 0.0;
        }
        __syncthreads();
        if (live) {
#pragma unroll 4
          for (int kk = 0; kk < kCB; ++kk) {
            const double l = (double)Lt[(long long)(k0 + kk) * r + i];
#pragma unroll
            for (int jj = 0; jj < kCB; ++jj) acc[jj] -= l * tile[jj][kk];
          }
        }
      }
      if (ib == j0) {
        // the chunk that holds the diagonal block: column by column, the finished column of the block
        // published in shared memory for the multiply-adds of the columns after it
#pragma unroll
        for (int jj = 0; jj < kCB; ++jj) {
          if (jj < nbw) {
            const int j = j0 + jj;
            if (live && i == j) {
              float d = (float)acc[jj];
              const float floor_pivot = fmaxf(kBreakdown * A[(long long)j * r + j], abs_floor);
              if (!(d > floor_pivot)) {  // also catches NaN
                atomicOr(status, LORDO_FLAG_QR_BREAKDOWN);
                d = floor_pivot;
              }
              pivot_s = sqrtf(d);
            }
            __syncthreads();
            const float piv = pivot_s;
            float lij = 0.f;
            if (live && i >= j) {
              lij = (i == j) ? piv : (float)acc[jj] / piv;
              Lt[(long long)j * r + i] = lij;
              if (i < j0 + nbw) dblk[i - j0][jj] = lij;
            }
            __syncthreads();
            if (live && i > j) {
#pragma unroll
              for (int j2 = jj + 1; j2 < kCB; ++j2)
                if (j2 < nbw) acc[j2] -= (double)lij * (double)dblk[j2][jj];
            }
          }
        }
      } else {
        // rows below the first chunk: the whole diagonal block is known
        __syncthreads();
        if (live) {
#pragma unroll
          for (int jj = 0; jj < kCB; ++jj) {
            if (jj < nbw) {
              const float lij = (float)acc[jj] / dblk[jj][jj];
              Lt[(long long)(j0 + jj) * r + i] = lij;
#pragma unroll
              for (int j2 = jj + 1; j2 < kCB; ++j2)
                if (j2 < nbw) acc[j2] -= (double)lij * (double)dblk[j2][jj];
            }
          }
        }
      }
    }
    __syncthreads();  // the panel's columns are in memory for everybody
  }

  // X = L^-1 (lower triangular), column c by thread c, 32 rows at a time:
  // X[i][c] = ([i == c] - sum_{k<i} L[i][k] X[k][c]) / L[i][i], zero above the diagonal.
  for (int c = t; c < r; c += nt)
    for (int i = 0; i < r; ++i)
      if (i < c) X[(long long)i * r + c] = 0.f;
  for (int i0 = 0; i0 < r; i0 += kCB) {
    const int nbw = r - i0 < kCB ? r - i0 : kCB;
    for (int cb = 0; cb < r; cb += nt) {
      const int c = cb + t;
      const bool live = c < r && c < i0 + nbw;  // columns right of the panel's last row are zero in it
      double sum[kCB];
#pragma unroll
      for (int ii = 0; ii < kCB; ++ii) sum[ii] = 0.0;
      for (int k0 = 0; k0 < i0; k0 += kCB) {
        __syncthreads();
        for (int e = t; e < kCB * kCB; e += nt) {
          const int ii = e / kCB, kk = e - ii * kCB;
          tile[ii][kk] = ii < nbw ? (double)Lt[(long long)(k0 + kk) * r + i0 + ii] : 0.0;
        }
        __syncthreads();
        if (live && c < k0 + kCB) {  // X[k][c] = 0 for k < c
#pragma unroll 4
          for (int kk = 0; kk < kCB; ++kk) {
            const double x = (double)X[(long long)(k0 + kk) * r + c];
#pragma unroll
            for (int ii = 0; ii < kCB; ++ii) sum[ii] += tile[ii][kk] * x;
          }
        }
      }
      __syncthreads();
      for (int e = t; e < kCB * kCB; e += nt) {
        const int ii = e / kCB, p = e - ii * kCB;
        dblk[ii][p] = (ii < nbw && p <= ii) ? Lt[(long long)(i0 + p) * r + i0 + ii] : 0.f;
      }
      __syncthreads();
      if (live) {
        float xs[kCB];
#pragma unroll
        for (int ii = 0; ii < kCB; ++ii) {
          xs[ii] = 0.f;
          if (ii < nbw) {
            const int i = i0 + ii;
            double s = sum[ii];
#pragma unroll
            for (int p = 0; p < ii; ++p) s += (double)dblk[ii][p] * (double)xs[p];
            xs[ii] = i < c ? 0.f : (float)(((i == c ? 1.0 : 0.0) - s) / (double)dblk[ii][ii]);
            X[(long long)i * r + c] = xs[ii];
          }
        }
      }
    }
  }
  __syncthreads();
  // R^-1 = (L^-1)^T : transpose X through Lt's storage (the factor is no longer needed)
  for (long long e = t; e < (long long)r * r; e += nt) Lt[e] = X[e];
  __syncthreads();
  for (long long e = t; e < (long long)r * r; e += nt) {
    const int i = (int)(e / r), c = (int)(e - (long long)i * r);
    X[e] = Lt[(long long)c * r + i];
  }
}

// ---------------------------------------------------------------------------------------------
// Parallel cyclic Jacobi eigen-solver of a small symmetric matrix + the projector it is wanted for.
// A sweep is w - 1 steps (w made even with a dummy index); a step rotates w/2 disjoint index pairs
// (round-robin tournament order). Rotations of disjoint pairs commute, so a step is
//   C <- J^T C J,  V^T <- J^T V^T,  J = product of the step's plane rotations,
// done pair by pair: a warp forms rows p and q of J^T C from the old rows p and q (coalesced reads),
// keeps them in shared memory, applies the column rotations there and writes the two new rows.
// Old and new matrices are separate buffers, swapped after every step.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) jacobi_projector_kernel(const EigProblem* __restrict__ probs) {
  extern __shared__ float jsm[];
  const EigProblem pb = probs[blockIdx.x];
  const int w = pb.w, r = pb.r;
  const int we = (w + 1) & ~1;           // even number of players
  float* cc = jsm;                       // [we] own-row coefficient
  float* ss = cc + we;                   // [we] partner-row coefficient
  int* partner = reinterpret_cast<int*>(ss + we);  // [we]
  float* rowbuf = reinterpret_cast<float*>(partner + we);  // [16][2][w]
  __shared__ double red[16];
  __shared__ int done_s;
  const int t = threadIdx.x, lane = t & 31, wp = t >> 5;
  float* Ca = pb.C;
  float* Cb = pb.work;
  float* Va = pb.work + (long long)w * w;
  float* Vb = pb.work + 2LL * w * w;
  for (long long e = t; e < (long long)w * w; e += 512) Va[e] = (e / w == e % w) ? 1.f : 0.f;  // V^T = I
  __syncthreads();

  for (int sweep = 0; sweep < 14; ++sweep) {
    // off-diagonal and diagonal weight: stop when the matrix is diagonal to fp32 accuracy
    double off = 0.0, dg = 0.0;
    for (long long e = t; e < (long long)w * w; e += 512) {
      const double x = (double)Ca[e];
      if (e / w == e % w) dg += x * x; else off += x * x;
    }
    for (int o = 16; o > 0; o >>= 1) { off += __shfl_xor_sync(0xffffffffu, off, o); dg += __shfl_xor_sync(0xffffffffu, dg, o); }
    if (lane == 0) red[wp] = off;
    __syncthreads();
    if (t == 0) { double s0 = 0.0; for (int k = 0; k < 16; ++k) s0 += red[k]; red[0] = s0; }
    __syncthreads();
    const double off_all = red[0];
    __syncthreads();
    if (lane == 0) red[wp] = dg;
    __syncthreads();
    if (t == 0) { double s0 = 0.0; for (int k = 0; k < 16; ++k) s0 += red[k]; done_s = off_all <= 1e-14 * (double)w * (double)w * s0; }
    __syncthreads();
    if (done_s) break;

    for (int step = 0; step < we - 1; ++step) {
      // ---- rotations of this step's pairs
      for (int k = t; k < we / 2; k += 512) {
        const int p = (step + k) % (we - 1);
        const int q = (k == 0) ? we - 1 : (step + we - 1 - k) % (we - 1);
        float c = 1.f, s = 0.f;
        if (p < w && q < w) {
          const double apq = (double)Ca[(long long)p * w + q];
          if (apq != 0.0) {
            const double app = (double)Ca[(long long)p * w + p], aqq = (double)Ca[(long long)q * w + q];
            const double theta = (aqq - app) / (2.0 * apq);
            const double tt = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
            const double cd = 1.0 / sqrt(tt * tt + 1.0);
            c = (float)cd; s = (float)(tt * cd);
          }
        }
        // new row p = c row p - s row q ; new row q = s row p + c row q
        if (p < we) { partner[p] = q; cc[p] = c; ss[p] = -s; }
        if (q < we) { partner[q] = p; cc[q] = c; ss[q] = s; }
      }
      __syncthreads();
      // ---- rows of J^T C J and of J^T V^T, a pair of rows per warp: both new rows come from the same two
      // old rows, which are read once
      float* rbp = rowbuf + wp * 2 * w;
      float* rbq = rbp + w;
      for (int k = wp; k < we / 2; k += 16) {
        int p = (step + k) % (we - 1);
        int q = (k == 0) ? we - 1 : (step + we - 1 - k) % (we - 1);
        float c = cc[p], sn = -ss[p];  // new row p = c row p - sn row q ; new row q = sn row p + c row q
        const bool single = q >= w || p >= w;  // paired with the dummy index: the row is copied
        if (p >= w) p = q;
        if (single) { q = p; c = 1.f; sn = 0.f; }
#pragma unroll 4
        for (int j = lane; j < w; j += 32) {
          const float cp = Ca[(long long)p * w + j], cq = Ca[(long long)q * w + j];
          const float vp = Va[(long long)p * w + j], vq = Va[(long long)q * w + j];
          rbp[j] = c * cp - sn * cq;
          rbq[j] = sn * cp + c * cq;
          Vb[(long long)p * w + j] = c * vp - sn * vq;
          if (!single) Vb[(long long)q * w + j] = sn * vp + c * vq;
        }
        __syncwarp();
#pragma unroll 4
        for (int j = lane; j < w; j += 32) {
          int pj = partner[j];
          float cj = cc[j], sj = ss[j];
          if (pj >= w) { pj = j; cj = 1.f; sj = 0.f; }
          Cb[(long long)p * w + j] = cj * rbp[j] + sj * rbp[pj];
          if (!single) Cb[(long long)q * w + j] = cj * rbq[j] + sj * rbq[pj];
        }
        __syncwarp();
      }
      __syncthreads();
      float* x = Ca; Ca = Cb; Cb = x;
      x = Va; Va = Vb; Vb = x;
    }
  }
  __syncthreads();
  // ---- eigenvalues = diagonal of Ca; rank of each (0 = largest), kept in `partner`
  for (int i = t; i < w; i += 512) {
    const float li = Ca[(long long)i * w + i];
    int rk = 0;
    for (int j = 0; j < w; ++j) {
      const float lj = Ca[(long long)j * w + j];
      rk += (lj > li || (lj == li && j < i)) ? 1 : 0;
    }
    partner[i] = rk;
  }
  __syncthreads();
  // ---- Mr[a][b] = sum over the r leading eigenvectors v of v[a] v[b], b < r  (rows of V^T are eigenvectors)
  for (long long e = t; e < (long long)w * r; e += 512) {
    const int a = (int)(e / r), b = (int)(e - (long long)a * r);
    double acc = 0.0;
    for (int i = 0; i < w; ++i)
      if (partner[i] < r) acc += (double)Va[(long long)i * w + a] * (double)Va[(long long)i * w + b];
    pb.Mr[e] = (float)acc;
  }
}

void launch_jacobi_projector(const EigProblem* probs, int nprobs, int w_max, cudaStream_t st) {
  const int we = (w_max + 1) & ~1;
  const size_t smem = sizeof(float) * (size_t)(3 * we + 32 * w_max);
  static bool configured = false;  // w <= 600 (checked at init): at most 84 KB
  if (!configured) {
    cudaFuncSetAttribute(jacobi_projector_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(float) * (3 * 600 + 32 * 600)));
    configured = true;
  }
  jacobi_projector_kernel<<<nprobs, 512, smem, st>>>(probs);
}

void launch_chol_inverse(const CholProblem* probs, int nprobs, int r_max, unsigned* status, cudaStream_t st) {
  (void)r_max;
  chol_inverse_kernel<<<nprobs, 512, 0, st>>>(probs, status);
}

}  // namespace lordo
