// Streaming (HBM-bound) kernels of the LoRDO hot path: clip norm, low-rank moment update,
// outer synchronisation, sketch generator. All grouped over the whole list of matrices.
#include "lordo_kernels.h"

namespace lordo {

// ---------------------------------------------------------------------------------------------
// Clip coefficient (Algorithm 1, line "clip"): c = min(1, rho / (||G_k||_2 + 1e-6))
// Pass 1: one partial sum of squares per block of kSqChunk elements. Pass 2: fixed-order sum.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) sumsq_partial_kernel(const MatDev* __restrict__ mats, const void* const* __restrict__ G,
                                                            const long long* __restrict__ chunk_start, int n_mats, int K,
                                                            int g_dt, double* __restrict__ partial) {
  const long long blk = blockIdx.x;
  const int i = find_segment(chunk_start, n_mats, blk);
  const long long elems = mats[i].m * mats[i].n;
  const long long chunks = (elems + kSqChunk - 1) / kSqChunk;
  const long long local = blk - chunk_start[i];
  const int k = (int)(local / chunks);
  const long long c = local - (long long)k * chunks;
  const long long begin = c * kSqChunk;
  long long end = begin + kSqChunk;
  if (end > elems) end = elems;
  const void* g = G[i];
  const long long base = (long long)k * elems;
  float acc = 0.f;
  for (long long e = begin + 4ll * threadIdx.x; e < end; e += 4ll * 256) {  // elems is a multiple of 8
    float4 x = load4(g, g_dt, base + e);
    acc += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
  }
  double d = (double)acc;
  for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
  __shared__ double warp_sum[8];
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = d;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += warp_sum[w];
    partial[blk] = s;
  }
}

// Step 1: one block per (matrix, replica) sums that pair's partials in a fixed order.
__global__ void __launch_bounds__(256) clip_matrix_sums_kernel(const MatDev* __restrict__ mats, const long long* __restrict__ chunk_start,
                                                               int K, const double* __restrict__ partial, float rho, int scope,
                                                               float* __restrict__ coef, double* __restrict__ sumsq) {
  const int i = blockIdx.x, k = blockIdx.y;
  __shared__ double red[256];
  const long long elems = mats[i].m * mats[i].n;
  const long long chunks = (elems + kSqChunk - 1) / kSqChunk;
  const double* p = partial + chunk_start[i] + (long long)k * chunks;
  double a = 0.0;
  for (long long c = threadIdx.x; c < chunks; c += 256) a += p[c];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double s_i = red[0];
    sumsq[(long long)i * K + k] = s_i;
    if (scope == 1) coef[(long long)i * K + k] = fminf(1.f, rho / ((float)sqrt(s_i) + 1e-6f));
  }
}

// Step 2: one block per replica adds the matrices' sums in matrix order (thread 0, so the order
// is fixed) and writes the coefficient of the per-worker norm.
__global__ void __launch_bounds__(256) clip_finalize_kernel(int n_mats, int K, float rho, int scope, float* __restrict__ coef,
                                                            const double* __restrict__ sumsq, unsigned* __restrict__ status) {
  const int k = blockIdx.x;
  __shared__ float c_s;
  if (threadIdx.x == 0) {
    double total = 0.0;
    for (int i = 0; i < n_mats; ++i) total += sumsq[(long long)i * K + k];
    if (!isfinite(total)) atomicOr(status, LORDO_FLAG_NONFINITE_GRAD);
    c_s = fminf(1.f, rho / ((float)sqrt(total) + 1e-6f));
  }
  __syncthreads();
  if (scope == 0)
    for (int i = threadIdx.x; i < n_mats; i += 256) coef[(long long)i * K + k] = c_s;
}

__global__ void fill_float_kernel(float* __restrict__ p, long long count, float value) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) p[i] = value;
}

// ---------------------------------------------------------------------------------------------
// Low-rank moment update (Algorithm 1: u, v lines and the bracket of the update cases).
//   u <- b1 u + (1-b1) g ; v <- b2 v + (1-b2) g*g ; u^ = u/(1-b1^s) ; v^ = v/(1-b2^s)
//   D = sqrt(v^) + eps ; U~ = u^/D (no / full-rank QHM) or (w u^ + (1-w) g)/D (low-rank QHM)
//   full-rank QHM also needs mu(D) = mean over the rank axis, one value per column.
// One block = 128 columns of one (matrix, replica); threadIdx.y strides over the r rows.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) moments_kernel(const MatDev* __restrict__ mats, const long long* __restrict__ tile_start,
                                                      int n_mats, StepScalars sc) {
  const long long blk = blockIdx.x;
  const int i = find_segment(tile_start, n_mats, blk);
  const MatDev md = mats[i];
  const long long n = md.ln;  // columns of the low-rank arrays
  const int r = md.r;
  const long long ctiles = (n + 127) / 128;
  const long long local = blk - tile_start[i];
  const int k = (int)(local / ctiles);
  const long long col = (local - (long long)k * ctiles) * 128 + 4ll * threadIdx.x;
  const bool active = col < n;
  const long long base = (long long)k * r * n + col;
  const float b1 = sc.beta1, b2 = sc.beta2, w = sc.omega;
  float dsum0 = 0.f, dsum1 = 0.f, dsum2 = 0.f, dsum3 = 0.f;
  if (active) {
#pragma unroll 2
    for (int a = threadIdx.y; a < r; a += 8) {
      const long long idx = base + (long long)a * n;
      const float4 g = *reinterpret_cast<const float4*>(md.ghat + idx);
      float4 u = *reinterpret_cast<const float4*>(md.u + idx);
      float4 v = *reinterpret_cast<const float4*>(md.v + idx);
      float4 o;
#define LORDO_MOM(c)                                                              \
  {                                                                               \
    u.c = b1 * u.c + (1.f - b1) * g.c;                                            \
    v.c = b2 * v.c + (1.f - b2) * g.c * g.c;                                      \
    const float uh = u.c * sc.inv_bc1;                                            \
    const float D = sqrtf(v.c * sc.inv_bc2) + sc.eps;                             \
    o.c = (sc.form == LORDO_QHM_LOW) ? (w * uh + (1.f - w) * g.c) / D : uh / D;   \
    dsum_##c += D;                                                                \
  }
      float dsum_x = 0.f, dsum_y = 0.f, dsum_z = 0.f, dsum_w = 0.f;
      LORDO_MOM(x) LORDO_MOM(y) LORDO_MOM(z) LORDO_MOM(w)
#undef LORDO_MOM
      dsum0 += dsum_x; dsum1 += dsum_y; dsum2 += dsum_z; dsum3 += dsum_w;
      *reinterpret_cast<float4*>(md.u + idx) = u;
      *reinterpret_cast<float4*>(md.v + idx) = v;
      *reinterpret_cast<float4*>(md.util + idx) = o;
      if (md.T) {  // up-link time buffer
        float4 tb = *reinterpret_cast<const float4*>(md.T + idx);
        tb.x += sc.lr * o.x; tb.y += sc.lr * o.y; tb.z += sc.lr * o.z; tb.w += sc.lr * o.w;
        *reinterpret_cast<float4*>(md.T + idx) = tb;
      }
    }
  }
  if (sc.form == LORDO_QHM_FULL) {  // uniform over the grid
    __shared__ float4 red[8][32];
    red[threadIdx.y][threadIdx.x] = make_float4(dsum0, dsum1, dsum2, dsum3);
    __syncthreads();
    if (threadIdx.y == 0 && active) {
      float4 s = red[0][threadIdx.x];
      for (int y = 1; y < 8; ++y) {
        const float4 t = red[y][threadIdx.x];
        s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
      }
      const float inv_r = 1.f / (float)r;
      s.x *= inv_r; s.y *= inv_r; s.z *= inv_r; s.w *= inv_r;
      *reinterpret_cast<float4*>(md.dcol + (long long)k * n + col) = s;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Outer synchronisation (Algorithm 1, synchronisation lines; appendix "Unrolled low-rank
// updates": Delta = old - new, theta <- theta - eta_s Delta).
// One thread = 4 consecutive weights of one matrix, all K replicas.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) outer_weights_kernel(const MatDev* __restrict__ mats, const long long* __restrict__ blk_start,
                                                            int n_mats, int K, int w_dt, int outer, float eta_s, float mu_s,
                                                            float delta_scale) {
  const long long blk = blockIdx.x;
  const int i = find_segment(blk_start, n_mats, blk);
  const MatDev md = mats[i];
  const long long elems = md.m * md.n;
  const long long e = ((blk - blk_start[i]) * 256 + threadIdx.x) * 4;
  if (e >= elems) return;
  const float4 x0 = *reinterpret_cast<const float4*>(md.X0 + e);
  float4 d, xn;
  if (delta_scale != 0.f) {  // the pseudo-gradient was rebuilt from the time buffers into Delta
    d = *reinterpret_cast<const float4*>(md.Delta + e);
    d.x *= delta_scale; d.y *= delta_scale; d.z *= delta_scale; d.w *= delta_scale;
  } else {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int k = 0; k < K; ++k) {
      const float4 w = load4(md.W, w_dt, (long long)k * elems + e);
      s.x += w.x; s.y += w.y; s.z += w.z; s.w += w.w;
    }
    const float inv_k = 1.f / (float)K;
    d.x = x0.x - s.x * inv_k; d.y = x0.y - s.y * inv_k; d.z = x0.z - s.z * inv_k; d.w = x0.w - s.w * inv_k;
  }
  if (outer == LORDO_OUTER_NESTEROV) {
    float4 b = *reinterpret_cast<const float4*>(md.B + e);
    b.x = mu_s * b.x + d.x; b.y = mu_s * b.y + d.y; b.z = mu_s * b.z + d.z; b.w = mu_s * b.w + d.w;
    *reinterpret_cast<float4*>(md.B + e) = b;
    xn.x = x0.x - eta_s * (d.x + mu_s * b.x); xn.y = x0.y - eta_s * (d.y + mu_s * b.y);
    xn.z = x0.z - eta_s * (d.z + mu_s * b.z); xn.w = x0.w - eta_s * (d.w + mu_s * b.w);
  } else {
    xn.x = x0.x - d.x; xn.y = x0.y - d.y; xn.z = x0.z - d.z; xn.w = x0.w - d.w;
  }
  *reinterpret_cast<float4*>(md.Delta + e) = d;
  *reinterpret_cast<float4*>(md.X0 + e) = xn;
#pragma unroll 4
  for (int k = 0; k < K; ++k) store4(md.W, w_dt, (long long)k * elems + e, xn);
}

// u, v <- mean over replicas (Algorithm 1, "Sync u / v" lines). which: bit 0 = u, bit 1 = v,
// bit 2 = the time buffers (Global rule: one basis, so their mean is all the rebuilt pseudo-gradient needs).
__global__ void __launch_bounds__(256) outer_states_kernel(const MatDev* __restrict__ mats, const long long* __restrict__ blk_start,
                                                           int n_mats, int K, int which) {
  const long long blk = blockIdx.x;
  const int i = find_segment(blk_start, n_mats, blk);
  const MatDev md = mats[i];
  const long long elems = (long long)md.r * md.ln;
  const long long e = ((blk - blk_start[i]) * 256 + threadIdx.x) * 4;
  if (e >= elems) return;
  const float inv_k = 1.f / (float)K;
  for (int t = 0; t < 3; ++t) {
    if (!((which >> t) & 1)) continue;
    float* p = t == 0 ? md.u : (t == 1 ? md.v : md.T);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int k = 0; k < K; ++k) {
      const float4 x = *reinterpret_cast<const float4*>(p + (long long)k * elems + e);
      s.x += x.x; s.y += x.y; s.z += x.z; s.w += x.w;
    }
    s.x *= inv_k; s.y *= inv_k; s.z *= inv_k; s.w *= inv_k;
#pragma unroll 4
    for (int k = 0; k < K; ++k) *reinterpret_cast<float4*>(p + (long long)k * elems + e) = s;
  }
}

// ---------------------------------------------------------------------------------------------
// init helpers
// ---------------------------------------------------------------------------------------------
// Copies W[0] to replicas 1..K-1 and to X0 (fp32).
__global__ void __launch_bounds__(256) init_weights_kernel(const MatDev* __restrict__ mats, const long long* __restrict__ blk_start,
                                                           int n_mats, int K, int w_dt) {
  const long long blk = blockIdx.x;
  const int i = find_segment(blk_start, n_mats, blk);
  const MatDev md = mats[i];
  const long long elems = md.m * md.n;
  const long long e = ((blk - blk_start[i]) * 256 + threadIdx.x) * 4;
  if (e >= elems) return;
  const float4 w = load4(md.W, w_dt, e);
  *reinterpret_cast<float4*>(md.X0 + e) = w;
  for (int k = 1; k < K; ++k) store4(md.W, w_dt, (long long)k * elems + e, w);
}

__global__ void identity_projection_kernel(float* __restrict__ P, long long m, int r, int copies) {
  const long long total = m * r * copies;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const long long within = idx % (m * r);
  const long long row = within / r;
  const int col = (int)(within - row * r);
  P[idx] = (row == col) ? 1.f : 0.f;
}

// out[c] = popcount(mix64(key + golden*(c+1))) - 32 ; batch entry b uses keys[b].
__global__ void __launch_bounds__(256) fill_random_kernel(float* __restrict__ out, long long count, long long batch_stride,
                                                          RandomKeys keys) {
  const long long c = (long long)blockIdx.x * 256 + threadIdx.x;
  if (c >= count) return;
  const unsigned long long w = mix64(keys.key[blockIdx.y] + kGolden * (unsigned long long)(c + 1));
  out[(long long)blockIdx.y * batch_stride + c] = (float)(__popcll(w) - 32);
}

// The same generator for many matrices in one launch; the key of each is derived on the device.
__global__ void __launch_bounds__(256) fill_random_grouped_kernel(const RandProblem* __restrict__ probs, int nprobs,
                                                                  unsigned long long seed, long long index) {
  const long long blk = blockIdx.x;
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].blk_start <= blk) lo = mid; else hi = mid - 1;
  }
  const RandProblem pb = probs[lo];
  const long long c0 = ((blk - pb.blk_start) * 256 + threadIdx.x) * 8;  // eight consecutive entries per thread (count is a multiple of 8)
  if (c0 >= pb.count) return;
  const unsigned long long key = stream_key(seed, pb.purpose, pb.mat, index, pb.replica);
  float val[8];
#pragma unroll
  for (int x = 0; x < 8; ++x) val[x] = (float)(__popcll(mix64(key + kGolden * (unsigned long long)(c0 + x + 1))) - 32);
  if (pb.out) {
    *reinterpret_cast<float4*>(pb.out + c0) = make_float4(val[0], val[1], val[2], val[3]);
    *reinterpret_cast<float4*>(pb.out + c0 + 4) = make_float4(val[4], val[5], val[6], val[7]);
  }
  if (pb.out16) {  // integers in [-32, 32]: exact in bf16
    store4(pb.out16, LORDO_BF16, c0, make_float4(val[0], val[1], val[2], val[3]));
    store4(pb.out16, LORDO_BF16, c0 + 4, make_float4(val[4], val[5], val[6], val[7]));
  }
}

// fp32 -> bf16 copies of many buffers in one launch (operands of the tensor-core sketch products)
__device__ __forceinline__ void split_store4(__nv_bfloat16* dst, long long plane, int planes, long long e, float4 v) {
  for (int p = 0; p < planes; ++p) {
    const float4 h = make_float4(__bfloat162float(__float2bfloat16_rn(v.x)), __bfloat162float(__float2bfloat16_rn(v.y)),
                                 __bfloat162float(__float2bfloat16_rn(v.z)), __bfloat162float(__float2bfloat16_rn(v.w)));
    store4(dst + p * plane, LORDO_BF16, e, h);
    v = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);  // exact: the residual of a rounding to 8 bits
  }
}

__global__ void __launch_bounds__(256) convert_grouped_kernel(const ConvProblem* __restrict__ probs, int nprobs, float inv_bc1, float inv_bc2,
                                                              float bc1, float bc2) {
  const long long blk = blockIdx.x;
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].blk_start <= blk) lo = mid; else hi = mid - 1;
  }
  const ConvProblem pb = probs[lo];
  const long long e = ((blk - pb.blk_start) * 256 + threadIdx.x) * 4;  // count is a multiple of 8
  if (e >= pb.count) return;
  if (pb.mode == CONV_ROT_T) {  // element e of the transposed matrix: (k, j) <- Rot[j][k]
    float t[4];
    for (int x = 0; x < 4; ++x) {
      const long long k = (e + x) / pb.ld, j = (e + x) - k * pb.ld;
      t[x] = pb.src[j * pb.ld + k];
    }
    split_store4(pb.dst, pb.plane, pb.planes, e, make_float4(t[0], t[1], t[2], t[3]));
    split_store4(pb.dst2, pb.plane, pb.planes, e, make_float4(t[0] * t[0], t[1] * t[1], t[2] * t[2], t[3] * t[3]));
    return;
  }
  const float4 v = *reinterpret_cast<const float4*>(pb.src + e);
  if (pb.mode == CONV_BF16) {
    store4(pb.dst, LORDO_BF16, e, v);
  } else if (pb.mode == CONV_SPLIT) {
    split_store4(pb.dst, pb.plane, pb.planes, e, v);
  } else if (pb.mode == CONV_STATES) {
    const float4 w = *reinterpret_cast<const float4*>(pb.src2 + e);
    const float4 uh = make_float4(inv_bc1 * v.x, inv_bc1 * v.y, inv_bc1 * v.z, inv_bc1 * v.w);
    split_store4(pb.dst, pb.plane, pb.planes, e, uh);
    split_store4(pb.dst2, pb.plane, pb.planes, e,
                 make_float4(inv_bc2 * w.x - uh.x * uh.x, inv_bc2 * w.y - uh.y * uh.y, inv_bc2 * w.z - uh.z * uh.z, inv_bc2 * w.w - uh.w * uh.w));
  } else {  // CONV_COMBINE
    const float4 w = *reinterpret_cast<const float4*>(pb.src2 + e);
    *reinterpret_cast<float4*>(pb.outf + e) = make_float4(bc1 * v.x, bc1 * v.y, bc1 * v.z, bc1 * v.w);
    *reinterpret_cast<float4*>(pb.outf2 + e) = make_float4(bc2 * fabsf(w.x + v.x * v.x), bc2 * fabsf(w.y + v.y * v.y),
                                                           bc2 * fabsf(w.z + v.z * v.z), bc2 * fabsf(w.w + v.w * v.w));
  }
}

__global__ void __launch_bounds__(256) colnorm_grouped_kernel(const NormProblem* __restrict__ probs, int nprobs) {
  __shared__ double part[8][32];
  const long long blk = blockIdx.x;
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].blk_start <= blk) lo = mid; else hi = mid - 1;
  }
  const NormProblem pb = probs[lo];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int col = (int)(blk - pb.blk_start) * 32 + lane;
  const bool live = col < pb.r;
  double s = 0.0;
  if (live)
    for (int row = w; row < pb.rows; row += 8) {
      const float x = pb.X[(long long)row * pb.r + col];
      s += (double)x * (double)x;
    }
  part[w][lane] = s;
  __syncthreads();
  if (w == 0) {
    double t = 0.0;
    for (int k = 0; k < 8; ++k) t += part[k][lane];
    part[0][lane] = t > 0.0 ? 1.0 / sqrt(t) : 1.0;
  }
  __syncthreads();
  const float sc = (float)part[0][lane];
  if (live)
    for (int row = w; row < pb.rows; row += 8) pb.X[(long long)row * pb.r + col] *= sc;
}

// Device-to-device copies of many buffers in one launch (16-byte chunks).
__global__ void __launch_bounds__(256) copy_grouped_kernel(const CopyProblem* __restrict__ probs, int nprobs) {
  const long long blk = blockIdx.x;
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].blk_start <= blk) lo = mid; else hi = mid - 1;
  }
  const CopyProblem pb = probs[lo];
  const long long c = ((blk - pb.blk_start) * 256 + threadIdx.x) * 4;
  const uint4* __restrict__ src = reinterpret_cast<const uint4*>(pb.src);
  uint4* __restrict__ dst = reinterpret_cast<uint4*>(pb.dst);
  uint4 v[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (c + i < pb.chunks) v[i] = src[c + i];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (c + i < pb.chunks) dst[c + i] = v[i];
}

// Mean squared singular value of Rot = P'^T P (the paper's MSSV metric): the sum of the squared
// singular values of a matrix is its squared Frobenius norm. One block per rotation matrix.
__global__ void __launch_bounds__(256) mssv_kernel(const DiagProblem* __restrict__ probs, float* __restrict__ out) {
  const DiagProblem pb = probs[blockIdx.x];
  const long long count = (long long)pb.r * pb.r;
  double a = 0.0;
  for (long long e = threadIdx.x; e < count; e += 256) { const double x = (double)pb.rot[e]; a += x * x; }
  __shared__ double red[256];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[blockIdx.x] = (float)(red[0] / (double)pb.r);
}

// ||E||_F of one (matrix, worker) per block.
__global__ void __launch_bounds__(256) error_norms_kernel(const MatDev* __restrict__ mats, int K, int e_dt, float* __restrict__ out) {
  const int i = blockIdx.x, k = blockIdx.y;
  const long long elems = mats[i].m * mats[i].n;
  const void* E = mats[i].E;
  double a = 0.0;
  for (long long e = 4ll * threadIdx.x; e < elems; e += 4ll * 256) {  // elems is a multiple of 8
    const float4 x = load4(E, e_dt, (long long)k * elems + e);
    a += (double)(x.x * x.x + x.y * x.y) + (double)(x.z * x.z + x.w * x.w);
  }
  __shared__ double red[256];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[(long long)i * K + k] = (float)sqrt(red[0]);
}

// ---------------------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------------------
void launch_mssv(const DiagProblem* probs, int nprobs, float* out, cudaStream_t st) { mssv_kernel<<<nprobs, 256, 0, st>>>(probs, out); }
void launch_error_norms(const MatDev* mats, int n_mats, int K, int e_dt, float* out, cudaStream_t st) {
  error_norms_kernel<<<dim3(n_mats, K), 256, 0, st>>>(mats, K, e_dt, out);
}
void launch_fill_random_grouped(const RandProblem* probs, int nprobs, long long total_blocks, unsigned long long seed, long long index,
                                cudaStream_t st) {
  fill_random_grouped_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(probs, nprobs, seed, index);
}
void launch_convert_grouped(const ConvProblem* probs, int nprobs, long long total_blocks, const GemmScalars& sc, cudaStream_t st) {
  convert_grouped_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(probs, nprobs, sc.inv_bc1, sc.inv_bc2, sc.bc1, sc.bc2);
}
void launch_colnorm_grouped(const NormProblem* probs, int nprobs, long long total_blocks, cudaStream_t st) {
  colnorm_grouped_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(probs, nprobs);
}
void launch_copy_grouped(const CopyProblem* probs, int nprobs, long long total_blocks, cudaStream_t st) {
  copy_grouped_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(probs, nprobs);
}
void launch_sumsq_partial(const MatDev* mats, const void* const* G, const long long* chunk_start, int n_mats, int K, int g_dt,
                          double* partial, long long total_chunks, cudaStream_t st) {
  sumsq_partial_kernel<<<(unsigned)total_chunks, 256, 0, st>>>(mats, G, chunk_start, n_mats, K, g_dt, partial);
}
void launch_clip_finalize(const MatDev* mats, const long long* chunk_start, int n_mats, int K, const double* partial, float rho,
                          int scope, float* coef, double* sumsq, unsigned* status, cudaStream_t st) {
  clip_matrix_sums_kernel<<<dim3(n_mats, K), 256, 0, st>>>(mats, chunk_start, K, partial, rho, scope, coef, sumsq);
  clip_finalize_kernel<<<K, 256, 0, st>>>(n_mats, K, rho, scope, coef, sumsq, status);
}
void launch_fill_float(float* p, long long count, float value, cudaStream_t st) {
  fill_float_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(p, count, value);
}
void launch_moments(const MatDev* mats, const long long* tile_start, int n_mats, long long total_tiles, const StepScalars& sc,
                    cudaStream_t st) {
  moments_kernel<<<(unsigned)total_tiles, dim3(32, 8), 0, st>>>(mats, tile_start, n_mats, sc);
}
void launch_outer_weights(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int w_dt,
                          int outer, float eta_s, float mu_s, float delta_scale, cudaStream_t st) {
  outer_weights_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(mats, blk_start, n_mats, K, w_dt, outer, eta_s, mu_s, delta_scale);
}
void launch_outer_states(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int which,
                         cudaStream_t st) {
  outer_states_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(mats, blk_start, n_mats, K, which);
}
void launch_init_weights(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int w_dt,
                         cudaStream_t st) {
  init_weights_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(mats, blk_start, n_mats, K, w_dt);
}
void launch_identity_projection(float* P, long long m, int r, int copies, cudaStream_t st) {
  const long long total = m * r * copies;
  identity_projection_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(P, m, r, copies);
}
void launch_fill_random(float* out, long long count, long long batch_stride, const RandomKeys& keys, int batch, cudaStream_t st) {
  fill_random_kernel<<<dim3((unsigned)((count + 255) / 256), batch), 256, 0, st>>>(out, count, batch_stride, keys);
}

}  // namespace lordo
