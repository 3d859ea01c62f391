// Internal interface between the host layer (lordo_api.cu) and the kernel files.
#pragma once
#include "lordo_common.cuh"

namespace lordo {

constexpr long long kSqChunk = 32768;  // elements per partial sum of squares

struct RandomKeys {
  unsigned long long key[64];
};

// ---------------------------------------------------------------------------------------------
// Grouped fp32 GEMM with fused operand formation and epilogues (FFMA path).
//   C[M x N] = A[M x Kd] * B[Kd x N]        (+ second accumulator: A' * B2, A' = A or A o A)
// B, B2 are stored row-major [Kd][N]. A is stored [M][Kd] (ATRANS = 0) or [Kd][M] (ATRANS = 1).
// ---------------------------------------------------------------------------------------------
enum OperandKind {
  OP_PLAIN = 0,  // (*s0_ptr) * p0[idx] + p1[idx]        (s0_ptr, p1 optional)
  OP_UHAT = 1,   // inv_bc1 * p0[idx]                      bias-corrected first moment
  OP_VRES = 2    // inv_bc2 * p1[idx] - (inv_bc1 * p0[idx])^2
};

struct Operand {
  const void* p0;
  const void* const* p0_ind;  // if set: p0 = *p0_ind (a per-call pointer table entry)
  long long p0_off;           // element offset added to p0
  const void* p1;
  const float* s0_ptr;
  long long ld;
  int dt0, dt1, kind, pad;
};

enum EpilogueKind { EPI_STORE = 0, EPI_APPLY = 1, EPI_ROTATE = 2 };

struct Epilogue {
  int kind, pad;
  float* C;         // STORE: C[row*ldc + col] = acc (pad != 0: += acc)
  long long ldc;
  // APPLY (Algorithm 1: error-feedback line and the model update), row = weight row, col = column
  void* W;
  void* E;
  const void* const* G_ind;
  long long G_off;
  const float* dcol;
  const float* cptr;
  // ROTATE (Algorithm 1: moment-rotation lines)
  float* u_out;
  float* v_out;
  // STORE and APPLY, a matrix projected from the right: output element (row, col) belongs to memory
  // element col * ldt + row (the product is formed for the transposed problem). STORE: ldt = ldc.
  int trans, pad2;
  long long ldt;
};

struct GemmProblem {
  int M, N, Kd, tiles_n;
  long long tile_start;  // first tile of this problem within its launch
  Operand A, B, B2;
  Epilogue epi;
};

struct GemmScalars {
  float lr, omega, inv_bc1, inv_bc2, bc1, bc2;
  int form, ef, w_dt, e_dt, g_dt, a_square;
};

void launch_gemm(const GemmProblem* probs, int nprobs, long long total_tiles, int atrans, int dual, int carry, const GemmScalars& sc,
                 cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Tensor-core path of the inner step (bf16 operands, fp32 accumulation), see lordo_tc.cu.
// One TcProblem per (matrix, worker); a launch covers `strips` 128-column strips in total.
// ---------------------------------------------------------------------------------------------
struct TcProblem {
  long long strip_start;       // first strip of this problem within the launch
  int m, n, r;
  int r_k;                     // r rounded up to 64: k extent of P16, gT16, uT16
  int r_n;                     // r rounded up to 16: rows of PT16
  int m_k;                     // m rounded up to 64: k extent of PT16, rows of P16
  const __nv_bfloat16* PT16;   // [r_n][m_k]  P^T, zero padded
  const __nv_bfloat16* P16;    // [m_k][r_k]  P, zero padded
  // Low-rank gradient and normalised low-rank update U~, transposed, private to the projection and
  // update kernels of one path. Register-staged kernels: [n][r_k]. TMA-fed kernels:
  // [strip][r_k/8][128 columns][8], i.e. the 16-byte pieces of one k-chunk of a strip's columns lie
  // side by side and a warp moves 512 contiguous bytes. Room for ceil(n/128)*128 columns either way.
  __nv_bfloat16* gT16;
  __nv_bfloat16* uT16;
  float* u;                    // [r][n] of this worker
  float* v;
  float* dcol;                 // [n]
  void* W;                     // [m][n] of this worker
  void* E;
  const void* const* G_ind;    // entry of the per-call gradient pointer table
  long long G_off;             // element offset of this worker inside it
  const float* cptr;           // clip coefficient
  int mat, replica, pcopy;     // matrix index, worker index, which copy of P (0 for Global)
  int tr;                      // 1: W, G, E are stored transposed with respect to this problem (a matrix projected from the
                               // right): m counts their columns, n their rows
  float* tb;                   // [r][n] time buffer of this worker (+= lr * U~ every step), or null
  // the projection's own numbering, in CTA pairs: nsplit pairs per 256 columns (2 when 256 < r <= 512: one
  // per half of the rank), and the second half's share of the column scale of the full-rank QHM term
  long long strip_start_p;
  float* dcol2;                // [n], or null when nsplit == 1
  int nsplit, pad2;
};

// Tensor maps (opaque 128-byte objects encoded on the host) of one matrix for the TMA-fed kernels.
// "sw": 64 x 64 boxes with the 128-byte swizzle (operands of the projection, and the tiles the update
// epilogue reads and writes in place); "st": 64 x 16 boxes with the same swizzle.
struct alignas(128) TmaMatMaps {
  unsigned char e_sw[128], pt[128], p16[128], w_sw[128];
  // a matrix projected from the right: W as 64 x 128 boxes, and stores of 32 rows of a 64-column tile
  unsigned char w_kb[128], e_st32[128], w_st32[128];
  // refresh: E and Delta16 as 64 x 128 swizzled boxes ("kb", rows of S as MMA rows), Delta16 as
  // 64 x 64 swizzled boxes, and the three bf16 right-hand sides [batch][Kd][r]
  unsigned char e_kb[128], d_kb[128], d_sw[128], om16[128], pn16[128], zq16[128];
  unsigned char e_st[128], w_st[128];  // stores of one row group of the update epilogue
  // refresh on tensor cores, all over hi|lo bf16 planes [2 x batch][rows][cols], 64 x 64 swizzled boxes
  // unless noted: the matrix being orthonormalised with m rows and with n rows (also as 64 x 128 boxes,
  // rows as MMA rows), R^-1, P, Rot^T, Rot^T o Rot^T, and the moment operands u^, v^ - u^ u^ as [r][n]
  unsigned char xm_sw[128], xm_kb[128], xn_sw[128], xn_kb[128], rinv_sw[128], phl_sw[128], rt_sw[128], sq_sw[128], uh_sw[128], wr_sw[128];
};
struct alignas(128) TmaGradMaps {  // re-encoded whenever the caller's gradient pointer changes
  unsigned char g_sw[128], g_kb[128];
};

struct TcPrep {
  const float* P;              // [m][r]
  __nv_bfloat16* P16;
  __nv_bfloat16* PT16;
  long long m;
  int r, r_k, m_k, pad;
};

cudaError_t tc_configure(int r_n_max, int r_k_max);
void launch_prep_projection(const TcPrep* items, const long long* blk_start, int nitems, long long total_blocks, cudaStream_t st);
// bf16 != 0: G, E, W are all bf16; else all fp32 (mixed storage runs on the fp32 path).
void launch_project_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_n_max, const StepScalars& sc, int bf16,
                       unsigned* status, cudaStream_t st);
void launch_apply_tc(const TcProblem* probs, int nprobs, long long total_strips, int r_k_max, const StepScalars& sc, int bf16,
                     unsigned* status, cudaStream_t st);

// TMA-fed persistent kernels for bf16 storage (lordo_tma.cu).
cudaError_t tma_configure();
void launch_project_tma(const TcProblem* probs, int nprobs, long long total_strips_p, const TmaMatMaps* maps, const TmaGradMaps* gmaps,
                        const StepScalars& sc, int grid, unsigned* status, cudaStream_t st);
// mode 0: r <= 256, one sweep; modes 1 and 2: the two sweeps for 256 < r <= 512. The launch covers the strips
// [strip_begin, strip_end) of `probs` (problems of one side only: tr = 0 stored as the problem, tr = 1 transposed).
void launch_apply_tma(const TcProblem* probs, int nprobs, long long strip_begin, long long strip_end, const TmaMatMaps* maps,
                      const TmaGradMaps* gmaps, const StepScalars& sc, int grid, int mode, int tr, unsigned* status, cudaStream_t st);

void launch_selftest_wait(unsigned* status, cudaStream_t st);

// Diagnostics: MSSV = ||Rot||_F^2 / r of every rotation matrix of the last refresh, and ||E||_F per
// (matrix, worker).
struct DiagProblem {
  const float* rot;  // r x r
  int r, pad;
};
void launch_mssv(const DiagProblem* probs, int nprobs, float* out, cudaStream_t st);
void launch_error_norms(const MatDev* mats, int n_mats, int K, int e_dt, float* out, cudaStream_t st);

// Cholesky factor of a batch of r x r Gram matrices and the inverse of its transpose:
// gram = R^T R (R upper triangular, positive diagonal); rinv = R^-1, row-major, zeros below the
// diagonal. lwork: r*r floats per problem. Strides in floats between batch entries.
struct CholProblem {
  const float* gram;
  float* lwork;
  float* rinv;
  int r, pad;
};
void launch_chol_inverse(const CholProblem* probs, int nprobs, int r_max, unsigned* status, cudaStream_t st);

// Rayleigh-Ritz truncation of an oversampled basis: C = (Q^T S)(Q^T S)^T is w x w symmetric (w = r + p
// <= 600). The kernel diagonalises C with a parallel cyclic Jacobi method (one CTA per problem) and
// writes Mr [w][r] = the first r columns of the projector V_r V_r^T onto the eigenvectors of the r
// largest eigenvalues. C is destroyed; work holds 3 w*w floats.
struct EigProblem {
  float* C;
  float* work;
  float* Mr;
  int w, r;
};
void launch_jacobi_projector(const EigProblem* probs, int nprobs, int w_max, cudaStream_t st);

// Grouped helpers of the refresh: random sketches and device-to-device copies for many matrices
// in one launch each. blk_start is the first 256-thread block of the entry within the launch.
struct RandProblem {
  float* out;            // fp32 output, may be null
  __nv_bfloat16* out16;  // bf16 output, may be null
  long long count, blk_start;
  int purpose, mat, replica, pad;
};
struct CopyProblem {
  void* dst;
  const void* src;
  long long chunks, blk_start;  // 16-byte chunks
};
void launch_fill_random_grouped(const RandProblem* probs, int nprobs, long long total_blocks, unsigned long long seed, long long index,
                                cudaStream_t st);
void launch_copy_grouped(const CopyProblem* probs, int nprobs, long long total_blocks, cudaStream_t st);
// Element-wise preparation of tensor-core operands, many buffers per launch (1024 elements per block).
// "Split" writes a value x as `planes` bf16 planes, plane p + 1 holding the rounding residual of the
// planes before it (x ~ p0 + p1 (+ p2)), `plane` elements apart. Products of split operands sum the
// plane pairs (0,0), (0,1), (1,0) [two planes: 16 bits of each operand] and (1,1), (0,2), (2,0)
// [three planes: 24 bits, the accuracy of an fp32 product].
enum ConvMode {
  CONV_BF16 = 0,     // dst = bf16(src)
  CONV_SPLIT = 1,    // dst = split(src)
  CONV_STATES = 2,   // dst = split(u^ = inv_bc1 src), dst2 = split(inv_bc2 src2 - u^ u^)
  CONV_ROT_T = 3,    // src is Rot [ld][ld]: dst = split(Rot^T), dst2 = split(Rot^T o Rot^T)
  CONV_COMBINE = 4   // outf = bc1 src, outf2 = bc2 |src2 + src src|   (rotated moments from the two products)
};
struct ConvProblem {
  const float* src;
  const float* src2;
  __nv_bfloat16 *dst, *dst2;
  float *outf, *outf2;
  long long count, blk_start;  // count is a multiple of 8
  long long plane;             // elements between the planes of dst and of dst2
  int mode, ld, planes, pad;
};
void launch_convert_grouped(const ConvProblem* probs, int nprobs, long long total_blocks, const GemmScalars& sc, cudaStream_t st);

// Columns of X [rows][r] scaled to unit length (sums of squares in fp64), one block per 32 columns.
// The tensor-core Gram matrix underestimates its diagonal (an fp32 accumulator that truncates, over
// thousands of positive addends), which leaves every column of Q a few 1e-5 too long; the
// off-diagonal part is already at fp32 level.
struct NormProblem {
  float* X;
  long long blk_start;
  int rows, r;
};
void launch_colnorm_grouped(const NormProblem* probs, int nprobs, long long total_blocks, cudaStream_t st);

// Tensor-core sketch products of the refresh (lordo_tma.cu): C[M x r] (fp32) = S * B with the big
// signal matrix S streamed by TMA as bf16 (optionally formed as c*G + E in shared memory) and
// B [Kd][r] in bf16. a_mn = 1: S is stored [Kd][M] (the product S^T P'); 0: stored [M][Kd].
struct SkProblem {
  long long tile_start;      // first 256-row tile (128 rows per CTA of a pair) of this problem within the launch
  int M, Kd, r, r_n;
  int a_mn, a_c2, b_c2;      // third TMA coordinate (worker / batch index) of A and of B
  int split;                 // 0: one product; 2 or 3: operands split in that many bf16 planes, 3 or 6 passes over k
  int a_pl, b_pl;            // third-coordinate distance between the planes of A and of B
  int c_trans, pad;          // 1: C is stored transposed, C[col * ldc + row]
  const void* map_a;         // 64 x 64 swizzled boxes (a_mn) or 64 x 128 swizzled boxes
  const void* map_e;         // same shape over E, or null
  const void* map_b;         // 64 x 64 swizzled boxes over B [batch][Kd][r]
  const float* cptr;         // scale of A when map_e is set (clip coefficient), else null
  float* C;
  long long ldc;
};
void launch_sketch_tma(const SkProblem* probs, int nprobs, long long total_tiles, int grid, int big, unsigned* status, cudaStream_t st);

// streaming kernels
void launch_sumsq_partial(const MatDev* mats, const void* const* G, const long long* chunk_start, int n_mats, int K, int g_dt,
                          double* partial, long long total_chunks, cudaStream_t st);
void launch_clip_finalize(const MatDev* mats, const long long* chunk_start, int n_mats, int K, const double* partial, float rho,
                          int scope, float* coef, double* sumsq, unsigned* status, cudaStream_t st);
void launch_fill_float(float* p, long long count, float value, cudaStream_t st);
void launch_moments(const MatDev* mats, const long long* tile_start, int n_mats, long long total_tiles, const StepScalars& sc,
                    cudaStream_t st);
void launch_outer_weights(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int w_dt,
                          int outer, float eta_s, float mu_s, float delta_scale, cudaStream_t st);
void launch_outer_states(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int which,
                         cudaStream_t st);
void launch_init_weights(const MatDev* mats, const long long* blk_start, int n_mats, long long total_blocks, int K, int w_dt,
                         cudaStream_t st);
void launch_identity_projection(float* P, long long m, int r, int copies, cudaStream_t st);
void launch_fill_random(float* out, long long count, long long batch_stride, const RandomKeys& keys, int batch, cudaStream_t st);

}  // namespace lordo
