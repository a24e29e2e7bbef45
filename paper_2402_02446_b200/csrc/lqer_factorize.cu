// Factor preparation on the GPU (paper Section 3.1: E_q = W - W_q, A_k = U_k, B_k = Sigma_k V_k^T; Section 3.2:
// SVD of S E_q, A_k = S^-1 U'_k, B_k = Sigma'_k V'_k^T; Appendix A: the calibration of S), so that the packed
// layer can be produced from the weight and a calibration batch alone.
//
//   s        per channel: mean |X| over the tokens of a sample, maximum over the samples, divided by
//            sqrt(min * max)                                                   (fp64 sums, fixed order)
//   G        = diag(s) (W - dq(q(W)))      fp32 [K, N]   (s = 1 for plain LQER)
//   top-k    singular triplets of G by randomised subspace iteration: Q = orth(G Omega); four rounds of
//            Z = orth(G^T Q), Q = orth(G Z); then Bt = G^T Q = Q_b R (Cholesky factor of Bt^T Bt), the right
//            singular vectors V of the small matrix R (one-sided Jacobi in one CTA), and
//            A = diag(1/s) Q V_k,   B = (Bt V_k)^T = Sigma_k V_k^T.
// The large products read G as fp32 and accumulate in fp64; everything of rank size is fp64.  orth() is
// Cholesky QR applied twice.  Omega (the random test matrix) is an input, so the caller owns the random numbers.
// None of this is on the inference path; the kernels are plain CUDA-core code built for clarity and a fixed
// summation order.
#include "lqer_common.cuh"

namespace lqer {
namespace fac {

constexpr int kOversample = 16;
constexpr int kIters = 4;
constexpr int kMaxR = 272;                 // 256 + oversample

// ---------------------------------------------------------------------------- calibration (Appendix A)
// Partial sums of |X| over a chunk of rows: grid (column blocks of 256, row chunks), one thread per column.
__global__ void __launch_bounds__(256) abs_sum_kernel(const float* __restrict__ X, int rows, int K, int rows_per_chunk,
                                                      double* __restrict__ part) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= K) return;
  const int r0 = blockIdx.y * rows_per_chunk, r1 = min(rows, r0 + rows_per_chunk);
  double acc = 0.0;
  for (int r = r0; r < r1; ++r) acc += (double)fabsf(X[(size_t)r * K + c]);
  part[(size_t)blockIdx.y * K + c] = acc;
}
// a_bar[c] = max(a_bar[c], sum of the chunks / rows)   (first sample: plain store)
__global__ void __launch_bounds__(256) abs_mean_max_kernel(const double* __restrict__ part, int chunks, int K, int rows,
                                                           int first, double* __restrict__ a_bar) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= K) return;
  double acc = 0.0;
  for (int q = 0; q < chunks; ++q) acc += part[(size_t)q * K + c];
  const double a = acc / (double)rows;
  a_bar[c] = first ? a : fmax(a_bar[c], a);
}
// s = a_bar / sqrt(min * max); one CTA.  status: 1 if a channel is identically zero (S is not invertible).
__global__ void __launch_bounds__(1024) normalise_scale_kernel(const double* __restrict__ a_bar, int K, double* __restrict__ s,
                                                               int* __restrict__ status) {
  __shared__ double s_min[1024], s_max[1024];
  double lo = 1e300, hi = 0.0;
  for (int c = threadIdx.x; c < K; c += 1024) { lo = fmin(lo, a_bar[c]); hi = fmax(hi, a_bar[c]); }
  s_min[threadIdx.x] = lo; s_max[threadIdx.x] = hi;
  __syncthreads();
  for (int w = 512; w > 0; w >>= 1) {
    if (threadIdx.x < w) {
      s_min[threadIdx.x] = fmin(s_min[threadIdx.x], s_min[threadIdx.x + w]);
      s_max[threadIdx.x] = fmax(s_max[threadIdx.x], s_max[threadIdx.x + w]);
    }
    __syncthreads();
  }
  lo = s_min[0]; hi = s_max[0];
  if (threadIdx.x == 0) *status = lo > 0.0 ? 0 : 1;
  const double norm = lo > 0.0 ? 1.0 / sqrt(lo * hi) : 0.0;
  for (int c = threadIdx.x; c < K; c += 1024) s[c] = lo > 0.0 ? a_bar[c] * norm : 1.0;
}
__global__ void fill_ones_kernel(double* s, int K) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < K) s[c] = 1.0;
}

// ---------------------------------------------------------------------------- G = diag(s) (W - dq(q(W)))
// One thread = one (column n, 16-block of K), as the packing kernel quantises it.
__global__ void __launch_bounds__(256) scaled_error_kernel(const float* __restrict__ W, int K, int N, int w_bits, int emin, int emax,
                                                           const double* __restrict__ s, float* __restrict__ G) {
  const int n = blockIdx.x * 256 + threadIdx.x;
  const int kb = blockIdx.y;
  if (n >= N) return;
  float v[16];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    v[i] = W[(size_t)(kb * 16 + i) * N + n];
    amax = fmaxf(amax, abs_ignore_nan(v[i]));
  }
  const int e = block_exponent(amax, emin, emax);
  const double step = pow2d(e - (w_bits - 2));
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const double err = (double)v[i] - (double)quant_mantissa(v[i], e, w_bits) * step;
    G[(size_t)(kb * 16 + i) * N + n] = (float)(s[kb * 16 + i] * err);
  }
}

// ---------------------------------------------------------------------------- products with G
// C[m, r] = op(G) X, fp64 accumulation.  TRANS = false: op(G) = G [m = K, inner = N], X [N, r].
// TRANS = true: op(G) = G^T [m = N, inner = K], X [K, r].  X may be fp32 (the test matrix) or fp64.
// CTA tile 64 (m) x 64 (r), inner step 16, 256 threads with 4 x 4 outputs each.
template <bool TRANS, typename XT>
__global__ void __launch_bounds__(256) g_times_kernel(const float* __restrict__ G, int K, int N, const XT* __restrict__ X, int r,
                                                      double* __restrict__ C) {
  __shared__ double s_g[16][65];     // [inner][m]
  __shared__ double s_x[16][65];     // [inner][r]
  const int m_total = TRANS ? N : K, inner = TRANS ? K : N;
  const int m0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  double acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
  for (int i0 = 0; i0 < inner; i0 += 16) {
    for (int q = threadIdx.x; q < 64 * 16; q += 256) {
      int mi, ii;
      if (TRANS) { mi = q & 63; ii = q >> 6; } else { ii = q & 15; mi = q >> 4; }   // coalesced along G's rows
      const int m = m0 + mi, i = i0 + ii;
      float g = 0.0f;
      if (m < m_total && i < inner) g = TRANS ? G[(size_t)i * N + m] : G[(size_t)m * N + i];
      s_g[ii][mi] = (double)g;
    }
    for (int q = threadIdx.x; q < 16 * 64; q += 256) {
      const int rr = q & 63, ii = q >> 6;
      const int i = i0 + ii, c = r0 + rr;
      s_x[ii][rr] = (i < inner && c < r) ? (double)X[(size_t)i * r + c] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int ii = 0; ii < 16; ++ii) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = s_g[ii][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = s_x[ii][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, c = r0 + tx * 4 + j;
      if (m < m_total && c < r) C[(size_t)m * r + c] = acc[i][j];
    }
}

// ---------------------------------------------------------------------------- tall-skinny helpers (fp64)
// Partial Gram matrices: part[chunk][r][r] = Y[rows of the chunk]^T Y[rows of the chunk].  grid (r tiles of 16,
// r tiles of 16, chunks), 256 threads = 16 x 16 outputs.
__global__ void __launch_bounds__(256) gram_partial_kernel(const double* __restrict__ Y, int m, int r, int rows_per_chunk,
                                                           double* __restrict__ part) {
  __shared__ double s_a[32][17], s_b[32][17];
  const int i0 = blockIdx.x * 16, j0 = blockIdx.y * 16;
  const int row_lo = blockIdx.z * rows_per_chunk, row_hi = min(m, row_lo + rows_per_chunk);
  const int ti = threadIdx.x & 15, tj = threadIdx.x >> 4;
  double acc = 0.0;
  for (int q0 = row_lo; q0 < row_hi; q0 += 32) {
    for (int q = threadIdx.x; q < 32 * 16; q += 256) {
      const int c = q & 15, rr = q >> 4;
      const int row = q0 + rr;
      s_a[rr][c] = (row < row_hi && i0 + c < r) ? Y[(size_t)row * r + i0 + c] : 0.0;
      s_b[rr][c] = (row < row_hi && j0 + c < r) ? Y[(size_t)row * r + j0 + c] : 0.0;
    }
    __syncthreads();
#pragma unroll 8
    for (int rr = 0; rr < 32; ++rr) acc = fma(s_a[rr][ti], s_b[rr][tj], acc);
    __syncthreads();
  }
  if (i0 + ti < r && j0 + tj < r) part[((size_t)blockIdx.z * r + i0 + ti) * r + j0 + tj] = acc;
}
__global__ void __launch_bounds__(256) gram_sum_kernel(const double* __restrict__ part, int chunks, int r, double* __restrict__ C) {
  const int idx = blockIdx.x * 256 + threadIdx.x;
  if (idx >= r * r) return;
  double acc = 0.0;
  for (int q = 0; q < chunks; ++q) acc += part[(size_t)q * r * r + idx];
  C[idx] = acc;
}
// C = R^T R (upper-triangular R by Cholesky), then Rinv = R^-1; one CTA, column by column.  A pivot that is not
// positive (rank-deficient Y) is replaced by a tiny one so that the run stays finite; status records it.
__global__ void __launch_bounds__(1024) cholesky_inverse_kernel(double* __restrict__ C, int r, double* __restrict__ Rinv,
                                                                int* __restrict__ status) {
  // in place: the upper triangle of C becomes R
  for (int j = 0; j < r; ++j) {
    __syncthreads();
    if (threadIdx.x == 0) {
      double d = C[(size_t)j * r + j];
      for (int p = 0; p < j; ++p) d -= C[(size_t)p * r + j] * C[(size_t)p * r + j];
      if (!(d > 0.0)) { d = 1e-300; atomicMax(status, 2); }
      C[(size_t)j * r + j] = sqrt(d);
    }
    __syncthreads();
    const double djj = C[(size_t)j * r + j];
    for (int c = j + 1 + threadIdx.x; c < r; c += 1024) {
      double v = C[(size_t)j * r + c];
      for (int p = 0; p < j; ++p) v -= C[(size_t)p * r + j] * C[(size_t)p * r + c];
      C[(size_t)j * r + c] = v / djj;
    }
  }
  __syncthreads();
  // Rinv: column c solves R x = e_c by back substitution (a thread per column)
  for (int c = threadIdx.x; c < r; c += 1024) {
    for (int i = r - 1; i >= 0; --i) {
      double v = i == c ? 1.0 : 0.0;
      if (i > c) { Rinv[(size_t)i * r + c] = 0.0; continue; }
      for (int p = i + 1; p <= c; ++p) v -= C[(size_t)i * r + p] * Rinv[(size_t)p * r + c];
      Rinv[(size_t)i * r + c] = v / C[(size_t)i * r + i];
    }
  }
}
// Out[m, c] = rowscale[m] * sum_j Y[m, j] T[j, c] for c < cols (T is [r, ldt]); fp64 in, OutT out, optionally
// written transposed (Out[c, m]).  One CTA = 64 rows; T's used columns are walked in tiles of 64.
template <typename OutT, bool TRANSPOSE_OUT>
__global__ void __launch_bounds__(256) tall_times_small_kernel(const double* __restrict__ Y, int m, int r, const double* __restrict__ T,
                                                               int ldt, int cols, const double* __restrict__ rowscale, int invert_scale,
                                                               OutT* __restrict__ Out) {
  __shared__ double s_y[16][65], s_t[16][65];
  const int m0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  double acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
  for (int j0 = 0; j0 < r; j0 += 16) {
    for (int q = threadIdx.x; q < 64 * 16; q += 256) {
      const int jj = q & 15, mi = q >> 4;
      s_y[jj][mi] = (m0 + mi < m && j0 + jj < r) ? Y[(size_t)(m0 + mi) * r + j0 + jj] : 0.0;
      const int cc = q & 63, j2 = q >> 6;
      s_t[j2][cc] = (j0 + j2 < r && c0 + cc < cols) ? T[(size_t)(j0 + j2) * ldt + c0 + cc] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int jj = 0; jj < 16; ++jj) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = s_y[jj][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = s_t[jj][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= m) continue;
    double sc = 1.0;
    if (rowscale != nullptr) sc = invert_scale ? 1.0 / rowscale[row] : rowscale[row];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + tx * 4 + j;
      if (c < cols) {
        if (TRANSPOSE_OUT) Out[(size_t)c * m + row] = (OutT)(sc * acc[i][j]);
        else Out[(size_t)row * cols + c] = (OutT)(sc * acc[i][j]);
      }
    }
  }
}

// ---------------------------------------------------------------------------- small SVD (one CTA)
// Right singular vectors and singular values of the r x r upper-triangular R (the Cholesky factor left in the upper
// triangle of C, row-major) by one-sided Jacobi: pairs of columns are rotated until all are mutually orthogonal,
// V collects the rotations.  A warp per pair, the pairs of a step disjoint (round-robin tournament).  Mt, Vt: r x r
// scratch, column-major.  Out: Vs row-major [r][r] with the columns in falling order of singular value, sigma[r].
__global__ void __launch_bounds__(1024) jacobi_right_kernel(const double* __restrict__ C, int r, double* __restrict__ Mt,
                                                            double* __restrict__ Vt, double* __restrict__ Vs, double* __restrict__ sigma,
                                                            int* __restrict__ status) {
  __shared__ int s_rotated;
  __shared__ double s_norm[kMaxR];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int q = tid; q < r * r; q += 1024) {
    const int col = q / r, row = q % r;
    Mt[q] = row <= col ? C[(size_t)row * r + col] : 0.0;
    Vt[q] = row == col ? 1.0 : 0.0;
  }
  const int n = r + (r & 1);                  // players of the tournament (one dummy if r is odd)
  const double tol = 1e-15;
  int sweeps = 0;
  for (; sweeps < 40; ++sweeps) {
    __syncthreads();
    if (tid == 0) s_rotated = 0;
    __syncthreads();
    for (int t = 0; t < n - 1; ++t) {
      for (int i = warp; i < n / 2; i += 32) {
        int a = i == 0 ? n - 1 : (t + i) % (n - 1);
        int b = i == 0 ? t % (n - 1) : (t + n - 1 - i) % (n - 1);
        if (a >= r || b >= r) continue;
        const int p = min(a, b), q = max(a, b);
        double* mp = Mt + (size_t)p * r;
        double* mq = Mt + (size_t)q * r;
        double alpha = 0.0, beta = 0.0, gamma = 0.0;
        for (int row = lane; row < r; row += 32) {
          const double x = mp[row], y = mq[row];
          alpha = fma(x, x, alpha); beta = fma(y, y, beta); gamma = fma(x, y, gamma);
        }
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) {
          alpha += __shfl_xor_sync(0xFFFFFFFFu, alpha, sft);
          beta += __shfl_xor_sync(0xFFFFFFFFu, beta, sft);
          gamma += __shfl_xor_sync(0xFFFFFFFFu, gamma, sft);
        }
        if (fabs(gamma) > tol * sqrt(alpha * beta)) {
          const double zeta = (beta - alpha) / (2.0 * gamma);
          const double tt = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
          const double c = 1.0 / sqrt(1.0 + tt * tt), s = c * tt;
          double* vp = Vt + (size_t)p * r;
          double* vq = Vt + (size_t)q * r;
          for (int row = lane; row < r; row += 32) {
            const double x = mp[row], y = mq[row];
            mp[row] = c * x - s * y; mq[row] = s * x + c * y;
            const double u = vp[row], w = vq[row];
            vp[row] = c * u - s * w; vq[row] = s * u + c * w;
          }
          if (lane == 0) s_rotated = 1;
        }
      }
      __syncthreads();
    }
    if (s_rotated == 0) break;
  }
  if (tid == 0 && sweeps >= 40) atomicMax(status, 3);
  // singular values = column norms; falling order (ties by index)
  for (int j = warp; j < r; j += 32) {
    double a = 0.0;
    for (int row = lane; row < r; row += 32) a = fma(Mt[(size_t)j * r + row], Mt[(size_t)j * r + row], a);
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, sft);
    if (lane == 0) s_norm[j] = a;
  }
  __syncthreads();
  for (int j = tid; j < r; j += 1024) {
    int rank = 0;
    for (int i = 0; i < r; ++i) rank += (s_norm[i] > s_norm[j] || (s_norm[i] == s_norm[j] && i < j)) ? 1 : 0;
    sigma[rank] = sqrt(s_norm[j]);
    for (int row = 0; row < r; ++row) Vs[(size_t)row * r + rank] = Vt[(size_t)j * r + row];
  }
}

}  // namespace fac

int factor_sketch_rank(int K, int N, int k) {
  int r = k + fac::kOversample;
  if (r > K) r = K;
  if (r > N) r = N;
  return r;
}

// Workspace of launch_factorize, in bytes (every piece 256-byte aligned).
size_t factor_workspace_bytes(int K, int N, int k, int max_calib_rows) {
  const int r = factor_sketch_rank(K, N, k);
  const size_t big = (size_t)(K > N ? K : N);
  auto al = [](size_t v) { return (v + 255) & ~(size_t)255; };
  size_t b = 0;
  b += al((size_t)K * N * 4);                     // G
  b += 2 * al((size_t)K * 8);                     // a_bar, s
  b += al((size_t)64 * K * 8);                    // partial column sums of |X| (64 row chunks)
  b += 2 * al(big * r * 8);                       // two tall buffers (ping-pong)
  b += al((size_t)N * r * 8);                     // Bt
  b += al((size_t)64 * r * r * 8);                // partial Gram matrices
  b += 5 * al((size_t)r * r * 8);                 // C, Rinv, Mt, Vt, Vs
  b += al((size_t)r * 8) + 256;                   // sigma, status
  b += al((size_t)K * k * 4) + al((size_t)k * N * 4);   // A, B (fp32) where the caller keeps none
  (void)max_calib_rows;
  return b;
}

static cudaError_t orthonormalise(const double* Yin, double* Yout, int m, int r, double* gram_part, double* C, double* Rinv,
                                  int* status, cudaStream_t s) {
  using namespace fac;
  // Cholesky QR, twice: Y = Q R with Q^T Q = I to rounding once the first pass has tamed the conditioning
  const double* src = Yin;
  double* bufs[2] = {Yout, const_cast<double*>(Yin)};
  for (int pass = 0; pass < 2; ++pass) {
    const int chunks = 64, rows_per_chunk = (m + chunks - 1) / chunks;
    const int rt = (r + 15) / 16;
    gram_partial_kernel<<<dim3(rt, rt, chunks), 256, 0, s>>>(src, m, r, rows_per_chunk, gram_part);
    gram_sum_kernel<<<(r * r + 255) / 256, 256, 0, s>>>(gram_part, chunks, r, C);
    cholesky_inverse_kernel<<<1, 1024, 0, s>>>(C, r, Rinv, status);
    double* dst = bufs[pass];
    tall_times_small_kernel<double, false><<<dim3((m + 63) / 64, (r + 63) / 64), 256, 0, s>>>(src, m, r, Rinv, r, r, nullptr, 0, dst);
    src = dst;
  }
  // after two passes the result sits in Yin's buffer; copy back to Yout so that the caller's view is uniform
  return cudaMemcpyAsync(Yout, src, (size_t)m * r * 8, cudaMemcpyDeviceToDevice, s);
}

// W [K,N], calibration samples Xs[i] [rows[i], K] (n_samples may be 0: plain LQER, S = I), Omega [N, r] fp32 with
// r = factor_sketch_rank.  Outputs A [K,k], B [k,N] fp32 (device).  status_out (device int, may be null inside ws).
cudaError_t launch_factorize(const float* W, const float* const* Xs, const int* rows, int n_samples, const float* Omega, int K,
                             int N, int k, int w_bits, int emin, int emax, float* A, float* B, void* workspace, int** status_dev,
                             float** A_used, float** B_used, cudaStream_t s) {
  using namespace fac;
  const int r = factor_sketch_rank(K, N, k);
  if (r > kMaxR || k < 1) return cudaErrorInvalidValue;
  const size_t big = (size_t)(K > N ? K : N);
  auto al = [](size_t v) { return (v + 255) & ~(size_t)255; };
  uint8_t* p = static_cast<uint8_t*>(workspace);
  float* G = reinterpret_cast<float*>(p); p += al((size_t)K * N * 4);
  double* a_bar = reinterpret_cast<double*>(p); p += al((size_t)K * 8);
  double* sc = reinterpret_cast<double*>(p); p += al((size_t)K * 8);
  double* colpart = reinterpret_cast<double*>(p); p += al((size_t)64 * K * 8);
  double* T0 = reinterpret_cast<double*>(p); p += al(big * r * 8);
  double* T1 = reinterpret_cast<double*>(p); p += al(big * r * 8);
  double* Bt = reinterpret_cast<double*>(p); p += al((size_t)N * r * 8);
  double* gram_part = reinterpret_cast<double*>(p); p += al((size_t)64 * r * r * 8);
  double* C = reinterpret_cast<double*>(p); p += al((size_t)r * r * 8);
  double* Rinv = reinterpret_cast<double*>(p); p += al((size_t)r * r * 8);
  double* Mt = reinterpret_cast<double*>(p); p += al((size_t)r * r * 8);
  double* Vt = reinterpret_cast<double*>(p); p += al((size_t)r * r * 8);
  double* Vs = reinterpret_cast<double*>(p); p += al((size_t)r * r * 8);
  double* sigma = reinterpret_cast<double*>(p); p += al((size_t)r * 8);
  int* status = reinterpret_cast<int*>(p); p += 256;
  if (status_dev != nullptr) *status_dev = status;
  if (A == nullptr) A = reinterpret_cast<float*>(p);
  p += al((size_t)K * k * 4);
  if (B == nullptr) B = reinterpret_cast<float*>(p);
  if (A_used != nullptr) *A_used = A;
  if (B_used != nullptr) *B_used = B;

  LaunchScope scope(kFamPrepare, s, 16 + 12 * kIters);
  cudaMemsetAsync(status, 0, 4, s);
  // ---- S (Appendix A), or the identity
  if (n_samples > 0) {
    for (int i = 0; i < n_samples; ++i) {
      const int chunks = rows[i] < 64 ? 1 : 64, rpc = (rows[i] + chunks - 1) / chunks;
      abs_sum_kernel<<<dim3((K + 255) / 256, chunks), 256, 0, s>>>(Xs[i], rows[i], K, rpc, colpart);
      abs_mean_max_kernel<<<(K + 255) / 256, 256, 0, s>>>(colpart, chunks, K, rows[i], i == 0 ? 1 : 0, a_bar);
    }
    normalise_scale_kernel<<<1, 1024, 0, s>>>(a_bar, K, sc, status);
  } else {
    fill_ones_kernel<<<(K + 255) / 256, 256, 0, s>>>(sc, K);
  }
  // ---- G = S (W - W_q)
  scaled_error_kernel<<<dim3((N + 255) / 256, K / 16), 256, 0, s>>>(W, K, N, w_bits, emin, emax, sc, G);
  // ---- subspace iteration
  const dim3 gK((K + 63) / 64, (r + 63) / 64), gN((N + 63) / 64, (r + 63) / 64);
  g_times_kernel<false, float><<<gK, 256, 0, s>>>(G, K, N, Omega, r, T0);             // Y = G Omega      [K, r]
  cudaError_t e = orthonormalise(T0, T1, K, r, gram_part, C, Rinv, status, s);           // Q in T1
  if (e != cudaSuccess) return e;
  for (int it = 0; it < kIters; ++it) {
    g_times_kernel<true, double><<<gN, 256, 0, s>>>(G, K, N, T1, r, T0);                // Z = G^T Q        [N, r]
    if ((e = orthonormalise(T0, Bt, N, r, gram_part, C, Rinv, status, s)) != cudaSuccess) return e;   // Z in Bt
    g_times_kernel<false, double><<<gK, 256, 0, s>>>(G, K, N, Bt, r, T0);               // Y = G Z          [K, r]
    if ((e = orthonormalise(T0, T1, K, r, gram_part, C, Rinv, status, s)) != cudaSuccess) return e;   // Q in T1
  }
  g_times_kernel<true, double><<<gN, 256, 0, s>>>(G, K, N, T1, r, Bt);                  // Bt = G^T Q       [N, r]
  // ---- small SVD: Bt^T Bt = R^T R, R = U Sigma V^T  ->  G ~ (Q V) Sigma (...)^T
  {
    const int chunks = 64, rpc = (N + chunks - 1) / chunks, rt = (r + 15) / 16;
    gram_partial_kernel<<<dim3(rt, rt, chunks), 256, 0, s>>>(Bt, N, r, rpc, gram_part);
    gram_sum_kernel<<<(r * r + 255) / 256, 256, 0, s>>>(gram_part, chunks, r, C);
    cholesky_inverse_kernel<<<1, 1024, 0, s>>>(C, r, Rinv, status);
    jacobi_right_kernel<<<1, 1024, 0, s>>>(C, r, Mt, Vt, Vs, sigma, status);
  }
  // ---- A = S^-1 Q V_k  [K, k];  B = (Bt V_k)^T  [k, N]
  tall_times_small_kernel<float, false><<<dim3((K + 63) / 64, (k + 63) / 64), 256, 0, s>>>(T1, K, r, Vs, r, k, sc, 1, A);
  tall_times_small_kernel<float, true><<<dim3((N + 63) / 64, (k + 63) / 64), 256, 0, s>>>(Bt, N, r, Vs, r, k, nullptr, 0, B);
  return cudaGetLastError();
}

}  // namespace lqer
