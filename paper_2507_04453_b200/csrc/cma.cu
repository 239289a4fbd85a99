// Search-distribution update on the device (Section 3, "Evolutionary optimization": after the rewards are known
// CMA-ES updates (m, sigma, C) from the reward ranking; Algorithm 1, the CMA-ES update every worker performs after
// the <seed, reward> exchange).  The paper gives no formulas (it cites Hansen's CMA-ES), so this is the
// (mu/mu_w, lambda)-CMA-ES of Hansen's tutorial with its default strategy parameters and non-negative weights:
//
//   rank the rewards (largest first; ties keep population order; NaN last)             cma_rank_kernel
//   y_i = (x_{i:lambda} - m) / sigma for the mu best                                     cma_steps_kernel
//   <y>_w = sum w_i y_i;  m += sigma <y>_w;  p_sigma, sigma, h_sigma, p_c                 cma_paths_kernel (one CTA)
//   C <- (1 - c_1 - c_mu + (1-h_sigma) c_1 c_c (2-c_c)) C + c_1 p_c p_c^T + c_mu sum w_i y_i y_i^T    cma_cov_kernel
//   C = B diag(D^2) B^T by one-sided Jacobi rotations (Hestenes), eigenvalues ascending    jacobi_* kernels
//
// Everything is fp64 on the CUDA cores (the work is small: d <= 1024); the state lives in device memory and the
// sampler reads its fp32 copies (mean, step, B, D), so ask -> rewards -> tell -> ask never leaves the device.
#include <cmath>
#include <new>
#include <vector>

#include "common.cuh"

struct essa_cma {
  int d = 0, lambda = 0, mu = 0;
  int generation = 0;
  // strategy parameters (host copies)
  double mu_eff = 0, c_sigma = 0, d_sigma = 0, c_c = 0, c_1 = 0, c_mu = 0, c_m = 1, chi_n = 0;
  // device state
  double* mean = nullptr;     // [d]
  double* sigma = nullptr;    // [1] global step size
  double* C = nullptr;        // [d][d] symmetric
  double* p_sigma = nullptr;  // [d]
  double* p_c = nullptr;      // [d]
  double* B = nullptr;        // [d][d] row-major, columns = eigenvectors
  double* D = nullptr;        // [d] square roots of the eigenvalues, ascending
  double* weights = nullptr;  // [mu]
  // fp32 copies the sampler reads
  float* mean32 = nullptr;
  float* step32 = nullptr;
  float* B32 = nullptr;
  float* D32 = nullptr;
  // scratch
  int32_t* order = nullptr;   // [lambda]
  double* Y = nullptr;        // [mu][d]
  double* yw = nullptr;       // [d] <y>_w, then work vectors
  double* hsig = nullptr;     // [1]
  double* G = nullptr;        // [d][d] column-major: C V during the decomposition
  double* V = nullptr;        // [d][d] column-major: accumulated rotations
  double* ev = nullptr;       // [d] eigenvalues before sorting
  int32_t* rot = nullptr;     // [kMaxSweeps + 1] rotations applied per sweep
  // host view of rot, copied back asynchronously after every sweep so that the host can stop issuing sweeps once
  // one of them found nothing to rotate (it never blocks on it: an answer that is late only costs no-op launches)
  int32_t* rot_host = nullptr;          // pinned, [kMaxSweeps]
  std::vector<cudaEvent_t> rot_events;  // one per sweep
};

namespace essa {
namespace {

constexpr int kMaxSweeps = 30;
constexpr int kMaxDim = 1024;
constexpr int kPathThreads = 512;

// order[r] = index of the candidate with the (r+1)-th largest reward; ties keep population order; NaN ranks last.
__global__ void cma_rank_kernel(const float* __restrict__ rewards, int lambda, int32_t* __restrict__ order) {
  for (int i = threadIdx.x; i < lambda; i += blockDim.x) {
    const float fi = rewards[i];
    const float ki = isnan(fi) ? -INFINITY : fi;
    int rank = 0;
    for (int j = 0; j < lambda; ++j) {
      const float fj = rewards[j];
      const float kj = isnan(fj) ? -INFINITY : fj;
      rank += (kj > ki || (kj == ki && j < i)) ? 1 : 0;
    }
    order[rank] = i;
  }
}

// Y[k][i] = (x[order[k]][i] - m[i]) / sigma for the mu best candidates.
__global__ void cma_steps_kernel(const float* __restrict__ pop, int ld, const int32_t* __restrict__ order, const double* __restrict__ mean,
                                 const double* __restrict__ sigma, int d, int mu, double* __restrict__ Y) {
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx >= (long long)mu * d) return;
  const int k = (int)(idx / d), i = (int)(idx % d);
  Y[idx] = ((double)pop[(size_t)order[k] * ld + i] - mean[i]) / *sigma;
}

__device__ double block_sum(double v, double* red) {
  __syncthreads();
  red[threadIdx.x] = v;
  __syncthreads();
  for (int s = blockDim.x / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  return red[0];
}

struct PathParams {
  int d, mu, generation;  // generation = count of updates done before this one
  double mu_eff, c_sigma, d_sigma, c_c, c_m, chi_n;
};

// One CTA: recombination, mean, conjugate evolution path, step size, stall indicator, evolution path.
__global__ void __launch_bounds__(kPathThreads) cma_paths_kernel(PathParams q, const double* __restrict__ Y, const double* __restrict__ w,
                                                                 const double* __restrict__ B, const double* __restrict__ D,
                                                                 double* __restrict__ mean, double* __restrict__ sigma,
                                                                 double* __restrict__ p_sigma, double* __restrict__ p_c,
                                                                 double* __restrict__ yw, double* __restrict__ hsig,
                                                                 float* __restrict__ mean32, float* __restrict__ step32) {
  __shared__ double red[kPathThreads];
  __shared__ double t_sh[kMaxDim];   // B^T <y>_w / D
  __shared__ double yw_sh[kMaxDim];
  const int d = q.d;
  const double sig_old = *sigma;
  // <y>_w and the mean
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    double acc = 0.0;
    for (int k = 0; k < q.mu; ++k) acc = fma(w[k], Y[(size_t)k * d + i], acc);
    yw_sh[i] = acc;
    yw[i] = acc;
    const double m = mean[i] + q.c_m * sig_old * acc;
    mean[i] = m;
    mean32[i] = (float)m;
  }
  __syncthreads();
  // t = D^-1 B^T <y>_w   (B row-major: column j is eigenvector j)
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    double acc = 0.0;
    for (int i = 0; i < d; ++i) acc = fma(B[(size_t)i * d + j], yw_sh[i], acc);
    t_sh[j] = acc / D[j];
  }
  __syncthreads();
  // p_sigma <- (1 - c_sigma) p_sigma + sqrt(c_sigma (2 - c_sigma) mu_eff) B t
  const double a_ps = sqrt(q.c_sigma * (2.0 - q.c_sigma) * q.mu_eff);
  double sq = 0.0;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) acc = fma(B[(size_t)i * d + j], t_sh[j], acc);
    const double ps = (1.0 - q.c_sigma) * p_sigma[i] + a_ps * acc;
    p_sigma[i] = ps;
    sq = fma(ps, ps, sq);
  }
  const double norm_ps = sqrt(block_sum(sq, red));
  const double sig_new = sig_old * exp((q.c_sigma / q.d_sigma) * (norm_ps / q.chi_n - 1.0));
  const double decay = sqrt(1.0 - pow(1.0 - q.c_sigma, 2.0 * (q.generation + 1)));
  const double h = norm_ps < (1.4 + 2.0 / (d + 1.0)) * q.chi_n * decay ? 1.0 : 0.0;
  const double a_pc = h * sqrt(q.c_c * (2.0 - q.c_c) * q.mu_eff);
  for (int i = threadIdx.x; i < d; i += blockDim.x) p_c[i] = (1.0 - q.c_c) * p_c[i] + a_pc * yw_sh[i];
  if (threadIdx.x == 0) {
    *sigma = sig_new;
    *step32 = (float)sig_new;
    *hsig = h;
  }
}

// C_ij <- a C_ij + c_1 p_c,i p_c,j + c_mu sum_k w_k Y_ki Y_kj,  a = 1 - c_1 - c_mu + (1 - h_sigma) c_1 c_c (2 - c_c).
// Every product of two vector entries is formed first (commutative, so entry (i,j) and (j,i) round alike) and
// then scaled, which keeps C symmetric bit for bit.
__global__ void cma_cov_kernel(int d, int mu, double c_1, double c_mu, double c_c, const double* __restrict__ hsig,
                               const double* __restrict__ p_c, const double* __restrict__ Y, const double* __restrict__ w,
                               double* __restrict__ C) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y * blockDim.y + threadIdx.y;
  if (i >= d || j >= d) return;
  const double a = 1.0 - c_1 - c_mu + (1.0 - *hsig) * c_1 * c_c * (2.0 - c_c);
  double acc = 0.0;
  for (int k = 0; k < mu; ++k) acc = fma(w[k], Y[(size_t)k * d + i] * Y[(size_t)k * d + j], acc);
  C[(size_t)i * d + j] = a * C[(size_t)i * d + j] + c_1 * (p_c[i] * p_c[j]) + c_mu * acc;
}

// ------------------------------------------------------------------------------------------------ decomposition
// One-sided Jacobi (Hestenes) on G = C V, V starting at I: a rotation of columns (p, q) of G and of V makes the two
// columns of G orthogonal; when every pair is orthogonal, G = V diag(lambda): the columns of V are the eigenvectors
// and lambda_j = v_j . g_j.  V is a product of plane rotations, so it stays orthonormal to rounding.  A sweep visits
// every pair once, in d - 1 (d even) rounds of d / 2 disjoint pairs (round-robin tournament); one launch per round,
// one CTA per pair.  A sweep that applies no rotation ends the iteration: later launches return at once.
__global__ void jacobi_init_kernel(int d, const double* __restrict__ C, double* __restrict__ G, double* __restrict__ V) {
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx >= (long long)d * d) return;
  const int col = (int)(idx / d), row = (int)(idx % d);
  G[idx] = C[(size_t)row * d + col];  // column-major copy (C is symmetric, but copy what is stored)
  V[idx] = row == col ? 1.0 : 0.0;
}

constexpr int kJacobiThreads = 128;
__global__ void __launch_bounds__(kJacobiThreads) jacobi_round_kernel(int d, int n_players, int round, int sweep, double* __restrict__ G,
                                                                      double* __restrict__ V, int32_t* __restrict__ rot) {
  if (sweep > 0 && rot[sweep - 1] == 0) return;  // the previous sweep found every pair orthogonal
  // pair of this CTA in this round: player n-1 stays, the others rotate
  const int m = n_players - 1;
  int p, q;
  if (blockIdx.x == 0) {
    p = m;
    q = round % m;
  } else {
    p = (round + (int)blockIdx.x) % m;
    q = (round - (int)blockIdx.x + m) % m;
  }
  if (p >= d || q >= d) return;  // the padding player of an odd dimension
  if (p > q) { const int t = p; p = q; q = t; }
  double* gp = G + (size_t)p * d;
  double* gq = G + (size_t)q * d;
  __shared__ double red[3][kJacobiThreads];
  double a = 0.0, b = 0.0, g = 0.0;
  for (int i = threadIdx.x; i < d; i += kJacobiThreads) {
    const double x = gp[i], y = gq[i];
    a = fma(x, x, a);
    b = fma(y, y, b);
    g = fma(x, y, g);
  }
  red[0][threadIdx.x] = a; red[1][threadIdx.x] = b; red[2][threadIdx.x] = g;
  __syncthreads();
  for (int s = kJacobiThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) {
      red[0][threadIdx.x] += red[0][threadIdx.x + s];
      red[1][threadIdx.x] += red[1][threadIdx.x + s];
      red[2][threadIdx.x] += red[2][threadIdx.x + s];
    }
    __syncthreads();
  }
  const double alpha = red[0][0], beta = red[1][0], gamma = red[2][0];
  if (!(fabs(gamma) > 1e-15 * sqrt(alpha * beta))) return;  // already orthogonal (or a zero column)
  if (threadIdx.x == 0) atomicAdd(rot + sweep, 1);
  const double zeta = (beta - alpha) / (2.0 * gamma);
  const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
  const double c = 1.0 / sqrt(1.0 + t * t), s = c * t;
  double* vp = V + (size_t)p * d;
  double* vq = V + (size_t)q * d;
  for (int i = threadIdx.x; i < d; i += kJacobiThreads) {
    const double x = gp[i], y = gq[i];
    gp[i] = c * x - s * y;
    gq[i] = s * x + c * y;
    const double u = vp[i], v = vq[i];
    vp[i] = c * u - s * v;
    vq[i] = s * u + c * v;
  }
}

// lambda_j = v_j . g_j
__global__ void jacobi_values_kernel(int d, const double* __restrict__ G, const double* __restrict__ V, double* __restrict__ ev) {
  const int j = blockIdx.x;
  __shared__ double red[kJacobiThreads];
  double acc = 0.0;
  for (int i = threadIdx.x; i < d; i += kJacobiThreads) acc = fma(V[(size_t)j * d + i], G[(size_t)j * d + i], acc);
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = kJacobiThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) ev[j] = red[0];
}

// Ascending order of the eigenvalues (ties keep column order): column j of V becomes column rank(j) of B (row-major);
// D = sqrt(max(lambda, 0)); fp32 copies for the sampler.
__global__ void jacobi_sort_kernel(int d, const double* __restrict__ ev, const double* __restrict__ V, double* __restrict__ B,
                                   double* __restrict__ D, float* __restrict__ B32, float* __restrict__ D32) {
  const int j = blockIdx.x;
  __shared__ int rank_sh;
  if (threadIdx.x == 0) {
    const double ej = ev[j];
    int rank = 0;
    for (int k = 0; k < d; ++k) rank += (ev[k] < ej || (ev[k] == ej && k < j)) ? 1 : 0;
    rank_sh = rank;
    const double dj = sqrt(ej > 0.0 ? ej : 0.0);
    D[rank] = dj;
    D32[rank] = (float)dj;
  }
  __syncthreads();
  const int rank = rank_sh;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const double v = V[(size_t)j * d + i];
    B[(size_t)i * d + rank] = v;
    B32[(size_t)i * d + rank] = (float)v;
  }
}

int32_t decompose(essa_ctx* ctx, essa_cma* s, cudaStream_t stream) {
  const int d = s->d;
  cudaError_t e = cudaMemsetAsync(s->rot, 0, (kMaxSweeps + 1) * sizeof(int32_t), stream);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cma: memset");
  const long long dd = (long long)d * d;
  jacobi_init_kernel<<<(unsigned)((dd + 255) / 256), 256, 0, stream>>>(d, s->C, s->G, s->V);
  ctx->launches += 1;
  if (d > 1) {
    const int n_players = d + (d & 1);
    for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
      bool converged = false;
      for (int t = 0; t < sweep && !converged; ++t)
        converged = cudaEventQuery(s->rot_events[t]) == cudaSuccess && s->rot_host[t] == 0;
      cudaGetLastError();  // cudaErrorNotReady is not an error here
      if (converged) break;
      for (int round = 0; round < n_players - 1; ++round) {
        jacobi_round_kernel<<<n_players / 2, kJacobiThreads, 0, stream>>>(d, n_players, round, sweep, s->G, s->V, s->rot);
        ctx->launches += 1;
      }
      s->rot_host[sweep] = -1;
      cudaMemcpyAsync(s->rot_host + sweep, s->rot + sweep, sizeof(int32_t), cudaMemcpyDeviceToHost, stream);
      cudaEventRecord(s->rot_events[sweep], stream);
    }
  }
  jacobi_values_kernel<<<d, kJacobiThreads, 0, stream>>>(d, s->G, s->V, s->ev);
  jacobi_sort_kernel<<<d, 128, 0, stream>>>(d, s->ev, s->V, s->B, s->D, s->B32, s->D32);
  ctx->launches += 2;
  return check_cuda(ctx, cudaGetLastError(), "cma: decomposition launches");
}

void free_state(essa_cma* s) {
  void* ptrs[] = {s->mean, s->sigma, s->C, s->p_sigma, s->p_c, s->B, s->D, s->weights, s->mean32, s->step32, s->B32, s->D32,
                  s->order, s->Y, s->yw, s->hsig, s->G, s->V, s->ev, s->rot};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  if (s->rot_host) cudaFreeHost(s->rot_host);
  for (cudaEvent_t ev : s->rot_events) cudaEventDestroy(ev);
  delete s;
}

}  // namespace
}  // namespace essa

using namespace essa;

extern "C" {

int32_t essa_cma_create(essa_ctx* ctx, int32_t d, int32_t lambda, const float* mean0_host, float step0, essa_cma** out) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!out || !mean0_host) return fail(ctx, ESSA_ERR_INVALID_ARG, "cma_create: NULL argument");
  *out = nullptr;
  if (d < 1 || lambda < 2 || !(step0 > 0.f)) return fail(ctx, ESSA_ERR_INVALID_ARG, "cma_create: need d >= 1, lambda >= 2, step0 > 0");
  if (d > kMaxDim) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "cma_create: d > 1024");
  if (lambda > 65536) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "cma_create: lambda > 65536");
  essa_cma* s = new (std::nothrow) essa_cma();
  if (!s) return fail(ctx, ESSA_ERR_ALLOC, "cma_create: host allocation failed");
  s->d = d;
  s->lambda = lambda;
  s->mu = lambda / 2;
  // default strategy parameters of the tutorial (alpha_cov = 2), non-negative weights
  std::vector<double> w((size_t)s->mu);
  double sum = 0.0, sum2 = 0.0;
  for (int i = 0; i < s->mu; ++i) {
    w[i] = std::log((lambda + 1) / 2.0) - std::log((double)(i + 1));
    sum += w[i];
  }
  for (int i = 0; i < s->mu; ++i) {
    w[i] /= sum;
    sum2 += w[i] * w[i];
  }
  const double n = d;
  s->mu_eff = 1.0 / sum2;
  s->c_sigma = (s->mu_eff + 2.0) / (n + s->mu_eff + 5.0);
  const double ds = std::sqrt((s->mu_eff - 1.0) / (n + 1.0)) - 1.0;
  s->d_sigma = 1.0 + 2.0 * (ds > 0.0 ? ds : 0.0) + s->c_sigma;
  s->c_c = (4.0 + s->mu_eff / n) / (n + 4.0 + 2.0 * s->mu_eff / n);
  s->c_1 = 2.0 / ((n + 1.3) * (n + 1.3) + s->mu_eff);
  const double cmu = 2.0 * (s->mu_eff - 2.0 + 1.0 / s->mu_eff) / ((n + 2.0) * (n + 2.0) + s->mu_eff);
  s->c_mu = cmu < 1.0 - s->c_1 ? cmu : 1.0 - s->c_1;
  s->c_m = 1.0;
  s->chi_n = std::sqrt(n) * (1.0 - 1.0 / (4.0 * n) + 1.0 / (21.0 * n * n));

  const size_t dd = (size_t)d * d;
  cudaError_t e = cudaSuccess;
  auto alloc = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
  alloc((void**)&s->mean, d * 8); alloc((void**)&s->sigma, 8); alloc((void**)&s->C, dd * 8);
  alloc((void**)&s->p_sigma, d * 8); alloc((void**)&s->p_c, d * 8); alloc((void**)&s->B, dd * 8); alloc((void**)&s->D, d * 8);
  alloc((void**)&s->weights, (size_t)s->mu * 8); alloc((void**)&s->mean32, d * 4); alloc((void**)&s->step32, 4);
  alloc((void**)&s->B32, dd * 4); alloc((void**)&s->D32, d * 4); alloc((void**)&s->order, (size_t)lambda * 4);
  alloc((void**)&s->Y, (size_t)s->mu * d * 8); alloc((void**)&s->yw, d * 8); alloc((void**)&s->hsig, 8);
  alloc((void**)&s->G, dd * 8); alloc((void**)&s->V, dd * 8); alloc((void**)&s->ev, d * 8);
  alloc((void**)&s->rot, (kMaxSweeps + 1) * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMallocHost((void**)&s->rot_host, kMaxSweeps * sizeof(int32_t));
  for (int i = 0; i < kMaxSweeps && e == cudaSuccess; ++i) {
    cudaEvent_t ev;
    e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    if (e == cudaSuccess) s->rot_events.push_back(ev);
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    free_state(s);
    return fail(ctx, ESSA_ERR_ALLOC, std::string("cma_create: allocation failed: ") + cudaGetErrorString(e));
  }
  // m_0 as given, sigma_0 = step0, C_0 = I (so B = I, D = 1), both paths zero
  std::vector<double> m64((size_t)d), eye(dd, 0.0), ones((size_t)d, 1.0);
  std::vector<float> eye32(dd, 0.f), ones32((size_t)d, 1.f);
  for (int i = 0; i < d; ++i) { m64[i] = mean0_host[i]; eye[(size_t)i * d + i] = 1.0; eye32[(size_t)i * d + i] = 1.f; }
  const double sig0 = step0;
  auto up = [&](void* dst, const void* src, size_t bytes) { if (e == cudaSuccess) e = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice); };
  up(s->mean, m64.data(), d * 8); up(s->sigma, &sig0, 8); up(s->C, eye.data(), dd * 8); up(s->B, eye.data(), dd * 8);
  up(s->D, ones.data(), d * 8); up(s->weights, w.data(), (size_t)s->mu * 8); up(s->mean32, mean0_host, d * 4);
  up(s->step32, &step0, 4); up(s->B32, eye32.data(), dd * 4); up(s->D32, ones32.data(), d * 4);
  if (e == cudaSuccess) e = cudaMemset(s->p_sigma, 0, d * 8);
  if (e == cudaSuccess) e = cudaMemset(s->p_c, 0, d * 8);
  if (e != cudaSuccess) {
    free_state(s);
    return check_cuda(ctx, e, "cma_create: initialisation");
  }
  *out = s;
  return ESSA_OK;
}

int32_t essa_cma_destroy(essa_ctx* ctx, essa_cma* s) {
  if (!ctx || !s) return ESSA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  free_state(s);
  return ESSA_OK;
}

int32_t essa_cma_ask(essa_ctx* ctx, essa_cma* s, uint64_t seed, int32_t k_begin, int32_t k_count, float* sigma_out, void* stream) {
  if (!ctx || !s) return ESSA_ERR_INVALID_ARG;
  if (k_begin < 0 || k_count < 0 || (k_count > 0 && !sigma_out)) return fail(ctx, ESSA_ERR_INVALID_ARG, "cma_ask: bad arguments");
  return launch_sampler(ctx, s->mean32, 0.f, s->B32, s->D32, s->d, seed, k_begin, k_count, nullptr, s->d, sigma_out,
                        static_cast<cudaStream_t>(stream), nullptr, nullptr, s->step32);
}

int32_t essa_tell(essa_ctx* ctx, essa_cma* s, const float* population, int32_t ld, const float* rewards, void* stream_v) {
  if (!ctx || !s) return ESSA_ERR_INVALID_ARG;
  if (!population || !rewards || ld < s->d) return fail(ctx, ESSA_ERR_INVALID_ARG, "tell: NULL buffer or ld < d");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const int d = s->d, mu = s->mu;
  cma_rank_kernel<<<1, 1024, 0, stream>>>(rewards, s->lambda, s->order);
  const long long md = (long long)mu * d;
  cma_steps_kernel<<<(unsigned)((md + 255) / 256), 256, 0, stream>>>(population, ld, s->order, s->mean, s->sigma, d, mu, s->Y);
  PathParams q{d, mu, s->generation, s->mu_eff, s->c_sigma, s->d_sigma, s->c_c, s->c_m, s->chi_n};
  cma_paths_kernel<<<1, kPathThreads, 0, stream>>>(q, s->Y, s->weights, s->B, s->D, s->mean, s->sigma, s->p_sigma, s->p_c, s->yw,
                                                   s->hsig, s->mean32, s->step32);
  dim3 blk(16, 16), grd((d + 15) / 16, (d + 15) / 16);
  cma_cov_kernel<<<grd, blk, 0, stream>>>(d, mu, s->c_1, s->c_mu, s->c_c, s->hsig, s->p_c, s->Y, s->weights, s->C);
  ctx->launches += 4;
  int32_t st = check_cuda(ctx, cudaGetLastError(), "tell: launches");
  if (st != ESSA_OK) return st;
  s->generation += 1;
  return decompose(ctx, s, stream);
}

int32_t essa_cma_set(essa_ctx* ctx, essa_cma* s, const double* mean, const double* step, const double* C, const double* p_sigma,
                     const double* p_c, int32_t generation, void* stream_v) {
  if (!ctx || !s) return ESSA_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const int d = s->d;
  cudaError_t e = cudaStreamSynchronize(stream);
  if (e == cudaSuccess && mean) {
    std::vector<float> m32((size_t)d);
    for (int i = 0; i < d; ++i) m32[i] = (float)mean[i];
    e = cudaMemcpy(s->mean, mean, d * 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s->mean32, m32.data(), d * 4, cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess && step) {
    if (!(*step > 0.0)) return fail(ctx, ESSA_ERR_INVALID_ARG, "cma_set: step must be positive");
    const float s32 = (float)*step;
    e = cudaMemcpy(s->sigma, step, 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(s->step32, &s32, 4, cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess && p_sigma) e = cudaMemcpy(s->p_sigma, p_sigma, d * 8, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && p_c) e = cudaMemcpy(s->p_c, p_c, d * 8, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && C) e = cudaMemcpy(s->C, C, (size_t)d * d * 8, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cma_set: copy");
  if (generation >= 0) s->generation = generation;
  return C ? decompose(ctx, s, stream) : ESSA_OK;
}

int32_t essa_cma_get(essa_ctx* ctx, essa_cma* s, double* mean, double* step, double* C, double* B, double* D, double* p_sigma,
                     double* p_c, int32_t* generation, int32_t* sweeps) {
  if (!ctx || !s) return ESSA_ERR_INVALID_ARG;
  const int d = s->d;
  cudaError_t e = cudaDeviceSynchronize();
  auto down = [&](void* dst, const void* src, size_t bytes) { if (e == cudaSuccess && dst) e = cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost); };
  down(mean, s->mean, d * 8); down(step, s->sigma, 8); down(C, s->C, (size_t)d * d * 8); down(B, s->B, (size_t)d * d * 8);
  down(D, s->D, d * 8); down(p_sigma, s->p_sigma, d * 8); down(p_c, s->p_c, d * 8);
  if (generation) *generation = s->generation;
  if (sweeps && e == cudaSuccess) {
    int32_t rot[kMaxSweeps + 1];
    e = cudaMemcpy(rot, s->rot, sizeof rot, cudaMemcpyDeviceToHost);
    int n = 0;
    while (n < kMaxSweeps && rot[n] != 0) ++n;
    *sweeps = n < kMaxSweeps ? n + 1 : kMaxSweeps;  // sweeps executed, the one that found nothing to rotate included
  }
  return check_cuda(ctx, e, "cma_get");
}

int32_t essa_cma_params(essa_cma* s, double* out9) {
  if (!s || !out9) return ESSA_ERR_INVALID_ARG;
  const double v[9] = {(double)s->mu, s->mu_eff, s->c_sigma, s->d_sigma, s->c_c, s->c_1, s->c_mu, s->c_m, s->chi_n};
  for (int i = 0; i < 9; ++i) out9[i] = v[i];
  return ESSA_OK;
}

}  // extern "C"
