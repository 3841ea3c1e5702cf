// SAP step 2, dense X: conflict bits of all candidate pairs from the candidate Gram
// G_ab = x_{c_a}^T x_{c_b} (Algorithm 1's rho test uses |x_j^T x_k| on standardised columns;
// here the cosine |G_ab| / (||x_a|| ||x_b||) so that columns need not be exactly unit norm).
//
// FP32 SIMT version: 128 x 128 output tiles over the upper triangle of tile pairs, 8 x 8 outputs
// per thread, K (= the N samples) in slices of 16 through double-buffered shared memory.  The
// operands are the candidate columns themselves (each is contiguous in a column-major X), fetched
// through the candidate list -- no packed copy.  The epilogue thresholds in FP64 and emits one bit
// per pair; the FP32 Gram is written only when a debug buffer is given.
#include "strads_internal.cuh"

namespace strads {
namespace {

constexpr int BM = 128, BK = 16, kThreads = 256;

__device__ __forceinline__ float4 load_k4(const float* col, long long k, long long N) {
  // col is 16-byte aligned and padded to a multiple of 4 floats, so a float4 that starts below N is in bounds
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col != nullptr && k < N) {
    v = __ldg(reinterpret_cast<const float4*>(col + k));
    if (k + 3 >= N) {
      if (k + 1 >= N) v.y = 0.f;
      if (k + 2 >= N) v.z = 0.f;
      v.w = 0.f;
    }
  }
  return v;
}

__global__ void __launch_bounds__(kThreads) k_gram_dense_simt(Problem p, const int* __restrict__ cand, int n_cand,
                                                               int n_tiles, float* __restrict__ gram_dbg) {
  chain_begin();
  if (blockIdx.x == 0 && threadIdx.x == 0) p.st->edges_off = 1;     // this kernel sets bits without listing the pairs
  __shared__ __align__(16) float As[2][BK][BM];
  __shared__ __align__(16) float Bs[2][BK][BM];
  __shared__ double n2a[BM], n2b[BM];
  __shared__ unsigned int bits[BM][4];

  // linear index -> (ti, tj) with ti <= tj
  int ti = 0, rem = blockIdx.x;
  while (rem >= n_tiles - ti) { rem -= n_tiles - ti; ++ti; }
  const int tj = ti + rem;

  const int tid = threadIdx.x;
  const int lrow = tid & 127, lhalf = tid >> 7;            // loader role: one tile row, 8 of the 16 k
  const int ty = tid >> 4, tx = tid & 15;                   // compute role

  const int ga = ti * BM + lrow, gb = tj * BM + lrow;
  const float* colA = ga < n_cand ? p.xv + (long long)cand[ga] * p.ld : nullptr;
  const float* colB = gb < n_cand ? p.xv + (long long)cand[gb] * p.ld : nullptr;
  if (tid < BM) {
    n2a[tid] = ga < n_cand ? coupling_n2(p, cand[ga]) : 0.0;
    n2b[tid] = gb < n_cand ? coupling_n2(p, cand[gb]) : 0.0;
    bits[tid][0] = bits[tid][1] = bits[tid][2] = bits[tid][3] = 0u;
  }

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  const long long N = p.N;
  const int n_slices = (int)((N + BK - 1) / BK);
  float4 ra0, ra1, rb0, rb1;
  {
    const long long k = lhalf * 8;
    ra0 = load_k4(colA, k, N); ra1 = load_k4(colA, k + 4, N);
    rb0 = load_k4(colB, k, N); rb1 = load_k4(colB, k + 4, N);
  }
  auto stash = [&](int buf) {
    const int k = lhalf * 8;
    As[buf][k + 0][lrow] = ra0.x; As[buf][k + 1][lrow] = ra0.y; As[buf][k + 2][lrow] = ra0.z; As[buf][k + 3][lrow] = ra0.w;
    As[buf][k + 4][lrow] = ra1.x; As[buf][k + 5][lrow] = ra1.y; As[buf][k + 6][lrow] = ra1.z; As[buf][k + 7][lrow] = ra1.w;
    Bs[buf][k + 0][lrow] = rb0.x; Bs[buf][k + 1][lrow] = rb0.y; Bs[buf][k + 2][lrow] = rb0.z; Bs[buf][k + 3][lrow] = rb0.w;
    Bs[buf][k + 4][lrow] = rb1.x; Bs[buf][k + 5][lrow] = rb1.y; Bs[buf][k + 6][lrow] = rb1.z; Bs[buf][k + 7][lrow] = rb1.w;
  };
  stash(0);
  __syncthreads();

  for (int s = 0; s < n_slices; ++s) {
    const int buf = s & 1;
    if (s + 1 < n_slices) {
      const long long k = (long long)(s + 1) * BK + lhalf * 8;
      ra0 = load_k4(colA, k, N); ra1 = load_k4(colA, k + 4, N);
      rb0 = load_k4(colB, k, N); rb1 = load_k4(colB, k + 4, N);
    }
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (s + 1 < n_slices) stash(buf ^ 1);
    __syncthreads();
  }

  // epilogue: |G_ab| >= rho sqrt(n_a n_b)  <=>  the pair may not be updated together
  const double rho = (double)p.rho;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int la = (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    const int a = ti * BM + la;
    unsigned int nib0 = 0u, nib1 = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int lb = (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
      const int b = tj * BM + lb;
      const double den = sqrt(n2a[la] * n2b[lb]);
      const bool hit = a < n_cand && b < n_cand && a != b && den > 0.0 && fabs((double)acc[i][j]) >= rho * den;
      if (j < 4) nib0 |= (unsigned)hit << j; else nib1 |= (unsigned)hit << (j - 4);
      if (gram_dbg != nullptr && a < n_cand && b < n_cand) {
        gram_dbg[(long long)a * n_cand + b] = acc[i][j];
        gram_dbg[(long long)b * n_cand + a] = acc[i][j];
      }
    }
    if (nib0) atomicOr(&bits[la][tx >> 3], nib0 << ((tx & 7) * 4));
    if (nib1) atomicOr(&bits[la][2 + (tx >> 3)], nib1 << ((tx & 7) * 4));
  }
  __syncthreads();
  for (int e = tid; e < BM * 4; e += kThreads) {
    const int la = e >> 2, w = e & 3;
    const int a = ti * BM + la, word = tj * 4 + w;
    if (a < n_cand && word < p.mask_words) p.conflict[(long long)a * p.mask_words + word] = bits[la][w];
  }
}

}  // namespace

cudaError_t launch_gram_dense_simt(const Problem& p, const int* cand, int n_cand, float* gram_dbg, cudaStream_t s) {
  const int n_tiles = (n_cand + BM - 1) / BM;
  const int blocks = n_tiles * (n_tiles + 1) / 2;
  return launch_chained(k_gram_dense_simt, blocks, kThreads, 0, s, p, cand, n_cand, n_tiles, gram_dbg);
}

}  // namespace strads
