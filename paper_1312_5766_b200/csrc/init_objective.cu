// Algorithm 1's initialisation (n_j = ||x_j||^2, r = y - X beta, delta_j = C) and the Lasso
// objective of Eq. 1 with squared loss, F = 1/2 ||r||^2 + lambda ||beta||_1.  Neither is on the
// per-round path; both accumulate in FP64 in a fixed order.
#include "strads_internal.cuh"

namespace strads {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the CTA (blockDim.x a multiple of 32, <= 1024); result valid in thread 0.
__device__ double block_sum(double v) {
  __shared__ double part[32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) part[wid] = v;
  __syncthreads();
  double s = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += part[w];
  return s;
}

// dense: one CTA per column (grid-strided); also tracks max |x|.
__global__ void __launch_bounds__(256) k_colnorm2_dense(Problem p) {
  for (long long j = blockIdx.x; j < p.J; j += gridDim.x) {
    const float* x = p.xv + j * p.ld;
    double acc = 0.0;
    const long long n4 = p.N >> 2;
    for (long long i = threadIdx.x; i < n4; i += blockDim.x) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i);
      acc += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
    }
    for (long long i = (n4 << 2) + threadIdx.x; i < p.N; i += blockDim.x) acc += (double)x[i] * x[i];
    const double s = block_sum(acc);
    if (threadIdx.x == 0) p.n2[j] = s;
  }
}

// CSC: one warp per column.
__global__ void __launch_bounds__(256) k_colnorm2_csc(Problem p) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  float amax = 0.f;
  for (long long j = warp; j < p.J; j += nwarps) {
    const long long b = p.xptr[j], e = p.xptr[j + 1];
    double acc = 0.0;
    for (long long q = b + lane; q < e; q += 32) {
      const float v = __ldg(p.xv + q);
      acc += (double)v * v;
      amax = fmaxf(amax, fabsf(v));
    }
    acc = warp_sum(acc);
    if (lane == 0) p.n2[j] = acc;
  }
  // max |x| (order-independent, so an integer atomic on the bit pattern of a non-negative float is exact)
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0 && amax > 0.f) atomicMax(reinterpret_cast<unsigned int*>(&p.st->x_abs_max), __float_as_uint(amax));
}

__global__ void k_fill_state(Problem p) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long j = i; j < p.J; j += stride) p.delta[j] = p.c_init;
  const bool logistic = (p.flags & STRADS_FLAG_LOGISTIC) != 0;        // margin 0: resid = y - sigma(0)
  for (long long r = i; r < p.N; r += stride) {
    p.resid[r] = logistic ? p.y[r] - 0.5f : p.y[r];
    if (logistic) p.margin[r] = 0.f;
  }
  if (i == 0) {
    DeviceState* st = p.st;
    st->round = 0;
    for (int k = 0; k < 4; ++k) { st->totals[k] = 0; st->counts[k] = 0; }
    st->status = 0; st->hist_ticket = 0; st->sure_count = 0; st->boundary_count = 0;
    st->objective = 0.0;
  }
  for (long long b = i; b < kHistBins; b += stride) p.hist[b] = 0;
  for (long long a = i; a < p.n_keep; a += stride) p.dot_ticket[a] = 0;
}

// r -= X beta for a non-zero starting point, dense: one thread per row, columns in index order.
__global__ void k_resid_dense(Problem p) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.N || !p.st->beta0_nonzero) return;
  double acc = 0.0;
  for (long long j = 0; j < p.J; ++j) {
    const float b = p.beta[j];
    if (b != 0.f) acc += (double)p.xv[j * p.ld + i] * (double)b;
  }
  if (p.flags & STRADS_FLAG_LOGISTIC) {
    p.margin[i] = (float)acc;
    p.resid[i] = (float)((double)p.y[i] - sigmoid64((double)(float)acc));
  } else {
    p.resid[i] = (float)((double)p.y[i] - acc);
  }
}

// CSC: one CTA walks the columns in index order; rows inside a column are distinct, so the
// threads of one column never collide and the order of additions per row is fixed.
__global__ void __launch_bounds__(1024) k_resid_csc(Problem p) {
  if (!p.st->beta0_nonzero) return;
  for (long long j = 0; j < p.J; ++j) {
    const float b = p.beta[j];
    if (b == 0.f) continue;
    for (long long q = p.xptr[j] + threadIdx.x; q < p.xptr[j + 1]; q += blockDim.x) {
      const int r = p.xrow[q];
      if (p.flags & STRADS_FLAG_LOGISTIC) p.margin[r] = (float)((double)p.margin[r] + (double)p.xv[q] * (double)b);
      else p.resid[r] = (float)((double)p.resid[r] - (double)p.xv[q] * (double)b);
    }
    __syncthreads();
  }
  if (p.flags & STRADS_FLAG_LOGISTIC)
    for (long long r = threadIdx.x; r < p.N; r += blockDim.x)
      p.resid[r] = (float)((double)p.y[r] - sigmoid64((double)p.margin[r]));
}

__global__ void k_any_nonzero(Problem p) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < p.J; j += stride)
    if (p.beta[j] != 0.f) p.st->beta0_nonzero = 1;
}

__global__ void __launch_bounds__(256) k_objective_partial(Problem p) {
  double sq = 0.0, l1 = 0.0;
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  if (p.flags & STRADS_FLAG_LOGISTIC) {                  // sum_i log(1 + exp(m_i)) - y_i m_i (twice: halved with the squares' 1/2)
    for (long long i = i0; i < p.N; i += stride) {
      const double m = p.margin[i];
      sq += 2.0 * ((m > 0.0 ? m : 0.0) + log1p(exp(-fabs(m))) - (double)p.y[i] * m);
    }
  } else {
    for (long long i = i0; i < p.N; i += stride) { const double r = p.resid[i]; sq += r * r; }
  }
  for (long long j = i0; j < p.J; j += stride) l1 += fabs((double)p.beta[j]);
  const double a = block_sum(sq);
  const double b = block_sum(l1);
  if (threadIdx.x == 0) { p.obj_partial[2 * blockIdx.x] = a; p.obj_partial[2 * blockIdx.x + 1] = b; }
}

__global__ void k_objective_final(Problem p) {
  if (threadIdx.x == 0) {
    double sq = 0.0, l1 = 0.0;
    for (int b = 0; b < kObjBlocks; ++b) { sq += p.obj_partial[2 * b]; l1 += p.obj_partial[2 * b + 1]; }
    p.st->objective = 0.5 * sq + (double)p.lambda * l1;
  }
}

// State of a further scheduler: zeroed like the first one's, with what init measured copied over and its
// first turn (round index = its own index).
__global__ void k_scheduler_state(Problem p, const DeviceState* first) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
  if (i == 0) {
    DeviceState* st = p.st;
    st->round = (unsigned long long)p.part_index;
    st->x_abs_max = first->x_abs_max;
    st->beta0_nonzero = first->beta0_nonzero;
  }
  for (int b = i; b < kHistBins; b += stride) p.hist[b] = 0;
  for (int a = i; a < p.n_keep; a += stride) p.dot_ticket[a] = 0;
}

}  // namespace

cudaError_t launch_init_scheduler(const Problem& p, const Problem& first, cudaStream_t s) {
  const cudaError_t e = cudaMemsetAsync(p.st, 0, sizeof(DeviceState), s);
  if (e != cudaSuccess) return e;
  k_scheduler_state<<<16, 256, 0, s>>>(p, first.st);
  return cudaGetLastError();
}

cudaError_t launch_init(const Problem& p, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(p.st, 0, sizeof(DeviceState), s);
  if (e != cudaSuccess) return e;
  k_fill_state<<<p.sm_count * 4, 256, 0, s>>>(p);
  if (p.layout == STRADS_DENSE_COLMAJOR) {
    const long long blocks = p.J < (long long)p.sm_count * 16 ? p.J : (long long)p.sm_count * 16;
    k_colnorm2_dense<<<(unsigned)blocks, 256, 0, s>>>(p);
  } else {
    k_colnorm2_csc<<<p.sm_count * 8, 256, 0, s>>>(p);
  }
  return cudaGetLastError();
}

// resid = y - X beta for beta != 0 (init already set resid = y; nothing happens when beta is all zero).
cudaError_t launch_resid_from_beta(const Problem& p, cudaStream_t s) {
  k_any_nonzero<<<p.sm_count * 4, 256, 0, s>>>(p);
  if (p.layout == STRADS_DENSE_COLMAJOR)
    k_resid_dense<<<(unsigned)((p.N + 127) / 128), 128, 0, s>>>(p);
  else
    k_resid_csc<<<1, 1024, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_objective(const Problem& p, cudaStream_t s) {
  k_objective_partial<<<kObjBlocks, 256, 0, s>>>(p);
  k_objective_final<<<1, 32, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace strads
