// Density-based centroid initialisation (DBCI, Section 3.1 of the LCD paper), offline, on a flat array of weights:
// sort; sigma from six nearest-rank percentiles; two seed clusters around the extreme weights; MinPts and eps from
// them; DBSCAN on the rest, which on sorted one-dimensional data is a neighbour count by two binary searches per
// point, a scan for the nearest core point on either side and a scan that numbers the clusters; lower medians.
// The sort and the scans are CUB device primitives; everything else is written here.  All comparisons and the
// few scalar operations are binary64 on the binary32 data, so every decision has one right answer.
#include <cuda_runtime.h>

#include <cub/device/device_radix_sort.cuh>
#include <cub/device/device_scan.cuh>

#include "common.h"

namespace lcd {

namespace {

struct DbciParams {        // device-side scalars shared by the kernels; mirrored into lcd_dbci_result at the end
  double sigma, eps;
  long long L, R;          // left cluster = sorted [0, L), right cluster = [R, n)
  long long min_pts;
  int n_mid;               // clusters found among the middle points
  int n_noise;
};

__device__ __forceinline__ long long lower_bound_d(const float* x, long long lo, long long hi, double v) {   // first >= v
  while (lo < hi) {
    const long long mid = (lo + hi) >> 1;
    if ((double)x[mid] < v) lo = mid + 1; else hi = mid;
  }
  return lo;
}
__device__ __forceinline__ long long upper_bound_d(const float* x, long long lo, long long hi, double v) {   // first > v
  while (lo < hi) {
    const long long mid = (lo + hi) >> 1;
    if ((double)x[mid] <= v) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void dbci_params_kernel(const float* __restrict__ x, long long n, DbciParams* __restrict__ P) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const long long first_pos = upper_bound_d(x, 0, n, 0.0);      // positives: [first_pos, n)
  const long long end_neg = lower_bound_d(x, 0, n, 0.0);        // negatives: [0, end_neg)
  const long long n_pos = n - first_pos, n_neg = end_neg;
  const double pct[3] = {0.6827, 0.9544, 0.9974};
  double sum = 0.0;
  for (int i = 0; i < 3; ++i) {
    if (n_pos > 0) {
      long long k = (long long)ceil(pct[i] * (double)n_pos) - 1;
      k = k < 0 ? 0 : (k > n_pos - 1 ? n_pos - 1 : k);
      sum += (double)x[first_pos + k];
    }
    if (n_neg > 0) {                                            // magnitudes ascending = values descending
      long long k = (long long)ceil(pct[i] * (double)n_neg) - 1;
      k = k < 0 ? 0 : (k > n_neg - 1 ? n_neg - 1 : k);
      sum += -(double)x[end_neg - 1 - k];
    }
  }
  const double sigma = sum / 12.0;
  long long L = upper_bound_d(x, 0, n, (double)x[0] + sigma);
  long long R = lower_bound_d(x, 0, n, (double)x[n - 1] - sigma);
  if (R < L) R = L;
  const long long min_pts = (n - R > 0) ? (L < n - R ? L : n - R) : L;
  P->sigma = sigma;
  P->eps = sigma / (double)min_pts;
  P->L = L;
  P->R = R;
  P->min_pts = min_pts;
  P->n_mid = 0;
  P->n_noise = 0;
}

// core flags of the middle points as scan inputs: fwd[i] = core ? i : -1, rev[m-1-i] = core ? (m-1-i) : -1 (indices in
// the reversed order, so that an inclusive max-scan of rev gives the nearest core at or after i)
__global__ void __launch_bounds__(256) dbci_core_kernel(const float* __restrict__ x, const DbciParams* __restrict__ P,
                                                        int* __restrict__ fwd, int* __restrict__ rev, long long cap) {
  const long long L = P->L, m = P->R - P->L;
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= cap) return;
  if (i >= m) { fwd[i] = -1; rev[i] = -1; return; }
  const float* y = x + L;
  const double v = (double)y[i], eps = P->eps;
  const long long min_pts = P->min_pts;
  bool core;
  if (min_pts <= 64) {
    // Only "at least MinPts neighbours" matters: count outwards over the sorted neighbours and stop at MinPts (the
    // same two comparisons as the searches below; MinPts is the size of the smaller outlier cluster, usually a few).
    const double a = v - eps, b = v + eps;
    long long cnt = 1;
    for (long long j = i - 1; j >= 0 && cnt < min_pts && !((double)y[j] < a); --j) ++cnt;
    for (long long j = i + 1; j < m && cnt < min_pts && (double)y[j] <= b; ++j) ++cnt;
    core = cnt >= min_pts;
  } else {
    const long long lo = lower_bound_d(y, 0, m, v - eps);
    const long long hi = upper_bound_d(y, 0, m, v + eps);
    core = hi - lo >= min_pts;
  }
  fwd[i] = core ? (int)i : -1;
  rev[m - 1 - i] = core ? (int)(m - 1 - i) : -1;
}

// start[i] = 1 when middle point i is a core point that no earlier core point reaches
__global__ void __launch_bounds__(256) dbci_start_kernel(const float* __restrict__ x, const DbciParams* __restrict__ P,
                                                         const int* __restrict__ prev_core, int* __restrict__ start,
                                                         long long cap) {
  const long long L = P->L, m = P->R - P->L;
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= cap) return;
  int s = 0;
  if (i < m && prev_core[i] == (int)i) {
    const int before = i > 0 ? prev_core[i - 1] : -1;
    s = (before < 0 || ((double)x[L + i] - (double)x[L + before]) > P->eps) ? 1 : 0;
  }
  start[i] = s;
}

struct MaxOp {
  __device__ __forceinline__ int operator()(int a, int b) const { return a > b ? a : b; }
};

// labels of all sorted points (0 left cluster, 1.. middle clusters in order, last = right cluster, -1 noise) and the
// first / last member of every cluster
__global__ void __launch_bounds__(256) dbci_label_kernel(const float* __restrict__ x, long long n, DbciParams* __restrict__ P,
                                                         const int* __restrict__ prev_core, const int* __restrict__ next_rev,
                                                         const int* __restrict__ cid1, int* __restrict__ labels,
                                                         int* __restrict__ first, int* __restrict__ last, int max_clusters) {
  const long long L = P->L, R = P->R, m = R - L;
  const long long g = (long long)blockIdx.x * 256 + threadIdx.x;
  const int n_mid = m > 0 ? cid1[m - 1] : 0;
  int lab = -2;                                  // -2: past the end of the array
  if (g < n) {
    if (g < L) lab = 0;
    else if (g >= R) lab = n_mid + 1;
    else {
      const long long i = g - L;
      const int pc = prev_core[i];
      const int nr = next_rev[m - 1 - i];
      const int nx = nr < 0 ? -1 : (int)(m - 1 - nr);
      if (pc == (int)i) {
        lab = cid1[i];
      } else {
        const double v = (double)x[g], eps = P->eps;
        const double dl = pc >= 0 ? v - (double)x[L + pc] : 1e300;
        const double dr = nx >= 0 ? (double)x[L + nx] - v : 1e300;
        if (dl <= eps && dl <= dr) lab = cid1[pc];
        else if (dr <= eps) lab = cid1[nx];
        else lab = -1;
      }
    }
    if (labels) labels[g] = lab;
  }
  // First and last member of every cluster, and the noise count.  Neighbours in the sorted array almost always share a
  // label, and millions of atomics on a handful of addresses serialise: a warp whose lanes agree sends one pair.
  const int lane = threadIdx.x & 31;
  const unsigned noise = __ballot_sync(0xffffffffu, lab == -1);
  if (lane == 0 && noise) atomicAdd(&P->n_noise, __popc(noise));
  const int lab0 = __shfl_sync(0xffffffffu, lab, 0);
  if (__all_sync(0xffffffffu, lab == lab0)) {
    if (lab0 >= 0 && lab0 < max_clusters) {
      if (lane == 0) atomicMin(first + lab0, (int)g);
      if (lane == 31) atomicMax(last + lab0, (int)g);
    }
  } else if (lab >= 0 && lab < max_clusters) {
    atomicMin(first + lab, (int)g);
    atomicMax(last + lab, (int)g);
  }
  if (g == 0) P->n_mid = n_mid;
}

__global__ void __launch_bounds__(256) dbci_fill_kernel(int* first, int* last, int count) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i < count) { first[i] = 0x7fffffff; last[i] = -1; }
}

// lower medians of the clusters in ascending order; result scalars
__global__ void dbci_centroid_kernel(const float* __restrict__ x, const DbciParams* __restrict__ P, const int* __restrict__ first,
                                     const int* __restrict__ last, int max_clusters, float* __restrict__ centroids,
                                     int max_centroids, lcd_dbci_result* __restrict__ out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int n_clusters = P->n_mid + 2;
  int w = 0;
  for (int c = 0; c < n_clusters && c < max_clusters; ++c) {
    if (last[c] < first[c]) continue;                      // the right cluster can be empty
    const int cnt = last[c] - first[c] + 1;
    if (w < max_centroids) centroids[w] = x[first[c] + (cnt - 1) / 2];
    ++w;
  }
  out->sigma = P->sigma;
  out->eps = P->eps;
  out->min_pts = P->min_pts;
  out->left = P->L;
  out->right = 0;          // filled by the caller-visible convention below
  out->n_centroids = w;
  out->n_noise = P->n_noise;
  out->n_clusters_found = n_clusters;
}

__global__ void dbci_right_kernel(const DbciParams* P, long long n, lcd_dbci_result* out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) out->right = n - P->R;
}

size_t al256(size_t v) { return (v + 255) & ~(size_t)255; }

struct DbciLayout {
  size_t sorted, fwd, rev, start, first, last, params, cub, total, cub_bytes;
};
DbciLayout dbci_layout(int64_t n, int max_clusters) {
  DbciLayout l;
  size_t off = 0;
  l.sorted = off; off += al256((size_t)n * sizeof(float));
  l.fwd = off; off += al256((size_t)n * sizeof(int));
  l.rev = off; off += al256((size_t)n * sizeof(int));
  l.start = off; off += al256((size_t)n * sizeof(int));
  l.first = off; off += al256((size_t)max_clusters * sizeof(int));
  l.last = off; off += al256((size_t)max_clusters * sizeof(int));
  l.params = off; off += al256(sizeof(DbciParams));
  size_t s1 = 0, s2 = 0, s3 = 0;
  cub::DeviceRadixSort::SortKeys(nullptr, s1, (const float*)nullptr, (float*)nullptr, (int)n);
  cub::DeviceScan::InclusiveScan(nullptr, s2, (int*)nullptr, (int*)nullptr, MaxOp(), (int)n);
  cub::DeviceScan::InclusiveSum(nullptr, s3, (int*)nullptr, (int*)nullptr, (int)n);
  l.cub_bytes = s1 > s2 ? (s1 > s3 ? s1 : s3) : (s2 > s3 ? s2 : s3);
  l.cub = off; off += al256(l.cub_bytes);
  l.total = off;
  return l;
}

}  // namespace

size_t dbci_workspace_bytes(int64_t n, int max_centroids) { return dbci_layout(n, max_centroids + 2).total; }

lcd_status launch_dbci(const float* weights, int64_t n, void* workspace, float* centroids, int max_centroids,
                       int32_t* labels, float* sorted_out, lcd_dbci_result* result, void* stream) {
  const int max_clusters = max_centroids + 2;
  const DbciLayout l = dbci_layout(n, max_clusters);
  uint8_t* base = static_cast<uint8_t*>(workspace);
  float* x = reinterpret_cast<float*>(base + l.sorted);
  int* fwd = reinterpret_cast<int*>(base + l.fwd);
  int* rev = reinterpret_cast<int*>(base + l.rev);
  int* start = reinterpret_cast<int*>(base + l.start);
  int* first = reinterpret_cast<int*>(base + l.first);
  int* last = reinterpret_cast<int*>(base + l.last);
  DbciParams* P = reinterpret_cast<DbciParams*>(base + l.params);
  void* tmp = base + l.cub;
  size_t tmp_bytes = l.cub_bytes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const unsigned blocks = (unsigned)((n + 255) / 256);
  cudaError_t e = cub::DeviceRadixSort::SortKeys(tmp, tmp_bytes, weights, x, (int)n, 0, 32, s);
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  dbci_params_kernel<<<1, 32, 0, s>>>(x, n, P);
  dbci_core_kernel<<<blocks, 256, 0, s>>>(x, P, fwd, rev, n);
  tmp_bytes = l.cub_bytes;
  e = cub::DeviceScan::InclusiveScan(tmp, tmp_bytes, fwd, fwd, MaxOp(), (int)n, s);       // nearest core at or before
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  tmp_bytes = l.cub_bytes;
  e = cub::DeviceScan::InclusiveScan(tmp, tmp_bytes, rev, rev, MaxOp(), (int)n, s);       // the same from the right
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  dbci_start_kernel<<<blocks, 256, 0, s>>>(x, P, fwd, start, n);
  tmp_bytes = l.cub_bytes;
  e = cub::DeviceScan::InclusiveSum(tmp, tmp_bytes, start, start, (int)n, s);             // cluster number (from 1)
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  dbci_fill_kernel<<<(unsigned)((max_clusters + 255) / 256), 256, 0, s>>>(first, last, max_clusters);
  dbci_label_kernel<<<blocks, 256, 0, s>>>(x, n, P, fwd, rev, start, labels, first, last, max_clusters);
  dbci_centroid_kernel<<<1, 32, 0, s>>>(x, P, first, last, max_clusters, centroids, max_centroids, result);
  dbci_right_kernel<<<1, 32, 0, s>>>(P, n, result);
  if (sorted_out) {
    e = cudaMemcpyAsync(sorted_out, x, (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) { set_cuda_error((int)e); return LCD_ERR_CUDA; }
  return LCD_OK;
}

}  // namespace lcd
