// lqsgd_orthonormalize_noalloc: column orthonormalisation of one n x r factor that needs no
// workspace from the caller and allocates nothing.
//
// Who this is for.  Everything else in this library works inside a workspace the caller
// allocates up front.  Some callers have no way to do that: code that runs where device memory
// may not be requested at all (every byte of the GPU already belongs to another allocator or
// to a fixed start-up budget), or where cudaMalloc is off limits because it stalls the whole
// device while it runs (a serving loop, a callback invoked from inside another library).  Such a
// caller still owns its input and its output; what it lacks is the few hundred kilobytes of
// intermediate storage CholeskyQR needs (per-block Gram matrices, R^-1).  Here that storage is a
// fixed array compiled into the library image, so the call can be made with nothing but the two
// tensors.
//
// Consequences of the fixed array, which the caller must know:
//  * it exists once per GPU that loads this library, for the life of the process (about 1 MiB);
//  * sizes beyond kNoAllocMaxRows rows or 16 columns are refused with LQSGD_ERR_TOO_LARGE;
//  * every call on a device uses the same array: two calls whose kernels can overlap on the GPU
//    (different streams without an ordering between them) race on it.  Calls on one stream are
//    ordered and safe.  The array keeps whatever the previous call left; the parts that must
//    start from zero (the status word) are cleared by the call itself;
//  * the first call on each device looks up the array's device address (a host-side symbol
//    query, no allocation).  Make that first call outside of any stream capture.
#include "../../include/lqsgd.h"

#include <cuda_runtime.h>
#include <math.h>

#include <mutex>

namespace lqsgd { int record_cuda_failure(cudaError_t e, const char* what); }   // lqsgd_api.cu: text for lqsgd_last_cuda_error()

namespace {

constexpr int kR = 16;                        // internal column padding (rank <= 16)
constexpr int kRowsPerBlock = 128;
constexpr int kNoAllocMaxRows = LQSGD_NOALLOC_MAX_ROWS;
constexpr int kMaxBlocks = kNoAllocMaxRows / kRowsPerBlock;
constexpr double kPivotEps = 1e-10;           // same dependence criterion as the workspace path

// Scratch layout, in doubles: [kMaxBlocks][kR*kR] block Gram matrices | [kR*kR] R^-1 | status word.
constexpr size_t kGramOff = 0;
constexpr size_t kRinvOff = (size_t)kMaxBlocks * kR * kR;
constexpr size_t kStatusOff = kRinvOff + kR * kR;
constexpr size_t kScratchDoubles = kStatusOff + 32;

// File-scope device storage.  In host code this name is only a handle for the symbol: the
// address kernels can use comes from cudaGetSymbolAddress (see scratch_for_current_device).
static __device__ __align__(256) double g_noalloc_scratch[kScratchDoubles];

// Gram matrix of one block of 128 rows, fp64, into scratch; block 0 also clears the status word.
__global__ void __launch_bounds__(256)
noalloc_gram_kernel(const float* __restrict__ p_in, int n, int r, double* scratch) {
  __shared__ float rows[kRowsPerBlock][kR];
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && tid == 0) *reinterpret_cast<unsigned int*>(scratch + kStatusOff) = 0u;
  if (tid < kRowsPerBlock) {
    const int row = blockIdx.x * kRowsPerBlock + tid;
#pragma unroll
    for (int j = 0; j < kR; ++j) rows[tid][j] = (row < n && j < r) ? p_in[(size_t)row * r + j] : 0.f;
  }
  __syncthreads();
  const int i = tid / kR, j = tid % kR;
  double s = 0.0;
  for (int k = 0; k < kRowsPerBlock; ++k) s = fma((double)rows[k][i], (double)rows[k][j], s);
  scratch[kGramOff + (size_t)blockIdx.x * (kR * kR) + tid] = s;
}

// Sum of the block Grams (in block order), Cholesky R^T R = Gram, R^-1; one block, warp 0 factors.
__global__ void __launch_bounds__(256)
noalloc_cholesky_kernel(int nblocks, int r, double* scratch, unsigned int* status_out) {
  __shared__ double A[kR][kR + 1];
  __shared__ double X[kR][kR + 1];
  __shared__ double diag0[kR];
  __shared__ int dead[kR];
  const int tid = threadIdx.x;
  {
    double s = 0.0;
    for (int b = 0; b < nblocks; ++b) s += scratch[kGramOff + (size_t)b * (kR * kR) + tid];
    A[tid / kR][tid % kR] = s;
    X[tid / kR][tid % kR] = 0.0;
  }
  __syncthreads();
  if (tid < kR) { diag0[tid] = A[tid][tid]; dead[tid] = 0; }
  __syncthreads();
  if (tid < 32) {
    const int i = tid;
    for (int j = 0; j < r; ++j) {
      const double d = A[j][j];
      __syncwarp();
      const bool ok = (d > kPivotEps * diag0[j]) && (d < INFINITY);
      double lij = 0.0;
      if (ok) {
        const double ljj = sqrt(d);
        if (i == j) A[j][j] = ljj;
        if (i > j && i < r) { lij = A[i][j] / ljj; A[i][j] = lij; }
      } else {
        if (i == j) { A[j][j] = 1.0; dead[j] = 1; }
        if (i > j && i < r) A[i][j] = 0.0;
      }
      __syncwarp();
      if (ok && i > j && i < r)
        for (int k = j + 1; k <= i; ++k) A[i][k] -= lij * A[k][j];
      __syncwarp();
    }
    const int c = tid;
    if (c < r) {
      for (int row = c; row < r; ++row) {
        double x = 0.0;
        if (!dead[row]) {
          double s = (row == c) ? 1.0 : 0.0;
          for (int k = c; k < row; ++k) s -= A[row][k] * X[c][k];
          x = s / A[row][row];
        }
        if (dead[c]) x = 0.0;
        X[c][row] = x;
      }
    }
  }
  __syncthreads();
  {
    const int k = tid / kR, j = tid % kR;
    scratch[kRinvOff + tid] = (k <= j && j < r) ? X[k][j] : 0.0;
  }
  if (tid == 0) {
    unsigned int st = 0;
    for (int j = 0; j < r; ++j) st |= dead[j] ? LQSGD_STATUS_DEPENDENT_COLUMN : 0u;
    for (int j = 0; j < r; ++j) st |= (diag0[j] < INFINITY) ? 0u : LQSGD_STATUS_NONFINITE;
    *reinterpret_cast<unsigned int*>(scratch + kStatusOff) = st;
    if (status_out) *status_out = st;
  }
}

// P_out = P_in R^-1, accumulated in fp64, one thread per row.
__global__ void __launch_bounds__(kRowsPerBlock)
noalloc_apply_kernel(const float* p_in, float* p_out, int n, int r, const double* scratch) {
  __shared__ double Rinv[kR * kR];
  for (int k = threadIdx.x; k < kR * kR; k += kRowsPerBlock) Rinv[k] = scratch[kRinvOff + k];
  __syncthreads();
  const int row = blockIdx.x * kRowsPerBlock + threadIdx.x;
  if (row >= n) return;
  float p[kR];
#pragma unroll
  for (int j = 0; j < kR; ++j) p[j] = (j < r) ? p_in[(size_t)row * r + j] : 0.f;
#pragma unroll
  for (int j = 0; j < kR; ++j) {
    double s = 0.0;
#pragma unroll
    for (int k = 0; k <= j; ++k) s = fma((double)p[k], Rinv[k * kR + j], s);
    if (j < r) p_out[(size_t)row * r + j] = (float)s;
  }
}

// Device address of the scratch array on the current device, looked up once per device.
cudaError_t scratch_for_current_device(double** out) {
  static std::mutex mu;
  static double* cached[64] = {nullptr};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    double* ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int lqsgd_orthonormalize_noalloc(const float* dev_p_in, float* dev_p_out, int32_t rows, int32_t rank,
                                            uint32_t* dev_status_out, void* cuda_stream) {
  if (!dev_p_in || !dev_p_out || rows < 1 || rank < 1) return LQSGD_ERR_INVALID_ARG;
  if (rows > kNoAllocMaxRows || rank > kR) return LQSGD_ERR_TOO_LARGE;
  if ((reinterpret_cast<uintptr_t>(dev_p_in) & 3) || (reinterpret_cast<uintptr_t>(dev_p_out) & 3))
    return LQSGD_ERR_MISALIGNED;
  double* scratch = nullptr;
  cudaError_t e = scratch_for_current_device(&scratch);
  if (e != cudaSuccess) return lqsgd::record_cuda_failure(e, "cudaGetSymbolAddress(scratch)");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int nblocks = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
  // every launch is checked by itself, so that the error reported is this call's own
  noalloc_gram_kernel<<<nblocks, 256, 0, st>>>(dev_p_in, rows, rank, scratch);
  if ((e = cudaPeekAtLastError()) != cudaSuccess) return lqsgd::record_cuda_failure(e, "noalloc_gram_kernel launch");
  noalloc_cholesky_kernel<<<1, 256, 0, st>>>(nblocks, rank, scratch, dev_status_out);
  if ((e = cudaPeekAtLastError()) != cudaSuccess) return lqsgd::record_cuda_failure(e, "noalloc_cholesky_kernel launch");
  noalloc_apply_kernel<<<nblocks, kRowsPerBlock, 0, st>>>(dev_p_in, dev_p_out, rows, rank, scratch);
  if ((e = cudaPeekAtLastError()) != cudaSuccess) return lqsgd::record_cuda_failure(e, "noalloc_apply_kernel launch");
  return LQSGD_OK;
}
