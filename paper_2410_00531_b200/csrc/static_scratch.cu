// Allocation-free variant of the row-sharded projection + star-allreduce step.
//
// Some callers of this library cannot obtain device memory at the moment they need this
// step: code running inside a memory-capped plug-in or a real-time loop where cudaMalloc is
// forbidden (it may synchronise the device or fail late), or a host that has handed its whole
// memory budget to another component.  For them the N per-shard partial sums live in a fixed
// array that is part of the library image itself, so the call needs nothing but its inputs
// and outputs.
//
// Facts a user must know:
//  * The array holds TPI_STATIC_SCRATCH_FLOATS floats (256 KiB).  Every GPU that loads this
//    library keeps that much memory until the process exits, whether or not the call is used.
//  * A call with n_shards * rows above that limit is rejected with TPI_ERR_NOMEM.
//  * All calls on one GPU share the array.  It keeps whatever the last call left in it; that
//    is harmless because each call overwrites every element it later reads (nothing has to
//    start at zero).  Two calls that overlap on the GPU (different streams, or different host
//    threads) race on it: keep calls to this entry point in one stream order per GPU.
//  * The first call on each GPU looks up the array's device address (once per device, with
//    that device current).  Make that first call before starting any stream capture.
//  * The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
#include <cuda_runtime.h>

#include "../../include/tpi.h"
#include "../../include/tpi_ops.h"
#include "kernels.h"

using namespace tpi;

#define TPI_STATIC_SCRATCH_FLOATS 65536

// In HOST code this name is only a stand-in for the symbol, not a device address: the address a
// kernel may use comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_partials[TPI_STATIC_SCRATCH_FLOATS];

extern "C" void tpi_internal_set_error(const char* msg);  // defined next to tpi_last_error()

namespace {
constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices] = {};  // per device; written once, then only read

int scratch_for_current_device(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    tpi_internal_set_error("static scratch: no current CUDA device (or device index >= 64)");
    return TPI_ERR_CUDA;
  }
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_partials);
    if (e != cudaSuccess || !p) {
      tpi_internal_set_error("static scratch: cudaGetSymbolAddress failed");
      return TPI_ERR_CUDA;
    }
    g_scratch_addr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_addr[dev];
  return TPI_OK;
}
}  // namespace

extern "C" size_t tpi_op_static_scratch_floats(void) { return TPI_STATIC_SCRATCH_FLOATS; }

extern "C" int tpi_op_rowshard_project_static(int dtype, const void* W, const float* x_in, int rows, int Ks,
                                              int n_shards, float eps, float* x, float* xhat, void* stream) {
  if (rows < 1 || n_shards < 1 || Ks < 1 || !W || !x_in || !x || !xhat) {
    tpi_internal_set_error("tpi_op_rowshard_project_static: rows, Ks and n_shards must be >= 1 and no pointer may be null");
    return TPI_ERR_INVALID_ARG;
  }
  if ((size_t)n_shards * (size_t)rows > (size_t)TPI_STATIC_SCRATCH_FLOATS) {
    tpi_internal_set_error(
        "tpi_op_rowshard_project_static: n_shards * rows exceeds the built-in scratch of 65536 floats; "
        "use tpi_op_rowshard_project with caller-provided scratch");
    return TPI_ERR_NOMEM;
  }
  float* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc) return rc;
  // same two kernels as tpi_op_rowshard_project: per-shard partial sums, then the rank-ordered sum
  const int r1 = tpi_op_gemv_partials(dtype, W, x_in, rows, Ks, n_shards, scratch, stream);
  if (r1) return r1;
  return tpi_op_reduce_residual(scratch, n_shards, rows, eps, x, xhat, stream);
}
