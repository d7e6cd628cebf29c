// Internal to the library: the model object behind the C ABI and the helpers its translation units share
// (api.cu: set-up and weight packing; window.cu: the block ring on CUDA streams and its diagnostics;
// step_decode.cu / step_prefill.cu: the step drivers; inspect.cu: taps, cache access, statistics).
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <chrono>
#include <new>
#include <thread>
#include <vector>

#include <cuda_bf16.h>

#include "../../include/tpi.h"
#include "kernels.h"
#include "plan.h"
#include "ring.h"


using namespace tpi;

// Everything declared from here on is internal: not exported from the shared library.
#pragma GCC visibility push(hidden)

// ------------------------------------------------------------------------------ errors
int fail(int code, const char* fmt, ...);  // records the message for tpi_last_error() and returns code
#define CK(call)                                                                                          \
  do {                                                                                                    \
    cudaError_t e_ = (call);                                                                              \
    if (e_ != cudaSuccess)                                                                                \
      return fail(TPI_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
  } while (0)
#define TRY(call)                  \
  do {                             \
    int rc_ = (call);              \
    if (rc_ != TPI_OK) return rc_; \
  } while (0)

// ------------------------------------------------------------------------------ model
struct tpi_model {
  tpi_config cfg{};
  tpi_resources res{};
  tpi_fill_fn fill = nullptr;
  void* user = nullptr;
  int N = 1, window = 0;
  bool host_images = false;
  Plan plan{};
  char* dev = nullptr;
  char* host = nullptr;
  cudaStream_t cs = nullptr, ps = nullptr;
  bool own_cs = false, own_ps = false;
  int opt_graph = 1, opt_pdl = 1, opt_profile = 0, opt_tensor = 1, opt_rowshard_fused = 1;
  int position = 0;
  // window ring
  Ring ring;
  // partition of the kv heads (with their query-head groups) and of the FFN columns over the shards: prefix sums,
  // N + 1 entries each.  unequal = false: the uniform p_i = 1/N.  With unequal proportions the QKV rows are packed
  // in the unsharded order (their results do not depend on who computes them) and the row-sharded O / down
  // matrices follow the partition, which is where it decides the grouping of the partial sums.
  std::vector<int> kv0, f0;
  bool unequal = false;
  int retain_T = 0;                  // keep the FFN block of every T-th layer resident beside the window (0: none)
  std::vector<char> retained;        // per block
  std::vector<size_t> retained_off;  // byte offset of a retained block after the window slots
  size_t retained_bytes = 0;
  std::vector<cudaEvent_t> ev_loaded, ev_released;
  uint64_t link_bytes = 0;
  // graph of one resident decode step
  cudaGraphExec_t graph_exec = nullptr;
  int graph_launches = 0;
  // timing
  cudaEvent_t ev_t0 = nullptr, ev_t1 = nullptr, ev_done = nullptr;
  std::vector<cudaEvent_t> prof_ev;  // pairs around gate/up GEMVs (profile mode)
  size_t prof_used = 0;
  double prof_ms_sum = 0;
  uint32_t prof_samples = 0;
  // scheduler diagnostics (profile mode, decode only): event pairs around each block's kernels on the
  // compute stream (kinds 0 attention, 1 FFN) and around each block copy on the copy stream (kinds 2, 3)
  struct TimedPair { cudaEvent_t a, b; int kind; };
  std::vector<TimedPair> sched_pending;
  std::vector<cudaEvent_t> sched_free;
  cudaEvent_t sched_open = nullptr;
  bool sched_rec = false;
  double sched_sum[4] = {0, 0, 0, 0};
  uint32_t sched_n[4] = {0, 0, 0, 0};
  std::vector<cudaEvent_t> stall_ev;  // pairs around window waits (profile mode)
  size_t stall_used = 0;
  double stall_ms = 0;
  tpi_stats st{};
  double wait_deadline_s = 900.0;
  bool debug = false;   // TPI_DEBUG=1 at load: guard zones after every arena buffer, checked after every step
  bool desync = false;  // a host wait timed out with work in flight; cleared by tpi_reset / tpi_set_position
};

template <typename T>
static T* dptr(tpi_model* m, size_t off) { return reinterpret_cast<T*>(m->dev + off); }


// ------------------------------------------------------------------------------ shared helpers
// api.cu
void uniform_partition(tpi_model* m);
int wait_event(tpi_model* m, cudaEvent_t ev);
char* host_image(tpi_model* m, int block);  // block = 2*layer + (0 attn | 1 ffn)
size_t block_size(const tpi_model* m, int block);
char* resident_block(tpi_model* m, int block);
char* slot_ptr(tpi_model* m, int slot);
int quiesce(tpi_model* m);
int write_position(tpi_model* m, int p);
int fill_canaries(tpi_model* m);
int enqueue_canary_check(tpi_model* m, LaunchCtx& lc);  // no-op unless the arena was built with guard zones
// window.cu
cudaEvent_t sched_event(tpi_model* m);
void sched_harvest(tpi_model* m);
int start_window(tpi_model* m);
struct BlockRef {
  char* base;
  int slot;
};
int acquire_block(tpi_model* m, int block, BlockRef* r);
int release_block(tpi_model* m, int block);
// step_decode.cu
void drop_graph(tpi_model* m);
void harvest_profile(tpi_model* m);
int check_device_error(tpi_model* m, const int* io_err);
void recover_after_failed_step(tpi_model* m);  // after an enqueue that failed part-way

#pragma GCC visibility pop
