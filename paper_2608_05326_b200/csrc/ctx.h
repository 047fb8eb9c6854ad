// Private definition of the cache handle, shared by the translation units of the host API.
#pragma once

#include <string>
#include <vector>

#include "decode_attn.cuh"
#include "kernels.cuh"

namespace qevict {

struct LayerMirror {  // what the host must know without reading device memory (same for every sequence)
  bool prefilled = false;
  bool has_open = false;
  int open_fill = 0;
  int n_windows = 0;
  int aged = 0;  // filled windows waiting for a routing event
};

constexpr int SM_COUNT_FALLBACK = 148;

// Makes the cache's device current for the duration of an API call and puts the caller's device back afterwards.
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) {
      err = cudaSetDevice(dev);
      switched = err == cudaSuccess;
    }
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
  DeviceGuard(const DeviceGuard&) = delete;
  DeviceGuard& operator=(const DeviceGuard&) = delete;
};

}  // namespace qevict

struct qevict_ctx {
  qevict_config cfg;
  qevict::Geometry geo;
  qevict::State st;
  std::vector<qevict::LayerMirror> layers;
  std::vector<uint32_t> mig_epoch;    // per layer: routing events launched with this layer first in the call
  std::string last_error;
  uint64_t launches = 0;
  uint64_t decode_steps = 0;
  qevict::decode_launch_fn decode_fn = nullptr;
  int forced_splits = 0;
  int sm_count = qevict::SM_COUNT_FALLBACK;
  bool timing = false;
  bool broken = false;                // a launch failed half way through a step: the tables and the host's mirror may
                                      // disagree from here on, every later call is refused
  std::vector<cudaEvent_t> ev_pool;   // start/stop pairs, reused
  std::vector<int> ev_kind;           // kernel index of each pair
  size_t ev_used = 0;
  cudaEvent_t out_ready = nullptr;  // recorded behind the last operation that writes a host entry point's `out`
  char* stage_q = nullptr;    // device staging for the host-buffer entry point
  char* stage_k = nullptr;
  char* stage_v = nullptr;
  char* stage_out = nullptr;
#ifdef QEVICT_TRACE
  uint32_t trace_calls = 0;   // API calls traced since the timeline was last read
#endif
};

namespace qevict {

// Splits per (unit, KV head) of the attention kernel for a call over `n_units` units.
int choose_splits(const qevict_ctx* h, int n_units);
// Argument and call-order checks of a decode step over layers [l0, l1); nullptr if the step may run (nothing is
// enqueued before this has passed), else the status in *st and the message.
const char* decode_precheck(const qevict_ctx* h, int layer, const void* q, const void* k_new, const void* v_new,
                            const void* out, int* l0, int* l1, qevict_status* st);

}  // namespace qevict
