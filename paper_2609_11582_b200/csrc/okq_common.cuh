// Host-side helpers: argument checks and CUDA error capture.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/okq.h"
#include "okq_layout.cuh"

namespace okq {

void set_last_cuda_error(int e);
int sm_count();   // SMs of the current device (cached per thread)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// shape checks shared by every entry point; `need_ptrs` also checks the buffers
okq_status check_cache(const okq_cache* c, bool need_ptrs);

inline CacheView make_view(const okq_cache* c) {
  CacheView v;
  v.n_layers = c->n_layers; v.batch = c->batch; v.n_kv_heads = c->n_kv_heads; v.n_q_heads = c->n_q_heads;
  v.capacity = c->capacity;
  v.fmt = c->meta_format;
  v.sched = c->schedule;
  v.records = static_cast<unsigned char*>(c->records);
  v.modality = c->modality;
  v.k_tail = static_cast<__half*>(c->k_tail);
  v.v_tail = static_cast<__half*>(c->v_tail);
  v.seq_len = c->seq_len;
  v.status = c->status;
  return v;
}

// Function attributes (dynamic shared memory size) are per device: `mask` remembers, per calling thread and
// call site, the devices on which they have been set.  Returns true when the current device still needs them.
inline bool attr_needed(unsigned long long& mask, int& dev_out) {
  int dev = 0;
  cudaGetDevice(&dev);
  dev_out = dev;
  return dev < 0 || dev >= 64 || !((mask >> dev) & 1ull);
}
inline void attr_done(unsigned long long& mask, int dev) {
  if (dev >= 0 && dev < 64) mask |= 1ull << dev;
}

inline okq_status launch_status() {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return OKQ_ERR_CUDA;
  }
  return OKQ_OK;
}

}  // namespace okq
