// Status strings, size helpers and argument validation of the C ABI.
#include "okq_common.cuh"

namespace okq {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

int sm_count() {
  static thread_local int cached_dev = -1, cached = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev != cached_dev) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached = n;
    cached_dev = dev;
  }
  return cached;
}

okq_status check_cache(const okq_cache* c, bool need_ptrs) {
  if (!c) return OKQ_ERR_INVALID_ARG;
  if (c->head_dim != OKQ_HEAD_DIM || c->window != OKQ_WINDOW) return OKQ_ERR_UNSUPPORTED;
  if (c->n_layers <= 0 || c->batch <= 0 || c->n_kv_heads <= 0 || c->n_q_heads <= 0 || c->capacity <= 0)
    return OKQ_ERR_INVALID_ARG;
  if (c->capacity % OKQ_WINDOW != 0) return OKQ_ERR_INVALID_ARG;
  if (c->meta_format != OKQ_META_FP16 && c->meta_format != OKQ_META_MXFP4) return OKQ_ERR_UNSUPPORTED;
  if (c->schedule != OKQ_SCHEDULE_WINDOW && c->schedule != OKQ_SCHEDULE_CAPTION) return OKQ_ERR_UNSUPPORTED;
  if (c->n_q_heads % c->n_kv_heads != 0 || c->n_q_heads / c->n_kv_heads > OKQ_MAX_GROUP) return OKQ_ERR_UNSUPPORTED;
  if (need_ptrs) {
    if (!c->records || !c->modality || !c->k_tail || !c->v_tail || !c->seq_len || !c->status)
      return OKQ_ERR_INVALID_ARG;
    if (!aligned16(c->records) || !aligned16(c->modality) || !aligned16(c->k_tail) || !aligned16(c->v_tail) ||
        !aligned16(c->seq_len) || !aligned16(c->status))
      return OKQ_ERR_ALIGNMENT;
  }
  return OKQ_OK;
}

}  // namespace okq

extern "C" {

const char* okq_status_string(okq_status s) {
  switch (s) {
    case OKQ_OK: return "ok";
    case OKQ_ERR_INVALID_ARG: return "invalid argument";
    case OKQ_ERR_UNSUPPORTED: return "unsupported shape (head_dim 128, window 32, GQA group <= 8 only)";
    case OKQ_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case OKQ_ERR_CAPACITY: return "sequence would exceed cache capacity";
    case OKQ_ERR_WORKSPACE: return "decode workspace too small";
    case OKQ_ERR_CUDA: return "CUDA runtime error";
    case OKQ_ERR_TIMEOUT: return "bounded device wait timed out";
  }
  return "unknown status";
}

int okq_last_cuda_error(void) { return okq::g_last_cuda_error; }

okq_status okq_cache_sizes(const okq_cache* c, size_t out[6]) {
  okq_status st = okq::check_cache(c, false);
  if (st != OKQ_OK) return st;
  if (!out) return OKQ_ERR_INVALID_ARG;
  size_t units = (size_t)c->n_layers * c->batch * c->n_kv_heads;
  okq::CacheView v{};
  v.capacity = c->capacity;
  v.fmt = c->meta_format;
  v.sched = c->schedule;
  out[0] = units * v.unit_bytes();
  out[0] = (out[0] + 15) & ~(size_t)15;
  out[1] = (size_t)c->batch * c->capacity;
  out[2] = units * (size_t)v.k_slots() * OKQ_HEAD_DIM * 2;
  out[3] = units * (size_t)v.v_slots() * OKQ_HEAD_DIM * 2;
  out[4] = (size_t)c->n_layers * c->batch * sizeof(int32_t);
  out[5] = 16;
  return OKQ_OK;
}

}  // extern "C"
