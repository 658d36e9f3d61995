// Context life cycle, cost tables, cross-step state and status of the CAST library.
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "cast_internal.h"

using namespace cast;

namespace {

__global__ void init_state_kernel(DevState* st, double* fifo_vals, int32_t* fifo_cnt, int nbuf, int R) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) {
    memset(st, 0, sizeof(DevState));
    st->u_last = 1.0;
  }
  if (i < nbuf) {  // every buffer A_i starts as {1}
    fifo_cnt[i] = 1;
    fifo_vals[(size_t)i * R] = 1.0;
    for (int k = 1; k < R; ++k) fifo_vals[(size_t)i * R + k] = 0.0;
  }
}

template <typename T>
cudaError_t dev_alloc(T** p, size_t n) {
  cudaError_t e = cudaMalloc((void**)p, n * sizeof(T));
  if (e == cudaSuccess) e = cudaMemset(*p, 0, n * sizeof(T));
  return e;
}

void free_all(cast_ctx* c) {
  cudaFree(c->pool_score); cudaFree(c->pool_token); cudaFree(c->pool_parent); cudaFree(c->pool_depth);
  cudaFree(c->pool_kept); cudaFree(c->retained); cudaFree(c->lsort); cudaFree(c->lscore); cudaFree(c->state);
  cudaFree(c->attn_worklist);
  cudaFree(c->layer_ticket); cudaFree(c->seq_ticket); cudaFree(c->tail_vs); cudaFree(c->tail_sorted); cudaFree(c->tail_tok);
  cudaFree(c->fifo_vals); cudaFree(c->fifo_cnt); cudaFree(c->sel_score); cudaFree(c->sel_value);
  cudaFree(c->sel_idx); cudaFree(c->acc_part); cudaFree(c->compact_ticket); cudaFree(c->attn_ws); cudaFree(c->attn_tc_ws);
  if (c->tables) {
    for (auto& kv : *c->tables) cudaFree(kv.second.storage);
    delete c->tables;
  }
}

}  // namespace

extern "C" const char* cast_status_string(cast_status s) {
  switch (s) {
    case CAST_OK: return "ok";
    case CAST_ERR_INVALID_ARG: return "invalid argument";
    case CAST_ERR_SHAPE: return "unsupported shape";
    case CAST_ERR_CAPACITY: return "capacity exceeded";
    case CAST_ERR_DTYPE: return "unsupported dtype";
    case CAST_ERR_COST_TABLE: return "cost table missing or not strictly increasing";
    case CAST_ERR_BAD_TREE: return "malformed tree";
    case CAST_ERR_BAD_PAGE: return "page index out of range";
    case CAST_ERR_NONFINITE: return "non-finite logits";
    case CAST_ERR_TIMEOUT: return "device wait timed out";
    case CAST_ERR_CUDA: return "CUDA error";
  }
  return "unknown";
}

extern "C" cast_status cast_create(const cast_config* cfg, cast_ctx** out) {
  if (!cfg || !out) return CAST_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->max_batch < 1 || cfg->vocab < 1 || cfg->top_k < 1 || cfg->max_depth < 1 || cfg->max_tree < 1 ||
      cfg->total_token < 1 || cfg->max_width < 0 || cfg->fifo_len < 1)
    return CAST_ERR_INVALID_ARG;
  if (cfg->pool_mode < 0 || cfg->pool_mode > 1) return CAST_ERR_INVALID_ARG;
  int W = cfg->max_width > 0 ? cfg->max_width : cfg->top_k;
  if (cfg->max_batch > CAST_MAX_BATCH || cfg->top_k > CAST_MAX_TOP_K || W > CAST_MAX_WIDTH ||
      cfg->max_depth > CAST_MAX_DEPTH || cfg->max_tree > CAST_MAX_TREE || cfg->total_token > cfg->max_tree ||
      cfg->top_k > cfg->vocab || cfg->fifo_len > kMaxFifo)
    return CAST_ERR_CAPACITY;
  if (!(cfg->C1 > 0) || !(cfg->C2 > 0) || !(cfg->C3 > 0)) return CAST_ERR_INVALID_ARG;

  cast_ctx* c = new (std::nothrow) cast_ctx();
  if (!c) return CAST_ERR_CUDA;
  memset(c, 0, sizeof(*c));
  c->cfg = *cfg;
  c->W = W;
  // layer 1 has one logits row (K candidates); layers 2..H have at most W rows each.
  c->P = 1 + cfg->top_k + (cfg->max_depth - 1) * W * cfg->top_k;
  c->words = (cfg->max_tree + 31) / 32;
  c->tables = new (std::nothrow) std::map<int, HostTable>();
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device);

  const size_t BP = (size_t)cfg->max_batch * c->P;
  const size_t rows = (size_t)cfg->max_batch * W;
  const size_t BN = (size_t)cfg->max_batch * cfg->max_tree;
  const int nbuf = cfg->max_depth > 1 ? cfg->max_depth - 1 : 1;
  if (e == cudaSuccess) e = dev_alloc(&c->pool_score, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->pool_token, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->pool_parent, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->pool_depth, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->pool_kept, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->retained, rows);
  if (e == cudaSuccess) e = dev_alloc(&c->lsort, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->lscore, BP);
  if (e == cudaSuccess) e = dev_alloc(&c->state, 1);
  if (e == cudaSuccess) e = dev_alloc(&c->attn_worklist, (size_t)kAttnWorkListCap * 8);
  if (e == cudaSuccess) e = dev_alloc(&c->layer_ticket, 1);
  if (e == cudaSuccess) e = dev_alloc(&c->seq_ticket, cfg->max_batch);
  if (e == cudaSuccess) e = dev_alloc(&c->tail_vs, (size_t)cfg->max_batch * CAST_MAX_WIDTH);
  if (e == cudaSuccess) e = dev_alloc(&c->tail_sorted, (size_t)cfg->max_batch * CAST_MAX_WIDTH);
  if (e == cudaSuccess) e = dev_alloc(&c->tail_tok, (size_t)cfg->max_batch * CAST_MAX_WIDTH);
  if (e == cudaSuccess) e = dev_alloc(&c->fifo_vals, (size_t)nbuf * cfg->fifo_len);
  if (e == cudaSuccess) e = dev_alloc(&c->fifo_cnt, nbuf);
  if (e == cudaSuccess) e = dev_alloc(&c->sel_score, BN);
  if (e == cudaSuccess) e = dev_alloc(&c->sel_value, BN);
  if (e == cudaSuccess) e = dev_alloc(&c->sel_idx, BN);
  if (e == cudaSuccess) e = dev_alloc(&c->acc_part, BN * kAcceptMaxChunks);
  if (e == cudaSuccess) e = dev_alloc(&c->compact_ticket, cfg->max_batch);
  if (e == cudaSuccess) {
    init_state_kernel<<<1, 64>>>(c->state, c->fifo_vals, c->fifo_cnt, nbuf, cfg->fifo_len);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess || !c->tables) {
    free_all(c);
    delete c;
    return CAST_ERR_CUDA;
  }
  c->cur_B = 0;
  c->next_layer = 0;
  *out = c;
  return CAST_OK;
}

extern "C" cast_status cast_destroy(cast_ctx* c) {
  if (!c) return CAST_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  free_all(c);
  delete c;
  return CAST_OK;
}

extern "C" cast_status cast_set_cost_tables(cast_ctx* c, int B, int L, int M, int Ntab, const double* fT,
                                            const double* fD) {
  if (!c || !fT || !fD || B < 1 || L < 1 || M < 1 || Ntab < 1) return CAST_ERR_INVALID_ARG;
  if (B > c->cfg.max_batch) return CAST_ERR_CAPACITY;
  const size_t n = (size_t)M * Ntab;
  for (int t = 0; t < 2; ++t) {
    const double* f = t ? fD : fT;
    for (int g = 0; g < M; ++g)
      for (int k = 0; k < Ntab; ++k) {
        double x = f[(size_t)g * Ntab + k];
        if (!isfinite(x) || x <= 0.0) return CAST_ERR_COST_TABLE;
        if (k > 0 && !(x > f[(size_t)g * Ntab + k - 1])) return CAST_ERR_COST_TABLE;
      }
  }
  CAST_CUDA_OK(cudaDeviceSynchronize());
  double* store = nullptr;
  CAST_CUDA_OK(cudaMalloc((void**)&store, 2 * n * sizeof(double)));
  cudaError_t e = cudaMemcpy(store, fT, n * sizeof(double), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(store + n, fD, n * sizeof(double), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    cudaFree(store);
    return CAST_ERR_CUDA;
  }
  auto it = c->tables->find(B);
  if (it != c->tables->end()) {
    cudaFree(it->second.storage);
    c->tables->erase(it);
  }
  HostTable ht;
  ht.storage = store;
  ht.dev.L = L; ht.dev.M = M; ht.dev.Ntab = Ntab;
  ht.dev.fT = store;
  ht.dev.fD = store + n;
  (*c->tables)[B] = ht;
  if (c->cur_B == B) c->cur_table = ht.dev;
  return CAST_OK;
}

extern "C" cast_status cast_state_export(cast_ctx* c, void* blob, size_t* bytes) {
  if (!c || !bytes) return CAST_ERR_INVALID_ARG;
  const int nbuf = c->cfg.max_depth - 1, R = c->cfg.fifo_len;
  const size_t need = 2 * sizeof(int32_t) + (size_t)nbuf * (sizeof(int32_t) + R * sizeof(double));
  if (!blob) { *bytes = need; return CAST_OK; }
  if (*bytes < need) return CAST_ERR_CAPACITY;
  *bytes = need;
  CAST_CUDA_OK(cudaDeviceSynchronize());
  std::vector<int32_t> cnt(nbuf > 0 ? nbuf : 1);
  std::vector<double> vals((size_t)(nbuf > 0 ? nbuf : 1) * R);
  if (nbuf > 0) {
    CAST_CUDA_OK(cudaMemcpy(cnt.data(), c->fifo_cnt, nbuf * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CAST_CUDA_OK(cudaMemcpy(vals.data(), c->fifo_vals, (size_t)nbuf * R * sizeof(double), cudaMemcpyDeviceToHost));
  }
  char* p = (char*)blob;
  int32_t hdr[2] = {nbuf, R};
  memcpy(p, hdr, sizeof(hdr)); p += sizeof(hdr);
  for (int i = 0; i < nbuf; ++i) {
    memcpy(p, &cnt[i], sizeof(int32_t)); p += sizeof(int32_t);
    memcpy(p, &vals[(size_t)i * R], R * sizeof(double)); p += R * sizeof(double);
  }
  return CAST_OK;
}

extern "C" cast_status cast_state_import(cast_ctx* c, const void* blob, size_t bytes) {
  if (!c || !blob) return CAST_ERR_INVALID_ARG;
  const int nbuf = c->cfg.max_depth - 1, R = c->cfg.fifo_len;
  const size_t need = 2 * sizeof(int32_t) + (size_t)nbuf * (sizeof(int32_t) + R * sizeof(double));
  if (bytes < need) return CAST_ERR_INVALID_ARG;
  const char* p = (const char*)blob;
  int32_t hdr[2];
  memcpy(hdr, p, sizeof(hdr)); p += sizeof(hdr);
  if (hdr[0] != nbuf || hdr[1] != R) return CAST_ERR_INVALID_ARG;
  std::vector<int32_t> cnt(nbuf > 0 ? nbuf : 1);
  std::vector<double> vals((size_t)(nbuf > 0 ? nbuf : 1) * R);
  for (int i = 0; i < nbuf; ++i) {
    memcpy(&cnt[i], p, sizeof(int32_t)); p += sizeof(int32_t);
    memcpy(&vals[(size_t)i * R], p, R * sizeof(double)); p += R * sizeof(double);
    if (cnt[i] < 1 || cnt[i] > R) return CAST_ERR_INVALID_ARG;
  }
  CAST_CUDA_OK(cudaDeviceSynchronize());
  if (nbuf > 0) {
    CAST_CUDA_OK(cudaMemcpy(c->fifo_cnt, cnt.data(), nbuf * sizeof(int32_t), cudaMemcpyHostToDevice));
    CAST_CUDA_OK(cudaMemcpy(c->fifo_vals, vals.data(), (size_t)nbuf * R * sizeof(double), cudaMemcpyHostToDevice));
  }
  return CAST_OK;
}

extern "C" cast_status cast_poll_status(cast_ctx* c, void* stream, cast_status* device_status, int32_t* detail) {
  if (!c || !device_status) return CAST_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t h[2] = {0, 0};
  CAST_CUDA_OK(cudaMemcpyAsync(h, c->state->status, sizeof(h), cudaMemcpyDeviceToHost, s));
  CAST_CUDA_OK(cudaMemsetAsync(c->state->status, 0, sizeof(h), s));
  CAST_CUDA_OK(cudaStreamSynchronize(s));
  *device_status = (cast_status)h[0];
  if (detail) *detail = h[1];
  return CAST_OK;
}

extern "C" cast_status cast_step_info(cast_ctx* c, void* stream, int32_t* info) {
  if (!c || !info) return CAST_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  DevState h;
  CAST_CUDA_OK(cudaMemcpyAsync(&h, c->state, sizeof(h), cudaMemcpyDeviceToHost, s));
  CAST_CUDA_OK(cudaStreamSynchronize(s));
  info[0] = h.layers_done;
  info[1] = h.pool_size;
  info[2] = h.n0;
  info[3] = h.n_tree;
  for (int i = 1; i <= c->cfg.max_depth; ++i) info[4 + i - 1] = i <= h.layers_done ? h.n_hist[i] : 0;
  return CAST_OK;
}
