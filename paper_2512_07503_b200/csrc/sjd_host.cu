// Host-buffer variant of the step (declared in include/sjd.h): device mirrors of every argument are
// allocated once per context; each call copies in, runs sjd_step() and copies out.
#include "../../include/sjd.h"

#include <cuda_runtime.h>

#include <cstdlib>
#include <cstring>

struct sjd_host_ctx {
  int32_t B, W, V, dtype, top_k, kcap;
  size_t rows, logits_bytes;
  void* d_cond;
  void* d_uncond;
  int32_t* d_drafts;
  sjd_probs d_q, d_out;
  int32_t *d_acc, *d_tokens, *d_flags, *d_status, *d_win, *d_pos, *d_iter;
  void* d_ws;
  size_t ws_bytes;
  cudaStream_t stream;
};

namespace {

template <typename T>
bool dev_alloc(T** p, size_t bytes) {
  return cudaMalloc(reinterpret_cast<void**>(p), bytes ? bytes : 16) == cudaSuccess;
}

bool alloc_probs(sjd_probs* p, size_t rows, size_t kcap) {
  return dev_alloc(&p->tok_prob, rows * 4) && dev_alloc(&p->ids, rows * kcap * 4) &&
         dev_alloc(&p->vals, rows * kcap * 4) && dev_alloc(&p->cnt, rows * 4);
}

void free_probs(sjd_probs* p) {
  cudaFree(p->tok_prob); cudaFree(p->ids); cudaFree(p->vals); cudaFree(p->cnt);
}

#define SJD_TRY(expr)                   \
  do {                                  \
    if ((expr) != cudaSuccess) return SJD_ERR_CUDA; \
  } while (0)

}  // namespace

extern "C" {

int sjd_host_ctx_create(const sjd_params* s, sjd_host_ctx** out_ctx) {
  if (!s || !out_ctx) return SJD_ERR_NULL;
  *out_ctx = nullptr;
  if (s->B < 1 || s->W < 1 || s->W > SJD_W_MAX || s->V < 8 || (s->V % 8) != 0 || s->top_k < 1) return SJD_ERR_SHAPE;
  if (s->logits_dtype != SJD_F32 && s->logits_dtype != SJD_BF16 && s->logits_dtype != SJD_F16) return SJD_ERR_DTYPE;
  sjd_host_ctx* c = static_cast<sjd_host_ctx*>(std::calloc(1, sizeof(sjd_host_ctx)));
  if (!c) return SJD_ERR_CUDA;
  c->B = s->B; c->W = s->W; c->V = s->V; c->dtype = s->logits_dtype; c->top_k = s->top_k;
  c->kcap = s->top_k < s->V ? s->top_k : s->V;
  c->rows = (size_t)s->B * s->W;
  c->logits_bytes = c->rows * (size_t)s->V * (s->logits_dtype == SJD_F32 ? 4 : 2);
  sjd_params shape;
  std::memset(&shape, 0, sizeof(shape));
  shape.B = s->B; shape.W = s->W;
  c->ws_bytes = sjd_workspace_bytes(&shape);
  const bool ok = dev_alloc(&c->d_cond, c->logits_bytes) && dev_alloc(&c->d_uncond, c->logits_bytes) &&
                  dev_alloc(&c->d_drafts, c->rows * 4) && alloc_probs(&c->d_q, c->rows, c->kcap) &&
                  alloc_probs(&c->d_out, c->rows, c->kcap) && dev_alloc(&c->d_acc, (size_t)s->B * 4) &&
                  dev_alloc(&c->d_tokens, c->rows * 4) && dev_alloc(&c->d_flags, c->rows * 4) &&
                  dev_alloc(&c->d_status, (size_t)s->B * 4) && dev_alloc(&c->d_win, (size_t)s->B * 4) &&
                  dev_alloc(&c->d_pos, (size_t)s->B * 4) && dev_alloc(&c->d_iter, (size_t)s->B * 4) &&
                  dev_alloc(&c->d_ws, c->ws_bytes) &&
                  cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking) == cudaSuccess;
  if (!ok) {
    sjd_host_ctx_destroy(c);
    return SJD_ERR_CUDA;
  }
  *out_ctx = c;
  return SJD_OK;
}

void sjd_host_ctx_destroy(sjd_host_ctx* c) {
  if (!c) return;
  if (c->stream) {
    cudaStreamSynchronize(c->stream);
    cudaStreamDestroy(c->stream);
  }
  cudaFree(c->d_cond); cudaFree(c->d_uncond); cudaFree(c->d_drafts);
  free_probs(&c->d_q); free_probs(&c->d_out);
  cudaFree(c->d_acc); cudaFree(c->d_tokens); cudaFree(c->d_flags); cudaFree(c->d_status);
  cudaFree(c->d_win); cudaFree(c->d_pos); cudaFree(c->d_iter); cudaFree(c->d_ws);
  std::free(c);
}

int sjd_step_host(sjd_host_ctx* c, const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                  const sjd_probs* q, const sjd_params* P, uint64_t seed, int32_t* out_accept_len,
                  int32_t* out_tokens, sjd_probs* out) {
  if (!c || !P || !logits_cond || !out_accept_len || !out_tokens || !out) return SJD_ERR_NULL;
  if (!out->tok_prob || !out->ids || !out->vals || !out->cnt) return SJD_ERR_NULL;
  if (P->struct_size != (int32_t)sizeof(sjd_params)) return SJD_ERR_STRUCT;
  if (P->B != c->B || P->W != c->W || P->V != c->V || P->logits_dtype != c->dtype || P->top_k != c->top_k)
    return SJD_ERR_SHAPE;
  const bool draft_all = (P->flags & SJD_FLAG_DRAFT_ALL) != 0;
  if (!draft_all && (!drafts || !q || !q->tok_prob || !q->ids || !q->vals || !q->cnt)) return SJD_ERR_NULL;
  cudaStream_t st = c->stream;
  const size_t rows = c->rows, kc = (size_t)c->kcap, B = (size_t)c->B;
  const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
  SJD_TRY(cudaMemcpyAsync(c->d_cond, logits_cond, c->logits_bytes, H2D, st));
  if (logits_uncond) SJD_TRY(cudaMemcpyAsync(c->d_uncond, logits_uncond, c->logits_bytes, H2D, st));
  if (!draft_all) {
    SJD_TRY(cudaMemcpyAsync(c->d_drafts, drafts, rows * 4, H2D, st));
    SJD_TRY(cudaMemcpyAsync(c->d_q.tok_prob, q->tok_prob, rows * 4, H2D, st));
    SJD_TRY(cudaMemcpyAsync(c->d_q.ids, q->ids, rows * kc * 4, H2D, st));
    SJD_TRY(cudaMemcpyAsync(c->d_q.vals, q->vals, rows * kc * 4, H2D, st));
    SJD_TRY(cudaMemcpyAsync(c->d_q.cnt, q->cnt, rows * 4, H2D, st));
  }
  if (P->win_len) SJD_TRY(cudaMemcpyAsync(c->d_win, P->win_len, B * 4, H2D, st));
  if (P->pos_base) SJD_TRY(cudaMemcpyAsync(c->d_pos, P->pos_base, B * 4, H2D, st));
  if (P->iteration) SJD_TRY(cudaMemcpyAsync(c->d_iter, P->iteration, B * 4, H2D, st));

  sjd_params D = *P;
  D.stride_b = (int64_t)c->W * c->V;
  D.stride_w = c->V;
  D.win_len = P->win_len ? c->d_win : nullptr;
  D.pos_base = P->pos_base ? c->d_pos : nullptr;
  D.iteration = P->iteration ? c->d_iter : nullptr;
  D.out_flags = P->out_flags ? c->d_flags : nullptr;
  D.status = P->status ? c->d_status : nullptr;
  D.workspace = c->d_ws;
  D.workspace_bytes = c->ws_bytes;
  D.stream = st;
  D.ev_rows_begin = nullptr;
  D.ev_rows_end = nullptr;
  const int rc = sjd_step(c->d_cond, logits_uncond ? c->d_uncond : nullptr, c->d_drafts, draft_all ? nullptr : &c->d_q,
                          &D, seed, c->d_acc, c->d_tokens, &c->d_out);
  if (rc != SJD_OK) {
    cudaStreamSynchronize(st);
    return rc;
  }
  SJD_TRY(cudaMemcpyAsync(out_accept_len, c->d_acc, B * 4, D2H, st));
  SJD_TRY(cudaMemcpyAsync(out_tokens, c->d_tokens, rows * 4, D2H, st));
  SJD_TRY(cudaMemcpyAsync(out->tok_prob, c->d_out.tok_prob, rows * 4, D2H, st));
  SJD_TRY(cudaMemcpyAsync(out->ids, c->d_out.ids, rows * kc * 4, D2H, st));
  SJD_TRY(cudaMemcpyAsync(out->vals, c->d_out.vals, rows * kc * 4, D2H, st));
  SJD_TRY(cudaMemcpyAsync(out->cnt, c->d_out.cnt, rows * 4, D2H, st));
  if (P->out_flags) SJD_TRY(cudaMemcpyAsync(P->out_flags, c->d_flags, rows * 4, D2H, st));
  if (P->status) SJD_TRY(cudaMemcpyAsync(P->status, c->d_status, B * 4, D2H, st));
  SJD_TRY(cudaStreamSynchronize(st));
  return SJD_OK;
}

}  // extern "C"
