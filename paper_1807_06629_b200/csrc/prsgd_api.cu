// C ABI of the PR-SGD library: host-side context, layout, schedule of
// Algorithm 1 and the kernel launches.  See include/prsgd.h for the contract.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "prsgd_common.cuh"
#include "kernels_f32.cuh"
#include "kernels_avg.cuh"
#include "kernels_bf16.cuh"

using namespace prsgd;

namespace {

thread_local std::string g_last_error;

int fail(prsgd_ctx* ctx, int code, const std::string& msg) {
  if (ctx) ctx->err = msg;
  g_last_error = msg;
  return code;
}

#define CUDA_TRY(ctx, expr)                                                                   \
  do {                                                                                        \
    cudaError_t e__ = (expr);                                                                 \
    if (e__ != cudaSuccess)                                                                   \
      return fail((ctx), PRSGD_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
  } while (0)

#define LAUNCH_CHECK(ctx)                                                                      \
  do {                                                                                         \
    cudaError_t e__ = cudaGetLastError();                                                      \
    if (e__ != cudaSuccess)                                                                    \
      return fail((ctx), PRSGD_ERR_CUDA, std::string("kernel launch: ") + cudaGetErrorString(e__)); \
    (ctx)->launches++;                                                                         \
    (ctx)->upper_weights_quiet = false;                                                        \
    prof_end(ctx);                                                                             \
  } while (0)

// The same for a launch whose timing interval stays open: the next launch overlaps it and is timed with it.
#define LAUNCH_CHECK_OPEN(ctx)                                                                 \
  do {                                                                                         \
    cudaError_t e__ = cudaGetLastError();                                                      \
    if (e__ != cudaSuccess)                                                                    \
      return fail((ctx), PRSGD_ERR_CUDA, std::string("kernel launch: ") + cudaGetErrorString(e__)); \
    (ctx)->launches++;                                                                         \
    (ctx)->open_launches++;                                                                    \
  } while (0)

// Optional per-kernel timing: an event pair around every launch of a family.
void prof_begin(prsgd_ctx* c, int kind) {
  if (!c->profile) return;
  cudaEvent_t a, b;
  if (!c->event_pool.empty()) {
    a = c->event_pool.back(); c->event_pool.pop_back();
    b = c->event_pool.back(); c->event_pool.pop_back();
  } else {
    if (cudaEventCreate(&a) != cudaSuccess) return;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return; }
  }
  cudaEventRecord(a, c->stream);
  c->open_kind = kind; c->open_a = a; c->open_b = b; c->open_launches = 0;
}

void prof_end(prsgd_ctx* c) {
  if (!c->profile || c->open_kind < 0) return;
  cudaEventRecord(c->open_b, c->stream);
  c->pending.push_back({c->open_kind, c->open_a, c->open_b, c->open_launches + 1});
  c->open_kind = -1;
}

int check_spec(const prsgd_model_spec* s, std::string* why) {
  if (!s || !s->dims) { *why = "spec or spec->dims is NULL"; return PRSGD_ERR_ARG; }
  if (s->n_layers < 1 || s->n_layers > PRSGD_MAX_LAYERS) { *why = "n_layers out of range"; return PRSGD_ERR_ARG; }
  for (int l = 0; l <= s->n_layers; ++l)
    if (s->dims[l] < 1 || s->dims[l] > (1 << 20)) { *why = "a layer width is out of range"; return PRSGD_ERR_ARG; }
  if (s->batch < 1 || s->batch > 256) { *why = "batch must be in 1..256"; return PRSGD_ERR_ARG; }
  if (s->pool_samples < s->batch || s->pool_samples % s->batch != 0) {
    *why = "pool_samples must be a positive multiple of batch"; return PRSGD_ERR_ARG;
  }
  if (s->pool_samples > 0x7fffffffll) { *why = "pool_samples must be below 2^31"; return PRSGD_ERR_SIZE; }
  if (s->precision != PRSGD_PRECISION_FP32 && s->precision != PRSGD_PRECISION_BF16) {
    *why = "unknown precision"; return PRSGD_ERR_ARG;
  }
  if (s->precision == PRSGD_PRECISION_BF16) {
    if (s->batch != 16 && s->batch != 32 && s->batch != 64) {
      *why = "BF16 precision needs batch 16, 32 or 64"; return PRSGD_ERR_ALIGN;
    }
    for (int l = 0; l < s->n_layers; ++l)
      if (s->dims[l] % 64 != 0) { *why = "BF16 precision needs d_0..d_{L-1} to be multiples of 64"; return PRSGD_ERR_ALIGN; }
  }
  return PRSGD_OK;
}

void compute_layout(const prsgd_model_spec* s, prsgd_layout_t* out) {
  int64_t off = 0, m = 0;
  for (int l = 0; l < s->n_layers; ++l) {
    const int64_t din = s->dims[l], dout = s->dims[l + 1];
    off = round_up(off, kSegAlign);
    out->w_off[l] = off;
    off += din * dout;
    off = round_up(off, kSegAlign);
    out->b_off[l] = off;
    off += dout;
    m += din * dout + dout;
  }
  out->m = m;
  out->m_pad = round_up(off, kSegAlign);
}

// Carve the scratch area.  With ctx == nullptr only the total is computed.
size_t carve_scratch(int N, const prsgd_model_spec* s, int64_t m_pad, prsgd_ctx* ctx) {
  size_t off = 0;
  unsigned char* base = ctx ? ctx->scratch : nullptr;
  auto take = [&](size_t bytes) -> unsigned char* {
    unsigned char* p = base ? base + off : nullptr;
    off += (size_t)round_up((int64_t)bytes, 256);
    return p;
  };
  const int L = s->n_layers, B = s->batch;
  auto status = take(sizeof(DeviceStatus));
  auto draws = take(sizeof(int32_t) * N);
  auto losses = take(sizeof(float) * (size_t)N * B);
  auto active = take((size_t)N);
  auto stage = take(sizeof(float) * (size_t)m_pad);
  auto canon = take(sizeof(float) * (size_t)m_pad);
  auto tdev = take(sizeof(int64_t));
  auto chain = take(sizeof(unsigned int) * ((size_t)kChainMax * N + 1));
  auto gmasks = take((size_t)kMaxGroups * N);
  if (ctx) {
    ctx->group_masks = gmasks;
    ctx->chain_ready = reinterpret_cast<unsigned int*>(chain);
    ctx->t_dev = reinterpret_cast<int64_t*>(tdev);
    ctx->status = reinterpret_cast<DeviceStatus*>(status);
    ctx->draws = reinterpret_cast<int32_t*>(draws);
    ctx->losses = reinterpret_cast<float*>(losses);
    ctx->active = active;
    ctx->stage_row = reinterpret_cast<float*>(stage);
    ctx->canon_row = reinterpret_cast<float*>(canon);
    std::memset(&ctx->buf, 0, sizeof(ctx->buf));
  }
  if (s->precision == PRSGD_PRECISION_FP32) {
    for (int l = 1; l <= L; ++l) {
      auto a = take(sizeof(float) * (size_t)N * B * s->dims[l]);
      auto d = take(sizeof(float) * (size_t)N * B * s->dims[l]);
      if (ctx) {
        ctx->buf.act_f32[l] = reinterpret_cast<float*>(a);
        ctx->buf.delta_f32[l] = reinterpret_cast<float*>(d);
        ctx->buf.ld[l] = s->dims[l];
      }
    }
  } else {
    // split blocks of the folded update kernels: two fp32 slots of [B][128] per CTA and a counter per block
    int wmax = 1;
    for (int l = 0; l <= L; ++l) wmax = s->dims[l] > wmax ? s->dims[l] : wmax;
    auto spart = take(sizeof(float) * 2 * (size_t)kSplitMaxCtas * B * 128);
    auto scount = take(sizeof(unsigned int) * (size_t)N * ((wmax + 63) / 64));
    auto tcount = take(sizeof(unsigned int));
    auto a1alt = take(L > 1 ? 2 * (size_t)N * B * (size_t)round_up(s->dims[1], 64) : 0);
    if (ctx) {
      ctx->split_part = reinterpret_cast<float*>(spart);
      ctx->split_count = reinterpret_cast<unsigned int*>(scount);
      ctx->tile_counter = reinterpret_cast<unsigned int*>(tcount);
    }
    for (int l = 1; l <= L; ++l) {
      const int ld = (int)round_up(s->dims[l], 64);
      const size_t e = (size_t)N * B * ld;
      unsigned char *abk = nullptr, *z = nullptr;
      if (l < L) abk = take(2 * e);
      else z = take(4 * e);                              // logits, fp32
      auto dbk = take(2 * e);
      if (ctx) {
        ctx->buf.ld[l] = ld;
        ctx->buf.act_bk[l] = reinterpret_cast<uint16_t*>(abk);
        ctx->buf.act_f32[l] = reinterpret_cast<float*>(z);
        ctx->buf.delta_bk[l] = reinterpret_cast<uint16_t*>(dbk);
      }
    }
    if (ctx) ctx->buf.act1_alt = L > 1 ? reinterpret_cast<uint16_t*>(a1alt) : nullptr;
  }
  return off;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int grid1d(int64_t n, int block) { return (int)((n + block - 1) / block); }

// ---- copies between the canonical (gap-free, row-major) order and the rows of the store ----------------
CanonArgs canon_args(const prsgd_ctx* c) {
  CanonArgs a{};
  a.L = c->L;
  int64_t pos = 0;
  for (int l = 0; l < c->L; ++l) {
    const Layer& ly = c->layer[l];
    a.w_off[l] = ly.w_off; a.b_off[l] = ly.b_off; a.d_out[l] = ly.d_out;
    a.wt[l].tiled = 0; a.wt[l].tn = ly.d_in / 64; a.wt[l].d_in = ly.d_in;
    if (c->precision == PRSGD_PRECISION_BF16) a.wt[l] = tc_wtile(c, l + 1);
    a.w_pos[l] = pos; pos += (int64_t)ly.d_in * ly.d_out;
    a.b_pos[l] = pos; pos += ly.d_out;
  }
  return a;
}

int launch_canonical(prsgd_ctx* c, float* store, int64_t store_stride, float* lin, int64_t lin_stride, int64_t nrows, bool to_store) {
  const CanonArgs a = canon_args(c);
  int64_t longest = 1;
  for (int l = 0; l < c->L; ++l) {
    const int64_t n = (int64_t)c->layer[l].d_in * c->layer[l].d_out;
    if (n > longest) longest = n;
  }
  int64_t blocks = (longest + 255) / 256;
  if (blocks > 2048) blocks = 2048;
  for (int64_t r0 = 0; r0 < nrows; r0 += 32768) {          // (grid z is limited to 65535)
    const int64_t nr = nrows - r0 < 32768 ? nrows - r0 : 32768;
    canonical_copy_kernel<<<dim3((unsigned)blocks, 2 * c->L, (unsigned)nr), 256, 0, c->stream>>>(
        store + r0 * store_stride, store_stride, lin + r0 * lin_stride, lin_stride, a, to_store ? 1 : 0);
    LAUNCH_CHECK(c);
  }
  return PRSGD_OK;
}

// rows [row0, row0 + nrows) of `store` (the parameters or the momentum buffers) <-> nrows * m floats at `lin`;
// host memory goes through one canonical row on the device
int copy_canonical(prsgd_ctx* c, float* store, float* lin, int64_t row0, int64_t nrows, bool to_store, bool lin_on_device) {
  float* rows = store + row0 * c->m_pad;
  if (lin_on_device) return launch_canonical(c, rows, c->m_pad, lin, c->m, nrows, to_store);
  if (c->readout_pending) {                     // (the canonical row still holds an asynchronous read-out)
    CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->readout_event, 0));
  }
  for (int64_t r = 0; r < nrows; ++r) {
    if (to_store) {
      CUDA_TRY(c, cudaMemcpyAsync(c->canon_row, lin + r * c->m, (size_t)c->m * 4, cudaMemcpyHostToDevice, c->stream));
      int rc = launch_canonical(c, rows + r * c->m_pad, c->m_pad, c->canon_row, c->m, 1, true);
      if (rc != PRSGD_OK) return rc;
    } else {
      int rc = launch_canonical(c, rows + r * c->m_pad, c->m_pad, c->canon_row, c->m, 1, false);
      if (rc != PRSGD_OK) return rc;
      CUDA_TRY(c, cudaMemcpyAsync(lin + r * c->m, c->canon_row, (size_t)c->m * 4, cudaMemcpyDeviceToHost, c->stream));
    }
  }
  return PRSGD_OK;
}

int refresh_shadow(prsgd_ctx* c) {
  if (c->precision != PRSGD_PRECISION_BF16) return PRSGD_OK;
  const int64_t total4 = (int64_t)c->N * c->m_pad / 4;
  prof_begin(c, PRSGD_KERNEL_MISC);
  refresh_shadow_kernel<<<grid1d(total4, 256), 256, 0, c->stream>>>(c->params, c->shadow, total4);
  LAUNCH_CHECK(c);
  return PRSGD_OK;
}

int check_device_status(prsgd_ctx* c) {
  DeviceStatus st;
  CUDA_TRY(c, cudaMemcpyAsync(&st, c->status, 4 * sizeof(unsigned int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  if (st.error != 0) {
    char msg[128];
    std::snprintf(msg, sizeof msg, "a bounded wait in a kernel expired (code %u, block %u)", st.error, st.where);
    return fail(c, PRSGD_ERR_DEVICE_TIMEOUT, msg);
  }
  return PRSGD_OK;
}

DrawArgs draw_args(const prsgd_ctx* c, int64_t t) {
  DrawArgs d;
  d.seed = c->seed; d.t = t; d.n_blocks = c->n_blocks; d.B = c->B; d.row_elems = c->dims[0]; d.worker0 = c->worker0;
  d.t_base = c->capturing ? c->t_dev : nullptr;      // while capturing, t is relative to the period's start
  return d;
}

template <int TM, bool A_PC, bool B_PC, int EPI, bool FUSE>
void launch_gemm_f32(prsgd_ctx* c, const GemmF32Args& g) {
  dim3 grid((g.Nn + 63) / 64, (g.M + TM - 1) / TM, FUSE ? 1 : g.N);
  launch_pdl(gemm_f32_kernel<TM, A_PC, B_PC, EPI, FUSE>, grid, dim3(256), 0, c->stream, g);
}

// One iteration of Algorithm 1 on the fp32-operand path.
int step_f32(prsgd_ctx* c, int64_t t, bool averaging) {
  const int L = c->L, B = c->B, N = c->N;
  const uint8_t* act_mask = c->has_mask ? c->active : nullptr;
  const bool fuse = averaging && c->fused_average && c->velocity == nullptr;   // the momentum step is not fused
  const DrawArgs dr = draw_args(c, t);
  const float* X = static_cast<const float*>(c->X);

  for (int l = 1; l <= L; ++l) {          // forward
    const Layer& ly = c->layer[l - 1];
    GemmF32Args g{};
    if (l == 1) g.A = {X, c->P * (int64_t)c->dims[0], ly.d_in, 1, 1};
    else        g.A = {c->buf.act_f32[l - 1], (int64_t)B * ly.d_in, ly.d_in, 1, 0};
    g.Bo = {c->params + ly.w_off, c->m_pad, 1, ly.d_in, 0};
    g.M = B; g.Nn = ly.d_out; g.K = ly.d_in; g.N = N; g.draw = dr;
    g.out = c->buf.act_f32[l]; g.out_worker_stride = (int64_t)B * ly.d_out;
    g.params = c->params; g.params_worker_stride = c->m_pad; g.b_off = ly.b_off;
    g.active = act_mask; g.status = c->status;
    prof_begin(c, PRSGD_KERNEL_FORWARD);
    if (l < L) {
      if (B <= 32) launch_gemm_f32<32, true, true, EPI_FWD_RELU, false>(c, g);
      else         launch_gemm_f32<64, true, true, EPI_FWD_RELU, false>(c, g);
    } else {
      if (B <= 32) launch_gemm_f32<32, true, true, EPI_FWD_LINEAR, false>(c, g);
      else         launch_gemm_f32<64, true, true, EPI_FWD_LINEAR, false>(c, g);
    }
    LAUNCH_CHECK(c);
  }
  {
    SoftmaxArgs a{};
    a.logits = c->buf.act_f32[L]; a.delta = c->buf.delta_f32[L]; a.ldz = c->dims[L];
    a.Y = c->Y; a.P = c->P; a.B = B; a.C = c->dims[L]; a.draw = dr;
    a.row_losses = c->losses; a.draws = c->draws; a.active = act_mask; a.status = c->status;
    prof_begin(c, PRSGD_KERNEL_SOFTMAX);
    launch_pdl(softmax_ce_kernel, dim3(N, (B + 7) / 8), dim3(256), 0, c->stream, a);
    LAUNCH_CHECK(c);
  }
  for (int l = L; l >= 1; --l) {          // backward, layer by layer: dX_l reads W_l before it is updated
    const Layer& ly = c->layer[l - 1];
    if (l > 1) {
      GemmF32Args g{};
      g.A = {c->buf.delta_f32[l], (int64_t)B * ly.d_out, ly.d_out, 1, 0};
      g.Bo = {c->params + ly.w_off, c->m_pad, ly.d_in, 1, 0};
      g.M = B; g.Nn = ly.d_in; g.K = ly.d_out; g.N = N; g.draw = dr;
      g.out = c->buf.delta_f32[l - 1]; g.out_worker_stride = (int64_t)B * ly.d_in;
      g.mask_src = c->buf.act_f32[l - 1];
      g.active = act_mask; g.status = c->status;
      prof_begin(c, PRSGD_KERNEL_DX);
      if (B <= 32) launch_gemm_f32<32, true, false, EPI_DX, false>(c, g);
      else         launch_gemm_f32<64, true, false, EPI_DX, false>(c, g);
      LAUNCH_CHECK(c);
    }
    GemmF32Args g{};
    g.A = {c->buf.delta_f32[l], (int64_t)B * ly.d_out, 1, ly.d_out, 0};
    if (l == 1) g.Bo = {X, c->P * (int64_t)c->dims[0], ly.d_in, 1, 1};
    else        g.Bo = {c->buf.act_f32[l - 1], (int64_t)B * ly.d_in, ly.d_in, 1, 0};
    g.M = ly.d_out; g.Nn = ly.d_in; g.K = B; g.N = N; g.draw = dr;
    g.out = c->params; g.out_worker_stride = c->m_pad; g.w_off = ly.w_off; g.b_off = ly.b_off;
    g.gamma = c->gamma; g.active = act_mask; g.vel = c->velocity; g.mu = c->mu; g.status = c->status;
    prof_begin(c, fuse ? PRSGD_KERNEL_UPDATE_AVERAGE : PRSGD_KERNEL_UPDATE);
    if (fuse) launch_gemm_f32<64, false, false, EPI_DW, true>(c, g);
    else      launch_gemm_f32<64, false, false, EPI_DW, false>(c, g);
    LAUNCH_CHECK(c);
  }
  return PRSGD_OK;
}

// One iteration of Algorithm 1 on the bf16-operand tensor-core path.
// `more_follow`: the caller runs iteration t + 1 right after this one (same call, nothing in between).
int step_bf16(prsgd_ctx* c, int64_t t, bool averaging, bool more_follow) {
  const int L = c->L, N = c->N;
  const uint8_t* act_mask = worker_mask(c);
  const bool fuse = averaging && c->fused_average;
  const bool avg_vel = c->velocity != nullptr && c->average_velocity;
  const DrawArgs dr = draw_args(c, t);
  // Layer 1's update can form a_1 of iteration t + 1 as well (its input is the data pool), which saves that
  // iteration's first forward launch and the write of W_1's shadow: only on a plain SGD iteration that is
  // not an averaging one and is followed by another one of the same call.
  const bool next_fwd = c->next_forward && more_follow && !averaging && L > 1 && tc_epilogues_fused(c);
  const bool skip_f1 = c->a1_ready;
  c->a1_ready = false;
  if (!skip_f1) c->a1_sel = 0;          // this iteration's first forward launch writes a_1: into the first buffer
  // The class layer as one launch of clusters (logits, softmax-CE gradient, step of W_L, dZ_{L-1}): whenever its
  // step is the plain one (a class layer large enough for the fused update + average keeps the separate launches).
  const bool head = tc_head_applies(c) && !(fuse && tc_layer_fuses_average(c, L));
  const bool head_fwd = head && tc_head_forward_stages(c) > 0 && !(skip_f1 && L == 2);   // ... and the forward GEMM below it
  const int l_fwd_last = head ? (head_fwd ? L - 2 : L - 1) : L;
  if (tc_chain_applies(c, skip_f1 ? 2 : 1, l_fwd_last)) {          // every remaining layer's forward GEMM in one launch
    prof_begin(c, PRSGD_KERNEL_FORWARD);
    tc_launch_forward_chain(c, skip_f1 ? 2 : 1, l_fwd_last, dr, act_mask);
    LAUNCH_CHECK(c);
  } else {
    for (int l = skip_f1 ? 2 : 1; l <= l_fwd_last; ++l) {
      prof_begin(c, PRSGD_KERNEL_FORWARD);
      tc_launch_forward(c, l, dr, act_mask);
      LAUNCH_CHECK(c);
    }
  }
  if (c->record_after_forward != nullptr) {             // the next worker group starts once this one's forward pass is enqueued
    cudaEventRecord(c->record_after_forward, c->stream);
    c->record_after_forward = nullptr;
  }
  const bool epi = tc_epilogues_fused(c);
  if (!epi) {
    SoftmaxArgs a{};
    a.logits = c->buf.act_f32[L]; a.ldz = c->buf.ld[L];
    a.delta_bk = c->buf.delta_bk[L]; a.ld_bf = c->buf.ld[L];
    a.Y = c->Y; a.P = c->P; a.B = c->B; a.C = c->dims[L]; a.draw = dr;
    a.row_losses = c->losses; a.draws = c->draws; a.active = act_mask; a.status = c->status;
    prof_begin(c, PRSGD_KERNEL_SOFTMAX);
    launch_pdl(softmax_ce_kernel, dim3(N, (c->B + 7) / 8), dim3(256), 0, c->stream, a);
    LAUNCH_CHECK(c);
  }
  // Layers >= 2 whose update is the plain SGD step: one launch forms dZ_{l-1} and applies the step of W_l (the
  // fused update + average of an averaging iteration owns a tile across workers instead and keeps dX separate).
  const bool dx_in_upd = c->dx_in_update && tc_epilogues_fused(c);
  if (head) {
    prof_begin(c, PRSGD_KERNEL_HEAD);
    tc_launch_head(c, dr, act_mask, head_fwd);
    LAUNCH_CHECK(c);
  }
  // (every worker active, layer 2 on separate dX and update launches, layer 1's launch the folded one)
  const bool overlap = c->overlap_update != 0 && next_fwd && L >= 3 && act_mask == nullptr &&
                       !(dx_in_upd && (c->dx_in_update == 2 || tc_layer_folds_dx(c, 2)));
  bool deferred = false;
  // Fused averaging iteration: the averages of the bias segments (and of the small weight segments) need every bias
  // step, i.e. every dX launch, but not layer 1's fused update + average, the iteration's last big launch.  They are
  // enqueued just before it and that launch starts beside them instead of being followed by them.
  const bool small_first = c->overlap_update != 0 && fuse && epi && L >= 2 && act_mask == nullptr && tc_layer_fuses_average(c, 1);
  bool small_done = false;
  auto small_averages = [&]() -> int {
    prof_begin(c, PRSGD_KERNEL_MISC);
    tc_launch_bias_average(c, c->params, c->merged_small_average != 0);
    LAUNCH_CHECK(c);
    if (avg_vel) {
      prof_begin(c, PRSGD_KERNEL_MISC);
      tc_launch_bias_average(c, c->velocity);
      LAUNCH_CHECK(c);
    }
    return PRSGD_OK;
  };
  int common_layers[PRSGD_MAX_LAYERS], n_common = 0;     // layers whose averaged step is formed from the common point, in one launch at the end
  for (int l = L; l >= 1; --l) {          // dX_l reads W_l before the update of layer l overwrites it
    const bool fuse_l = fuse && tc_layer_fuses_average(c, l);
    if (l == L && head) {
      // (forward, step and dZ_{L-1} of this layer were the head launch)
    } else if (fuse_l && n_common < kCommonMax && tc_layer_takes_common_point(c, l, act_mask)) {
      if (l > 1) {
        prof_begin(c, PRSGD_KERNEL_DX);
        tc_launch_dx(c, l, dr, act_mask);
        LAUNCH_CHECK(c);
      }
      common_layers[n_common++] = l;      // (needs only dZ_l and a_{l-1}, which nothing later in the iteration changes)
    } else if (l > 1 && dx_in_upd && !fuse_l && (c->dx_in_update == 2 || tc_layer_folds_dx(c, l))) {
      prof_begin(c, PRSGD_KERNEL_UPDATE);
      tc_launch_update_dx(c, l);
      LAUNCH_CHECK(c);
    } else {
      // Layer 2's plain update waits for nothing that layer 1's launch produces, and that launch (whole row blocks
      // per CTA) often leaves SMs idle: layer 2's update is enqueued after it, in the form that starts beside it.
      const bool defer = l == 2 && overlap;
      if (l > 1) {
        prof_begin(c, PRSGD_KERNEL_DX);
        tc_launch_dx(c, l, dr, act_mask, defer ? c->tile_counter : nullptr);
        LAUNCH_CHECK(c);
      }
      if (defer) {
        deferred = true;
      } else {
        bool late = false;
        if (l == 1 && small_first && fuse_l && n_common == 0) {   // (with layers waiting for the common-point launch: before that one)
          const int rc = small_averages();
          if (rc != PRSGD_OK) return rc;
          small_done = late = true;
        }
        prof_begin(c, fuse_l ? PRSGD_KERNEL_UPDATE_AVERAGE : PRSGD_KERNEL_UPDATE);
        if (l == 1 && next_fwd) {
          tc_launch_update_next(c, dr, deferred);         // (deferred: a_1 of iteration t + 1 goes to the other buffer)
          c->a1_ready = true;
          if (deferred) {
            LAUNCH_CHECK_OPEN(c);
            tc_launch_update(c, 2, dr, act_mask, false, true);     // still reads this iteration's a_1
            c->a1_sel ^= 1;
            c->no_early_once = true;
          }
        } else {
          tc_launch_update(c, l, dr, act_mask, fuse_l, false, late);
        }
        LAUNCH_CHECK(c);
      }
    }
    if (fuse && !fuse_l) {
      if (!c->merged_small_average) {        // (else with the bias segments, in the iteration's last launch)
        prof_begin(c, PRSGD_KERNEL_AVERAGE);
        tc_launch_weight_average(c, l);
        LAUNCH_CHECK(c);
      }
      if (avg_vel) {
        prof_begin(c, PRSGD_KERNEL_AVERAGE);
        tc_launch_velocity_segment_average(c, l);
        LAUNCH_CHECK(c);
      }
    }
  }
  if (n_common > 0) {
    bool late = false;
    if (small_first && !small_done) {
      const int rc = small_averages();
      if (rc != PRSGD_OK) return rc;
      small_done = late = true;
    }
    prof_begin(c, PRSGD_KERNEL_UPDATE_AVERAGE);
    tc_launch_update_common(c, common_layers, n_common, dr, late);
    LAUNCH_CHECK(c);
  }
  if (!epi) {
    prof_begin(c, PRSGD_KERNEL_MISC);
    tc_launch_bias(c, act_mask);
    LAUNCH_CHECK(c);
  }
  if (fuse && !small_done) {
    const int rc = small_averages();
    if (rc != PRSGD_OK) return rc;
  }
  // a plain iteration ends with layer 1's update: nothing in flight writes W_2..W_L, unless layer 2's update was
  // enqueued last; a fused averaging iteration ends with launches that write them
  c->upper_weights_quiet = !deferred && !fuse;
  return PRSGD_OK;
}

int launch_average(prsgd_ctx* c) {
  const bool narrow = c->m_pad < kAvgNarrowLaneBelow;      // m_pad is a multiple of 32: no scalar tail either way
  const int64_t threads = narrow ? c->m_pad / 2 : c->m_pad / 4;
  prof_begin(c, PRSGD_KERNEL_AVERAGE);
  if (c->precision == PRSGD_PRECISION_BF16) {
    if (narrow)
      average_rows_kernel<0, true, 2><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                                 nullptr, c->shadow, c->status);
    else
      average_rows_kernel<0, true><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                              nullptr, c->shadow, c->status);
  } else {
    if (narrow)
      average_rows_kernel<0, false, 2><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                                  nullptr, nullptr, c->status);
    else
      average_rows_kernel<0, false><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                               nullptr, nullptr, c->status);
  }
  LAUNCH_CHECK(c);
  if (c->velocity != nullptr && c->average_velocity) {     // momentum buffers averaged like the models
    prof_begin(c, PRSGD_KERNEL_AVERAGE);
    average_rows_kernel<0, false><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->velocity, c->N, c->m_pad, c->m_pad,
                                                                             nullptr, nullptr, c->status);
    LAUNCH_CHECK(c);
  }
  c->rows_identical = true;      // N copies of y
  return PRSGD_OK;
}

}  // namespace

// =====================================================================================
extern "C" {

const char* prsgd_last_error(prsgd_ctx* ctx) { return ctx ? ctx->err.c_str() : g_last_error.c_str(); }

uint64_t prsgd_draw_block(uint64_t seed, int32_t worker, int64_t t, uint64_t n_blocks) {
  if (n_blocks == 0 || n_blocks > 0xffffffffull) return 0;
  return draw_block(seed, worker, t, (uint32_t)n_blocks);
}

int prsgd_layout(const prsgd_model_spec* spec, prsgd_layout_t* out) {
  std::string why;
  int rc = check_spec(spec, &why);
  if (rc != PRSGD_OK) return fail(nullptr, rc, why);
  if (!out) return fail(nullptr, PRSGD_ERR_ARG, "out is NULL");
  std::memset(out, 0, sizeof *out);
  compute_layout(spec, out);
  return PRSGD_OK;
}

int prsgd_workspace_bytes(int32_t N, const prsgd_model_spec* spec, size_t* params_bytes, size_t* shadow_bytes,
                          size_t* scratch_bytes) {
  std::string why;
  int rc = check_spec(spec, &why);
  if (rc != PRSGD_OK) return fail(nullptr, rc, why);
  if (N < 1 || N > 65536) return fail(nullptr, PRSGD_ERR_ARG, "N must be in 1..65536");
  prsgd_layout_t lay;
  compute_layout(spec, &lay);
  if (params_bytes) *params_bytes = (size_t)N * lay.m_pad * 4;
  if (shadow_bytes) *shadow_bytes = spec->precision == PRSGD_PRECISION_BF16 ? (size_t)N * lay.m_pad * 2 : 0;
  if (scratch_bytes) *scratch_bytes = carve_scratch(N, spec, lay.m_pad, nullptr);
  return PRSGD_OK;
}

int prsgd_create(int32_t N, const prsgd_model_spec* spec, float gamma, int32_t I, void* d_params, void* d_shadow,
                 void* d_scratch, void* cuda_stream, prsgd_ctx** out) {
  std::string why;
  int rc = check_spec(spec, &why);
  if (rc != PRSGD_OK) return fail(nullptr, rc, why);
  if (!out) return fail(nullptr, PRSGD_ERR_ARG, "out is NULL");
  *out = nullptr;
  if (N < 1 || N > 65536) return fail(nullptr, PRSGD_ERR_ARG, "N must be in 1..65536");
  if (!(gamma > 0.f)) return fail(nullptr, PRSGD_ERR_ARG, "gamma must be > 0");
  if (I < 0) return fail(nullptr, PRSGD_ERR_ARG, "I must be >= 0");
  if (!d_params || !d_scratch) return fail(nullptr, PRSGD_ERR_ARG, "d_params / d_scratch is NULL");
  if (spec->precision == PRSGD_PRECISION_BF16 && !d_shadow)
    return fail(nullptr, PRSGD_ERR_ARG, "BF16 precision needs d_shadow");
  if (!aligned(d_params, 256) || !aligned(d_scratch, 256) || !aligned(d_shadow, 256))
    return fail(nullptr, PRSGD_ERR_ALIGN, "device buffers must be 256-byte aligned");

  prsgd_ctx* c = new (std::nothrow) prsgd_ctx();
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "out of host memory");
  c->N = N; c->L = spec->n_layers; c->B = spec->batch; c->precision = spec->precision;
  for (int l = 0; l <= c->L; ++l) c->dims[l] = spec->dims[l];
  c->P = spec->pool_samples; c->n_blocks = (uint32_t)(spec->pool_samples / spec->batch);
  c->seed = spec->draw_seed; c->gamma = gamma; c->I = I;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  prsgd_layout_t lay;
  compute_layout(spec, &lay);
  c->m = lay.m; c->m_pad = lay.m_pad;
  for (int l = 0; l < c->L; ++l) c->layer[l] = {c->dims[l], c->dims[l + 1], lay.w_off[l], lay.b_off[l]};
  c->params = static_cast<float*>(d_params);
  c->shadow = static_cast<uint16_t*>(d_shadow);
  c->scratch = static_cast<unsigned char*>(d_scratch);
  c->scratch_bytes = carve_scratch(N, spec, c->m_pad, c);

  auto bail = [&](int code) { delete c; return code; };
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->params, 0, (size_t)N * c->m_pad * 4, c->stream);
  if (e == cudaSuccess && c->shadow) e = cudaMemsetAsync(c->shadow, 0, (size_t)N * c->m_pad * 2, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->scratch, 0, c->scratch_bytes, c->stream);
  if (e != cudaSuccess) return bail(fail(nullptr, PRSGD_ERR_CUDA, std::string("create: ") + cudaGetErrorString(e)));
  if (c->precision == PRSGD_PRECISION_BF16) {
    std::string terr;
    int trc = tc_create(c, &terr);
    if (trc != PRSGD_OK) return bail(fail(nullptr, trc, terr));
  }
  *out = c;
  return PRSGD_OK;
}

int prsgd_destroy(prsgd_ctx* ctx) {
  if (!ctx) return PRSGD_OK;
  tc_destroy(ctx);
  for (auto& p : ctx->pending) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (auto e : ctx->event_pool) cudaEventDestroy(e);
  for (auto& g : ctx->graphs) cudaGraphExecDestroy(g.exec);
  if (ctx->mean_ready_event) cudaEventDestroy(ctx->mean_ready_event);
  if (ctx->readout_event) cudaEventDestroy(ctx->readout_event);
  if (ctx->staged_event) cudaEventDestroy(ctx->staged_event);
  if (ctx->free_event) cudaEventDestroy(ctx->free_event);
  if (ctx->group_fork) cudaEventDestroy(ctx->group_fork);
  for (int g = 0; g < kMaxGroups; ++g) {
    if (ctx->group_join[g]) cudaEventDestroy(ctx->group_join[g]);
    if (ctx->group_stagger[g]) cudaEventDestroy(ctx->group_stagger[g]);
    if (ctx->group_stream[g]) cudaStreamDestroy(ctx->group_stream[g]);
  }
  delete ctx;
  return PRSGD_OK;
}

int prsgd_bind_data(prsgd_ctx* c, const void* d_X, int32_t x_dtype, const int32_t* d_Y) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!d_X || !d_Y) return fail(c, PRSGD_ERR_ARG, "d_X / d_Y is NULL");
  const int want = c->precision == PRSGD_PRECISION_BF16 ? PRSGD_X_BF16 : PRSGD_X_FP32;
  if (x_dtype != want) return fail(c, PRSGD_ERR_ARG, "x_dtype does not match the context's precision");
  if (!aligned(d_X, 256) || !aligned(d_Y, 256)) return fail(c, PRSGD_ERR_ALIGN, "pools must be 256-byte aligned");
  c->X = d_X; c->x_dtype = x_dtype; c->Y = d_Y;
  if (c->precision == PRSGD_PRECISION_BF16) {
    std::string terr;
    int trc = tc_bind_data(c, &terr);
    if (trc != PRSGD_OK) return fail(c, trc, terr);
  }
  return PRSGD_OK;
}

int prsgd_upload_data(prsgd_ctx* c, const void* h_X, const int32_t* h_Y) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!c->X) return fail(c, PRSGD_ERR_STATE, "bind_data must come first");
  if (!h_X || !h_Y) return fail(c, PRSGD_ERR_ARG, "h_X / h_Y is NULL");
  const size_t esz = c->x_dtype == PRSGD_X_BF16 ? 2 : 4;
  CUDA_TRY(c, cudaMemcpyAsync(const_cast<void*>(c->X), h_X, (size_t)c->N * c->P * c->dims[0] * esz,
                              cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(const_cast<int32_t*>(c->Y), h_Y, (size_t)c->N * c->P * 4, cudaMemcpyHostToDevice,
                              c->stream));
  return PRSGD_OK;
}

int prsgd_stage_data(prsgd_ctx* c, const void* h_X, const int32_t* h_Y, void* d_X_spare, int32_t* d_Y_spare,
                     void* copy_stream) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!c->X) return fail(c, PRSGD_ERR_STATE, "bind_data must come first");
  if (!h_X || !h_Y || !d_X_spare || !d_Y_spare) return fail(c, PRSGD_ERR_ARG, "NULL pointer");
  if (d_X_spare == c->X || d_Y_spare == c->Y) return fail(c, PRSGD_ERR_ARG, "the spare pools must not be the bound pools");
  if (!aligned(d_X_spare, 256) || !aligned(d_Y_spare, 256)) return fail(c, PRSGD_ERR_ALIGN, "pools must be 256-byte aligned");
  cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
  if (!c->staged_event) CUDA_TRY(c, cudaEventCreateWithFlags(&c->staged_event, cudaEventDisableTiming));
  if (c->free_event) CUDA_TRY(c, cudaStreamWaitEvent(cs, c->free_event, 0));   // the spare pools are no longer read
  const size_t esz = c->x_dtype == PRSGD_X_BF16 ? 2 : 4;
  CUDA_TRY(c, cudaMemcpyAsync(d_X_spare, h_X, (size_t)c->N * c->P * c->dims[0] * esz, cudaMemcpyHostToDevice, cs));
  CUDA_TRY(c, cudaMemcpyAsync(d_Y_spare, h_Y, (size_t)c->N * c->P * 4, cudaMemcpyHostToDevice, cs));
  CUDA_TRY(c, cudaEventRecord(c->staged_event, cs));
  c->staged_X = d_X_spare; c->staged_Y = d_Y_spare;
  return PRSGD_OK;
}

int prsgd_swap_data(prsgd_ctx* c) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!c->staged_X) return fail(c, PRSGD_ERR_STATE, "nothing staged: prsgd_stage_data must come first");
  if (!c->free_event) CUDA_TRY(c, cudaEventCreateWithFlags(&c->free_event, cudaEventDisableTiming));
  CUDA_TRY(c, cudaEventRecord(c->free_event, c->stream));                 // everything that read the old pools
  CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->staged_event, 0));        // later work sees the staged pools
  c->X = c->staged_X; c->Y = c->staged_Y;
  c->staged_X = nullptr; c->staged_Y = nullptr;
  if (c->precision == PRSGD_PRECISION_BF16) {
    std::string terr;
    int trc = tc_bind_data(c, &terr);
    if (trc != PRSGD_OK) return fail(c, trc, terr);
  }
  return PRSGD_OK;
}

int prsgd_set_params(prsgd_ctx* c, const float* src, int32_t worker, int src_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!src) return fail(c, PRSGD_ERR_ARG, "src is NULL");
  if (worker < -1 || worker >= c->N) return fail(c, PRSGD_ERR_ARG, "worker out of range");
  int rc = copy_canonical(c, c->params, const_cast<float*>(src), worker < 0 ? 0 : worker, 1, true, src_on_device != 0);
  if (rc != PRSGD_OK) return rc;
  if (worker < 0 && c->N > 1) {
    prof_begin(c, PRSGD_KERNEL_MISC);
    broadcast_row0_kernel<<<grid1d(c->m_pad / 4, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad / 4, c->m_pad / 4);
    LAUNCH_CHECK(c);
  }
  if (!src_on_device) CUDA_TRY(c, cudaStreamSynchronize(c->stream));   // src may be reused by the caller
  c->rows_identical = worker < 0 || c->N == 1;
  c->a1_ready = false;
  return refresh_shadow(c);
}

int prsgd_set_params_stacked(prsgd_ctx* c, const float* src, int src_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!src) return fail(c, PRSGD_ERR_ARG, "src is NULL");
  int rc = copy_canonical(c, c->params, const_cast<float*>(src), 0, c->N, true, src_on_device != 0);
  if (rc != PRSGD_OK) return rc;
  if (!src_on_device) CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  c->rows_identical = c->N == 1;
  c->a1_ready = false;
  return refresh_shadow(c);
}

int prsgd_get_params_stacked(prsgd_ctx* c, float* dst, int dst_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!dst) return fail(c, PRSGD_ERR_ARG, "dst is NULL");
  int rc = copy_canonical(c, c->params, dst, 0, c->N, false, dst_on_device != 0);
  if (rc != PRSGD_OK) return rc;
  return check_device_status(c);
}

int prsgd_get_params(prsgd_ctx* c, float* dst, int32_t worker, int dst_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!dst) return fail(c, PRSGD_ERR_ARG, "dst is NULL");
  if (worker < 0 || worker >= c->N) return fail(c, PRSGD_ERR_ARG, "worker out of range");
  int rc = copy_canonical(c, c->params, dst, worker, 1, false, dst_on_device != 0);
  if (rc != PRSGD_OK) return rc;
  return check_device_status(c);
}

namespace {

// iterations t_first .. t_first + count - 1, launched directly
int run_iterations_on_stream(prsgd_ctx* c, int64_t t_first, int64_t count, int64_t t_call_end) {
  for (int64_t t = t_first; t < t_first + count; ++t) {
    const bool averaging = c->I > 0 && (t % c->I) == 0;
    const bool more_follow = t + 1 < t_call_end;
    int rc = c->precision == PRSGD_PRECISION_BF16 ? step_bf16(c, t, averaging, more_follow) : step_f32(c, t, averaging);
    // (the fp32 path has no fused form for the momentum step)
    const bool separate_average = !c->fused_average || (c->velocity != nullptr && c->precision == PRSGD_PRECISION_FP32);
    if (rc == PRSGD_OK && averaging && separate_average) rc = launch_average(c);
    if (rc != PRSGD_OK) {
      c->a1_ready = false;      // a launch failed: the next iteration must not count on an a_1 formed ahead
      c->rows_identical = false;
      return rc;
    }
    c->rows_identical = averaging;     // an averaging iteration leaves N copies of y, any other one N different points
    c->assigned_upto = -1;
  }
  return PRSGD_OK;
}

// Worker groups: inside an epoch the workers need no synchronisation (the text after Algorithm 1), so a run of
// plain iterations can be enqueued as G independent chains of launches, one per group of workers, each on a
// stream of its own; the launches of a chain skip the other groups' workers (the per-worker flags of Algorithm
// 3's mask).  While one group's long update kernels run, another group's short, latency-bound launches find
// free SMs.  The chains fork from the context's stream and join it again before the next averaging iteration.
int ensure_group_resources(prsgd_ctx* c) {
  for (int g = 0; g < c->worker_groups; ++g) {
    if (!c->group_stream[g]) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->group_stream[g], cudaStreamNonBlocking));
    if (!c->group_join[g]) CUDA_TRY(c, cudaEventCreateWithFlags(&c->group_join[g], cudaEventDisableTiming));
    if (!c->group_stagger[g]) CUDA_TRY(c, cudaEventCreateWithFlags(&c->group_stagger[g], cudaEventDisableTiming));
  }
  if (!c->group_fork) CUDA_TRY(c, cudaEventCreateWithFlags(&c->group_fork, cudaEventDisableTiming));
  return PRSGD_OK;
}

int run_iterations(prsgd_ctx* c, int64_t t_first, int64_t count) {
  const int64_t t_end = t_first + count;
  int64_t t = t_first;
  while (t < t_end) {
    // the run of plain iterations that starts here
    int64_t plain = 0;
    while (t + plain < t_end && !(c->I > 0 && ((t + plain) % c->I) == 0)) ++plain;
    const bool grouped = c->worker_groups > 1 && c->precision == PRSGD_PRECISION_BF16 && !c->has_mask && !c->profile &&
                         plain >= 2 && c->N >= 2 * c->worker_groups;
    if (!grouped) {
      const int64_t n = plain > 0 ? plain : 1;           // the plain run, or the averaging iteration it ends at
      int rc = run_iterations_on_stream(c, t, n, t_end);
      if (rc != PRSGD_OK) return rc;
      t += n;
      continue;
    }
    int rc = ensure_group_resources(c);
    if (rc != PRSGD_OK) return rc;
    cudaStream_t main_stream = c->stream;
    const bool a1_0 = c->a1_ready, ident_0 = c->rows_identical, quiet_0 = c->upper_weights_quiet;
    CUDA_TRY(c, cudaEventRecord(c->group_fork, main_stream));
    for (int g = 0; g < c->worker_groups && rc == PRSGD_OK; ++g) {
      cudaStream_t gs = c->group_stream[g];
      CUDA_TRY(c, cudaStreamWaitEvent(gs, c->group_fork, 0));
      if (g > 0) CUDA_TRY(c, cudaStreamWaitEvent(gs, c->group_stagger[g - 1], 0));   // half a step behind the group before
      c->stream = gs;
      c->group_active = c->group_masks + (size_t)g * c->N;
      c->a1_ready = a1_0; c->rows_identical = ident_0; c->upper_weights_quiet = quiet_0;
      c->record_after_forward = g + 1 < c->worker_groups ? c->group_stagger[g] : nullptr;
      rc = run_iterations_on_stream(c, t, plain, t_end);
      c->stream = main_stream;
      c->group_active = nullptr;
      c->record_after_forward = nullptr;
      if (rc == PRSGD_OK) {
        CUDA_TRY(c, cudaEventRecord(c->group_join[g], gs));
        CUDA_TRY(c, cudaStreamWaitEvent(main_stream, c->group_join[g], 0));
      }
    }
    if (rc != PRSGD_OK) return rc;
    t += plain;
  }
  return PRSGD_OK;
}

void period_key(const prsgd_ctx* c, uint64_t (&key)[13]) {
  uint32_t gbits, mbits;
  std::memcpy(&gbits, &c->gamma, 4);
  std::memcpy(&mbits, &c->mu, 4);
  key[0] = gbits; key[1] = (uint64_t)c->I; key[2] = (uint64_t)c->fused_average; key[3] = (uint64_t)c->upd_tile;
  key[4] = c->has_mask ? 1 : 0; key[5] = reinterpret_cast<uint64_t>(c->velocity); key[6] = mbits;
  key[7] = (uint64_t)c->average_velocity; key[8] = reinterpret_cast<uint64_t>(c->X);
  key[9] = reinterpret_cast<uint64_t>(c->Y); key[10] = (uint64_t)c->worker0; key[11] = (uint64_t)c->fused_epilogues | ((uint64_t)c->early_loads << 1) | ((uint64_t)c->next_forward << 2) | ((uint64_t)c->dx_in_update << 3);
  key[12] = (c->rows_identical ? 1u : 0u) | ((uint64_t)c->shared_restart << 1) | ((uint64_t)c->forward_chain << 2) |
            ((uint64_t)c->worker_groups << 3) | ((uint64_t)c->dx_shared_pair << 6) | ((uint64_t)c->head_kernel << 7) |
            ((uint64_t)c->common_point << 9) | ((uint64_t)c->split_blocks << 11) | ((uint64_t)c->head_forward << 13) |
            ((uint64_t)c->merged_small_average << 14) | ((uint64_t)c->tiled_weights << 15) | ((uint64_t)c->overlap_update << 16);      // (rows_identical: the period's first iteration may share reads)
}

// One whole averaging period (I iterations starting right after an average) as a CUDA graph: the
// kernels take the iteration number as device counter + offset, so one capture serves every period.
// Returns nullptr when capture is not possible (the caller then launches directly).
prsgd_ctx::PeriodGraph* get_period_graph(prsgd_ctx* c) {
  uint64_t key[13];
  period_key(c, key);
  for (auto& g : c->graphs)
    if (std::memcmp(g.key, key, sizeof key) == 0) return &g;
  if (c->graphs.size() >= 8) {                          // settings keep changing: start over
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.exec);
    c->graphs.clear();
  }
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    c->use_graph = 0;
    return nullptr;
  }
  const int64_t launches0 = c->launches;
  const bool identical0 = c->rows_identical;
  c->capturing = true;
  int rc = run_iterations(c, 1, c->I);                  // offsets 1..I; offset I is the averaging iteration
  if (rc == PRSGD_OK) {
    counter_add_kernel<<<1, 1, 0, c->stream>>>(c->t_dev, (int64_t)c->I);
    if (cudaGetLastError() != cudaSuccess) rc = PRSGD_ERR_CUDA;
  }
  c->capturing = false;
  const int64_t per_replay = c->launches - launches0;
  c->launches = launches0;
  cudaGraph_t graph = nullptr;
  cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
  cudaGraphExec_t exec = nullptr;
  if (rc == PRSGD_OK && e == cudaSuccess && graph != nullptr) e = cudaGraphInstantiate(&exec, graph, 0);
  if (graph) cudaGraphDestroy(graph);
  c->a1_ready = false;     // launches recorded into a capture have not run: no a_1 has been formed ahead
  c->rows_identical = identical0;
  if (rc != PRSGD_OK || e != cudaSuccess || exec == nullptr) {
    cudaGetLastError();
    c->use_graph = 0;                                   // do not try again on this context
    return nullptr;
  }
  prsgd_ctx::PeriodGraph g;
  std::memcpy(g.key, key, sizeof key);
  g.exec = exec; g.launches = per_replay;
  c->graphs.push_back(g);
  return &c->graphs.back();
}

}  // namespace

int prsgd_local_steps(prsgd_ctx* c, int64_t k) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (k < 0) return fail(c, PRSGD_ERR_ARG, "k must be >= 0");
  if (!c->X || !c->Y) return fail(c, PRSGD_ERR_STATE, "bind_data must come before local_steps");
  while (k > 0) {
    // whole periods that start right after an average are replayed from a captured graph
    if (c->use_graph && !c->profile && c->I > 0 && k >= c->I && (c->t % c->I) == 0) {
      prsgd_ctx::PeriodGraph* g = get_period_graph(c);
      if (g != nullptr) {
        if (c->t_dev_after != c->t) {                  // (a replayed period leaves the counter at the next period's start)
          counter_set_kernel<<<1, 1, 0, c->stream>>>(c->t_dev, c->t);
          CUDA_TRY(c, cudaGetLastError());
          c->launches += 1;
        }
        c->t_dev_after = -1;
        CUDA_TRY(c, cudaGraphLaunch(g->exec, c->stream));
        c->t_dev_after = c->t + c->I;
        c->rows_identical = true;                      // a period ends with the node average
        c->launches += g->launches;
        c->t += c->I;
        k -= c->I;
        continue;
      }
    }
    // otherwise: directly, up to the next period boundary (or the end of the request)
    int64_t n = k;
    if (c->I > 0) {
      const int64_t to_boundary = c->I - (c->t % c->I);
      if (to_boundary < n) n = to_boundary;
    }
    int rc = run_iterations(c, c->t + 1, n);
    if (rc != PRSGD_OK) return rc;
    c->t += n;
    k -= n;
  }
  return PRSGD_OK;
}

int prsgd_average(prsgd_ctx* c) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  return launch_average(c);
}

int prsgd_local_steps_sum(prsgd_ctx* c, int64_t k) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (k < 1) return fail(c, PRSGD_ERR_ARG, "k must be >= 1");
  if (c->I != 0) return fail(c, PRSGD_ERR_STATE, "prsgd_local_steps_sum needs I = 0: the caller drives the averages");
  if (!c->X || !c->Y) return fail(c, PRSGD_ERR_STATE, "bind_data must come before local steps");
  if (c->velocity != nullptr && c->average_velocity)
    return fail(c, PRSGD_ERR_STATE, "averaged momentum buffers have no row-sum form");
  const int64_t t_end = c->t + k + 1;                  // (exclusive) so that iteration t + k - 1 knows another one follows
  int rc = k > 1 ? run_iterations_on_stream(c, c->t + 1, k - 1, t_end) : PRSGD_OK;
  if (rc != PRSGD_OK) return rc;
  // iteration t + k: the local step in its fused form, with the summed rows divided by 1 instead of N
  c->avg_divisor = 1.f;
  const int fused_keep = c->fused_average;
  if (c->precision == PRSGD_PRECISION_BF16) {
    c->fused_average = 1;
    rc = step_bf16(c, c->t + k, /*averaging=*/true, /*more_follow=*/false);
  } else {
    rc = step_f32(c, c->t + k, /*averaging=*/false);   // plain step, then every row <- sum of the rows
    if (rc == PRSGD_OK) {
      const int64_t threads = c->m_pad / 4;
      prof_begin(c, PRSGD_KERNEL_AVERAGE);
      average_rows_kernel<0, false><<<grid1d(threads, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad, nullptr,
                                                                               nullptr, c->status, 1.f);
      LAUNCH_CHECK(c);
    }
  }
  c->fused_average = fused_keep;
  c->avg_divisor = 0.f;
  c->a1_ready = false;
  c->rows_identical = rc == PRSGD_OK;                  // every row holds the same bits: the row sum
  c->assigned_upto = -1;
  if (rc != PRSGD_OK) return rc;
  c->t += k;
  return PRSGD_OK;
}

int prsgd_get_average_async(prsgd_ctx* c, float* h_dst, void* copy_stream) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!h_dst) return fail(c, PRSGD_ERR_ARG, "h_dst is NULL");
  cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
  if (cs == c->stream) return fail(c, PRSGD_ERR_ARG, "copy_stream must differ from the context's stream");
  if (!c->mean_ready_event) CUDA_TRY(c, cudaEventCreateWithFlags(&c->mean_ready_event, cudaEventDisableTiming));
  if (!c->readout_event) CUDA_TRY(c, cudaEventCreateWithFlags(&c->readout_event, cudaEventDisableTiming));
  // the staging row is free again once the previous asynchronous read-out has left it
  if (c->readout_pending) CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->readout_event, 0));
  if (c->rows_identical) {
    // right after an average every row IS the node average: snapshot row 0 instead of summing N equal rows
    CUDA_TRY(c, cudaMemcpyAsync(c->stage_row, c->params, (size_t)c->m_pad * 4, cudaMemcpyDeviceToDevice, c->stream));
  } else {
    prof_begin(c, PRSGD_KERNEL_AVERAGE);
    average_rows_kernel<1, false><<<grid1d(c->m_pad / 4, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                                c->stage_row, nullptr);
    LAUNCH_CHECK(c);
  }
  {   // the mean in canonical order, still on the training stream; one copy to the host on the caller's stream
    int rc = launch_canonical(c, c->stage_row, c->m_pad, c->canon_row, c->m, 1, false);
    if (rc != PRSGD_OK) return rc;
  }
  CUDA_TRY(c, cudaEventRecord(c->mean_ready_event, c->stream));
  CUDA_TRY(c, cudaStreamWaitEvent(cs, c->mean_ready_event, 0));
  CUDA_TRY(c, cudaMemcpyAsync(h_dst, c->canon_row, (size_t)c->m * 4, cudaMemcpyDeviceToHost, cs));
  CUDA_TRY(c, cudaEventRecord(c->readout_event, cs));
  c->readout_pending = true;
  return PRSGD_OK;
}

int prsgd_get_average(prsgd_ctx* c, float* dst, int dst_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!dst) return fail(c, PRSGD_ERR_ARG, "dst is NULL");
  if (c->readout_pending) CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->readout_event, 0));   // staging row in use
  const float* mean = c->stage_row;
  if (c->rows_identical) {
    mean = c->params;            // right after an average every row IS the node average: row 0, as it stands
  } else {
    prof_begin(c, PRSGD_KERNEL_AVERAGE);
    average_rows_kernel<1, false><<<grid1d(c->m_pad / 4, 256), 256, 0, c->stream>>>(c->params, c->N, c->m_pad, c->m_pad,
                                                                                c->stage_row, nullptr);
    LAUNCH_CHECK(c);
  }
  if (dst_on_device) return launch_canonical(c, const_cast<float*>(mean), c->m_pad, dst, c->m, 1, false);
  {
    int rc = launch_canonical(c, const_cast<float*>(mean), c->m_pad, c->canon_row, c->m, 1, false);
    if (rc != PRSGD_OK) return rc;
  }
  CUDA_TRY(c, cudaMemcpyAsync(dst, c->canon_row, (size_t)c->m * 4, cudaMemcpyDeviceToHost, c->stream));
  return check_device_status(c);
}

int prsgd_enable_momentum(prsgd_ctx* c, float mu, void* d_velocity, int average_velocity) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (d_velocity == nullptr) {                 // back to plain SGD
    c->velocity = nullptr; c->mu = 0.f; c->average_velocity = 0;
    return PRSGD_OK;
  }
  if (!(mu >= 0.f && mu < 1.f)) return fail(c, PRSGD_ERR_ARG, "mu must be in [0, 1)");
  if (!aligned(d_velocity, 256)) return fail(c, PRSGD_ERR_ALIGN, "d_velocity must be 256-byte aligned");
  CUDA_TRY(c, cudaMemsetAsync(d_velocity, 0, (size_t)c->N * c->m_pad * 4, c->stream));
  c->velocity = static_cast<float*>(d_velocity); c->mu = mu; c->average_velocity = average_velocity != 0;
  if (c->precision == PRSGD_PRECISION_BF16) {
    std::string terr;
    int trc = tc_bind_velocity(c, &terr);
    if (trc != PRSGD_OK) { c->velocity = nullptr; c->mu = 0.f; return fail(c, trc, terr); }
  }
  return PRSGD_OK;
}

int prsgd_get_velocity_stacked(prsgd_ctx* c, float* dst, int dst_on_device) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!dst) return fail(c, PRSGD_ERR_ARG, "dst is NULL");
  if (!c->velocity) return fail(c, PRSGD_ERR_STATE, "momentum is not enabled");
  int rc = copy_canonical(c, c->velocity, dst, 0, c->N, false, dst_on_device != 0);   // same row layout as the store
  if (rc != PRSGD_OK) return rc;
  return check_device_status(c);
}

int prsgd_set_worker_offset(prsgd_ctx* c, int32_t first_worker) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (first_worker < 0) return fail(c, PRSGD_ERR_ARG, "first_worker must be >= 0");
  c->worker0 = first_worker;
  return PRSGD_OK;
}

int prsgd_set_global_workers(prsgd_ctx* c, int32_t N_global) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (N_global != 0 && N_global < c->worker0 + c->N)
    return fail(c, PRSGD_ERR_ARG, "N_global must be 0 or at least first_worker + the context's own N");
  c->N_global = N_global;
  return PRSGD_OK;
}

namespace {
int check_cols(prsgd_ctx* c, const void* p, int64_t col0, int64_t ncols) {
  if (!p) return fail(c, PRSGD_ERR_ARG, "NULL row pointer");
  if (col0 < 0 || ncols < 0 || col0 + ncols > c->m_pad) return fail(c, PRSGD_ERR_ARG, "column range outside [0, m_pad)");
  if ((col0 % 4) != 0 || (ncols % 4) != 0 || !aligned(p, 16))
    return fail(c, PRSGD_ERR_ALIGN, "col0 and ncols must be multiples of 4 and the row 16-byte aligned");
  return PRSGD_OK;
}
}  // namespace

int prsgd_partial_sum(prsgd_ctx* c, float* d_dst, int64_t col0, int64_t ncols) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  int rc = check_cols(c, d_dst, col0, ncols);
  if (rc != PRSGD_OK || ncols == 0) return rc;
  prof_begin(c, PRSGD_KERNEL_AVERAGE);
  average_rows_kernel<2, false><<<grid1d(ncols / 4, 256), 256, 0, c->stream>>>(c->params + col0, c->N, ncols, c->m_pad,
                                                                            d_dst + col0, nullptr, c->status);
  LAUNCH_CHECK(c);
  return PRSGD_OK;
}

int prsgd_assign_rows(prsgd_ctx* c, const float* d_src, float divisor, int64_t col0, int64_t ncols) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  int rc = check_cols(c, d_src, col0, ncols);
  if (rc != PRSGD_OK || ncols == 0) return rc;
  if (!(divisor > 0.f)) return fail(c, PRSGD_ERR_ARG, "divisor must be > 0");
  prof_begin(c, PRSGD_KERNEL_AVERAGE);
  if (c->precision == PRSGD_PRECISION_BF16)
    assign_rows_kernel<true><<<grid1d(ncols / 4, 256), 256, 0, c->stream>>>(c->params + col0, c->shadow + col0, d_src + col0,
                                                                         divisor, c->N, ncols / 4, c->m_pad / 4, c->status);
  else
    assign_rows_kernel<false><<<grid1d(ncols / 4, 256), 256, 0, c->stream>>>(c->params + col0, nullptr, d_src + col0, divisor,
                                                                          c->N, ncols / 4, c->m_pad / 4, c->status);
  LAUNCH_CHECK(c);
  // chunks assigned in ascending order since the last local step: once they cover the row, all rows are equal
  if (col0 == 0) c->assigned_upto = ncols;
  else if (col0 == c->assigned_upto) c->assigned_upto += ncols;
  else c->assigned_upto = -1;
  if (c->assigned_upto == c->m_pad) c->rows_identical = true;
  return PRSGD_OK;
}

int prsgd_get_losses(prsgd_ctx* c, float* h_dst) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!h_dst) return fail(c, PRSGD_ERR_ARG, "h_dst is NULL");
  std::vector<float> rows((size_t)c->N * c->B);
  CUDA_TRY(c, cudaMemcpyAsync(rows.data(), c->losses, sizeof(float) * rows.size(), cudaMemcpyDeviceToHost, c->stream));
  int rc = check_device_status(c);
  if (rc != PRSGD_OK) return rc;
  for (int n = 0; n < c->N; ++n) {          // mean over the minibatch, rows added in order
    float s = 0.f;
    for (int b = 0; b < c->B; ++b) s += rows[(size_t)n * c->B + b];
    h_dst[n] = s / (float)c->B;
  }
  return PRSGD_OK;
}

int prsgd_get_draws(prsgd_ctx* c, int32_t* h_dst) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!h_dst) return fail(c, PRSGD_ERR_ARG, "h_dst is NULL");
  CUDA_TRY(c, cudaMemcpyAsync(h_dst, c->draws, sizeof(int32_t) * c->N, cudaMemcpyDeviceToHost, c->stream));
  return check_device_status(c);
}

int prsgd_alg2_schedule(int32_t N, int64_t s, int64_t* K_s, float* gamma_s) {
  if (N < 1 || s < 1) return fail(nullptr, PRSGD_ERR_ARG, "need N >= 1 and s >= 1");
  // cube root of s, exact at perfect cubes
  double root = std::cbrt((double)s);
  const int64_t r = (int64_t)std::llround(root);
  if (r * r * r == s) root = (double)r;
  if (K_s) *K_s = (int64_t)std::ceil(root / (double)N);
  if (gamma_s) *gamma_s = (float)((double)N / (root * root));
  return PRSGD_OK;
}

int prsgd_run_time_varying(prsgd_ctx* c, int64_t s_begin, int64_t s_end, float gamma_scale) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (s_begin < 1 || s_end < s_begin) return fail(c, PRSGD_ERR_ARG, "need 1 <= s_begin <= s_end");
  if (!(gamma_scale > 0.f)) return fail(c, PRSGD_ERR_ARG, "gamma_scale must be > 0");
  if (c->N_global > c->N)
    return fail(c, PRSGD_ERR_STATE, "this context holds a shard of the workers: the epoch's starting average needs "
                                    "every shard; drive the epochs with prsgd_alg2_schedule(N_global, s)");
  const int I_keep = c->I;
  const float g_keep = c->gamma;
  c->I = 0;                                          // epochs are driven here, not by t mod I
  int rc = PRSGD_OK;
  for (int64_t s = s_begin; s <= s_end && rc == PRSGD_OK; ++s) {
    int64_t K = 0; float g = 0.f;
    prsgd_alg2_schedule(c->N_global > 0 ? c->N_global : c->N, s, &K, &g);   // Theorem 2's N counts every worker
    rc = launch_average(c);                          // x_i^{s,0} = node average of the previous epoch's end points
    if (rc != PRSGD_OK) break;
    c->gamma = g * gamma_scale;
    rc = prsgd_local_steps(c, K);
  }
  c->I = I_keep;
  c->gamma = g_keep;
  return rc;
}

int prsgd_run_heterogeneous_epoch(prsgd_ctx* c, const int32_t* h_I_i) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!h_I_i) return fail(c, PRSGD_ERR_ARG, "h_I_i is NULL");
  int32_t Imax = 0;
  for (int i = 0; i < c->N; ++i) {
    if (h_I_i[i] < 0) return fail(c, PRSGD_ERR_ARG, "epoch lengths must be >= 0");
    if (h_I_i[i] > Imax) Imax = h_I_i[i];
  }
  const int I_keep = c->I;
  const bool mask_keep = c->has_mask;
  std::vector<uint8_t> mask((size_t)c->N), old_mask((size_t)c->N);
  if (mask_keep) {
    CUDA_TRY(c, cudaMemcpyAsync(old_mask.data(), c->active, (size_t)c->N, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  }
  c->I = 0;
  int rc = launch_average(c);                        // x_i^{s,0} = node average
  for (int32_t k = 1; k <= Imax && rc == PRSGD_OK; ++k) {
    bool all = true;
    for (int i = 0; i < c->N; ++i) { mask[i] = k <= h_I_i[i] ? 1 : 0; all = all && mask[i]; }
    rc = prsgd_set_active(c, all ? nullptr : mask.data());
    if (rc == PRSGD_OK) rc = prsgd_local_steps(c, 1);
  }
  c->I = I_keep;
  int rc2 = prsgd_set_active(c, mask_keep ? old_mask.data() : nullptr);
  return rc != PRSGD_OK ? rc : rc2;
}

int prsgd_set_lr(prsgd_ctx* c, float gamma) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!(gamma > 0.f)) return fail(c, PRSGD_ERR_ARG, "gamma must be > 0");
  c->gamma = gamma;
  return PRSGD_OK;
}

int prsgd_set_interval(prsgd_ctx* c, int32_t I) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (I < 0) return fail(c, PRSGD_ERR_ARG, "I must be >= 0");
  c->I = I;
  return PRSGD_OK;
}

int prsgd_set_active(prsgd_ctx* c, const uint8_t* h_mask) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (!h_mask) { c->has_mask = false; return PRSGD_OK; }
  CUDA_TRY(c, cudaMemcpyAsync(c->active, h_mask, (size_t)c->N, cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  c->has_mask = true;
  return PRSGD_OK;
}

int prsgd_get_step(prsgd_ctx* c, int64_t* t) {
  if (!c || !t) return fail(c, PRSGD_ERR_ARG, "NULL argument");
  *t = c->t;
  return PRSGD_OK;
}

int prsgd_set_step(prsgd_ctx* c, int64_t t) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (t < 0) return fail(c, PRSGD_ERR_ARG, "t must be >= 0");
  c->t = t;
  return PRSGD_OK;
}

int prsgd_set_option(prsgd_ctx* c, int32_t option, int64_t value) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (option == PRSGD_OPT_FUSED_AVERAGE) { c->fused_average = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_PROFILE) { c->profile = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_GRAPH) { c->use_graph = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_FUSED_EPILOGUES) { c->fused_epilogues = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_EARLY_LOADS) { c->early_loads = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_NEXT_FORWARD) { c->next_forward = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_CHECK_FINITE) { c->check_finite = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_SHARED_RESTART) { c->shared_restart = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_FORWARD_CHAIN) { c->forward_chain = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_DX_SHARED_PAIR) { c->dx_shared_pair = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_TILED_WEIGHTS) {
    const int want = value != 0 ? 1 : 0;
    if (want == c->tiled_weights || c->precision != PRSGD_PRECISION_BF16) { c->tiled_weights = want; return PRSGD_OK; }
    // re-order the store in place: every row through the canonical order, old order out, new order in
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (c->readout_pending) CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->readout_event, 0));
    float* stores[2] = {c->params, c->velocity};
    for (int r = 0; r < c->N; ++r) {
      for (int k = 0; k < 2; ++k) {
        if (stores[k] == nullptr) continue;
        c->tiled_weights = 1 - want;
        int rc = launch_canonical(c, stores[k] + (int64_t)r * c->m_pad, c->m_pad, c->canon_row, c->m, 1, false);
        c->tiled_weights = want;
        if (rc == PRSGD_OK) rc = launch_canonical(c, stores[k] + (int64_t)r * c->m_pad, c->m_pad, c->canon_row, c->m, 1, true);
        if (rc != PRSGD_OK) return rc;
      }
    }
    std::string terr;
    int trc = tc_make_weight_maps(c, &terr);
    if (trc != PRSGD_OK) return fail(c, trc, terr);
    c->a1_ready = false;
    return refresh_shadow(c);
  }
  if (option == PRSGD_OPT_COMMON_POINT) {
    if (value < 0 || value > 2) return fail(c, PRSGD_ERR_ARG, "PRSGD_OPT_COMMON_POINT takes 0, 1 or 2");
    c->common_point = (int)value;
    return PRSGD_OK;
  }
  if (option == PRSGD_OPT_HEAD_FORWARD) { c->head_forward = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_OVERLAP_UPDATE) { c->overlap_update = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_MERGED_SMALL_AVERAGE) { c->merged_small_average = value != 0; return PRSGD_OK; }
  if (option == PRSGD_OPT_SPLIT_BLOCKS) {
    if (value < 0 || value > 2) return fail(c, PRSGD_ERR_ARG, "PRSGD_OPT_SPLIT_BLOCKS takes 0, 1 or 2");
    c->split_blocks = (int)value;
    return PRSGD_OK;
  }
  if (option == PRSGD_OPT_HEAD_KERNEL) {
    if (value < 0 || value > 2) return fail(c, PRSGD_ERR_ARG, "PRSGD_OPT_HEAD_KERNEL takes 0, 1 or 2");
    c->head_kernel = (int)value;
    return PRSGD_OK;
  }
  if (option == PRSGD_OPT_WORKER_GROUPS) {
    if (value < 1 || value > kMaxGroups) return fail(c, PRSGD_ERR_ARG, "PRSGD_OPT_WORKER_GROUPS takes 1..4");
    // group g holds the contiguous workers [g N / G, (g + 1) N / G)
    std::vector<uint8_t> m((size_t)kMaxGroups * c->N, 0);
    for (int i = 0; i < c->N; ++i) m[(size_t)((int64_t)i * value / c->N) * c->N + i] = 1;
    CUDA_TRY(c, cudaMemcpyAsync(c->group_masks, m.data(), m.size(), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    c->worker_groups = (int)value;
    return PRSGD_OK;
  }
  if (option == PRSGD_OPT_DX_IN_UPDATE) {
    if (value < 0 || value > 2) return fail(c, PRSGD_ERR_ARG, "PRSGD_OPT_DX_IN_UPDATE takes 0, 1 or 2");
    c->dx_in_update = (int)value;
    return PRSGD_OK;
  }
  if (option == PRSGD_OPT_UPDATE_TILE) {
    if (value != 0 && value != 64 && value != 128) return fail(c, PRSGD_ERR_ARG, "update tile width must be 0, 64 or 128");
    c->upd_tile = (int)value;
    return PRSGD_OK;
  }
  return fail(c, PRSGD_ERR_ARG, "unknown option");
}

int prsgd_get_launch_count(prsgd_ctx* c, int64_t* count) {
  if (!c || !count) return fail(c, PRSGD_ERR_ARG, "NULL argument");
  *count = c->launches;
  return PRSGD_OK;
}

int prsgd_get_profile(prsgd_ctx* c, int32_t family, double* ms_total, int64_t* launches) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (family < 0 || family >= PRSGD_KERNEL_FAMILIES) return fail(c, PRSGD_ERR_ARG, "unknown kernel family");
  if (!c->pending.empty()) {
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (auto& p : c->pending) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, p.a, p.b) == cudaSuccess) { c->prof_ms[p.kind] += ms; c->prof_count[p.kind] += p.launches; }
      c->event_pool.push_back(p.a);
      c->event_pool.push_back(p.b);
    }
    c->pending.clear();
  }
  if (ms_total) *ms_total = c->prof_ms[family];
  if (launches) *launches = c->prof_count[family];
  c->prof_ms[family] = 0.0;
  c->prof_count[family] = 0;
  return PRSGD_OK;
}

int prsgd_selftest_wait_expiry(prsgd_ctx* c, int32_t limit_us) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  if (limit_us < 1 || limit_us > 1000000) return fail(c, PRSGD_ERR_ARG, "limit_us must be in 1..1000000");
  prof_begin(c, PRSGD_KERNEL_MISC);
  wait_expiry_kernel<<<1, 32, 0, c->stream>>>(c->status, (long long)limit_us * 2000ll);
  LAUNCH_CHECK(c);
  return PRSGD_OK;
}

int prsgd_clear_device_error(prsgd_ctx* c) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  CUDA_TRY(c, cudaMemsetAsync(c->status, 0, sizeof(DeviceStatus), c->stream));
  // an interrupted forward chain may have left its counters half way
  CUDA_TRY(c, cudaMemsetAsync(c->chain_ready, 0, sizeof(unsigned int) * ((size_t)kChainMax * c->N + 1), c->stream));
  if (c->split_count != nullptr) {   // ... and an interrupted split launch the counters of its cut blocks
    int wmax = 1;
    for (int l = 0; l <= c->L; ++l) wmax = c->dims[l] > wmax ? c->dims[l] : wmax;
    CUDA_TRY(c, cudaMemsetAsync(c->split_count, 0, sizeof(unsigned int) * (size_t)c->N * ((wmax + 63) / 64), c->stream));
  }
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  c->err.clear();
  c->rows_identical = false;     // whatever the interrupted launches left
  c->a1_ready = false;
  return PRSGD_OK;
}

int prsgd_check_finite(prsgd_ctx* c, int64_t* count, int32_t* first_worker) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  CUDA_TRY(c, cudaMemsetAsync(&c->status->nonfinite, 0, sizeof(unsigned int), c->stream));
  CUDA_TRY(c, cudaMemsetAsync(&c->status->nonfinite_row, 0xFF, sizeof(unsigned int), c->stream));
  const int64_t row4 = c->m_pad / 4;
  const int64_t total4 = (int64_t)c->N * row4;
  const int grid = (int)std::min<int64_t>((total4 + 1023) / 1024, 148 * 16);
  for (const float* store : {(const float*)c->params, (const float*)c->velocity}) {
    if (store == nullptr) continue;
    prof_begin(c, PRSGD_KERNEL_MISC);
    finite_check_kernel<<<grid, 256, 0, c->stream>>>(store, total4, row4, c->status);
    LAUNCH_CHECK(c);
  }
  DeviceStatus st;
  CUDA_TRY(c, cudaMemcpyAsync(&st, c->status, 4 * sizeof(unsigned int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  if (count) *count = (int64_t)st.nonfinite;
  if (first_worker) *first_worker = st.nonfinite != 0u ? (int32_t)st.nonfinite_row : -1;
  if (st.nonfinite != 0u) {
    char msg[160];
    std::snprintf(msg, sizeof msg, "%u non-finite value(s) in the parameter store, the first in worker %u's row",
                  st.nonfinite, st.nonfinite_row);
    return fail(c, PRSGD_ERR_NONFINITE, msg);
  }
  return PRSGD_OK;
}

int prsgd_sync(prsgd_ctx* c) {
  if (!c) return fail(nullptr, PRSGD_ERR_ARG, "ctx is NULL");
  int rc = check_device_status(c);
  if (rc == PRSGD_OK && c->check_finite) rc = prsgd_check_finite(c, nullptr, nullptr);
  return rc;
}

int prsgd_average_rows(float* d_P, int64_t N, int64_t m, int64_t row_stride, void* cuda_stream) {
  if (!d_P) return fail(nullptr, PRSGD_ERR_ARG, "d_P is NULL");
  if (N < 1 || m < 0 || row_stride < m) return fail(nullptr, PRSGD_ERR_ARG, "need N >= 1, m >= 0, row_stride >= m");
  if (!aligned(d_P, 16) || (row_stride % 4) != 0)
    return fail(nullptr, PRSGD_ERR_ALIGN, "d_P must be 16-byte aligned and row_stride a multiple of 4");
  if (m == 0) return PRSGD_OK;
  // Launched as a programmatic dependent: its blocks may become resident while the kernel before it in
  // the stream drains (they touch no memory before griddepcontrol.wait), which hides the launch latency
  // of back-to-back calls on short rows.
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (m < kAvgNarrowLaneBelow) {
    const int64_t threads = m / 2 + (m & 1);
    launch_pdl(average_rows_kernel<0, false, 2>, grid1d(threads, 256), dim3(256), 0, st, d_P, N, m, row_stride,
               (float*)nullptr, (uint16_t*)nullptr, (const DeviceStatus*)nullptr, 0.f);
  } else {
    const int64_t threads = m / 4 + (m & 3);
    if ((threads + 255) / 256 > 0x7fffffffll) return fail(nullptr, PRSGD_ERR_SIZE, "m too large");
    launch_pdl(average_rows_kernel<0, false>, grid1d(threads, 256), dim3(256), 0, st, d_P, N, m, row_stride,
               (float*)nullptr, (uint16_t*)nullptr, (const DeviceStatus*)nullptr, 0.f);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, PRSGD_ERR_CUDA, std::string("average_rows: ") + cudaGetErrorString(e));
  return PRSGD_OK;
}

// ---- allocation-free node average ------------------------------------------------------
// Staging row for prsgd_mean_rows_noalloc.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernel must be given the device address looked up below.
static __device__ __align__(256) float g_noalloc_row[PRSGD_NOALLOC_MAX_M];

namespace {
constexpr int kMaxDevices = 64;
float* g_noalloc_addr[kMaxDevices] = {nullptr};
std::mutex g_noalloc_mutex;
}  // namespace

int prsgd_mean_rows_noalloc(const float* d_P, int64_t N, int64_t m, int64_t row_stride, float* dst, int dst_on_device,
                            void* cuda_stream) {
  if (!d_P || !dst) return fail(nullptr, PRSGD_ERR_ARG, "d_P / dst is NULL");
  if (N < 1 || m < 0 || row_stride < m) return fail(nullptr, PRSGD_ERR_ARG, "need N >= 1, m >= 0, row_stride >= m");
  if (m > PRSGD_NOALLOC_MAX_M)
    return fail(nullptr, PRSGD_ERR_SIZE, "m exceeds PRSGD_NOALLOC_MAX_M (" + std::to_string(PRSGD_NOALLOC_MAX_M) +
                                             " floats), the size of the library's fixed staging row");
  if (!aligned(d_P, 16) || (row_stride % 4) != 0)
    return fail(nullptr, PRSGD_ERR_ALIGN, "d_P must be 16-byte aligned and row_stride a multiple of 4");
  if (m == 0) return PRSGD_OK;
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(nullptr, PRSGD_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, PRSGD_ERR_ARG, "device ordinal out of range");
  float* row = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_addr[dev]) {                 // once per device, with that device current
      float* p = nullptr;
      e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_row);
      if (e != cudaSuccess || !p)
        return fail(nullptr, PRSGD_ERR_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
      g_noalloc_addr[dev] = p;
    }
    row = g_noalloc_addr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t threads = m / 4 + (m & 3);
  // MODE 1 only reads P; every entry of row[0, m) is written before the copy below reads it
  average_rows_kernel<1, false><<<grid1d(threads, 256), 256, 0, st>>>(const_cast<float*>(d_P), N, m, row_stride, row, nullptr);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, PRSGD_ERR_CUDA, std::string("mean_rows_noalloc: ") + cudaGetErrorString(e));
  e = cudaMemcpyAsync(dst, row, (size_t)m * 4, dst_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess && !dst_on_device) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(nullptr, PRSGD_ERR_CUDA, std::string("mean_rows_noalloc copy: ") + cudaGetErrorString(e));
  return PRSGD_OK;
}

}  // extern "C"
