// fp32-operand path: grouped (one problem per worker) GEMMs on the CUDA cores
// with the forward, backward and SGD-update epilogues fused in, and the
// softmax cross-entropy gradient.  All sums run in a fixed order.
#pragma once
#include "prsgd_common.cuh"

namespace prsgd {

// One operand of a grouped GEMM, element (a, b) of worker n at
//   base + n * worker_stride + [pool ? block(n) * B * ld_pool : 0] + a * s0 + b * s1.
struct OperandF32 {
  const float* base;
  int64_t worker_stride;
  int64_t s0, s1;
  int pool;              // 1: rows come from the worker's data pool, offset by its drawn block
};

struct DrawArgs {
  uint64_t seed;
  int64_t t;
  uint32_t n_blocks;
  int B;                 // rows per block
  int64_t row_elems;     // d_0
  int worker0;           // global index of local row 0 (workers sharded over several GPUs)
  const int64_t* t_base; // nullptr, or a device counter added to t (a captured period is replayed with a new base)
};

__device__ __forceinline__ int64_t draw_t(const DrawArgs& d) { return d.t + (d.t_base != nullptr ? *d.t_base : 0); }

enum { EPI_FWD_RELU = 0, EPI_FWD_LINEAR = 1, EPI_DX = 2, EPI_DW = 3 };

struct GemmF32Args {
  OperandF32 A;          // A(i, p), i < M, p < K
  OperandF32 Bo;         // B(p, j), p < K, j < Nn
  int M, Nn, K, N;       // N = workers
  DrawArgs draw;
  // epilogue
  float* out;            // FWD/DX: [N][M][Nn]; DW: parameter store (row n at out + n*out_worker_stride)
  int64_t out_worker_stride;
  int64_t w_off, b_off;  // DW: offsets of W_l and b_l inside a row; FWD: b_off used for the bias
  const float* params;   // FWD: parameter store (bias source); stride = params_worker_stride
  int64_t params_worker_stride;
  const float* mask_src; // DX: a_{l-1} of the same shape as out (ReLU mask: a > 0)
  float gamma;
  const uint8_t* active; // per-worker flag or nullptr
  float* vel;            // DW: momentum buffers laid out like the store, or nullptr
  float mu;
  const DeviceStatus* status;   // a recorded expired wait turns the launch into a no-op
};

__device__ __forceinline__ const float* operand_ptr(const OperandF32& o, int n, const DrawArgs& d) {
  const float* p = o.base + (int64_t)n * o.worker_stride;
  if (o.pool) p += (int64_t)draw_block(d.seed, d.worker0 + n, draw_t(d), d.n_blocks) * d.B * d.row_elems;
  return p;
}

// C(i, j) = sum_p A(i, p) B(p, j); tile TM x 64 x 32, 256 threads, (TM/16) x 4 outputs per thread.
// A_PC / B_PC: the contraction index p is the contiguous one of that operand.
template <int TM, bool A_PC, bool B_PC, int EPI, bool FUSE>
__global__ void __launch_bounds__(256) gemm_f32_kernel(const GemmF32Args g) {
  constexpr int TN = 64, TK = 32, RM = TM / 16;
  constexpr int LA = TM * TK / 256, LB = TN * TK / 256;   // elements each thread moves per K chunk
  __shared__ float As[2][TK][TM + 1];
  __shared__ __align__(16) float Bs[2][TK][TN + 4];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");   // no-op unless launched as a programmatic dependent
  if (g.status != nullptr && g.status->error != 0u) return;   // uniform over the grid: leave everything alone

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int i0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
  const int n_begin = FUSE ? 0 : (int)blockIdx.z;
  const int n_end = FUSE ? g.N : n_begin + 1;
  const bool do_bias = (EPI == EPI_DW) && blockIdx.x == 0;

  float sum[RM][4];
  float bias_sum_all = 0.f;
#pragma unroll
  for (int r = 0; r < RM; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) sum[r][c] = 0.f;

  for (int n = n_begin; n < n_end; ++n) {
    const bool is_active = g.active == nullptr || g.active[n] != 0;
    if (!FUSE && !is_active) return;          // an inactive worker keeps its point
    float acc[RM][4];
#pragma unroll
    for (int r = 0; r < RM; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
    float bsum = 0.f;

    if (is_active) {
      const float* Ap = operand_ptr(g.A, n, g.draw);
      const float* Bp = operand_ptr(g.Bo, n, g.draw);
      // software pipeline: the next K chunk travels global -> registers while the current one is
      // consumed from shared memory; two shared buffers, one barrier per chunk
      float ra[LA], rb[LB];
      auto gload = [&](int k0) {
#pragma unroll
        for (int r = 0; r < LA; ++r) {
          const int e = tid + 256 * r;
          const int i = A_PC ? e / TK : e % TM;
          const int p = A_PC ? e % TK : e / TM;
          ra[r] = (i0 + i < g.M && k0 + p < g.K) ? Ap[(int64_t)(i0 + i) * g.A.s0 + (int64_t)(k0 + p) * g.A.s1] : 0.f;
        }
#pragma unroll
        for (int r = 0; r < LB; ++r) {
          const int e = tid + 256 * r;
          const int j = B_PC ? e / TK : e % TN;
          const int p = B_PC ? e % TK : e / TN;
          rb[r] = (j0 + j < g.Nn && k0 + p < g.K) ? Bp[(int64_t)(k0 + p) * g.Bo.s0 + (int64_t)(j0 + j) * g.Bo.s1] : 0.f;
        }
      };
      auto sstore = [&](int buf) {
#pragma unroll
        for (int r = 0; r < LA; ++r) {
          const int e = tid + 256 * r;
          As[buf][A_PC ? e % TK : e / TM][A_PC ? e / TK : e % TM] = ra[r];
        }
#pragma unroll
        for (int r = 0; r < LB; ++r) {
          const int e = tid + 256 * r;
          Bs[buf][B_PC ? e % TK : e / TN][B_PC ? e / TK : e % TN] = rb[r];
        }
      };
      gload(0);
      sstore(0);
      __syncthreads();
      int buf = 0;
      for (int k0 = 0; k0 < g.K; k0 += TK) {
        const bool more = k0 + TK < g.K;
        if (more) gload(k0 + TK);
#pragma unroll
        for (int p = 0; p < TK; ++p) {
          float a[RM];
#pragma unroll
          for (int r = 0; r < RM; ++r) a[r] = As[buf][p][ty * RM + r];
          const float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][p][tx * 4]);
          const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
          for (int r = 0; r < RM; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
        }
        if (do_bias && tid < TM) {
#pragma unroll
          for (int p = 0; p < TK; ++p) bsum += As[buf][p][tid];
        }
        if (more) sstore(buf ^ 1);
        __syncthreads();
        buf ^= 1;
      }
    }

    // ---- epilogue for worker n
    if (EPI == EPI_FWD_RELU || EPI == EPI_FWD_LINEAR) {
      const float* bias = g.params + (int64_t)n * g.params_worker_stride + g.b_off;
      float* o = g.out + (int64_t)n * g.out_worker_stride;
#pragma unroll
      for (int r = 0; r < RM; ++r) {
        int i = i0 + ty * RM + r;
        if (i >= g.M) continue;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int j = j0 + tx * 4 + c;
          if (j >= g.Nn) continue;
          float v = acc[r][c] + bias[j];
          if (EPI == EPI_FWD_RELU) v = fmaxf(v, 0.f);
          o[(int64_t)i * g.Nn + j] = v;
        }
      }
    } else if (EPI == EPI_DX) {
      float* o = g.out + (int64_t)n * g.out_worker_stride;
      const float* msk = g.mask_src + (int64_t)n * g.out_worker_stride;
#pragma unroll
      for (int r = 0; r < RM; ++r) {
        int i = i0 + ty * RM + r;
        if (i >= g.M) continue;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int j = j0 + tx * 4 + c;
          if (j >= g.Nn) continue;
          o[(int64_t)i * g.Nn + j] = msk[(int64_t)i * g.Nn + j] > 0.f ? acc[r][c] : 0.f;
        }
      }
    } else {  // EPI_DW: x <- x - gamma * G in place (Eq. parallel-sgd-x-update)
      float* row = g.out + (int64_t)n * g.out_worker_stride;
      float* W = row + g.w_off;
#pragma unroll
      for (int r = 0; r < RM; ++r) {
        int i = i0 + ty * RM + r;
        if (i >= g.M) continue;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int j = j0 + tx * 4 + c;
          if (j >= g.Nn) continue;
          float w = W[(int64_t)i * g.Nn + j];
          float step = acc[r][c];
          if (g.vel != nullptr && is_active) {             // v <- mu v + G ; x <- x - gamma v
            float* vp = g.vel + (int64_t)n * g.out_worker_stride + g.w_off + (int64_t)i * g.Nn + j;
            step = fmaf(g.mu, *vp, step);
            *vp = step;
          }
          float xi = is_active ? fmaf(-g.gamma, step, w) : w;
          if (FUSE) sum[r][c] += xi;
          else W[(int64_t)i * g.Nn + j] = xi;
        }
      }
      if (do_bias && tid < TM && i0 + tid < g.M) {
        float* bp = row + g.b_off + i0 + tid;
        float bstep = bsum;
        if (g.vel != nullptr && is_active) {
          float* vp = g.vel + (int64_t)n * g.out_worker_stride + g.b_off + i0 + tid;
          bstep = fmaf(g.mu, *vp, bstep);
          *vp = bstep;
        }
        float xi = is_active ? fmaf(-g.gamma, bstep, *bp) : *bp;
        if (FUSE) bias_sum_all += xi;
        else *bp = xi;
      }
    }
  }

  if (FUSE && EPI == EPI_DW) {
    // node average of the freshly updated models, written to every row
    const float fN = (float)g.N;
#pragma unroll
    for (int r = 0; r < RM; ++r) {
      int i = i0 + ty * RM + r;
      if (i >= g.M) continue;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int j = j0 + tx * 4 + c;
        if (j >= g.Nn) continue;
        float y = __fdiv_rn(sum[r][c], fN);
        for (int n = 0; n < g.N; ++n)
          g.out[(int64_t)n * g.out_worker_stride + g.w_off + (int64_t)i * g.Nn + j] = y;
      }
    }
    if (do_bias && tid < TM && i0 + tid < g.M) {
      float y = __fdiv_rn(bias_sum_all, fN);
      for (int n = 0; n < g.N; ++n) g.out[(int64_t)n * g.out_worker_stride + g.b_off + i0 + tid] = y;
    }
  }
}

// delta_L = (softmax(z_L) - onehot(y)) / B and the per-sample losses.
// Grid (N, ceil(B / 8)), 256 threads: one warp per minibatch row.
struct SoftmaxArgs {
  const float* logits;   // [N][B][ldz]
  float* delta;          // [N][B][ldz]  (fp32), may be nullptr
  uint16_t* delta_bk;    // bf16 [N][B][ld_bf] or nullptr
  int ld_bf;
  int ldz;
  const int32_t* Y;      // [N][P]
  int64_t P;
  int B, C;
  DrawArgs draw;
  float* row_losses;     // [N][B]: logsumexp(z_b) - z_b[y_b]; the caller averages them in row order
  int32_t* draws;        // [N]
  const uint8_t* active;
  const DeviceStatus* status;   // tensor-core path: a recorded expired wait turns the launch into a no-op
};

__device__ __forceinline__ uint16_t f32_to_bf16_rn(float f) {
  uint32_t u = __float_as_uint(f);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

__global__ void __launch_bounds__(256) softmax_ce_kernel(const SoftmaxArgs a) {
  asm volatile("griddepcontrol.wait;" ::: "memory");   // no-op unless launched as a programmatic dependent
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // after the wait: see tc_stream_kernel
  const int n = blockIdx.x;
  if (a.active != nullptr && a.active[n] == 0) return;
  if (a.status != nullptr && a.status->error != 0u) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y * 8 + warp;
  const uint32_t blk = draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks);
  if (blockIdx.y == 0 && threadIdx.x == 0) a.draws[n] = (int32_t)blk;
  if (b >= a.B) return;
  const float invB = 1.f / (float)a.B;
  const float* z = a.logits + ((int64_t)n * a.B + b) * a.ldz;
  float mx = -INFINITY;
  for (int c = lane; c < a.C; c += 32) mx = fmaxf(mx, z[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float s = 0.f;
  for (int c = lane; c < a.C; c += 32) s += expf(z[c] - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float lse = mx + logf(s);
  const int label = a.Y[(int64_t)n * a.P + (int64_t)blk * a.B + b];
  for (int c = lane; c < a.C; c += 32) {
    float d = (expf(z[c] - lse) - (c == label ? 1.f : 0.f)) * invB;
    if (a.delta) a.delta[((int64_t)n * a.B + b) * a.ldz + c] = d;
    if (a.delta_bk) a.delta_bk[((int64_t)n * a.B + b) * a.ld_bf + c] = f32_to_bf16_rn(d);
  }
  if (lane == 0) a.row_losses[(int64_t)n * a.B + b] = lse - z[label];
}

}  // namespace prsgd
