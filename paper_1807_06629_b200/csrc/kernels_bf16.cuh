// bf16-operand tensor-core path (sm_100a): grouped GEMMs on tcgen05 with TMEM
// accumulators, operands staged by TMA, one problem per worker.
//
//   stream kernel  : forward  Z^T[d_out, B]  = W[d_out, d_in] A^T[d_in, B]      (+bias, ReLU)   (persistent)
//                    backward dA^T[d_in, B]  = W^T[d_in, d_out] dZ^T[d_out, B]  (ReLU mask)
//                    The layer width sits on the MMA's M axis (128 rows per CTA) and the
//                    minibatch on its N axis, because B = 16..64 is too small for M.
//   update kernel  : dW[d_out, d_in] = dZ^T A over K = B, then x <- x - gamma dW in the
//                    epilogue, in place, fp32 master and bf16 shadow written by TMA.
//                    A bandwidth kernel: the MMA is tiny, the epilogue moves 10 B per parameter.
//                    FUSE: the node average of the updated models is formed in registers over
//                    all workers and written to every worker's rows (Algorithm 1, averaging step).
#pragma once
#include <new>
#include "prsgd_common.cuh"
#include "kernels_f32.cuh"
#include "kernels_avg.cuh"
#include "tc_ptx.cuh"

namespace prsgd {

// ---------------------------------------------------------------------------------------------
// host-side state: tensor maps
// ---------------------------------------------------------------------------------------------
struct TcLayerMaps {
  CUtensorMap shadow_k;     // bf16 W_l  dims {d_in, d_out, N}, box {64, 128, 1}: forward A tiles, shadow stores
  CUtensorMap shadow_mn;    // same tensor, box {64, 64, 1}: backward A tiles (W^T, MN-major)
  CUtensorMap master;       // fp32 W_l  dims {d_in, d_out, N}, box {32, 128, 1}: update loads and stores
  CUtensorMap velocity;     // fp32 momentum buffer of W_l, same geometry as master (valid once momentum is enabled)
  CUtensorMap act_in;       // bf16 a_{l-1} dims {ld, B, N}, box {64, B, 1} (layer 1: the data pool {d0, P, N})
  CUtensorMap delta_out;    // bf16 dZ_l  dims {ld, B, N}, box {64, B, 1}
};

struct TcState {
  TcLayerMaps layer[PRSGD_MAX_LAYERS];
  CUtensorMap head_shadow;  // bf16 W_L, box {64, ceil16(d_L), 1}: tiles of tc_head_kernel (valid when head_rows > 0)
  CUtensorMap head_master;  // fp32 W_L, box {32, ceil16(d_L), 1}
  CUtensorMap act1_alt;     // a_1 in its second buffer, same geometry as layer[1].act_in (valid when L >= 2)
  int head_rows = 0;
  int num_sms = 148;
  bool pool_bound = false;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn(std::string* err) {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
    *err = "cuTensorMapEncodeTiled is not available from the driver";
    return nullptr;
  }
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// 3-D tiled map with 128-byte swizzle; dims/box innermost first; strides in bytes for dims 1 and 2.
inline int make_map3(CUtensorMap* m, bool fp32, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                     uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, std::string* err) {
  EncodeTiledFn enc = get_encode_fn(err);
  if (!enc) return PRSGD_ERR_CUDA;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {b0, b1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                   const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    *err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return PRSGD_ERR_CUDA;
  }
  return PRSGD_OK;
}

// ---------------------------------------------------------------------------------------------
// stream kernel: forward and backward-data GEMMs
// ---------------------------------------------------------------------------------------------
enum { TC_FWD_RELU = 0, TC_FWD_LINEAR = 1, TC_DX = 2 };

struct StreamArgs {
  int B, N;
  int k_steps;             // pipeline steps per item: ceil(contraction length / 128)
  int tiles_m;             // 128-row tiles of the output features
  int M_total;             // valid output features
  int stages;
  int pool;                // operand B rows come from the data pool at the drawn block
  DrawArgs draw;
  uint16_t* out_bk;        // bf16 [N][B][ld_out]
  float* out_f32;          // fp32 [N][B][ld_out] (logits)
  int ld_out;
  const float* bias;       // params + b_off; worker stride bias_stride
  int64_t bias_stride;
  const uint16_t* mask_src;  // bf16 a_{l-1} [N][B][ld_out] (TC_DX)
  const uint8_t* active;
  DeviceStatus* status;
  // Bias step folded into the epilogue that produces dZ of the output layer (TC_DX: the layer below;
  // TC_FWD_LINEAR with `softmax`: the last layer): b <- b - gamma sum_b dZ[b, :]
  float* bias_rw;            // params + b_off of that layer (worker stride bias_stride), or nullptr
  float* bias_vel;           // its momentum segment, or nullptr
  float gamma, mu;
  // Softmax cross-entropy gradient in the epilogue of the last forward GEMM (needs tiles_m == 1)
  WTile wt;                  // order of the weight segment's elements
  int prefetch;              // 1: the weight tiles may be requested before the previous launch has completed
  int shared_w;              // 1: every worker's weights hold the same bits (the launch follows a node average with
                             // nothing in between), so every item reads worker 0's tiles: one HBM read serves all N
  int softmax;
  const int32_t* Y;          // labels [N][P]
  int64_t P;
  uint16_t* delta_bk;        // bf16 dZ_L [N][B][ld_delta]
  int ld_delta;
  float* row_losses;         // [N][B]
  int32_t* draws;            // [N]
  unsigned int* zero_word;   // not nullptr: block 0 clears this word after its dependency wait (the item counter of an
                             // overlapped update launched later in the iteration)
};

// Persistent: one CTA per SM walks (tile, worker) items.  Warp 0 issues TMA, warp 1 issues MMAs,
// warps 2..5 run the epilogue of item i from one TMEM accumulator while the loads and MMAs of
// item i + 1 fill the other, so the weight stream never pauses at an item boundary.
// A stage holds TWO 64-wide K blocks (>= 40 KB per barrier phase): a single issuing thread
// sustains only ~2 barrier phases per microsecond, so small stages would cap the stream.
constexpr int kStreamThreads = 192;
constexpr uint32_t kTileA = 16384;   // 128 x 64 bf16

constexpr int kLogitLd = 129;        // row pitch (floats) of the logits tile the softmax epilogue keeps in shared memory

__host__ __device__ inline uint32_t stream_stage_bytes(int B) { return 2u * (kTileA + (uint32_t)B * 128u); }
__host__ __device__ inline uint32_t stream_logit_bytes(int B, bool softmax) { return softmax ? (uint32_t)B * kLogitLd * 4u : 0u; }
inline int stream_stages(int B, bool softmax = false) {
  int s = (int)((200000u - stream_logit_bytes(B, softmax)) / stream_stage_bytes(B));
  return s > 6 ? 6 : s;
}
inline size_t stream_smem_bytes(int B, bool softmax = false) {
  return (size_t)stream_stages(B, softmax) * stream_stage_bytes(B) + 1024 + 256 + stream_logit_bytes(B, softmax);
}

template <int MODE>
__global__ void __launch_bounds__(kStreamThreads, 1) tc_stream_kernel(const __grid_constant__ CUtensorMap mapW,
                                                                      const __grid_constant__ CUtensorMap mapB,
                                                                      const StreamArgs a) {
  using namespace ptx;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t stage_bytes = stream_stage_bytes(a.B);
  const uint32_t b_box = (uint32_t)a.B * 128u;
  const int S = a.stages;
  const uint32_t bar0 = base + (uint32_t)S * stage_bytes;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int q) { return bar0 + 128u + 8u * q; };
  auto acc_empty = [&](int q) { return bar0 + 144u + 8u * q; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + (size_t)S * stage_bytes + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (size_t)S * stage_bytes + 164);
  float* zs = reinterpret_cast<float*>(gen + (size_t)S * stage_bytes + 256);   // [B][kLogitLd], softmax epilogue only

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t ncols = 2 * a.B < 32 ? 32u : (uint32_t)(2 * a.B);   // two accumulators of B columns

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int q = 0; q < 2; ++q) { mbar_init(acc_full(q), 1); mbar_init(acc_empty(q), 128); }
    // A wait that expired in an earlier launch turns this one into a no-op.  The word is read here, off
    // the critical path: a launch whose set-up overlapped the failing one may miss it and run (its own
    // waits are bounded too); every launch after that sees it.
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;
    fence_mbar_init();
    prefetch_tensormap(&mapW);
    prefetch_tensormap(&mapB);
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), ncols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Weight tiles of a pipeline step (two 64-wide K blocks of the 128-row tile of worker n).
  auto load_weights = [&](int s, int ks, int m0, int n) {
    const uint32_t sa = base + (uint32_t)s * stage_bytes;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int k0 = (2 * ks + j) * 64;              // a block past the end of K is zero-filled by TMA
      if (MODE == TC_DX) {
        tma_load_w(sa + j * kTileA, &mapW, full_bar(s), a.wt, m0, k0, n);
        tma_load_w(sa + j * kTileA + 8192u, &mapW, full_bar(s), a.wt, m0 + 64, k0, n);
      } else {
        tma_load_w(sa + j * kTileA, &mapW, full_bar(s), a.wt, k0, m0, n);
      }
    }
  };
  auto load_operand = [&](int s, int ks, int row0, int n) {
    const uint32_t sb = base + (uint32_t)s * stage_bytes + 2u * kTileA;
#pragma unroll
    for (int j = 0; j < 2; ++j) tma_load_3d(sb + j * b_box, &mapB, full_bar(s), (2 * ks + j) * 64, row0, n);
  };
  // The weights this launch reads were last written before the previous launch began (the host sets
  // `prefetch` only then), so the first stages' weight tiles are requested while that launch drains.
  // Item -> (worker, row tile).  Worker-major as a rule; with shared weights tile-major, so that the N items
  // that read the same tile run at about the same time and all but the first find it in L2.
  auto item_worker = [&](int item) { return a.shared_w ? item % a.N : item / a.tiles_m; };
  auto item_row0 = [&](int item) { return (a.shared_w ? item / a.N : item % a.tiles_m) * 128; };
  uint32_t pre = 0;
  if (warp == 0 && lane == 0 && a.prefetch != 0 && (int)blockIdx.x < a.tiles_m * a.N) {
    const int n = a.shared_w ? 0 : item_worker((int)blockIdx.x), m0 = item_row0((int)blockIdx.x);
    pre = (uint32_t)(a.k_steps < S ? a.k_steps : S);
    for (uint32_t ks = 0; ks < pre; ++ks) {
      mbar_expect_tx(full_bar(ks), stage_bytes);
      load_weights((int)ks, (int)ks, m0, n);
    }
  }
  pdl_wait();            // everything above overlapped the previous kernel's tail; dependent memory is touched below
  pdl_trigger();         // only now: the next launch's early loads may overlap this launch, never an older one
  if (a.zero_word != nullptr && blockIdx.x == 0 && tid == 0) *a.zero_word = 0u;
  const uint32_t tmem = *tmem_slot;
  const int total_items = *abort_flag != 0 ? 0 : a.tiles_m * a.N;
  auto item_active = [&](int n) { return a.active == nullptr || a.active[n] != 0; };

  if (warp == 0 && lane == 0) {
    // ---------------- producer: per step two weight K blocks and two activation K blocks
    uint32_t g = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const int n = item_worker(item), m0 = item_row0(item);
      if (!item_active(n)) continue;
      const int row0 = a.pool ? (int)draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks) * a.B : 0;
      for (int ks = 0; ks < a.k_steps; ++ks, ++g) {
        const int s = g % S;
        const uint32_t ph = (g / S) & 1u;
        if (g >= pre) {                               // (the early steps already have their weights under way)
          ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, a.status, 0x101);
          if (!ok) break;
          mbar_expect_tx(full_bar(s), stage_bytes);
          load_weights(s, ks, m0, a.shared_w ? 0 : n);
        }
        load_operand(s, ks, row0, n);
      }
    }
    if (total_items == 0 && pre > 0) {   // nothing will consume the early tiles: complete their stages
      for (uint32_t ks = 0; ks < pre; ++ks) load_operand((int)ks, (int)ks, 0, item_worker((int)blockIdx.x));
      g = pre;
    }
    if (*abort_flag && g > 0) {   // let the copies already in flight land before the CTA goes away
      const uint32_t first = g > (uint32_t)S ? g - (uint32_t)S : 0u;
      for (uint32_t q = first; q < g; ++q) {
        const long long t0 = clock64();
        while (!mbar_try_wait(full_bar(q % S), (q / S) & 1u) && clock64() - t0 < 200000000ll) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    constexpr int A_MN = MODE == TC_DX ? 1 : 0;
    const uint32_t idesc = idesc_bf16(128, a.B, A_MN, 0);
    uint32_t g = 0, it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      if (!item_active(item_worker(item))) continue;
      const int q = it & 1;
      ok = mbar_wait(acc_empty(q), ((it >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x104);
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = tmem + (uint32_t)(q * a.B);
      for (int ks = 0; ks < a.k_steps; ++ks, ++g) {
        const int s = g % S;
        ok = mbar_wait(full_bar(s), (g / S) & 1u, abort_flag, a.status, 0x102);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + 2u * kTileA;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t aj = sa + j * kTileA, bj = sb + j * b_box;
            const uint64_t da = A_MN ? smem_desc_sw128(aj + k * 2048u, 8192u, 1024u) : smem_desc_sw128(aj + k * 32u, 16u, 1024u);
            const uint64_t db = smem_desc_sw128(bj + k * 32u, 16u, 1024u);
            mma_bf16(acc, da, db, idesc, (ks | j | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(empty_bar(s));
      }
      if (ok) mma_commit(acc_full(q));
      ++it;
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: thread <-> output feature, its B accumulators sit in one TMEM lane.
    // Work goes in batches of 16 minibatch columns; the ReLU-mask values a batch needs (TC_DX) are
    // fetched one batch ahead, the first of them before the accumulator is even ready, so that no
    // global-load latency sits between the accumulator and the stores.
    const int q4 = warp & 3;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const int batches = a.B / 16;
    uint32_t it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const int n = item_worker(item);
      if (!item_active(n)) continue;
      const int m = item_row0(item) + q4 * 32 + lane;
      const bool valid = m < a.M_total;
      auto mask_fetch = [&](int bi, uint16_t (&mk)[16]) {
        if (MODE == TC_DX && bi < batches && valid) {
#pragma unroll
          for (int j = 0; j < 16; ++j) mk[j] = __ldg(a.mask_src + ((int64_t)n * a.B + bi * 16 + j) * a.ld_out + m);
        }
      };
      uint16_t mk_cur[16], mk_next[16];
      mask_fetch(0, mk_cur);
      float bias = 0.f;
      if (MODE != TC_DX && valid) bias = a.bias[(int64_t)n * a.bias_stride + m];
      const bool smx = MODE == TC_FWD_LINEAR && a.softmax != 0;
      float gsum = 0.f;                                   // sum over the minibatch of this feature's dZ
      const int etid = tid - 64;                          // 0..127 among the epilogue threads
      uint32_t blk = 0;
      int label = 0;
      if (MODE == TC_FWD_LINEAR && smx) {                 // the label of this thread's row, fetched ahead of the wait
        blk = draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks);
        label = a.Y[(int64_t)n * a.P + (int64_t)blk * a.B + etid / (128 / a.B)];
      }
      const int q = it & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(acc_full(q), (it >> 1) & 1u, abort_flag, a.status, 0x103));
      if (!ok) break;
      tc_fence_after();
      for (int bi = 0; bi < batches; ++bi) {
        const int c0 = bi * 16;
        uint32_t v[16];
        tmem_ld16(tmem + lane_off + (uint32_t)(q * a.B + c0), v);
        mask_fetch(bi + 1, mk_next);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int64_t o = ((int64_t)n * a.B + c0 + j) * a.ld_out + m;
            const float x = __uint_as_float(v[j]);
            if (MODE == TC_FWD_RELU) {
              a.out_bk[o] = f32_to_bf16_rn(fmaxf(x + bias, 0.f));
            } else if (MODE == TC_FWD_LINEAR) {
              if (smx) zs[(c0 + j) * kLogitLd + m] = x + bias;
              else a.out_f32[o] = x + bias;
            } else {
              const float d = (mk_cur[j] & 0x7FFFu) != 0 ? x : 0.f;
              gsum += d;
              a.out_bk[o] = f32_to_bf16_rn(d);
            }
          }
        }
        if (MODE == TC_DX) {
#pragma unroll
          for (int j = 0; j < 16; ++j) mk_cur[j] = mk_next[j];
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty(q));
      ++it;
      if (MODE == TC_FWD_LINEAR && smx) {
        // Softmax cross-entropy gradient dZ_L = (softmax(z) - onehot(y)) / B and the per-sample loss.
        // The logits of the whole minibatch sit in shared memory; row b belongs to the T = 128 / B
        // neighbouring threads etid = b T .. b T + T - 1, each of which takes every T-th class.
        named_bar_sync(1, 128);
        const int C = a.M_total;
        const int T = 128 / a.B, sub = etid % T, b = etid / T;
        const float invB = 1.f / (float)a.B;
        float* z = zs + b * kLogitLd;
        float mx = -INFINITY;
        for (int cc = sub; cc < C; cc += T) mx = fmaxf(mx, z[cc]);
        for (int o = T >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int cc = sub; cc < C; cc += T) se += expf(z[cc] - mx);
        for (int o = T >> 1; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float lse = mx + logf(se);
        const float zl = z[label];
        __syncwarp();
        for (int cc = sub; cc < C; cc += T) z[cc] = (expf(z[cc] - lse) - (cc == label ? 1.f : 0.f)) * invB;
        if (sub == 0) a.row_losses[(int64_t)n * a.B + b] = lse - zl;
        if (etid == 0) a.draws[n] = (int32_t)blk;
        named_bar_sync(1, 128);
        if (valid) {
          for (int bb = 0; bb < a.B; ++bb) gsum += zs[bb * kLogitLd + m];
        }
        uint16_t* dn = a.delta_bk + (int64_t)n * a.B * a.ld_delta;
        for (int idx = etid; idx < a.B * C; idx += 128) {
          const int bb = idx / C, cc = idx - bb * C;
          dn[bb * a.ld_delta + cc] = f32_to_bf16_rn(zs[bb * kLogitLd + cc]);
        }
        named_bar_sync(1, 128);                           // the tile is free for the next item
      }
      if ((MODE == TC_DX || smx) && a.bias_rw != nullptr && valid) {
        float* bp = a.bias_rw + (int64_t)n * a.bias_stride + m;
        if (a.bias_vel != nullptr) {                      // momentum form of the local step
          float* vp = a.bias_vel + (int64_t)n * a.bias_stride + m;
          gsum = fmaf(a.mu, *vp, gsum);
          *vp = gsum;
        }
        *bp = fmaf(-a.gamma, gsum, *bp);
      }
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, ncols);
}

// ---------------------------------------------------------------------------------------------
// forward chain: the forward GEMMs of consecutive layers l_first..L in ONE launch
// ---------------------------------------------------------------------------------------------
// The items of all layers form one list (layer by layer); a CTA walks its share of the list with the same
// TMA / MMA / epilogue pipeline as tc_stream_kernel and never drains between layers.  Workers are independent
// inside an iteration, so an item of layer l only needs a_{l-1} of ITS worker: a counter per (layer, worker)
// counts the finished row tiles, the epilogue adds to it once an item's activations are in global memory,
// and the loader waits for it (bounded) before it requests the activation tiles; the weight tiles, which do
// not depend on this launch, are requested first.  Items are walked in list order and every grid has at
// most one CTA per SM, all resident, so the oldest unfinished item can always run: no wait can be circular.
// The last CTA to finish zeroes the counters for the next launch.
constexpr int kChainMax = 8;

struct ChainSeg {
  int k_steps, tiles_m, M_total, ld_out;
  int linear;                // 0: bias + ReLU, bf16 out; 1: the last layer (fp32 logits, or the softmax epilogue)
  int pool;                  // operand B rows come from the data pool at the drawn block (layer 1)
  int prefetch;              // the weight tiles may be requested before the previous launch has completed
  int item0;                 // index of the layer's first item in the list
  WTile wt;                  // order of the weight segment's elements
  uint16_t* out_bk;          // bf16 [N][B][ld_out]
  float* out_f32;            // fp32 [N][B][ld_out] (logits without the softmax epilogue)
  const float* bias;         // params + b_off; worker stride ChainArgs::bias_stride
};

struct ChainMaps {
  CUtensorMap w[kChainMax];  // bf16 W_l, box {64, 128, 1}
  CUtensorMap b[kChainMax];  // bf16 a_{l-1} (the data pool for layer 1), box {64, B, 1}
};

struct ChainArgs {
  int B, N, stages, n_seg, total_items;
  int shared_w;              // every worker's weights hold the same bits: read worker 0's tiles (see StreamArgs)
  int softmax;               // the last layer's epilogue forms the softmax cross-entropy gradient
  DrawArgs draw;
  const uint8_t* active;
  DeviceStatus* status;
  int64_t bias_stride;
  unsigned int* ready;       // [n_seg][N] finished row tiles of (layer, worker); zero between launches
  unsigned int* done;        // CTAs that have finished; zero between launches
  float* bias_rw; float* bias_vel; float gamma, mu;     // step of b_L in the softmax epilogue
  const int32_t* Y; int64_t P; uint16_t* delta_bk; int ld_delta; float* row_losses; int32_t* draws;
  ChainSeg seg[kChainMax];
};

__global__ void __launch_bounds__(kStreamThreads, 1) tc_forward_chain_kernel(const __grid_constant__ ChainMaps maps,
                                                                             const __grid_constant__ ChainArgs a) {
  using namespace ptx;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t stage_bytes = stream_stage_bytes(a.B);
  const uint32_t b_box = (uint32_t)a.B * 128u;
  const int S = a.stages;
  const uint32_t bar0 = base + (uint32_t)S * stage_bytes;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int q) { return bar0 + 128u + 8u * q; };
  auto acc_empty = [&](int q) { return bar0 + 144u + 8u * q; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + (size_t)S * stage_bytes + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (size_t)S * stage_bytes + 164);
  float* zs = reinterpret_cast<float*>(gen + (size_t)S * stage_bytes + 256);   // [B][kLogitLd], softmax epilogue only

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t ncols = 2 * a.B < 32 ? 32u : (uint32_t)(2 * a.B);   // two accumulators of B columns

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int q = 0; q < 2; ++q) { mbar_init(acc_full(q), 1); mbar_init(acc_empty(q), 128); }
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    for (int i = 0; i < a.n_seg; ++i) { prefetch_tensormap(&maps.w[i]); prefetch_tensormap(&maps.b[i]); }
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), ncols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  auto seg_of = [&](int item) { int si = 0; while (si + 1 < a.n_seg && item >= a.seg[si + 1].item0) ++si; return si; };
  // worker-major inside a layer as a rule; tile-major with shared weights (see tc_stream_kernel)
  auto item_worker = [&](const ChainSeg& g, int item) { const int r = item - g.item0; return a.shared_w ? r % a.N : r / g.tiles_m; };
  auto item_row0 = [&](const ChainSeg& g, int item) { const int r = item - g.item0; return (a.shared_w ? r / a.N : r % g.tiles_m) * 128; };
  auto load_weights = [&](int si, int s, int ks, int m0, int n) {
    const uint32_t sa = base + (uint32_t)s * stage_bytes;
#pragma unroll
    for (int j = 0; j < 2; ++j) tma_load_w(sa + j * kTileA, &maps.w[si], full_bar(s), a.seg[si].wt, (2 * ks + j) * 64, m0, n);
  };
  auto load_operand = [&](int si, int s, int ks, int row0, int n) {
    const uint32_t sb = base + (uint32_t)s * stage_bytes + 2u * kTileA;
#pragma unroll
    for (int j = 0; j < 2; ++j) tma_load_3d(sb + j * b_box, &maps.b[si], full_bar(s), (2 * ks + j) * 64, row0, n);
  };
  // early weight loads of this CTA's first item (see tc_stream_kernel), when its layer allows them
  uint32_t pre = 0;
  if (warp == 0 && lane == 0 && (int)blockIdx.x < a.total_items) {
    const int si = seg_of((int)blockIdx.x);
    const ChainSeg& g = a.seg[si];
    if (g.prefetch != 0) {
      const int n = a.shared_w ? 0 : item_worker(g, (int)blockIdx.x), m0 = item_row0(g, (int)blockIdx.x);
      pre = (uint32_t)(g.k_steps < S ? g.k_steps : S);
      for (uint32_t ks = 0; ks < pre; ++ks) {
        mbar_expect_tx(full_bar(ks), stage_bytes);
        load_weights(si, (int)ks, (int)ks, m0, n);
      }
    }
  }
  pdl_wait();
  pdl_trigger();
  const uint32_t tmem = *tmem_slot;
  const int total_items = *abort_flag != 0 ? 0 : a.total_items;
  auto item_active = [&](int n) { return a.active == nullptr || a.active[n] != 0; };

  if (warp == 0 && lane == 0) {
    // ---------------- producer
    uint32_t g = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const int si = seg_of(item);
      const ChainSeg& sg = a.seg[si];
      const int n = item_worker(sg, item), m0 = item_row0(sg, item);
      if (!item_active(n)) continue;
      const int row0 = sg.pool ? (int)draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks) * a.B : 0;
      for (int ks = 0; ks < sg.k_steps; ++ks, ++g) {
        const int s = g % S;
        const uint32_t ph = (g / S) & 1u;
        if (g >= pre) {
          ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, a.status, 0x601);
          if (!ok) break;
          mbar_expect_tx(full_bar(s), stage_bytes);
          load_weights(si, s, ks, m0, a.shared_w ? 0 : n);
        }
        if (ks == 0 && si > 0) {
          // a_{l-1} of this worker: every row tile of the layer below must be in global memory
          ok = flag_wait(a.ready + (size_t)(si - 1) * a.N + n, (unsigned)a.seg[si - 1].tiles_m, abort_flag, a.status, 0x605);
          if (!ok) break;
          fence_proxy_async_all();                      // written by other CTAs' plain stores, read below by TMA
        }
        load_operand(si, s, ks, row0, n);
      }
    }
    if (total_items == 0 && pre > 0) {   // nothing will consume the early tiles: complete their stages
      const int si = seg_of((int)blockIdx.x);
      for (uint32_t ks = 0; ks < pre; ++ks) load_operand(si, (int)ks, (int)ks, 0, 0);
      g = pre;
    }
    if (*abort_flag && g > 0) {   // let the copies already in flight land before the CTA goes away
      const uint32_t first = g > (uint32_t)S ? g - (uint32_t)S : 0u;
      for (uint32_t q = first; q < g; ++q) {
        const long long t0 = clock64();
        while (!mbar_try_wait(full_bar(q % S), (q / S) & 1u) && clock64() - t0 < 200000000ll) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = idesc_bf16(128, a.B, 0, 0);
    uint32_t g = 0, it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const ChainSeg& sg = a.seg[seg_of(item)];
      if (!item_active(item_worker(sg, item))) continue;
      const int q = it & 1;
      ok = mbar_wait(acc_empty(q), ((it >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x604);
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = tmem + (uint32_t)(q * a.B);
      for (int ks = 0; ks < sg.k_steps; ++ks, ++g) {
        const int s = g % S;
        ok = mbar_wait(full_bar(s), (g / S) & 1u, abort_flag, a.status, 0x602);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = base + (uint32_t)s * stage_bytes, sb = sa + 2u * kTileA;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t aj = sa + j * kTileA, bj = sb + j * b_box;
            mma_bf16(acc, smem_desc_sw128(aj + k * 32u, 16u, 1024u), smem_desc_sw128(bj + k * 32u, 16u, 1024u), idesc,
                     (ks | j | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(empty_bar(s));
      }
      if (ok) mma_commit(acc_full(q));
      ++it;
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: thread <-> output feature (see tc_stream_kernel)
    const int q4 = warp & 3;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const int batches = a.B / 16;
    const int etid = tid - 64;                            // 0..127 among the epilogue threads
    uint32_t it = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const int si = seg_of(item);
      const ChainSeg& sg = a.seg[si];
      const int n = item_worker(sg, item);
      if (!item_active(n)) continue;
      const int m = item_row0(sg, item) + q4 * 32 + lane;
      const bool valid = m < sg.M_total;
      const float bias = valid ? sg.bias[(int64_t)n * a.bias_stride + m] : 0.f;
      const bool smx = sg.linear != 0 && a.softmax != 0;
      float gsum = 0.f;                                   // sum over the minibatch of this feature's dZ
      uint32_t blk = 0;
      int label = 0;
      if (smx) {                                          // the label of this thread's row, fetched ahead of the wait
        blk = draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks);
        label = a.Y[(int64_t)n * a.P + (int64_t)blk * a.B + etid / (128 / a.B)];
      }
      const int q = it & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(acc_full(q), (it >> 1) & 1u, abort_flag, a.status, 0x603));
      if (!ok) break;
      tc_fence_after();
      for (int bi = 0; bi < batches; ++bi) {
        const int c0 = bi * 16;
        uint32_t v[16];
        tmem_ld16(tmem + lane_off + (uint32_t)(q * a.B + c0), v);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int64_t o = ((int64_t)n * a.B + c0 + j) * sg.ld_out + m;
            const float x = __uint_as_float(v[j]) + bias;
            if (sg.linear == 0) sg.out_bk[o] = f32_to_bf16_rn(fmaxf(x, 0.f));
            else if (smx) zs[(c0 + j) * kLogitLd + m] = x;
            else sg.out_f32[o] = x;
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty(q));
      ++it;
      if (si + 1 < a.n_seg) {
        // this row tile of a_l is in global memory: count it for the items of layer l + 1 of this worker
        __threadfence();
        named_bar_sync(2, 128);
        if (etid == 0) red_release_add(a.ready + (size_t)si * a.N + n, 1u);
      }
      if (smx) {
        // softmax cross-entropy gradient and the step of b_L (see tc_stream_kernel)
        named_bar_sync(1, 128);
        const int C = sg.M_total;
        const int T = 128 / a.B, sub = etid % T, b = etid / T;
        const float invB = 1.f / (float)a.B;
        float* z = zs + b * kLogitLd;
        float mx = -INFINITY;
        for (int cc = sub; cc < C; cc += T) mx = fmaxf(mx, z[cc]);
        for (int o = T >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int cc = sub; cc < C; cc += T) se += expf(z[cc] - mx);
        for (int o = T >> 1; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float lse = mx + logf(se);
        const float zl = z[label];
        __syncwarp();
        for (int cc = sub; cc < C; cc += T) z[cc] = (expf(z[cc] - lse) - (cc == label ? 1.f : 0.f)) * invB;
        if (sub == 0) a.row_losses[(int64_t)n * a.B + b] = lse - zl;
        if (etid == 0) a.draws[n] = (int32_t)blk;
        named_bar_sync(1, 128);
        if (valid) {
          for (int bb = 0; bb < a.B; ++bb) gsum += zs[bb * kLogitLd + m];
        }
        uint16_t* dn = a.delta_bk + (int64_t)n * a.B * a.ld_delta;
        for (int idx = etid; idx < a.B * C; idx += 128) {
          const int bb = idx / C, cc = idx - bb * C;
          dn[bb * a.ld_delta + cc] = f32_to_bf16_rn(zs[bb * kLogitLd + cc]);
        }
        named_bar_sync(1, 128);                           // the tile is free for the next item
        if (a.bias_rw != nullptr && valid) {
          float* bp = a.bias_rw + (int64_t)n * a.bias_stride + m;
          if (a.bias_vel != nullptr) {                    // momentum form of the local step
            float* vp = a.bias_vel + (int64_t)n * a.bias_stride + m;
            gsum = fmaf(a.mu, *vp, gsum);
            *vp = gsum;
          }
          *bp = fmaf(-a.gamma, gsum, *bp);
        }
      }
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, ncols);
  if (tid == 0) {
    // the last CTA to get here has seen every other CTA finish all its waits: zero the counters for the next launch
    __threadfence();
    const unsigned int before = atomicAdd(a.done, 1u);
    if (before == gridDim.x - 1) {
      for (int i = 0; i < a.n_seg * a.N; ++i) a.ready[i] = 0u;
      *a.done = 0u;
      __threadfence();
    }
  }
}

// ---------------------------------------------------------------------------------------------
// update kernel: dW GEMM (K = B) + in-place SGD step, optionally fused with the node average
// ---------------------------------------------------------------------------------------------
struct UpdateArgs {
  int B, N;
  int tiles_m, tiles_n;
  float gamma;
  float mu;
  int pool;
  DrawArgs draw;
  const uint8_t* active;
  DeviceStatus* status;
  WTile wt;                // order of the weight segment's elements
  int prefetch;            // 1: master tiles may be requested before the previous launch has completed
  float divisor;           // fused form: the summed models are divided by this (N; 1 leaves the local row SUM in every
                           // row, the first half of an average whose other rows live on other GPUs)
  int avg_vel;             // fused form with momentum, 1: the momentum buffers are averaged like the models
  int shared_w;            // fused form only, 1: every worker's master tile holds the same bits (the launch follows a
                           // node average with nothing in between): all N loads of a tile read worker 0's copy, which
                           // nobody overwrites before the CTA that owns the tile has summed all N workers
  // Overlapped form (plain step only, no worker mask): the launch just before this one does not produce anything
  // this one reads and has passed its own dependency wait in every CTA before this one starts, so this kernel
  // begins WITHOUT a dependency wait, beside that launch, and takes the wait before it exits (whoever waits for
  // this launch thereby waits for both).  CTAs become resident as SMs fall free, so items are not dealt out by
  // block index: the loader claims the next one from *next_item (zero at launch) and hands the index to the other
  // roles through a ring in shared memory.
  unsigned int* next_item;
  // 1: the same start and end (no dependency wait until just before the exit) with items dealt out by block index:
  // for a launch enqueued right after a small one that it does not depend on (the averages of the bias segments),
  // whose CTAs have all passed their own dependency wait before this one starts.
  int late;
};

constexpr int kUpdSchedSlots = 8;         // ring of claimed item indices (>= twice the stage count)

constexpr int kUpdThreads = 224;          // warp 0 loader, 1 MMA, 2 storer, 3..6 epilogue
// The two folded update kernels end every block of tiles (a column block's dX, a row block's next forward)
// with an epilogue of its own; four more warps (7..10) run it, so that the tile epilogue warps go straight
// on to the next block's tiles and the weight stream does not pause at a block boundary.
constexpr int kUpdBlkThreads = 352;

// One pipeline stage of the update kernel for a 128 x TN tile: the fp32 master tile (TN/32 boxes of
// 128 x 32) followed by a region that first holds the operands (two dZ boxes and TN/64 activation
// boxes of {64, B}) and later, once the MMA has consumed them, the bf16 output tile (TN/64 boxes
// of 128 x 64).  TN = 64 gives four stages, TN = 128 two.
template <int TN, bool MOM> struct UpdCfg {
  static constexpr int kStages = (TN == 64 && !MOM) ? 4 : 2;
  static constexpr uint32_t kMaster = 128u * TN * 4u;
  static constexpr uint32_t kVel = MOM ? kMaster : 0u;          // momentum tile right after the master tile
  static constexpr uint32_t kOut = 128u * TN * 2u;
  __host__ __device__ static uint32_t ops_bytes(int B) { return (uint32_t)(2 + TN / 64) * (uint32_t)B * 128u; }
  __host__ __device__ static uint32_t region(int B) { return ops_bytes(B) > kOut ? ops_bytes(B) : kOut; }
  __host__ __device__ static uint32_t stage(int B) { return kMaster + kVel + region(B); }
  static size_t smem(int B) { return (size_t)kStages * stage(B) + 1024 + 384; }
};

// MOM: the local step of the paper's experiment, v <- mu v + G, x <- x - gamma v; the momentum tile
// travels with the master tile (loaded, updated in shared memory, stored back).  FUSE with MOM: every worker's
// new momentum tile goes back to its own row as the CTA walks the workers (avg_vel = 0), or a second set of
// running sums averages the momentum tiles as well and the mean goes to every row with the models (avg_vel = 1).
template <bool FUSE, int TN, bool MOM>
__global__ void __launch_bounds__(kUpdThreads, 1) tc_update_kernel(const __grid_constant__ CUtensorMap mapDelta,
                                                                   const __grid_constant__ CUtensorMap mapAct,
                                                                   const __grid_constant__ CUtensorMap mapMaster,
                                                                   const __grid_constant__ CUtensorMap mapShadow,
                                                                   const __grid_constant__ CUtensorMap mapVel,
                                                                   const UpdateArgs a) {
  using namespace ptx;
  using Cfg = UpdCfg<TN, MOM>;
  // Fused form, plain step, 64-wide tiles: the averaged tile (fp32 + bf16, 48 KB) is written to a buffer of its
  // own that takes the place of the fourth pipeline stage.  Its N row stores last ~17 us at one SM's share of
  // the HBM bandwidth; from a stage they would stall the loader for that long, from the buffer the three
  // remaining stages keep cycling through the next tile's workers meanwhile.
  constexpr bool kOutBuf = FUSE && !MOM && TN == 64;
  constexpr int S = kOutBuf ? Cfg::kStages - 1 : Cfg::kStages;
  constexpr int NB32 = TN / 32, NB64 = TN / 64;
  // Fused form on shared weights (every worker's master tile holds the same bits): all loads of a tile read
  // worker 0's copy; with 64-wide tiles and the plain step the tile is loaded ONCE, by its first worker, and
  // kept in registers while the CTA walks the other workers (wider tiles and the momentum step reload it from L2).
  constexpr bool kShareOnce = FUSE && !MOM && TN == 64;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t stage_bytes = Cfg::stage(a.B);
  auto master_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes; };
  auto vel_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster; };
  auto ops_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster + Cfg::kVel; };
  const uint32_t bar0 = base + (uint32_t)Cfg::kStages * stage_bytes;
  auto full_ops = [&](int s) { return bar0 + 8u * s; };
  auto full_w = [&](int s) { return bar0 + 32u + 8u * s; };
  auto stage_empty = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int s) { return bar0 + 96u + 8u * s; };
  auto acc_empty = [&](int s) { return bar0 + 128u + 8u * s; };
  auto tile_ready = [&](int s) { return bar0 + 160u + 8u * s; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + (size_t)Cfg::kStages * stage_bytes + 192);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (size_t)Cfg::kStages * stage_bytes + 196);
  const uint32_t out_free = bar0 + 200u;               // kOutBuf: the row stores have read the output buffer
  const uint32_t out_u32 = base + (uint32_t)S * stage_bytes;     // kOutBuf: fp32 tile, then the bf16 tile
  constexpr uint32_t R = (uint32_t)kUpdSchedSlots;
  auto sched_full = [&](uint32_t i) { return bar0 + 208u + 8u * i; };   // overlapped form: slot i of the ring holds an item index
  volatile int* sched = reinterpret_cast<volatile int*>(gen + (size_t)Cfg::kStages * stage_bytes + 272);
  const bool dyn = !FUSE && a.next_item != nullptr;
  const bool late = dyn || a.late != 0;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t op_box = (uint32_t)a.B * 128u;       // one {64, B} box
  const int tiles = a.tiles_m * a.tiles_n;
  const int items_all = FUSE ? tiles : tiles * a.N;    // FUSE: a CTA owns a tile and walks all workers

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_ops(s), 1); mbar_init(full_w(s), 1); mbar_init(stage_empty(s), 1);
      mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 128); mbar_init(tile_ready(s), 128);
    }
    mbar_init(out_free, 1);
    for (uint32_t i = 0; i < R; ++i) mbar_init(sched_full(i), 1);
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    prefetch_tensormap(&mapDelta); prefetch_tensormap(&mapAct);
    prefetch_tensormap(&mapMaster); prefetch_tensormap(&mapShadow);
    if (MOM) prefetch_tensormap(&mapVel);
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 256u); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // (with shared weights the master tile comes from worker 0's row; the momentum tile is always the worker's own)
  auto load_master = [&](int s, int m0, int n0, int n) {
    mbar_expect_tx(full_w(s), Cfg::kMaster + Cfg::kVel);
    const int nm = (FUSE && a.shared_w) ? 0 : n;
#pragma unroll
    for (int q = 0; q < NB32; ++q) tma_load_w(master_u32(s) + q * 16384u, &mapMaster, full_w(s), a.wt, n0 + 32 * q, m0, nm);
    if (MOM) {
#pragma unroll
      for (int q = 0; q < NB32; ++q) tma_load_w(vel_u32(s) + q * 16384u, &mapVel, full_w(s), a.wt, n0 + 32 * q, m0, n);
    }
  };
  // The master (and momentum) tiles were last written an iteration ago, so those of the first items
  // are requested while the previous launch (which only reads the bf16 shadow) drains; `prefetch` is
  // set by the host when no worker mask is in use, so item k of this CTA is known without reading memory.
  uint32_t pre = 0;
  if (warp == 0 && lane == 0 && a.prefetch != 0 && !dyn) {
    for (int k = 0; k < S; ++k) {
      const int w = FUSE ? (int)blockIdx.x : (int)blockIdx.x + k * (int)gridDim.x;
      const int n = FUSE ? k : w / tiles;
      if (w >= items_all || n >= a.N) break;
      const int tile = FUSE ? w : w % tiles;
      if (kShareOnce && a.shared_w && n > 0) mbar_arrive(full_w(k));     // the common master tile is read once per tile
      else load_master(k, (tile / a.tiles_n) * 128, (tile % a.tiles_n) * TN, n);
      ++pre;
    }
  }
  if (!late) {
    pdl_wait();          // set-up above overlapped the previous kernel's tail; dependent memory is touched below
    pdl_trigger();       // only now: the next launch's early loads may overlap this launch, never an older one
  }
  const uint32_t tmem = *tmem_slot;
  const int total_items = *abort_flag != 0 ? 0 : items_all;

  // Every role walks the same sequence of (tile, worker) items; `it` counts the items it has handled,
  // item `it` lives in stage it % S and TMEM columns (it % S) * TN.
  auto item_active = [&](int n) { return FUSE || a.active == nullptr || a.active[n] != 0; };
  // Item k of this CTA's sequence (-1: the sequence has ended): dealt out by block index, or, in the overlapped
  // form, whatever the loader claimed k-th (every role but the loader reads it from the ring).
  auto item_of = [&](uint32_t k, bool& ok) -> int {
    if (!dyn) {
      const int64_t w = (int64_t)blockIdx.x + (int64_t)k * (int64_t)gridDim.x;
      return w < (int64_t)total_items ? (int)w : -1;
    }
    ok = mbar_wait(sched_full(k % R), (k / R) & 1u, abort_flag, a.status, 0x20B);
    return ok ? sched[k % R] : -1;
  };

  if (warp == 0 && lane == 0) {
    // ---------------- loader
    uint32_t it = 0;
    bool ok = true;
    for (uint32_t k = 0; ok; ++k) {
      int w;
      if (dyn) {
        // the stage first, the claim last: a CTA that waits for room in its ring leaves the items to the others
        ok = mbar_wait(stage_empty(k % S), ((k / S) & 1u) ^ 1u, abort_flag, a.status, 0x201);
        if (!ok) break;
        w = total_items > 0 ? (int)atomicAdd(a.next_item, 1u) : -1;
        if (w >= total_items) w = -1;
        sched[k % R] = w;
        mbar_arrive(sched_full(k % R));
      } else {
        w = item_of(k, ok);
      }
      if (w < 0) break;
      const int tile = FUSE ? w : w % tiles;
      const int n_begin = FUSE ? 0 : w / tiles, n_end = FUSE ? a.N : n_begin + 1;
      const int m0 = (tile / a.tiles_n) * 128, n0 = (tile % a.tiles_n) * TN;
      for (int n = n_begin; n < n_end; ++n) {
        if (!item_active(n)) continue;
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        if (it >= pre && !dyn) {                          // (the early items already have their master tiles under way)
          ok = mbar_wait(stage_empty(s), ph ^ 1u, abort_flag, a.status, 0x201);
          if (!ok) break;
        }
        const int row0 = a.pool ? (int)draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks) * a.B : 0;
        const uint32_t ops = ops_u32(s);
        mbar_expect_tx(full_ops(s), (2u + NB64) * op_box);
        tma_load_3d(ops, &mapDelta, full_ops(s), m0, 0, n);
        tma_load_3d(ops + op_box, &mapDelta, full_ops(s), m0 + 64, 0, n);
#pragma unroll
        for (int h = 0; h < NB64; ++h) tma_load_3d(ops + (2u + h) * op_box, &mapAct, full_ops(s), n0 + 64 * h, row0, n);
        if (it >= pre) {
          if (kShareOnce && a.shared_w && n > n_begin) mbar_arrive(full_w(s));   // (its first worker has brought it)
          else load_master(s, m0, n0, n);
        }
        ++it;
      }
    }
    if (it < pre) it = pre;        // early tiles that nothing will consume (the launch turned into a no-op)
    if (*abort_flag && it > 0) {   // let the copies already in flight land before the CTA goes away
      const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
      for (uint32_t q = first; q < it; ++q) {
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(full_w(q % S), (q / S) & 1u) && globaltimer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = idesc_bf16(128, TN, 1, 1);
    const int ksteps = a.B / 16;
    uint32_t it = 0;
    bool ok = true;
    for (uint32_t k = 0; ok; ++k) {
      const int w = item_of(k, ok);
      if (w < 0) break;
      const int n_begin = FUSE ? 0 : w / tiles, n_end = FUSE ? a.N : n_begin + 1;
      for (int n = n_begin; n < n_end; ++n) {
        if (!item_active(n)) continue;
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(acc_empty(s), ph ^ 1u, abort_flag, a.status, 0x202) &&
             mbar_wait(full_ops(s), ph, abort_flag, a.status, 0x203);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = ops_u32(s), sb = sa + 2u * op_box;
        for (int k = 0; k < ksteps; ++k)
          mma_bf16(tmem + (uint32_t)(s * TN), smem_desc_sw128(sa + k * 2048u, op_box, 1024u),
                   smem_desc_sw128(sb + k * 2048u, op_box, 1024u), idesc, k != 0 ? 1u : 0u);
        mma_commit(acc_full(s));
        ++it;
      }
    }
  } else if (warp == 2 && lane == 0) {
    // ---------------- storer: TMA stores of finished tiles, then hands the stage back to the loader
    uint32_t it = 0, tile_it = 0;
    bool ok = true;
    auto store_tile = [&](int s, int m0, int n0, int n) {
#pragma unroll
      for (int q = 0; q < NB32; ++q) tma_store_w(&mapMaster, master_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
      if (MOM) {
#pragma unroll
        for (int q = 0; q < NB32; ++q) tma_store_w(&mapVel, vel_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
      }
#pragma unroll
      for (int h = 0; h < NB64; ++h) tma_store_w(&mapShadow, ops_u32(s) + h * 16384u, a.wt, n0 + 64 * h, m0, n);
    };
    for (uint32_t k = 0; ok; ++k) {
      const int w = item_of(k, ok);
      if (w < 0) break;
      const int tile = FUSE ? w : w % tiles;
      const int m0 = (tile / a.tiles_n) * 128, n0 = (tile % a.tiles_n) * TN;
      if (!FUSE) {
        const int n = w / tiles;
        if (!item_active(n)) continue;
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(tile_ready(s), ph, abort_flag, a.status, 0x204);
        if (!ok) break;
        store_tile(s, m0, n0, n);
        tma_commit_group();
        tma_wait_group_read0();
        mbar_arrive(stage_empty(s));
        ++it;
      } else if (kOutBuf) {
        ok = mbar_wait(tile_ready(0), tile_it & 1u, abort_flag, a.status, 0x209);
        if (!ok) break;
        // one row at a time: a burst of all N rows would sit in the copy engine's queue ahead of the next
        // tile's operand loads for as long as the memory system takes to absorb it
        for (int n = 0; n < a.N; ++n) {
#pragma unroll
          for (int q = 0; q < NB32; ++q) tma_store_w(&mapMaster, out_u32 + q * 16384u, a.wt, n0 + 32 * q, m0, n);
#pragma unroll
          for (int h = 0; h < NB64; ++h) tma_store_w(&mapShadow, out_u32 + Cfg::kMaster + h * 16384u, a.wt, n0 + 64 * h, m0, n);
          tma_commit_group();
          tma_wait_group_read0();
        }
        mbar_arrive(out_free);
        ++tile_it;
      } else if (MOM && a.avg_vel == 0) {
        // every worker's new momentum tile goes back to its own row; the last worker's stage also holds the
        // averaged models, which go to every row
        for (int n = 0; n < a.N && ok; ++n, ++it) {
          const int s = it % S;
          const uint32_t ph = (it / S) & 1u;
          ok = mbar_wait(tile_ready(s), ph, abort_flag, a.status, 0x208);
          if (!ok) break;
          if (n == a.N - 1) {
            for (int rr = 0; rr < a.N; ++rr) {
#pragma unroll
              for (int q = 0; q < NB32; ++q) tma_store_w(&mapMaster, master_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, rr);
#pragma unroll
              for (int h = 0; h < NB64; ++h) tma_store_w(&mapShadow, ops_u32(s) + h * 16384u, a.wt, n0 + 64 * h, m0, rr);
            }
          }
#pragma unroll
          for (int q = 0; q < NB32; ++q) tma_store_w(&mapVel, vel_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
          tma_commit_group();
          tma_wait_group_read0();
          mbar_arrive(stage_empty(s));
        }
      } else {
        it += (uint32_t)a.N;
        const int s = (it - 1) % S;                       // stage of the tile's last worker
        ok = mbar_wait(tile_ready(0), tile_it & 1u, abort_flag, a.status, 0x205);
        if (!ok) break;
        for (int n = 0; n < a.N; ++n) {                   // one row at a time (see the buffered form above)
          store_tile(s, m0, n0, n);
          tma_commit_group();
          tma_wait_group_read0();
        }
        mbar_arrive(stage_empty(s));
        ++tile_it;
      }
    }
    tma_wait_group0();
  } else if (warp >= 3) {
    // ---------------- epilogue: row r of the tile <-> TMEM lane r
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const uint32_t row_off = (uint32_t)r * 128u;
    const uint32_t sw = (uint32_t)(r & 7);
    const int etid = tid - 96;                            // 0..127 among the epilogue threads
    const float fN = (float)a.N;
    const float fD = a.divisor;
    constexpr int NSUM = FUSE ? TN : 1;
    constexpr int NVSUM = (FUSE && MOM) ? TN : 1;
    constexpr int NXR = kShareOnce ? TN : 1;
    const bool shared_x = kShareOnce && a.shared_w != 0;
    const bool avg_vel = FUSE && MOM && a.avg_vel != 0;
    const bool vel_per_worker = FUSE && MOM && a.avg_vel == 0;      // the storer takes every worker's momentum tile
    uint32_t it = 0, tile_it = 0;
    bool ok = true;
    for (uint32_t k = 0; ok; ++k, ++tile_it) {
      const int w = item_of(k, ok);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok || w < 0) break;
      const int n_begin = FUSE ? 0 : w / tiles, n_end = FUSE ? a.N : n_begin + 1;
      float sum[NSUM], vsum[NVSUM];
      float xr[NXR];                                        // shared weights: the tile every worker starts from
#pragma unroll
      for (int i = 0; i < NSUM; ++i) sum[i] = 0.f;
#pragma unroll
      for (int i = 0; i < NVSUM; ++i) vsum[i] = 0.f;
      for (int n = n_begin; n < n_end; ++n) {
        if (!item_active(n)) continue;
        const bool upd = a.active == nullptr || a.active[n] != 0;
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(full_w(s), ph, abort_flag, a.status, 0x206) &&
             mbar_wait(acc_full(s), ph, abort_flag, a.status, 0x207);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint8_t* mst = gen + (size_t)s * stage_bytes;
        uint8_t* stg = mst + Cfg::kMaster + Cfg::kVel;
        const bool last = FUSE && n == a.N - 1;
        uint8_t* dst_w = mst;                               // where the tile to be stored is written
        if (kOutBuf && last) {
          dst_w = gen + (size_t)S * stage_bytes;
          stg = dst_w + Cfg::kMaster;
          if (tile_it > 0) {                                // the previous tile's row stores have read the buffer
            ok = __all_sync(0xffffffffu, mbar_wait(out_free, (tile_it - 1) & 1u, abort_flag, a.status, 0x20A));
            if (!ok) break;
          }
        }
#pragma unroll
        for (int c = 0; c < NB32; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_off + (uint32_t)(s * TN + c * 32), v);
          tmem_ld_wait();
          uint2 lo = make_uint2(0u, 0u);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float4* pw = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)j ^ sw) << 4));
            float4 x;
            if (kShareOnce && shared_x) {                   // worker 0's load brought the common tile: keep it in registers
              constexpr int F = kShareOnce ? 1 : 0;
              float* xp = &xr[F * (c * 32 + 4 * j)];
              if (n == 0) { x = *pw; xp[0] = x.x; xp[F * 1] = x.y; xp[F * 2] = x.z; xp[F * 3] = x.w; }
              else x = make_float4(xp[0], xp[F * 1], xp[F * 2], xp[F * 3]);
            } else {
              x = *pw;
            }
            float4 g4 = make_float4(__uint_as_float(v[4 * j + 0]), __uint_as_float(v[4 * j + 1]),
                                    __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
            if (MOM) {                                      // v <- mu v + G, kept in place next to the master tile
              float4* pv = reinterpret_cast<float4*>(mst + Cfg::kMaster + c * 16384 + row_off + (((uint32_t)j ^ sw) << 4));
              const float4 vo = *pv;
              if (!FUSE || upd) {
                g4.x = fmaf(a.mu, vo.x, g4.x); g4.y = fmaf(a.mu, vo.y, g4.y);
                g4.z = fmaf(a.mu, vo.z, g4.z); g4.w = fmaf(a.mu, vo.w, g4.w);
              } else {
                g4 = vo;                                    // an inactive worker keeps its momentum (and its point)
              }
              float4 vst = g4;
              if (FUSE && MOM && avg_vel) {                 // running sums of the momentum tiles, worker order
                constexpr int F = (FUSE && MOM) ? 1 : 0;
                float* vp = &vsum[F * (c * 32 + 4 * j)];
                vp[0] += g4.x; vp[F * 1] += g4.y; vp[F * 2] += g4.z; vp[F * 3] += g4.w;
                if (last) {
                  vst.x = __fdiv_rn(vp[0], fN); vst.y = __fdiv_rn(vp[F * 1], fN);
                  vst.z = __fdiv_rn(vp[F * 2], fN); vst.w = __fdiv_rn(vp[F * 3], fN);
                }
              }
              if (!avg_vel || last) *pv = vst;
            }
            if (upd) {
              x.x = fmaf(-a.gamma, g4.x, x.x);
              x.y = fmaf(-a.gamma, g4.y, x.y);
              x.z = fmaf(-a.gamma, g4.z, x.z);
              x.w = fmaf(-a.gamma, g4.w, x.w);
            }
            if (FUSE) {
              constexpr int F = FUSE ? 1 : 0;
              float* sp = &sum[F * (c * 32 + 4 * j)];
              sp[0] += x.x; sp[F * 1] += x.y; sp[F * 2] += x.z; sp[F * 3] += x.w;
              if (last) {
                x.x = __fdiv_rn(sp[0], fD); x.y = __fdiv_rn(sp[F * 1], fD);
                x.z = __fdiv_rn(sp[F * 2], fD); x.w = __fdiv_rn(sp[F * 3], fD);
              }
            }
            if (!FUSE || last) {
              *reinterpret_cast<float4*>(dst_w + c * 16384 + row_off + (((uint32_t)j ^ sw) << 4)) = x;
              // two neighbouring fp32 chunks make one 16-byte bf16 chunk: a single conflict-free store
              if ((j & 1) == 0) {
                lo = make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
              } else {
                const uint32_t chunk = (uint32_t)((c & 1) * 4 + (j >> 1));
                *reinterpret_cast<uint4*>(stg + (c >> 1) * 16384 + row_off + ((chunk ^ sw) << 4)) =
                    make_uint4(lo.x, lo.y, pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
              }
            }
          }
        }
        tc_fence_before();
        mbar_arrive(acc_empty(s));
        if (!FUSE || vel_per_worker) {
          fence_proxy_async();
          mbar_arrive(tile_ready(s));
        } else if (last && !kOutBuf) {
          fence_proxy_async();
          mbar_arrive(tile_ready(0));
        } else {
          if (kOutBuf && last) {                            // the averaged tile sits in its own buffer: hand it over
            fence_proxy_async();
            mbar_arrive(tile_ready(0));
          }
          named_bar_sync(1, 128);                         // every epilogue thread is done reading stage s
          if (etid == 0) mbar_arrive(stage_empty(s));
        }
        ++it;
      }
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256u);
  if (late) {            // the overlapped forms: only now the launch before this one has to have completed
    pdl_wait();
    pdl_trigger();
  }
}

// v <- mu v + G on two neighbouring 16-byte chunks (j, j + 1) of a 128-byte-swizzled fp32 row of the momentum
// tile, in place; G is replaced by the new v, which the caller then applies as the step direction.
__device__ __forceinline__ void momentum_pair(uint8_t* vrow, uint32_t j, uint32_t sw, float mu, float4& gx, float4& gy) {
  float4* q0 = reinterpret_cast<float4*>(vrow + ((j ^ sw) << 4));
  float4* q1 = reinterpret_cast<float4*>(vrow + (((j + 1u) ^ sw) << 4));
  const float4 v0 = *q0, v1 = *q1;
  gx.x = fmaf(mu, v0.x, gx.x); gx.y = fmaf(mu, v0.y, gx.y); gx.z = fmaf(mu, v0.z, gx.z); gx.w = fmaf(mu, v0.w, gx.w);
  gy.x = fmaf(mu, v1.x, gy.x); gy.y = fmaf(mu, v1.y, gy.y); gy.z = fmaf(mu, v1.z, gy.z); gy.w = fmaf(mu, v1.w, gy.w);
  *q0 = gx; *q1 = gy;
}

// ---------------------------------------------------------------------------------------------
// update of layer 1 with the next iteration's first forward GEMM folded in
// ---------------------------------------------------------------------------------------------
// The first layer's input is the data pool, so once a tile of W_1 has taken its step the product of
// that tile with the NEXT minibatch can be formed straight from the bf16 tile the epilogue has just
// written to shared memory.  A CTA therefore owns whole row blocks (128 output features of one
// worker), walks their column tiles left to right, accumulates z_1 = W_1 x' over them in a second
// TMEM accumulator and finishes the row block with the forward epilogue (bias, ReLU, bf16 a_1).
// The forward launch of layer 1 in the next iteration is then skipped, and W_1's bf16 shadow, which
// only that launch reads, is not written (the host uses the ordinary update on the last iteration of
// a call, so the shadow is valid whenever control returns to the caller).
// The (block, first tile, end tile) segments one CTA of a block-walking kernel handles.  A block is a row block
// of tc_update_next_kernel (its tiles = the column tiles the forward product accumulates over).  Plain form: whole
// blocks, blockIdx.x, + gridDim.x, ...  Split form: the tiles of all blocks, in block-major order, are cut into
// runs of `chunk` tiles, one run per CTA, so every CTA streams the same number of tiles however the block count
// divides by the CTA count; a block cut by a run boundary is finished by whichever of its CTAs comes last
// (see SplitArgs).
struct BlockWalk {
  int tn, split, nblocks, stride;
  int64_t t, t1;
  int rb, k0, k1;
  __device__ BlockWalk(int tiles_per_block, int blocks, int split_, int chunk)
      : tn(tiles_per_block), split(split_), nblocks(blocks), stride((int)gridDim.x), rb((int)blockIdx.x - (int)gridDim.x), k0(0), k1(0) {
    t = (int64_t)blockIdx.x * chunk;
    t1 = t + chunk;
    const int64_t all = (int64_t)blocks * tiles_per_block;
    if (t1 > all) t1 = all;
  }
  __device__ bool next() {
    if (split) {
      if (t >= t1) return false;
      rb = (int)(t / tn);
      k0 = (int)(t - (int64_t)rb * tn);
      k1 = (int64_t)k0 + (t1 - t) < (int64_t)tn ? k0 + (int)(t1 - t) : tn;
      t += k1 - k0;
      return true;
    }
    rb += stride; k0 = 0; k1 = tn;
    return rb < nblocks;
  }
  __device__ bool whole() const { return k0 == 0 && k1 == tn; }
};

// Split form: a CTA that holds only part of a block's accumulator writes it, as fp32, to a slot of its own in
// global memory (slot 2 c for the first segment of CTA c, 2 c + 1 for a later one: a run has at most one cut
// block at each end), raises the block's counter, and the CTA that finds the counter complete adds the parts in
// run order, applies the block epilogue and zeroes the counter again.  Nobody waits for anybody, and the order of
// the additions is fixed, so the result does not depend on which CTA comes last.
struct SplitArgs {
  int on;                    // 0: whole blocks per CTA
  int chunk;                 // tiles per CTA
  float* part;               // [2 * CTAs][B][128] fp32
  unsigned int* count;       // [blocks], zero between launches
};

struct UpdateNextArgs {
  int B, N;
  int tiles_m, tiles_n;
  float gamma;
  DrawArgs draw;             // iteration t; the next minibatch is the draw of t + 1
  DeviceStatus* status;
  int stages;
  uint16_t* next_out;        // bf16 a_1 [N][B][next_ld]
  int next_ld;
  const float* bias;         // params + b_off of layer 1 (already stepped by this iteration's dX epilogue)
  int64_t bias_stride;
  int M_total;               // d_1
  float mu;                  // momentum form: v <- mu v + G, x <- x - gamma v
  const uint8_t* active;     // per-worker flag or nullptr: an inactive worker's row blocks are skipped
  SplitArgs split;           // row blocks cut at run boundaries (never together with a worker mask)
  WTile wt;                  // order of the weight segment's elements
};

template <int TN, bool MOM> struct UpdNextCfg {
  static constexpr uint32_t kMaster = 128u * TN * 4u;
  static constexpr uint32_t kVel = MOM ? kMaster : 0u;          // momentum tile right after the master tile
  static constexpr uint32_t kOut = 128u * TN * 2u;
  // per stage: the minibatch boxes of the tile's columns (later the bf16 output tile), then the next minibatch's
  __host__ __device__ static uint32_t ops_bytes(int B) { return (uint32_t)(TN / 64) * (uint32_t)B * 128u; }
  __host__ __device__ static uint32_t region(int B) { return ops_bytes(B) > kOut ? ops_bytes(B) : kOut; }
  __host__ __device__ static uint32_t next_bytes(int B) { return (uint32_t)(TN / 64) * (uint32_t)B * 128u; }
  __host__ __device__ static uint32_t stage(int B) { return kMaster + kVel + region(B) + next_bytes(B); }
  // behind the stages: the two dZ boxes of a row block, which every column tile of the block uses, loaded once
  // per block (two buffers, so that the next block's boxes arrive while this block's last tiles are multiplied)
  __host__ __device__ static uint32_t dz_bytes(int B) { return 4u * (uint32_t)B * 128u; }
  static int stages(int B) {
    int s = (int)((227u * 1024u - 2048u - dz_bytes(B)) / stage(B));
    return s > 4 ? 4 : s;
  }
  static size_t smem(int B) { return (size_t)stages(B) * stage(B) + dz_bytes(B) + 1024 + 512; }
};

template <int TN, bool MOM>
__global__ void __launch_bounds__(kUpdBlkThreads, 1) tc_update_next_kernel(const __grid_constant__ CUtensorMap mapDelta,
                                                                        const __grid_constant__ CUtensorMap mapPool,
                                                                        const __grid_constant__ CUtensorMap mapMaster,
                                                                        const __grid_constant__ CUtensorMap mapVel,
                                                                        const UpdateNextArgs a) {
  using namespace ptx;
  using Cfg = UpdNextCfg<TN, MOM>;
  constexpr int NB32 = TN / 32, NB64 = TN / 64;
  constexpr uint32_t kFwdCol = 256u;                    // TMEM: dW accumulators in columns [0, 256), forward ones behind
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int S = a.stages;
  const uint32_t stage_bytes = Cfg::stage(a.B);
  const uint32_t op_box = (uint32_t)a.B * 128u;         // one {64, B} box
  auto master_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes; };
  auto vel_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster; };
  auto ops_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster + Cfg::kVel; };
  auto next_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster + Cfg::kVel + Cfg::region(a.B); };
  auto dz_u32 = [&](int q) { return base + (uint32_t)S * stage_bytes + (uint32_t)q * 2u * op_box; };
  const uint32_t bar0 = base + (uint32_t)S * stage_bytes + Cfg::dz_bytes(a.B);
  auto full_ops = [&](int s) { return bar0 + 8u * s; };
  auto full_w = [&](int s) { return bar0 + 32u + 8u * s; };
  auto stage_empty = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int s) { return bar0 + 96u + 8u * s; };
  auto acc_empty = [&](int s) { return bar0 + 128u + 8u * s; };
  auto tile_ready = [&](int s) { return bar0 + 160u + 8u * s; };
  auto fwd_done = [&](int s) { return bar0 + 192u + 8u * s; };      // forward MMAs have read the stage's bf16 tile
  auto facc_full = [&](int q) { return bar0 + 224u + 8u * q; };
  auto facc_empty = [&](int q) { return bar0 + 240u + 8u * q; };
  auto dz_full = [&](int q) { return bar0 + 272u + 8u * q; };       // the row block's dZ boxes have arrived
  auto dz_empty = [&](int q) { return bar0 + 288u + 8u * q; };      // every dW product of the block has read them
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + (bar0 - base) + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (bar0 - base) + 260);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row_blocks = a.tiles_m * a.N;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_ops(s), 1); mbar_init(full_w(s), 1); mbar_init(stage_empty(s), 1);
      mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 128); mbar_init(tile_ready(s), 128);
      mbar_init(fwd_done(s), 1);
    }
    for (int q = 0; q < 2; ++q) {
      mbar_init(facc_full(q), 1); mbar_init(facc_empty(q), 128);
      mbar_init(dz_full(q), 1); mbar_init(dz_empty(q), 1);
    }
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    prefetch_tensormap(&mapDelta); prefetch_tensormap(&mapPool);
    prefetch_tensormap(&mapMaster);
    if (MOM) prefetch_tensormap(&mapVel);
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 512u); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  pdl_trigger();
  const uint32_t tmem = *tmem_slot;
  const int total_rb = *abort_flag != 0 ? 0 : row_blocks;
  auto item_active = [&](int n) { return a.active == nullptr || a.active[n] != 0; };

  // Every role walks the same sequence of tiles: row blocks rb = blockIdx.x, + gridDim.x, ..., and inside a
  // row block the column tiles kb = 0 .. tiles_n - 1; `it` counts tiles, tile `it` lives in stage it % S.
  if (warp == 0 && lane == 0) {
    // ---------------- loader
    uint32_t it = 0, rbi = 0;
    bool ok = true;
    BlockWalk wk(a.tiles_n, total_rb, a.split.on, a.split.chunk);
    while (ok && wk.next()) {
      const int rb = wk.rb;
      const int n = rb / a.tiles_m, m0 = (rb % a.tiles_m) * 128;
      if (!item_active(n)) continue;
      const int64_t t = draw_t(a.draw);
      const int row0 = (int)draw_block(a.draw.seed, a.draw.worker0 + n, t, a.draw.n_blocks) * a.B;
      const int row1 = (int)draw_block(a.draw.seed, a.draw.worker0 + n, t + 1, a.draw.n_blocks) * a.B;
      {   // the block's two dZ boxes, once for all its column tiles
        const int q = rbi & 1;
        ok = mbar_wait(dz_empty(q), ((rbi >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x40B);
        if (!ok) break;
        mbar_expect_tx(dz_full(q), 2u * op_box);
        tma_load_3d(dz_u32(q), &mapDelta, dz_full(q), m0, 0, n);
        tma_load_3d(dz_u32(q) + op_box, &mapDelta, dz_full(q), m0 + 64, 0, n);
        ++rbi;
      }
      for (int kb = wk.k0; kb < wk.k1; ++kb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(stage_empty(s), ph ^ 1u, abort_flag, a.status, 0x401);
        if (!ok) break;
        const int n0 = kb * TN;
        const uint32_t ops = ops_u32(s), nx = next_u32(s);
        mbar_expect_tx(full_ops(s), 2u * NB64 * op_box);
#pragma unroll
        for (int h = 0; h < NB64; ++h) {
          tma_load_3d(ops + h * op_box, &mapPool, full_ops(s), n0 + 64 * h, row0, n);
          tma_load_3d(nx + h * op_box, &mapPool, full_ops(s), n0 + 64 * h, row1, n);
        }
        mbar_expect_tx(full_w(s), Cfg::kMaster + Cfg::kVel);
#pragma unroll
        for (int q = 0; q < NB32; ++q) tma_load_w(master_u32(s) + q * 16384u, &mapMaster, full_w(s), a.wt, n0 + 32 * q, m0, n);
        if (MOM) {
#pragma unroll
          for (int q = 0; q < NB32; ++q) tma_load_w(vel_u32(s) + q * 16384u, &mapVel, full_w(s), a.wt, n0 + 32 * q, m0, n);
        }
      }
    }
    if (*abort_flag && it > 0) {   // let the copies already in flight land before the CTA goes away
      const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
      for (uint32_t q = first; q < it; ++q) {
        const uint64_t t0 = globaltimer_ns();
        while (!(mbar_try_wait(full_w(q % S), (q / S) & 1u) && mbar_try_wait(full_ops(q % S), (q / S) & 1u)) &&
               globaltimer_ns() - t0 < 100000000ull) {}
      }
    }
    if (*abort_flag && rbi > 0) {
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(dz_full((rbi - 1) & 1), ((rbi - 1) >> 1) & 1u) && globaltimer_ns() - t0 < 100000000ull) {}
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer: dW of tile `it`, then the forward product of tile it - 1 (whose
    // stepped bf16 tile the epilogue has finished meanwhile)
    const uint32_t idesc_dw = idesc_bf16(128, TN, 1, 1);
    const uint32_t idesc_fw = idesc_bf16(128, a.B, 0, 0);
    const int ksteps = a.B / 16;
    uint32_t it = 0, rbi = 0;
    bool ok = true;
    bool have_prev = false;
    uint32_t p_it = 0, p_rbi = 0;
    bool p_first = false, p_last = false;
    // forward product of tile j; `first` / `last`: the tile opens / closes its segment of the row block
    auto forward_of = [&](uint32_t j, bool first, bool last, uint32_t rj) -> bool {
      const int s = j % S, q = rj & 1;
      if (first && !mbar_wait(facc_empty(q), ((rj >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x402)) return false;
      if (!mbar_wait(tile_ready(s), (j / S) & 1u, abort_flag, a.status, 0x403)) return false;
      tc_fence_after();
      const uint32_t acc = tmem + kFwdCol + (uint32_t)(q * a.B);
#pragma unroll
      for (int h = 0; h < NB64; ++h) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_bf16(acc, smem_desc_sw128(ops_u32(s) + h * 16384u + k * 32u, 16u, 1024u),
                   smem_desc_sw128(next_u32(s) + h * op_box + k * 32u, 16u, 1024u), idesc_fw, (!first || (h | k) != 0) ? 1u : 0u);
      }
      mma_commit(fwd_done(s));
      if (last) mma_commit(facc_full(q));
      return true;
    };
    BlockWalk wk(a.tiles_n, total_rb, a.split.on, a.split.chunk);
    while (ok && wk.next()) {
      if (!item_active(wk.rb / a.tiles_m)) continue;
      for (int kb = wk.k0; kb < wk.k1 && ok; ++kb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        const int dq = rbi & 1;
        if (kb == wk.k0) {
          ok = mbar_wait(dz_full(dq), (rbi >> 1) & 1u, abort_flag, a.status, 0x40C);
          if (!ok) break;
        }
        ok = mbar_wait(acc_empty(s), ph ^ 1u, abort_flag, a.status, 0x404) &&
             mbar_wait(full_ops(s), ph, abort_flag, a.status, 0x405);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = dz_u32(dq), sb = ops_u32(s);
        for (int k = 0; k < ksteps; ++k)
          mma_bf16(tmem + (uint32_t)(s * TN), smem_desc_sw128(sa + k * 2048u, op_box, 1024u),
                   smem_desc_sw128(sb + k * 2048u, op_box, 1024u), idesc_dw, k != 0 ? 1u : 0u);
        mma_commit(acc_full(s));
        if (kb == wk.k1 - 1) mma_commit(dz_empty(dq));          // the block's dZ boxes are free once these products are done
        if (have_prev) ok = forward_of(p_it, p_first, p_last, p_rbi);
        p_it = it; p_first = kb == wk.k0; p_last = kb == wk.k1 - 1; p_rbi = rbi; have_prev = true;
      }
      ++rbi;                                              // counts the segments actually walked
    }
    if (ok && have_prev) forward_of(p_it, p_first, p_last, p_rbi);
  } else if (warp == 2 && lane == 0) {
    // ---------------- storer: TMA stores of finished tiles; the stage goes back to the loader once the
    // forward MMAs have consumed its bf16 tile too
    uint32_t it = 0;
    bool ok = true;
    BlockWalk wk(a.tiles_n, total_rb, a.split.on, a.split.chunk);
    while (ok && wk.next()) {
      const int rb = wk.rb;
      const int n = rb / a.tiles_m, m0 = (rb % a.tiles_m) * 128;
      if (!item_active(n)) continue;
      for (int kb = wk.k0; kb < wk.k1; ++kb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        const int n0 = kb * TN;
        ok = mbar_wait(tile_ready(s), ph, abort_flag, a.status, 0x406);
        if (!ok) break;
#pragma unroll
        for (int q = 0; q < NB32; ++q) tma_store_w(&mapMaster, master_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
        if (MOM) {
#pragma unroll
          for (int q = 0; q < NB32; ++q) tma_store_w(&mapVel, vel_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
        }
        tma_commit_group();
        tma_wait_group_read0();
        ok = mbar_wait(fwd_done(s), ph, abort_flag, a.status, 0x407);
        if (!ok) break;
        mbar_arrive(stage_empty(s));
      }
    }
    tma_wait_group0();
  } else if (warp >= 3 && warp < 7) {
    // ---------------- tile epilogue: row r of the tile <-> TMEM lane r
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const uint32_t row_off = (uint32_t)r * 128u;
    const uint32_t sw = (uint32_t)(r & 7);
    uint32_t it = 0;
    bool ok = true;
    BlockWalk wk(a.tiles_n, total_rb, a.split.on, a.split.chunk);
    while (ok && wk.next()) {
      if (!item_active(wk.rb / a.tiles_m)) continue;
      for (int kb = wk.k0; kb < wk.k1; ++kb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(full_w(s), ph, abort_flag, a.status, 0x408) &&
             mbar_wait(acc_full(s), ph, abort_flag, a.status, 0x409);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint8_t* mst = gen + (size_t)s * stage_bytes;
        uint8_t* stg = mst + Cfg::kMaster + Cfg::kVel;
#pragma unroll
        for (int c = 0; c < NB32; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_off + (uint32_t)(s * TN + c * 32), v);
          tmem_ld_wait();
#pragma unroll
          for (int jp = 0; jp < 4; ++jp) {                  // two 16-byte fp32 chunks = one 16-byte bf16 chunk
            float4* p0 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp) ^ sw) << 4));
            float4* p1 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp + 1) ^ sw) << 4));
            float4 x = *p0, y = *p1;
            float4 gx = make_float4(__uint_as_float(v[8 * jp + 0]), __uint_as_float(v[8 * jp + 1]),
                                    __uint_as_float(v[8 * jp + 2]), __uint_as_float(v[8 * jp + 3]));
            float4 gy = make_float4(__uint_as_float(v[8 * jp + 4]), __uint_as_float(v[8 * jp + 5]),
                                    __uint_as_float(v[8 * jp + 6]), __uint_as_float(v[8 * jp + 7]));
            if (MOM) momentum_pair(mst + Cfg::kMaster + c * 16384 + row_off, (uint32_t)(2 * jp), sw, a.mu, gx, gy);
            x.x = fmaf(-a.gamma, gx.x, x.x); x.y = fmaf(-a.gamma, gx.y, x.y);
            x.z = fmaf(-a.gamma, gx.z, x.z); x.w = fmaf(-a.gamma, gx.w, x.w);
            y.x = fmaf(-a.gamma, gy.x, y.x); y.y = fmaf(-a.gamma, gy.y, y.y);
            y.z = fmaf(-a.gamma, gy.z, y.z); y.w = fmaf(-a.gamma, gy.w, y.w);
            *p0 = x; *p1 = y;
            const uint32_t chunk = (uint32_t)((c & 1) * 4 + jp);
            *reinterpret_cast<uint4*>(stg + (c >> 1) * 16384 + row_off + ((chunk ^ sw) << 4)) =
                make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w), pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
          }
        }
        tc_fence_before();
        mbar_arrive(acc_empty(s));
        fence_proxy_async();
        mbar_arrive(tile_ready(s));
      }
    }
  } else if (warp >= 7) {
    // ---------------- block epilogue: forward epilogue of every row block, a_1[., m] = relu(z + b_1[m]) for
    // the next iteration, while the tile epilogue warps are already on the next row block
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const int batches = a.B / 16;
    uint32_t rbi = 0;
    bool ok = true;
    const int etid = tid - 224;                           // 0..127 among these warps
    volatile unsigned int* last_flag = reinterpret_cast<volatile unsigned int*>(gen + (bar0 - base) + 264);
    BlockWalk wk(a.tiles_n, total_rb, a.split.on, a.split.chunk);
    while (ok && wk.next()) {
      const int rb = wk.rb;
      const int n = rb / a.tiles_m, m = (rb % a.tiles_m) * 128 + r;
      if (!item_active(n)) continue;
      const int q = rbi & 1;
      const bool valid = m < a.M_total;
      const float bias = valid ? a.bias[(int64_t)n * a.bias_stride + m] : 0.f;
      ok = __all_sync(0xffffffffu, mbar_wait(facc_full(q), (rbi >> 1) & 1u, abort_flag, a.status, 0x40A));
      if (!ok) break;
      tc_fence_after();
      if (wk.whole()) {
        for (int bi = 0; bi < batches; ++bi) {
          uint32_t v[16];
          tmem_ld16(tmem + lane_off + kFwdCol + (uint32_t)(q * a.B + bi * 16), v);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              a.next_out[((int64_t)n * a.B + bi * 16 + j) * a.next_ld + m] = f32_to_bf16_rn(fmaxf(__uint_as_float(v[j]) + bias, 0.f));
          }
        }
        tc_fence_before();
        mbar_arrive(facc_empty(q));
      } else {
        // part of a row block: this CTA's share of z_1 goes to its slot; whoever completes the block's counter
        // adds the shares in run order and applies bias and ReLU
        float* mine = a.split.part + ((int64_t)(2 * blockIdx.x + (rbi == 0 ? 0 : 1)) * a.B) * 128 + r;
        for (int bi = 0; bi < batches; ++bi) {
          uint32_t v[16];
          tmem_ld16(tmem + lane_off + kFwdCol + (uint32_t)(q * a.B + bi * 16), v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) __stcg(mine + (bi * 16 + j) * 128, __uint_as_float(v[j]));
        }
        tc_fence_before();
        mbar_arrive(facc_empty(q));
        __threadfence();
        named_bar_sync(2, 128);
        const int64_t tb = (int64_t)rb * a.tiles_n;          // first tile of the block in the global order
        const int c_first = (int)(tb / a.split.chunk), c_last = (int)((tb + a.tiles_n - 1) / a.split.chunk);
        if (etid == 0) *last_flag = atomicAdd(a.split.count + rb, 1u) == (unsigned int)(c_last - c_first) ? 1u : 0u;
        named_bar_sync(2, 128);
        if (*last_flag != 0u) {
          __threadfence();
          for (int b0 = 0; b0 < a.B; b0 += 16) {             // sixteen rows at a time: their loads are in flight together
            float z[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) z[j] = 0.f;
            for (int cc = c_first; cc <= c_last; ++cc) {     // CTA cc's segment of this block is its first one unless its run began earlier
              const int slot = 2 * cc + ((int64_t)cc * a.split.chunk < tb ? 1 : 0);
              const float* src = a.split.part + ((int64_t)slot * a.B + b0) * 128 + r;
              float v[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] = __ldcg(src + j * 128);
#pragma unroll
              for (int j = 0; j < 16; ++j) z[j] += v[j];
            }
            if (valid) {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                a.next_out[((int64_t)n * a.B + b0 + j) * a.next_ld + m] = f32_to_bf16_rn(fmaxf(z[j] + bias, 0.f));
            }
          }
          if (etid == 0) a.split.count[rb] = 0u;
        }
        named_bar_sync(2, 128);                             // (the flag is read by all before the next block overwrites it)
      }
      ++rbi;
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512u);
}

// ---------------------------------------------------------------------------------------------
// update of a layer l >= 2 with its input-gradient GEMM folded in
// ---------------------------------------------------------------------------------------------
// dZ_{l-1} = (dZ_l W_l) (.) relu' needs the bf16 value of every weight BEFORE its step, and the update
// kernel has the fp32 master tile of exactly those weights in shared memory.  Its epilogue therefore
// writes two bf16 tiles, the old values and the stepped ones; the old tile (MN-major A operand, the
// layer's input features on the MMA's M axis) and the dZ_l boxes already loaded for dW (K-major B
// operand) feed a second accumulator dZ_{l-1}^T[64, B].  A CTA owns a 64-wide column block of one
// worker, walks its row tiles top to bottom so that the contraction over d_l completes in TMEM, and
// ends the block with the dX epilogue (ReLU mask, bf16 dZ_{l-1}, bias step of layer l-1).  That saves
// the separate dX launch and its second read of the layer's bf16 weights.
// The accumulator has 128 lanes but the block only 64 features: the descriptor's second 64-row
// half points at other shared memory of the stage and lanes 64..127 are never read.
struct UpdateDxArgs {
  int B, N;
  int tiles_m, tiles_n;      // 128-row tiles of d_l, 64-column tiles of d_{l-1}
  float gamma;
  DeviceStatus* status;
  int stages;
  uint16_t* out_bk;          // bf16 dZ_{l-1} [N][B][ld_out]
  const uint16_t* mask_src;  // bf16 a_{l-1}  [N][B][ld_out]
  int ld_out;
  int M_total;               // d_{l-1}
  float* bias_rw;            // params + b_off of layer l-1 (worker stride bias_stride), or nullptr
  int64_t bias_stride;
  float mu;                  // momentum form: v <- mu v + G, x <- x - gamma v
  float* bias_vel;           // momentum segment of b_{l-1}, or nullptr
  const uint8_t* active;     // per-worker flag or nullptr: an inactive worker's column blocks are skipped
  WTile wt;                  // order of the weight segment's elements
};

// Two stage layouts.  Own pair (SP = false): every stage holds fp32 master | momentum | bf16 old | bf16 new (first
// the a_{l-1} box) | two dZ_l boxes.  Shared pair (SP = true): only what has a long latency is staged (master |
// dZ_l boxes | a_{l-1} boxes) and ONE pair of bf16 tiles behind the stages is shared: the epilogue of a tile
// waits until the pair of the tile before it has been read by its TMA store and its dX MMAs.  The shared pair
// makes room for more stages (64-wide: four instead of three at B = 32, three instead of two at B = 64), and it
// is the only way 128-wide tiles fit at all (512-byte rows, which the memory system serves ~7 % faster than
// 256-byte ones; two stages, B <= 32).  The momentum form keeps its own pairs.
template <int TN, bool MOM, bool SP = (TN == 128)> struct UpdDxCfg {
  static_assert(TN == 64 || !MOM, "the momentum form uses 64-wide tiles");
  static_assert(!(SP && MOM), "the momentum form keeps a pair of bf16 tiles per stage");
  static_assert(TN == 64 || SP, "128-wide tiles need the shared pair");
  static constexpr bool kSharedPair = SP;
  static constexpr uint32_t kMaster = 128u * TN * 4u;      // fp32 master tile
  static constexpr uint32_t kVel = MOM ? kMaster : 0u;     // fp32 momentum tile right behind it
  static constexpr uint32_t kOld = 128u * TN * 2u;         // bf16 of the weights before the step
  static constexpr uint32_t kNew = 128u * TN * 2u;         // bf16 of the stepped weights
  __host__ __device__ static uint32_t delta_bytes(int B) { return 2u * (uint32_t)B * 128u; }
  __host__ __device__ static uint32_t act_bytes(int B) { return (uint32_t)(TN / 64) * (uint32_t)B * 128u; }
  __host__ __device__ static uint32_t stage(int B) {
    return kSharedPair ? kMaster + delta_bytes(B) + act_bytes(B) : kMaster + kVel + kOld + kNew + delta_bytes(B);
  }
  __host__ __device__ static uint32_t shared_bytes() { return kSharedPair ? kOld + kNew : 0u; }
  static int stages(int B) {
    int s = (int)((227u * 1024u - 2048u - shared_bytes()) / stage(B));
    if (s < 2) return 0;                       // (a tile's dX product is issued after the next tile's dW: two stages at least)
    return s > 4 ? 4 : s;
  }
  static size_t smem(int B) { return (size_t)stages(B) * stage(B) + shared_bytes() + 1024 + 512; }
};

template <int TN, bool MOM, bool SP = (TN == 128)>
__global__ void __launch_bounds__(kUpdBlkThreads, 1) tc_update_dx_kernel(const __grid_constant__ CUtensorMap mapDelta,
                                                                      const __grid_constant__ CUtensorMap mapAct,
                                                                      const __grid_constant__ CUtensorMap mapMaster,
                                                                      const __grid_constant__ CUtensorMap mapShadow,
                                                                      const __grid_constant__ CUtensorMap mapVel,
                                                                      const UpdateDxArgs a) {
  using namespace ptx;
  using Cfg = UpdDxCfg<TN, MOM, SP>;
  constexpr int NB32 = TN / 32, NB64 = TN / 64;
  constexpr bool kSharedPair = Cfg::kSharedPair;
  constexpr uint32_t kDxCol = 256u;                     // TMEM: dW accumulators in columns [0, 256), dX ones behind
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int S = a.stages;
  const uint32_t stage_bytes = Cfg::stage(a.B);
  const uint32_t op_box = (uint32_t)a.B * 128u;         // one {64, B} box
  auto master_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes; };
  auto vel_u32 = [&](int s) { return base + (uint32_t)s * stage_bytes + Cfg::kMaster; };
  const uint32_t pair0 = base + (uint32_t)S * stage_bytes;            // the shared bf16 pair (TN = 128)
  auto old_u32 = [&](int s) { return kSharedPair ? pair0 : base + (uint32_t)s * stage_bytes + Cfg::kMaster + Cfg::kVel; };
  auto new_u32 = [&](int s) { return old_u32(s) + Cfg::kOld; };
  auto delta_u32 = [&](int s) {
    return base + (uint32_t)s * stage_bytes + (kSharedPair ? Cfg::kMaster : Cfg::kMaster + Cfg::kVel + Cfg::kOld + Cfg::kNew);
  };
  auto act_u32 = [&](int s) { return kSharedPair ? delta_u32(s) + 2u * op_box : new_u32(s); };
  const uint32_t bar0 = pair0 + Cfg::shared_bytes();
  auto full_ops = [&](int s) { return bar0 + 8u * s; };
  auto full_w = [&](int s) { return bar0 + 32u + 8u * s; };
  auto stage_empty = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int s) { return bar0 + 96u + 8u * s; };
  auto acc_empty = [&](int s) { return bar0 + 128u + 8u * s; };
  auto tile_ready = [&](int s) { return bar0 + 160u + 8u * s; };
  auto dx_done = [&](int s) { return bar0 + 192u + 8u * s; };       // the dX MMAs have read the stage's old tile and dZ boxes
  auto dacc_full = [&](int q) { return bar0 + 224u + 8u * q; };
  auto dacc_empty = [&](int q) { return bar0 + 240u + 8u * q; };
  uint8_t* tail = gen + (size_t)S * stage_bytes + Cfg::shared_bytes();
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 260);
  const uint32_t pair_free = bar0 + 264u;      // shared pair: the store of the tile's new half and its dX MMAs are done

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col_blocks = a.tiles_n * a.N;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_ops(s), 1); mbar_init(full_w(s), 1); mbar_init(stage_empty(s), 1);
      mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 128); mbar_init(tile_ready(s), 128);
      mbar_init(dx_done(s), 1);
    }
    for (int q = 0; q < 2; ++q) { mbar_init(dacc_full(q), 1); mbar_init(dacc_empty(q), 128); }
    mbar_init(pair_free, 2);
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    prefetch_tensormap(&mapDelta); prefetch_tensormap(&mapAct);
    prefetch_tensormap(&mapMaster); prefetch_tensormap(&mapShadow);
    if (MOM) prefetch_tensormap(&mapVel);
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 512u); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  pdl_trigger();
  const uint32_t tmem = *tmem_slot;
  const int total_cb = *abort_flag != 0 ? 0 : col_blocks;
  auto item_active = [&](int n) { return a.active == nullptr || a.active[n] != 0; };

  // Every role walks the same sequence of tiles: column blocks cb = blockIdx.x, + gridDim.x, ..., and inside
  // a column block the row tiles mb = 0 .. tiles_m - 1; `it` counts tiles, tile `it` lives in stage it % S.
  if (warp == 0 && lane == 0) {
    // ---------------- loader
    uint32_t it = 0;
    bool ok = true;
    for (int cb = blockIdx.x; cb < total_cb && ok; cb += gridDim.x) {
      const int n = cb / a.tiles_n, n0 = (cb % a.tiles_n) * TN;
      if (!item_active(n)) continue;
      for (int mb = 0; mb < a.tiles_m; ++mb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(stage_empty(s), ph ^ 1u, abort_flag, a.status, 0x501);
        if (!ok) break;
        const int m0 = mb * 128;
        mbar_expect_tx(full_ops(s), (2u + NB64) * op_box);
        tma_load_3d(delta_u32(s), &mapDelta, full_ops(s), m0, 0, n);
        tma_load_3d(delta_u32(s) + op_box, &mapDelta, full_ops(s), m0 + 64, 0, n);
#pragma unroll
        for (int h = 0; h < NB64; ++h) tma_load_3d(act_u32(s) + h * op_box, &mapAct, full_ops(s), n0 + 64 * h, 0, n);
        mbar_expect_tx(full_w(s), Cfg::kMaster + Cfg::kVel);
#pragma unroll
        for (int q = 0; q < NB32; ++q) tma_load_w(master_u32(s) + q * 16384u, &mapMaster, full_w(s), a.wt, n0 + 32 * q, m0, n);
        if (MOM) {
          tma_load_w(vel_u32(s), &mapVel, full_w(s), a.wt, n0, m0, n);
          tma_load_w(vel_u32(s) + 16384u, &mapVel, full_w(s), a.wt, n0 + 32, m0, n);
        }
      }
    }
    if (*abort_flag && it > 0) {   // let the copies already in flight land before the CTA goes away
      const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
      for (uint32_t q = first; q < it; ++q) {
        const uint64_t t0 = globaltimer_ns();
        while (!(mbar_try_wait(full_w(q % S), (q / S) & 1u) && mbar_try_wait(full_ops(q % S), (q / S) & 1u)) &&
               globaltimer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer: dW of tile `it`, then the dX contribution of tile it - 1 (whose bf16
    // tiles the epilogue has finished meanwhile)
    const uint32_t idesc_dw = idesc_bf16(128, TN, 1, 1);
    const uint32_t idesc_dx = idesc_bf16(128, a.B, 1, 0);
    const int ksteps = a.B / 16;
    uint32_t it = 0, cbi = 0;
    bool ok = true;
    bool have_prev = false;
    uint32_t p_it = 0, p_cbi = 0;
    int p_mb = 0;
    auto dx_of = [&](uint32_t j, int mb, uint32_t cj) -> bool {
      const int s = j % S, q = cj & 1;
      if (mb == 0 && !mbar_wait(dacc_empty(q), ((cj >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x502)) return false;
      if (!mbar_wait(tile_ready(s), (j / S) & 1u, abort_flag, a.status, 0x503)) return false;
      tc_fence_after();
      const uint32_t acc = tmem + kDxCol + (uint32_t)(q * a.B);
#pragma unroll
      for (int h = 0; h < 2; ++h) {                       // the tile's two 64-row halves = the two dZ_l boxes
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_bf16(acc, smem_desc_sw128(old_u32(s) + (uint32_t)(h * 4 + k) * 2048u, 16384u, 1024u),
                   smem_desc_sw128(delta_u32(s) + h * op_box + k * 32u, 16u, 1024u), idesc_dx, (mb | h | k) != 0 ? 1u : 0u);
      }
      mma_commit(dx_done(s));
      if (kSharedPair) mma_commit(pair_free);
      if (mb == a.tiles_m - 1) mma_commit(dacc_full(q));
      return true;
    };
    for (int cb = blockIdx.x; cb < total_cb && ok; cb += gridDim.x) {
      if (!item_active(cb / a.tiles_n)) continue;
      for (int mb = 0; mb < a.tiles_m && ok; ++mb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(acc_empty(s), ph ^ 1u, abort_flag, a.status, 0x504) &&
             mbar_wait(full_ops(s), ph, abort_flag, a.status, 0x505);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = delta_u32(s), sb = act_u32(s);
        for (int k = 0; k < ksteps; ++k)
          mma_bf16(tmem + (uint32_t)(s * TN), smem_desc_sw128(sa + k * 2048u, op_box, 1024u),
                   smem_desc_sw128(sb + k * 2048u, op_box, 1024u), idesc_dw, k != 0 ? 1u : 0u);
        mma_commit(acc_full(s));
        if (have_prev) ok = dx_of(p_it, p_mb, p_cbi);
        p_it = it; p_mb = mb; p_cbi = cbi; have_prev = true;
      }
      ++cbi;                                              // counts the column blocks actually walked
    }
    if (ok && have_prev) dx_of(p_it, p_mb, p_cbi);
  } else if (warp == 2 && lane == 0) {
    // ---------------- storer
    uint32_t it = 0;
    bool ok = true;
    for (int cb = blockIdx.x; cb < total_cb && ok; cb += gridDim.x) {
      const int n = cb / a.tiles_n, n0 = (cb % a.tiles_n) * TN;
      if (!item_active(n)) continue;
      for (int mb = 0; mb < a.tiles_m; ++mb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        const int m0 = mb * 128;
        ok = mbar_wait(tile_ready(s), ph, abort_flag, a.status, 0x506);
        if (!ok) break;
#pragma unroll
        for (int h = 0; h < NB64; ++h) tma_store_w(&mapShadow, new_u32(s) + h * 16384u, a.wt, n0 + 64 * h, m0, n);
        if (kSharedPair) tma_commit_group();              // a group of its own: the shared pair is released first
#pragma unroll
        for (int q = 0; q < NB32; ++q) tma_store_w(&mapMaster, master_u32(s) + q * 16384u, a.wt, n0 + 32 * q, m0, n);
        if (MOM) {
          tma_store_w(&mapVel, vel_u32(s), a.wt, n0, m0, n);
          tma_store_w(&mapVel, vel_u32(s) + 16384u, a.wt, n0 + 32, m0, n);
        }
        tma_commit_group();
        if (kSharedPair) {
          tma_wait_group_read1();
          mbar_arrive(pair_free);
        }
        tma_wait_group_read0();
        ok = mbar_wait(dx_done(s), ph, abort_flag, a.status, 0x507);
        if (!ok) break;
        mbar_arrive(stage_empty(s));
      }
    }
    tma_wait_group0();
  } else if (warp >= 3 && warp < 7) {
    // ---------------- tile epilogue: row r of the tile <-> TMEM lane r
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const uint32_t row_off = (uint32_t)r * 128u;
    const uint32_t sw = (uint32_t)(r & 7);
    uint32_t it = 0;
    bool ok = true;
    for (int cb = blockIdx.x; cb < total_cb && ok; cb += gridDim.x) {
      if (!item_active(cb / a.tiles_n)) continue;
      for (int mb = 0; mb < a.tiles_m; ++mb, ++it) {
        const int s = it % S;
        const uint32_t ph = (it / S) & 1u;
        ok = mbar_wait(full_w(s), ph, abort_flag, a.status, 0x508) &&
             mbar_wait(acc_full(s), ph, abort_flag, a.status, 0x509);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (kSharedPair && it > 0) {            // the one bf16 pair is free once the tile before has let go of it
          ok = __all_sync(0xffffffffu, mbar_wait(pair_free, (it - 1) & 1u, abort_flag, a.status, 0x50B));
          if (!ok) break;
        }
        uint8_t* mst = gen + (size_t)s * stage_bytes;
        uint8_t* old = kSharedPair ? gen + (size_t)S * stage_bytes : mst + Cfg::kMaster + Cfg::kVel;
        uint8_t* stg = old + Cfg::kOld;
#pragma unroll
        for (int c = 0; c < NB32; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_off + (uint32_t)(s * TN + c * 32), v);
          tmem_ld_wait();
#pragma unroll
          for (int jp = 0; jp < 4; ++jp) {                  // two 16-byte fp32 chunks = one 16-byte bf16 chunk
            float4* p0 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp) ^ sw) << 4));
            float4* p1 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp + 1) ^ sw) << 4));
            float4 x = *p0, y = *p1;
            const uint32_t boff = (uint32_t)(c >> 1) * 16384u + row_off + (((uint32_t)((c & 1) * 4 + jp) ^ sw) << 4);
            *reinterpret_cast<uint4*>(old + boff) = make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w),
                                                               pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
            float4 gx = make_float4(__uint_as_float(v[8 * jp + 0]), __uint_as_float(v[8 * jp + 1]),
                                    __uint_as_float(v[8 * jp + 2]), __uint_as_float(v[8 * jp + 3]));
            float4 gy = make_float4(__uint_as_float(v[8 * jp + 4]), __uint_as_float(v[8 * jp + 5]),
                                    __uint_as_float(v[8 * jp + 6]), __uint_as_float(v[8 * jp + 7]));
            if (MOM) momentum_pair(mst + Cfg::kMaster + c * 16384 + row_off, (uint32_t)(2 * jp), sw, a.mu, gx, gy);
            x.x = fmaf(-a.gamma, gx.x, x.x); x.y = fmaf(-a.gamma, gx.y, x.y);
            x.z = fmaf(-a.gamma, gx.z, x.z); x.w = fmaf(-a.gamma, gx.w, x.w);
            y.x = fmaf(-a.gamma, gy.x, y.x); y.y = fmaf(-a.gamma, gy.y, y.y);
            y.z = fmaf(-a.gamma, gy.z, y.z); y.w = fmaf(-a.gamma, gy.w, y.w);
            *p0 = x; *p1 = y;
            *reinterpret_cast<uint4*>(stg + boff) = make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w),
                                                               pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
          }
        }
        tc_fence_before();
        mbar_arrive(acc_empty(s));
        fence_proxy_async();
        mbar_arrive(tile_ready(s));
      }
    }
  } else if (warp >= 7) {
    // ---------------- block epilogue: dX epilogue of every column block (ReLU mask, bf16 dZ_{l-1}, bias step of
    // layer l-1), feature c = n0 + r (lanes 0..TN-1 only), while the tile epilogue warps are already on the
    // next column block
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const int batches = a.B / 16;
    uint32_t cbi = 0;
    bool ok = true;
    for (int cb = blockIdx.x; cb < total_cb && ok; cb += gridDim.x) {
      const int n = cb / a.tiles_n, n0 = (cb % a.tiles_n) * TN;
      if (!item_active(n)) continue;
      const int q = cbi & 1;
      const int cfeat = n0 + r;
      const bool valid = r < TN && cfeat < a.M_total;
      // Everything this epilogue reads from global memory (the ReLU-mask values of the whole minibatch, the bias
      // and its momentum) is requested before the accumulator wait: a layer of one row tile per block (the class
      // layer) runs at the pace of this epilogue, and three dependent load latencies per block were most of it.
      uint16_t mk[4][16];                                 // B <= 64: at most four batches of 16
      if (valid) {
#pragma unroll
        for (int bi = 0; bi < 4; ++bi) {
          if (bi < batches) {
#pragma unroll
            for (int j = 0; j < 16; ++j) mk[bi][j] = __ldg(a.mask_src + ((int64_t)n * a.B + bi * 16 + j) * a.ld_out + cfeat);
          }
        }
      }
      const bool step_bias = valid && a.bias_rw != nullptr;
      float* bp = a.bias_rw + (int64_t)n * a.bias_stride + cfeat;
      float* vp = a.bias_vel + (int64_t)n * a.bias_stride + cfeat;
      float b_old = 0.f, v_old = 0.f;
      if (step_bias) {
        b_old = *bp;
        if (a.bias_vel != nullptr) v_old = *vp;
      }
      ok = __all_sync(0xffffffffu, mbar_wait(dacc_full(q), (cbi >> 1) & 1u, abort_flag, a.status, 0x50A));
      if (!ok) break;
      tc_fence_after();
      float gsum = 0.f;
#pragma unroll
      for (int bi = 0; bi < 4; ++bi) {
        if (bi < batches) {
          uint32_t v[16];
          tmem_ld16(tmem + lane_off + kDxCol + (uint32_t)(q * a.B + bi * 16), v);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float d = (mk[bi][j] & 0x7FFFu) != 0 ? __uint_as_float(v[j]) : 0.f;
              gsum += d;
              a.out_bk[((int64_t)n * a.B + bi * 16 + j) * a.ld_out + cfeat] = f32_to_bf16_rn(d);
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(dacc_empty(q));
      if (step_bias) {
        if (a.bias_vel != nullptr) {                      // momentum form of the bias step
          gsum = fmaf(a.mu, v_old, gsum);
          *vp = gsum;
        }
        *bp = fmaf(-a.gamma, gsum, b_old);
      }
      ++cbi;
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512u);
}

// b_l <- b_l - gamma * sum_b dZ_l[b, :] (the bias part of Eq. parallel-sgd-x-update) for every layer in
// one launch: grid (ceil(max d_l / 128), N, L), one thread per (layer, worker, j).
struct BiasArgs {
  float* params;
  int64_t m_pad;
  int L, B;
  float gamma;
  const uint8_t* active;
  int64_t b_off[PRSGD_MAX_LAYERS];
  int d_out[PRSGD_MAX_LAYERS];
  int ld[PRSGD_MAX_LAYERS];
  const uint16_t* delta_bk[PRSGD_MAX_LAYERS];
  const DeviceStatus* status;
  float* vel;              // momentum buffers laid out like the store, or nullptr
  float mu;
};

__global__ void __launch_bounds__(128) bias_update_kernel(const BiasArgs a) {
  ptx::pdl_wait();
  ptx::pdl_trigger();     // after the wait: a later launch's early loads overlap this launch only
  const int l = blockIdx.z, n = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= a.d_out[l] || (a.active != nullptr && a.active[n] == 0) || a.status->error != 0u) return;
  const uint16_t* d = a.delta_bk[l] + (int64_t)n * a.B * a.ld[l] + j;
  float g = 0.f;
  for (int b0 = 0; b0 < a.B; b0 += 16) {            // B is a multiple of 16: 16 loads in flight, added in order
    uint16_t v[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) v[u] = __ldg(d + (int64_t)(b0 + u) * a.ld[l]);
#pragma unroll
    for (int u = 0; u < 16; ++u) g += __uint_as_float((uint32_t)v[u] << 16);
  }
  float* bp = a.params + (int64_t)n * a.m_pad + a.b_off[l] + j;
  if (a.vel != nullptr) {
    float* vp = a.vel + (int64_t)n * a.m_pad + a.b_off[l] + j;
    g = fmaf(a.mu, *vp, g);
    *vp = g;
  }
  *bp = fmaf(-a.gamma, g, *bp);
}

// Node average of every layer's bias segment in one launch (averaging iteration of the fused form), plus the
// weight segments of the layers that are too small for the fused update + average (the class layer): grid
// (blocks, L + weight segments), one thread per entry (grid-stride over a weight segment), the same arithmetic as
// average_rows_kernel (fp32 sum in worker order, one division), so the bits equal update-then-average.
struct BiasAverageArgs {
  float* params;             // the store, or the momentum buffers (same layout)
  int64_t m_pad;
  int N, L;
  int64_t b_off[PRSGD_MAX_LAYERS];
  int d_out[PRSGD_MAX_LAYERS];
  const DeviceStatus* status;
  float divisor;             // N, or 1 to leave the row sum
  int n_seg;                 // weight segments averaged in the same launch (blockIdx.y = L + k)
  int64_t seg_off[PRSGD_MAX_LAYERS];
  int64_t seg_len[PRSGD_MAX_LAYERS];
  uint16_t* shadow;          // bf16 copy of the store: the averaged weight segments are written there too
};

__global__ void __launch_bounds__(128) bias_average_kernel(const BiasAverageArgs a) {
  ptx::pdl_wait();
  ptx::pdl_trigger();     // after the wait: a later launch's early loads overlap this launch only
  if (a.status->error != 0u) return;
  const int y = blockIdx.y;
  const int64_t off = y < a.L ? a.b_off[y] : a.seg_off[y - a.L];
  const int64_t len = y < a.L ? (int64_t)a.d_out[y] : a.seg_len[y - a.L];
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < len; j += (int64_t)gridDim.x * blockDim.x) {
    float* p = a.params + off + j;
    float s = 0.f;
    int i = 0;
    for (; i + 8 <= a.N; i += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = p[(int64_t)(i + u) * a.m_pad];
#pragma unroll
      for (int u = 0; u < 8; ++u) s += v[u];
    }
    for (; i < a.N; ++i) s += p[(int64_t)i * a.m_pad];
    const float mean = __fdiv_rn(s, a.divisor);
    for (int r = 0; r < a.N; ++r) p[(int64_t)r * a.m_pad] = mean;
    if (y >= a.L && a.shadow != nullptr) {
      const uint16_t h = (uint16_t)(pack_bf16x2(mean, 0.f) & 0xFFFFu);
      uint16_t* q = a.shadow + off + j;
      for (int r = 0; r < a.N; ++r) q[(int64_t)r * a.m_pad] = h;
    }
  }
}

}  // namespace prsgd
#include "kernels_head.cuh"
#include "kernels_update_common.cuh"
namespace prsgd {

// Self-test of the failure path: waits on an mbarrier that nothing ever arrives on, with a short
// limit, so that the wait expires, the status word is set and the kernel returns normally.
__global__ void __launch_bounds__(32) wait_expiry_kernel(DeviceStatus* status, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_mbar_init();
    ptx::mbar_wait(ptx::smem_u32(&bar), 0u, &abort_flag, status, 0x301, limit_cycles);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// Order of layer l's weight segment (1-based l): tile-major for hidden layers whose height is a multiple of 128
// (the class layer, whose tiles the head kernel loads with only as many rows as it has, stays row-major).
inline bool tc_layer_tiled(const prsgd_ctx* c, int l) {
  const Layer& ly = c->layer[l - 1];
  return c->precision == PRSGD_PRECISION_BF16 && c->tiled_weights != 0 && l < c->L && ly.d_out % 128 == 0 && ly.d_in % 64 == 0;
}
inline WTile tc_wtile(const prsgd_ctx* c, int l) {
  WTile t;
  t.tiled = tc_layer_tiled(c, l) ? 1 : 0; t.tn = c->layer[l - 1].d_in / 64; t.d_in = c->layer[l - 1].d_in;
  return t;
}

// tensor maps over a weight segment of layer l: {d_in, d_out, N} row-major, {64, tiles * 128, N} tile-major
inline int tc_make_weight_map(const prsgd_ctx* c, CUtensorMap* m, bool fp32, const void* seg, int l, uint32_t b0, uint32_t b1, std::string* err) {
  const Layer& ly = c->layer[l - 1];
  const uint64_t esz = fp32 ? 4 : 2;
  if (tc_layer_tiled(c, l)) {
    const uint64_t tiles = (uint64_t)(ly.d_out / 128) * (uint64_t)(ly.d_in / 64);
    return make_map3(m, fp32, seg, 64, tiles * 128, (uint64_t)c->N, 64 * esz, (uint64_t)c->m_pad * esz, b0, b1, err);
  }
  return make_map3(m, fp32, seg, (uint64_t)ly.d_in, (uint64_t)ly.d_out, (uint64_t)c->N, (uint64_t)ly.d_in * esz, (uint64_t)c->m_pad * esz, b0, b1, err);
}

// (re)builds the maps of all weight segments: at creation and whenever the order of the segments changes
inline int tc_make_weight_maps(prsgd_ctx* c, std::string* err) {
  TcState* st = static_cast<TcState*>(c->tc);
  int rc = PRSGD_OK;
  for (int l = 1; l <= c->L && rc == PRSGD_OK; ++l) {
    const Layer& ly = c->layer[l - 1];
    TcLayerMaps& mp = st->layer[l - 1];
    rc = tc_make_weight_map(c, &mp.shadow_k, false, c->shadow + ly.w_off, l, 64, 128, err);
    if (rc == PRSGD_OK) rc = tc_make_weight_map(c, &mp.shadow_mn, false, c->shadow + ly.w_off, l, 64, 64, err);
    if (rc == PRSGD_OK) rc = tc_make_weight_map(c, &mp.master, true, c->params + ly.w_off, l, 32, 128, err);
    if (rc == PRSGD_OK && c->velocity != nullptr) rc = tc_make_weight_map(c, &mp.velocity, true, c->velocity + ly.w_off, l, 32, 128, err);
  }
  return rc;
}

inline int tc_create(prsgd_ctx* c, std::string* err) {
  if (c->B > 64) { *err = "BF16 precision supports batch 16, 32 or 64"; return PRSGD_ERR_ALIGN; }
  TcState* st = new (std::nothrow) TcState();
  if (!st) { *err = "out of host memory"; return PRSGD_ERR_ARG; }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device) == cudaSuccess && sms > 0) st->num_sms = sms;
  const uint64_t N = c->N, B = c->B;
  int rc = PRSGD_OK;
  c->tc = st;
  rc = tc_make_weight_maps(c, err);
  c->tc = nullptr;
  for (int l = 1; l <= c->L && rc == PRSGD_OK; ++l) {
    TcLayerMaps& mp = st->layer[l - 1];
    const uint64_t ld = c->buf.ld[l];
    if (rc == PRSGD_OK) rc = make_map3(&mp.delta_out, false, c->buf.delta_bk[l], ld, B, N, ld * 2, B * ld * 2, 64, (uint32_t)B, err);
    if (rc == PRSGD_OK && l > 1) {
      const uint64_t ldi = c->buf.ld[l - 1];
      rc = make_map3(&mp.act_in, false, c->buf.act_bk[l - 1], ldi, B, N, ldi * 2, B * ldi * 2, 64, (uint32_t)B, err);
      if (rc == PRSGD_OK && l == 2)
        rc = make_map3(&st->act1_alt, false, c->buf.act1_alt, ldi, B, N, ldi * 2, B * ldi * 2, 64, (uint32_t)B, err);
    }
  }
  if (rc == PRSGD_OK && c->L >= 2 && c->dims[c->L] <= 128) {      // the class layer's tiles with only as many rows as it has
    const Layer& ly = c->layer[c->L - 1];
    const uint64_t din = ly.d_in, dout = ly.d_out;
    const uint32_t rows = (uint32_t)((ly.d_out + 15) / 16 * 16);
    rc = make_map3(&st->head_shadow, false, c->shadow + ly.w_off, din, dout, N, din * 2, (uint64_t)c->m_pad * 2, 64, rows, err);
    if (rc == PRSGD_OK) rc = make_map3(&st->head_master, true, c->params + ly.w_off, din, dout, N, din * 4, (uint64_t)c->m_pad * 4, 32, rows, err);
    st->head_rows = (int)rows;
  }
  if (rc != PRSGD_OK) { delete st; return rc; }
  cudaError_t e = cudaSuccess;
  const int big = (int)stream_smem_bytes(c->B);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_stream_kernel<TC_FWD_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  const int big_sm = (int)stream_smem_bytes(c->B, true);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_stream_kernel<TC_FWD_LINEAR>, cudaFuncAttributeMaxDynamicSharedMemorySize, big > big_sm ? big : big_sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_stream_kernel<TC_DX>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_forward_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big > big_sm ? big : big_sm);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<false, 64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<64, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<true, 64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<64, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<false, 128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<128, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<true, 128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<128, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<false, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<64, true>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_kernel<true, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCfg<64, true>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_dx_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdDxCfg<64, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_dx_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdDxCfg<64, true>::smem(c->B));
  if (e == cudaSuccess && UpdDxCfg<128, false>::stages(c->B) >= 2)
    e = cudaFuncSetAttribute(tc_update_dx_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdDxCfg<128, false>::smem(c->B));
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc_update_dx_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdDxCfg<64, false, true>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_next_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdNextCfg<64, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_next_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdNextCfg<128, false>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_next_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdNextCfg<64, true>::smem(c->B));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_update_common_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UpdCommonCfg::smem(c->B));
  if (e == cudaSuccess && st->head_rows > 0)
    e = cudaFuncSetAttribute(tc_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)head_smem_bytes(c->B, st->head_rows, 4) > 227 * 1024
                                 ? 227 * 1024 : (int)head_smem_bytes(c->B, st->head_rows, 4));
  if (e != cudaSuccess) {
    *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
    delete st;
    return PRSGD_ERR_CUDA;
  }
  c->tc = st;
  return PRSGD_OK;
}

inline void tc_destroy(prsgd_ctx* c) {
  delete static_cast<TcState*>(c->tc);
  c->tc = nullptr;
}

inline int tc_bind_velocity(prsgd_ctx* c, std::string* err) { return tc_make_weight_maps(c, err); }

inline int tc_bind_data(prsgd_ctx* c, std::string* err) {
  TcState* st = static_cast<TcState*>(c->tc);
  const uint64_t d0 = c->dims[0];
  int rc = make_map3(&st->layer[0].act_in, false, c->X, d0, (uint64_t)c->P, (uint64_t)c->N, d0 * 2,
                     (uint64_t)c->P * d0 * 2, 64, (uint32_t)c->B, err);
  st->pool_bound = rc == PRSGD_OK;
  return rc;
}

// The softmax cross-entropy gradient and every bias step run inside GEMM epilogues when the class
// count fits one 128-row tile (and PRSGD_OPT_FUSED_EPILOGUES is on); otherwise as kernels of their own.
// a_1 lives in one of two buffers (prsgd_ctx::a1_sel names the one of the current iteration); every other
// activation has one.  tc_act_in: a_{l-1} as the operand of layer l's GEMMs; tc_act_ptr: a_l as plain memory.
inline const CUtensorMap& tc_act_in(const prsgd_ctx* c, int l) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  return (l == 2 && c->a1_sel != 0) ? st->act1_alt : st->layer[l - 1].act_in;
}
inline uint16_t* tc_act_ptr(const prsgd_ctx* c, int l) {
  return (l == 1 && c->a1_sel != 0) ? c->buf.act1_alt : c->buf.act_bk[l];
}

// Early weight loads of the forward launch being enqueued: not right after an overlapped update, which may still
// be writing the weights of layer 2 when that launch's CTAs start (the flag is consumed by the first launch).
inline bool tc_forward_early_loads(prsgd_ctx* c) {
  const bool quiet = !c->no_early_once;
  c->no_early_once = false;
  return c->early_loads != 0 && quiet;
}

inline bool tc_epilogues_fused(const prsgd_ctx* c) { return c->fused_epilogues != 0 && c->dims[c->L] <= 128; }

// Right after a node average every worker's row holds the same bits (Algorithm 1: all workers restart from y),
// so the launches of the iteration that follows may read worker 0's weights for every worker.  Safe for
// launches that only read the weights (forward, dX) and for the fused update + average, whose CTA has read all
// N copies of a tile before it writes any; NOT for the plain in-place update, where worker 0's row changes
// while other workers' items are still to come.
inline bool tc_shared_restart(const prsgd_ctx* c, const uint8_t* active) {
  return c->shared_restart != 0 && c->rows_identical && active == nullptr && c->N > 1;
}

// forward GEMM of layer l (1-based)
inline void tc_launch_forward(prsgd_ctx* c, int l, const DrawArgs& dr, const uint8_t* active) {
  TcState* st = static_cast<TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  StreamArgs a{};
  a.B = c->B; a.N = c->N; a.k_steps = (ly.d_in / 64 + 1) / 2; a.M_total = ly.d_out; a.tiles_m = (ly.d_out + 127) / 128;
  a.stages = stream_stages(c->B); a.wt = tc_wtile(c, l);
  a.pool = l == 1; a.draw = dr; a.ld_out = c->buf.ld[l];
  a.out_bk = tc_act_ptr(c, l); a.out_f32 = c->buf.act_f32[l];
  a.bias = c->params + ly.b_off; a.bias_stride = c->m_pad;
  a.active = active; a.status = c->status;
  const bool early = tc_forward_early_loads(c);
  a.prefetch = (l > 1 && active == nullptr && early) ? 1 : 0;   // W_1 was written by the launch just before
  a.shared_w = tc_shared_restart(c, active) ? 1 : 0;
  const bool softmax = l == c->L && tc_epilogues_fused(c);
  if (softmax) {        // the softmax-CE gradient, the loss and the step of b_L happen in this launch's epilogue
    a.softmax = 1; a.stages = stream_stages(c->B, true);
    a.Y = c->Y; a.P = c->P; a.delta_bk = c->buf.delta_bk[l]; a.ld_delta = c->buf.ld[l];
    a.row_losses = c->losses; a.draws = c->draws;
    a.bias_rw = c->params + ly.b_off; a.gamma = c->gamma; a.mu = c->mu;
    a.bias_vel = c->velocity != nullptr ? c->velocity + ly.b_off : nullptr;
  }
  const int items = a.tiles_m * c->N;
  dim3 grid(items < st->num_sms ? items : st->num_sms);
  const size_t smem = stream_smem_bytes(c->B, softmax);
  if (l < c->L)
    launch_pdl(tc_stream_kernel<TC_FWD_RELU>, grid, kStreamThreads, smem, c->stream, st->layer[l - 1].shadow_k, tc_act_in(c, l), a);
  else
    launch_pdl(tc_stream_kernel<TC_FWD_LINEAR>, grid, kStreamThreads, smem, c->stream, st->layer[l - 1].shadow_k, tc_act_in(c, l), a);
}

// The class layer's forward GEMM, softmax-CE gradient, step and dZ of the layer below as one launch of
// clusters (tc_head_kernel): plain SGD step, at most 128 classes, d_{L-1} = 128 x {1, 2, 4, 8}, and the
// options that the two launches it replaces depend on left at their defaults.  One CTA per (worker, 128
// features) runs its code once, from a cold instruction cache: that pays while all CTAs are resident at the
// same time (one wave); with more workers the persistent kernels, whose CTAs walk several items, are faster
// (64 workers x 8 slices: 68 us against 39 us), unless PRSGD_OPT_HEAD_KERNEL = 2 asks for it regardless.
inline bool tc_head_applies(const prsgd_ctx* c) {
  if (c->head_kernel == 0 || c->L < 2 || !tc_epilogues_fused(c) || c->dx_in_update != 1 || c->velocity != nullptr) return false;
  const TcState* st = static_cast<const TcState*>(c->tc);
  const int din = c->layer[c->L - 1].d_in;
  if (st->head_rows == 0 || !(din == 128 || din == 256 || din == 512 || din == 1024)) return false;
  return c->head_kernel == 2 || (int64_t)c->N * (din / 128) <= (int64_t)st->num_sms;
}

// The forward GEMM of layer L - 1 inside the head launch (PRSGD_OPT_HEAD_FORWARD): at least three layers (layer
// L - 1's input is then an activation buffer, not the data pool) and room for a ring of two or more stages behind
// the head's own shared memory.
inline int tc_head_forward_stages(const prsgd_ctx* c) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  if (c->head_forward == 0 || c->L < 3 || st->head_rows == 0) return 0;
  const int64_t room = 227 * 1024 - (int64_t)head_smem_bytes(c->B, st->head_rows, 0);
  int stages = (int)(room / (int64_t)head_fwd_stage_bytes(c->B));
  if (stages > 4) stages = 4;
  return stages >= 2 ? stages : 0;
}

inline void tc_launch_head(prsgd_ctx* c, const DrawArgs& dr, const uint8_t* active, bool with_forward) {
  TcState* st = static_cast<TcState*>(c->tc);
  const int L = c->L;
  const Layer& ly = c->layer[L - 1];
  HeadArgs a{};
  a.B = c->B; a.N = c->N; a.C = ly.d_out; a.Cp = st->head_rows; a.gamma = c->gamma; a.draw = dr; a.active = active; a.status = c->status;
  a.prefetch = (active == nullptr && c->early_loads) ? 1 : 0;
  a.bias_rw = c->params + ly.b_off; a.bias_lo_rw = c->params + c->layer[L - 2].b_off; a.bias_stride = c->m_pad;
  a.Y = c->Y; a.P = c->P; a.row_losses = c->losses; a.draws = c->draws;
  a.out_bk = c->buf.delta_bk[L - 1]; a.ld_out = c->buf.ld[L - 1];
  if (with_forward) {
    a.fwd = 1; a.fwd_stages = tc_head_forward_stages(c);
    a.fwd_ksteps = (c->layer[L - 2].d_in / 64 + 1) / 2;
    a.fwd_prefetch = (active == nullptr && tc_forward_early_loads(c)) ? 1 : 0;
    a.fwd_shared_w = tc_shared_restart(c, active) ? 1 : 0;
    a.wt_lo = tc_wtile(c, L - 1);
  }
  const unsigned cl = (unsigned)(ly.d_in / 128);
  const TcLayerMaps& lo = st->layer[L >= 2 ? L - 2 : 0];
  launch_pdl_cluster(tc_head_kernel, dim3(cl, (unsigned)c->N), dim3(kHeadThreads), head_smem_bytes(c->B, st->head_rows, a.fwd_stages),
                     c->stream, cl, st->head_shadow, tc_act_in(c, L), st->head_master, lo.shadow_k, tc_act_in(c, L - 1), a);
}

// The per-worker flags the launches being enqueued honour: Algorithm 3's mask, or the mask of a worker group.
inline const uint8_t* worker_mask(const prsgd_ctx* c) {
  if (c->group_active != nullptr) return c->group_active;
  return c->has_mask ? c->active : nullptr;
}

// forward GEMMs of layers l_first..L as one launch (tc_forward_chain_kernel)
inline bool tc_chain_applies(const prsgd_ctx* c, int l_first, int l_last) {
  const int n_seg = l_last - l_first + 1;
  return c->forward_chain != 0 && n_seg >= 2 && n_seg <= kChainMax && c->group_active == nullptr;   // (its counters serve one chain at a time)
}

inline void tc_launch_forward_chain(prsgd_ctx* c, int l_first, int l_last, const DrawArgs& dr, const uint8_t* active) {
  TcState* st = static_cast<TcState*>(c->tc);
  ChainMaps maps;
  ChainArgs a{};
  a.B = c->B; a.N = c->N; a.n_seg = l_last - l_first + 1;
  a.shared_w = tc_shared_restart(c, active) ? 1 : 0;
  a.softmax = (l_last == c->L && tc_epilogues_fused(c)) ? 1 : 0;
  a.stages = stream_stages(c->B, a.softmax != 0);
  a.draw = dr; a.active = active; a.status = c->status; a.bias_stride = c->m_pad;
  a.ready = c->chain_ready; a.done = c->chain_ready + (size_t)kChainMax * c->N;
  int items = 0;
  const bool early = tc_forward_early_loads(c);
  for (int l = l_first; l <= l_last; ++l) {
    const Layer& ly = c->layer[l - 1];
    ChainSeg& g = a.seg[l - l_first];
    g.k_steps = (ly.d_in / 64 + 1) / 2; g.tiles_m = (ly.d_out + 127) / 128; g.M_total = ly.d_out; g.ld_out = c->buf.ld[l];
    g.linear = l == c->L ? 1 : 0; g.pool = l == 1 ? 1 : 0; g.wt = tc_wtile(c, l);
    // early weight loads overlap whatever launch precedes the whole forward pass: only when that launch is known
    // to leave the weights of layers >= 2 alone (the layer-1 update or a bias launch that ended the iteration before)
    g.prefetch = (l > 1 && active == nullptr && early && c->upper_weights_quiet) ? 1 : 0;
    g.item0 = items;
    g.out_bk = tc_act_ptr(c, l); g.out_f32 = c->buf.act_f32[l]; g.bias = c->params + ly.b_off;
    items += g.tiles_m * c->N;
    maps.w[l - l_first] = st->layer[l - 1].shadow_k;
    maps.b[l - l_first] = tc_act_in(c, l);
  }
  for (int i = a.n_seg; i < kChainMax; ++i) { maps.w[i] = maps.w[0]; maps.b[i] = maps.b[0]; }
  a.total_items = items;
  if (a.softmax) {
    const Layer& ly = c->layer[c->L - 1];
    a.Y = c->Y; a.P = c->P; a.delta_bk = c->buf.delta_bk[c->L]; a.ld_delta = c->buf.ld[c->L];
    a.row_losses = c->losses; a.draws = c->draws;
    a.bias_rw = c->params + ly.b_off; a.gamma = c->gamma; a.mu = c->mu;
    a.bias_vel = c->velocity != nullptr ? c->velocity + ly.b_off : nullptr;
  }
  dim3 grid(items < st->num_sms ? items : st->num_sms);
  launch_pdl(tc_forward_chain_kernel, grid, kStreamThreads, stream_smem_bytes(c->B, a.softmax != 0), c->stream, maps, a);
}

// dZ_{l-1} from dZ_l through W_l (l >= 2)
inline void tc_launch_dx(prsgd_ctx* c, int l, const DrawArgs& dr, const uint8_t* active, unsigned int* zero_word = nullptr) {
  TcState* st = static_cast<TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  StreamArgs a{};
  a.B = c->B; a.N = c->N; a.k_steps = (c->buf.ld[l] / 64 + 1) / 2; a.M_total = ly.d_in; a.tiles_m = (ly.d_in + 127) / 128;
  a.stages = stream_stages(c->B); a.wt = tc_wtile(c, l);
  a.pool = 0; a.draw = dr; a.ld_out = c->buf.ld[l - 1];
  a.out_bk = c->buf.delta_bk[l - 1]; a.mask_src = tc_act_ptr(c, l - 1);
  a.active = active; a.status = c->status; a.zero_word = zero_word;
  a.prefetch = (active == nullptr && c->early_loads) ? 1 : 0;
  a.shared_w = tc_shared_restart(c, active) ? 1 : 0;
  if (tc_epilogues_fused(c)) {      // the step of b_{l-1} rides on the epilogue that forms dZ_{l-1}
    a.bias_rw = c->params + c->layer[l - 2].b_off; a.bias_stride = c->m_pad; a.gamma = c->gamma; a.mu = c->mu;
    a.bias_vel = c->velocity != nullptr ? c->velocity + c->layer[l - 2].b_off : nullptr;
  }
  const int items = a.tiles_m * c->N;
  dim3 grid(items < st->num_sms ? items : st->num_sms);
  launch_pdl(tc_stream_kernel<TC_DX>, grid, kStreamThreads, stream_smem_bytes(c->B), c->stream, st->layer[l - 1].shadow_mn,
             st->layer[l - 1].delta_out, a);
}

template <int TN, bool MOM>
inline void tc_launch_update_tn(prsgd_ctx* c, int l, const DrawArgs& dr, const uint8_t* active, bool fuse, bool overlapped, bool late) {
  TcState* st = static_cast<TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  UpdateArgs a{};
  a.B = c->B; a.N = c->N; a.tiles_m = (ly.d_out + 127) / 128; a.tiles_n = (ly.d_in + TN - 1) / TN;
  a.gamma = c->gamma; a.mu = c->mu; a.pool = l == 1; a.draw = dr; a.active = active; a.status = c->status;
  a.prefetch = (active == nullptr && c->early_loads && !overlapped) ? 1 : 0;
  a.next_item = overlapped ? c->tile_counter : nullptr;       // (the caller has checked: no mask, not fused)
  a.late = late ? 1 : 0;
  a.shared_w = (fuse && tc_shared_restart(c, active)) ? 1 : 0; a.wt = tc_wtile(c, l);
  a.avg_vel = c->average_velocity ? 1 : 0;
  a.divisor = c->avg_divisor > 0.f ? c->avg_divisor : (float)c->N;
  const int items = a.tiles_m * a.tiles_n * (fuse ? 1 : c->N);
  const int grid = items < st->num_sms ? items : st->num_sms;
  const TcLayerMaps& mp = st->layer[l - 1];
  const size_t smem = UpdCfg<TN, MOM>::smem(c->B);
  if constexpr (MOM) {
    if (fuse)
      launch_pdl(tc_update_kernel<true, TN, true>, dim3(grid), kUpdThreads, smem, c->stream, mp.delta_out, tc_act_in(c, l), mp.master, mp.shadow_k, mp.velocity, a);
    else
      launch_pdl(tc_update_kernel<false, TN, true>, dim3(grid), kUpdThreads, smem, c->stream, mp.delta_out, tc_act_in(c, l), mp.master, mp.shadow_k, mp.velocity, a);
  } else {
    if (fuse)
      launch_pdl(tc_update_kernel<true, TN, false>, dim3(grid), kUpdThreads, smem, c->stream, mp.delta_out, tc_act_in(c, l), mp.master, mp.shadow_k, mp.master, a);
    else
      launch_pdl(tc_update_kernel<false, TN, false>, dim3(grid), kUpdThreads, smem, c->stream, mp.delta_out, tc_act_in(c, l), mp.master, mp.shadow_k, mp.master, a);
  }
}

// The folded form gives a CTA whole 64-wide column blocks of one worker (all row tiles of the block), so it
// needs several blocks per SM to balance; with fewer the separate dX and update launches (one tile per
// item) are faster.  A layer of a single row tile (the class layer) has one tile per block anyway and is
// latency-bound: there one launch instead of two always wins.
inline bool tc_layer_folds_dx(const prsgd_ctx* c, int l) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  const int64_t blocks = (int64_t)((c->layer[l - 1].d_in + 63) / 64) * c->N;
  return blocks >= 3 * (int64_t)st->num_sms || c->layer[l - 1].d_out <= 128;
}

// Update of layer l >= 2 that also forms dZ_{l-1} (tc_update_dx_kernel): replaces dX_l + update_l.
template <int TN, bool MOM, bool SP = (TN == 128)>
inline void tc_launch_update_dx_m(prsgd_ctx* c, int l) {
  TcState* st = static_cast<TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  UpdateDxArgs a{};
  a.B = c->B; a.N = c->N; a.tiles_m = (ly.d_out + 127) / 128; a.tiles_n = (ly.d_in + TN - 1) / TN;
  a.gamma = c->gamma; a.status = c->status; a.stages = UpdDxCfg<TN, MOM, SP>::stages(c->B); a.wt = tc_wtile(c, l);
  a.out_bk = c->buf.delta_bk[l - 1]; a.mask_src = tc_act_ptr(c, l - 1); a.ld_out = c->buf.ld[l - 1]; a.M_total = ly.d_in;
  a.bias_rw = c->params + c->layer[l - 2].b_off; a.bias_stride = c->m_pad;
  a.mu = c->mu; a.bias_vel = MOM ? c->velocity + c->layer[l - 2].b_off : nullptr;
  a.active = worker_mask(c);
  const int items = a.tiles_n * c->N;
  const int grid = items < st->num_sms ? items : st->num_sms;
  const TcLayerMaps& mp = st->layer[l - 1];
  launch_pdl(tc_update_dx_kernel<TN, MOM, SP>, dim3(grid), kUpdBlkThreads, UpdDxCfg<TN, MOM, SP>::smem(c->B), c->stream, mp.delta_out,
             tc_act_in(c, l), mp.master, mp.shadow_k, MOM ? mp.velocity : mp.master, a);
}

// 128-wide column blocks when every SM has a long queue of them and the operand boxes leave room for two
// stages (B <= 32); 64-wide ones otherwise and for the momentum form.
inline void tc_launch_update_dx(prsgd_ctx* c, int l) {
  if (c->velocity != nullptr) { tc_launch_update_dx_m<64, true>(c, l); return; }
  const TcState* st = static_cast<const TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  int tile = c->upd_tile;
  if (tile == 0) {
    const int64_t blocks128 = (int64_t)((ly.d_in + 127) / 128) * c->N;
    // (a layer of one row tile, the class layer, has one tile per block: the wide form halves the number of blocks,
    // and with them the block epilogues that set its pace)
    tile = (blocks128 >= 4 * (int64_t)st->num_sms && ly.d_out > 128) ||
           (ly.d_out <= 128 && c->B <= 32 && blocks128 >= 2 * (int64_t)st->num_sms) ? 128 : 64;
  }
  if (tile == 128 && UpdDxCfg<128, false>::stages(c->B) >= 2) tc_launch_update_dx_m<128, false>(c, l);
  else if (c->dx_shared_pair) tc_launch_update_dx_m<64, false, true>(c, l);      // more stages (see UpdDxCfg)
  else tc_launch_update_dx_m<64, false, false>(c, l);
}

// Whether a block-walking launch of `blocks` blocks of `tn` tiles runs in its split form (PRSGD_OPT_SPLIT_BLOCKS,
// off by default), and with what run length: only without a worker mask, only when equal runs shorten the longest
// CTA's walk by 5 % or more, and (unless the option says 2) only for launches of at least eight tiles per SM.
// Measured: layer 1 of a 16-worker 3072-1024 net (128 row blocks on 148 SMs) 121 us split, 119 us whole; of a
// 64-worker 1024-2048 net (3.46 rounds of blocks) within 0.5 %: the launch is bound by the memory system, which
// the remaining CTAs of a short last round saturate just as well.
inline SplitArgs tc_split_plan(const prsgd_ctx* c, int64_t blocks, int tn, const uint8_t* active, int* grid) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  SplitArgs sp{};
  sp.part = c->split_part; sp.count = c->split_count;
  const int64_t tiles = blocks * tn;
  const int g_whole = blocks < st->num_sms ? (int)blocks : st->num_sms;
  *grid = g_whole;
  if (c->split_blocks == 0 || active != nullptr || st->num_sms > kSplitMaxCtas || blocks <= 0) return sp;
  const int g = tiles < st->num_sms ? (int)tiles : st->num_sms;
  const int64_t chunk = (tiles + g - 1) / g;
  const int64_t whole_walk = (blocks + g_whole - 1) / g_whole * tn;
  const bool pays = 20 * chunk <= 19 * whole_walk && (c->split_blocks == 2 || tiles >= 8 * (int64_t)st->num_sms);
  if (!pays) return sp;
  sp.on = 1; sp.chunk = (int)chunk;
  *grid = (int)((tiles + chunk - 1) / chunk);
  return sp;
}

// Update of layer 1 that also forms a_1 of the next iteration (tc_update_next_kernel).
template <int TN, bool MOM>
inline void tc_launch_update_next_tn(prsgd_ctx* c, const DrawArgs& dr, bool other_a1) {
  TcState* st = static_cast<TcState*>(c->tc);
  const Layer& ly = c->layer[0];
  UpdateNextArgs a{};
  a.B = c->B; a.N = c->N; a.tiles_m = (ly.d_out + 127) / 128; a.tiles_n = (ly.d_in + TN - 1) / TN;
  a.gamma = c->gamma; a.mu = c->mu; a.draw = dr; a.status = c->status;
  a.active = worker_mask(c);
  a.stages = UpdNextCfg<TN, MOM>::stages(c->B); a.wt = tc_wtile(c, 1);
  // (other_a1: something launched after this still reads the current a_1, so the next one goes to the other buffer)
  a.next_out = other_a1 ? (c->a1_sel != 0 ? c->buf.act_bk[1] : c->buf.act1_alt) : tc_act_ptr(c, 1);
  a.next_ld = c->buf.ld[1];
  a.bias = c->params + ly.b_off; a.bias_stride = c->m_pad; a.M_total = ly.d_out;
  int grid = 1;
  a.split = tc_split_plan(c, (int64_t)a.tiles_m * c->N, a.tiles_n, a.active, &grid);
  const TcLayerMaps& mp = st->layer[0];
  launch_pdl(tc_update_next_kernel<TN, MOM>, dim3(grid), kUpdBlkThreads, UpdNextCfg<TN, MOM>::smem(c->B), c->stream, mp.delta_out,
             mp.act_in, mp.master, MOM ? mp.velocity : mp.master, a);
}

inline void tc_launch_update_next(prsgd_ctx* c, const DrawArgs& dr, bool other_a1 = false) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  const Layer& ly = c->layer[0];
  if (c->velocity != nullptr) {            // momentum step: 64-wide tiles (two stages of master + momentum tiles)
    tc_launch_update_next_tn<64, true>(c, dr, other_a1);
    return;
  }
  int tile = c->upd_tile;
  if (tile == 0) {
    const int64_t tiles128 = (int64_t)((ly.d_out + 127) / 128) * ((ly.d_in + 127) / 128);
    tile = (c->B <= 32 && tiles128 * c->N >= 32 * (int64_t)st->num_sms) ? 128 : 64;
  }
  if (tile == 128 && UpdNextCfg<128, false>::stages(c->B) >= 2) tc_launch_update_next_tn<128, false>(c, dr, other_a1);
  else tc_launch_update_next_tn<64, false>(c, dr, other_a1);
}

inline bool tc_layer_fuses_average(const prsgd_ctx* c, int l);

// Fused update + average from a common starting point for the layers in `layers` (n of them, 1-based, any order):
// one weight-gradient GEMM per tile over the minibatches of all workers (tc_update_common_kernel), all layers'
// tiles in one launch, the tiles of the last partly filled round cut into row ranges.
inline void tc_launch_update_common(prsgd_ctx* c, const int* layers, int n, const DrawArgs& dr, bool late = false) {
  TcState* st = static_cast<TcState*>(c->tc);
  CommonMaps maps;
  UpdateCommonArgs a{};
  a.B = c->B; a.N = c->N; a.n_seg = n;
  a.gamma = c->gamma; a.draw = dr; a.status = c->status;
  a.prefetch = c->early_loads ? 1 : 0; a.late = late ? 1 : 0;
  a.divisor = c->avg_divisor > 0.f ? c->avg_divisor : (float)c->N;
  a.stages = UpdCommonCfg::stages(c->B);
  a.m_pad = c->m_pad;
  int tiles = 0;
  for (int i = 0; i < n; ++i) {
    const int l = layers[i];
    const Layer& ly = c->layer[l - 1];
    CommonSeg& g = a.seg[i];
    g.tiles_n = (ly.d_in + 63) / 64; g.tile0 = tiles; g.pool = l == 1 ? 1 : 0; g.d_in = ly.d_in; g.d_out = ly.d_out;
    g.params = c->params + ly.w_off; g.shadow = c->shadow + ly.w_off; g.wt = tc_wtile(c, l);
    tiles += ((ly.d_out + 127) / 128) * g.tiles_n;
    maps.delta[i] = st->layer[l - 1].delta_out; maps.act[i] = tc_act_in(c, l); maps.master[i] = st->layer[l - 1].master;
  }
  for (int i = n; i < kCommonMax; ++i) { maps.delta[i] = maps.delta[0]; maps.act[i] = maps.act[0]; maps.master[i] = maps.master[0]; }
  a.tiles = tiles;
  const int grid = tiles < st->num_sms ? tiles : st->num_sms;
  a.full_tiles = tiles / grid * grid;
  const int rest = tiles - a.full_tiles;                       // tiles of the last, partly filled round
  a.split = rest > 0 ? grid / rest : 1;
  if (a.split > c->N) a.split = c->N;
  if (a.split < 1 || c->common_point == 2) a.split = 1;        // (2: whole tiles only)
  launch_pdl(tc_update_common_kernel, dim3(grid), kUpdCommonThreads, UpdCommonCfg::smem(c->B), c->stream, maps, a);
}

// Whether the averaging iteration being enqueued forms layer l's step from the common point in the one launch
// that follows the dX launches.
inline bool tc_layer_takes_common_point(const prsgd_ctx* c, int l, const uint8_t* active) {
  return c->common_point != 0 && c->velocity == nullptr && tc_shared_restart(c, active) && tc_layer_fuses_average(c, l);
}

// Tile width: forced by PRSGD_OPT_UPDATE_TILE, else chosen per launch.  Wide tiles need fewer TMA
// operations per byte and win when every SM has a long queue of them; narrow tiles give four
// pipeline stages and twice as many work items, which wins on small stores and on the fused form,
// where a launch has only one item per tile.
inline void tc_launch_update(prsgd_ctx* c, int l, const DrawArgs& dr, const uint8_t* active, bool fuse, bool overlapped = false,
                             bool late = false) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  if (c->velocity != nullptr) {            // momentum step: 64-wide tiles (two stages of master + momentum + output)
    tc_launch_update_tn<64, true>(c, l, dr, active, fuse, overlapped, late);
    return;
  }
  int tile = c->upd_tile;
  if (tile == 0) {
    const int64_t tiles128 = (int64_t)((ly.d_out + 127) / 128) * ((ly.d_in + 127) / 128);
    // (fused form: a CTA owns a tile across all workers; wide tiles once one round of them nearly fills the GPU)
    if (fuse) tile = (2 * tiles128 >= 3 * (int64_t)st->num_sms || (c->B <= 32 && 5 * tiles128 >= 4 * (int64_t)st->num_sms)) ? 128 : 64;
    else tile = (c->B <= 32 && tiles128 * c->N >= 32 * (int64_t)st->num_sms) ? 128 : 64;
  }
  if (tile == 128) tc_launch_update_tn<128, false>(c, l, dr, active, fuse, overlapped, late);
  else tc_launch_update_tn<64, false>(c, l, dr, active, fuse, overlapped, late);
}

// Bias step of all layers (after the last dZ has been formed).  On an averaging iteration it is followed
// by the node average of each bias segment (same arithmetic as the stand-alone averaging kernel, so
// the bits agree with update-then-average).
inline void tc_launch_bias(prsgd_ctx* c, const uint8_t* active) {
  BiasArgs a{};
  a.params = c->params; a.m_pad = c->m_pad; a.L = c->L; a.B = c->B; a.gamma = c->gamma; a.active = active;
  a.status = c->status; a.vel = c->velocity; a.mu = c->mu;
  int dmax = 1;
  for (int l = 1; l <= c->L; ++l) {
    const Layer& ly = c->layer[l - 1];
    a.b_off[l - 1] = ly.b_off; a.d_out[l - 1] = ly.d_out; a.ld[l - 1] = c->buf.ld[l]; a.delta_bk[l - 1] = c->buf.delta_bk[l];
    if (ly.d_out > dmax) dmax = ly.d_out;
  }
  launch_pdl(bias_update_kernel, dim3((dmax + 127) / 128, c->N, c->L), dim3(128), 0, c->stream, a);
}

// A layer with few tiles gives the fused update + average too few CTAs (each walks all N workers of
// its tile), so such a layer takes the plain update followed by the node average of its weight segment.
inline bool tc_layer_fuses_average(const prsgd_ctx* c, int l) {
  const TcState* st = static_cast<const TcState*>(c->tc);
  const Layer& ly = c->layer[l - 1];
  const int64_t tiles64 = (int64_t)((ly.d_out + 127) / 128) * ((ly.d_in + 63) / 64);
  return 2 * tiles64 >= (int64_t)st->num_sms;
}

inline void tc_launch_weight_average(prsgd_ctx* c, int l) {
  const Layer& ly = c->layer[l - 1];
  const int64_t cols = (int64_t)ly.d_out * ly.d_in;          // a multiple of 64, like every input width of this path
  launch_pdl(average_rows_kernel<0, true, 2>, dim3((unsigned)((cols / 2 + (cols & 1) + 255) / 256)), dim3(256), 0, c->stream,
             c->params + ly.w_off, (int64_t)c->N, cols, c->m_pad, (float*)nullptr, c->shadow + ly.w_off,
             (const DeviceStatus*)c->status, c->avg_divisor);
}

// the same segment of the momentum buffers, when they are averaged with the models
inline void tc_launch_velocity_segment_average(prsgd_ctx* c, int l) {
  const Layer& ly = c->layer[l - 1];
  const int64_t cols = (int64_t)ly.d_out * ly.d_in;
  launch_pdl(average_rows_kernel<0, false, 2>, dim3((unsigned)((cols / 2 + (cols & 1) + 255) / 256)), dim3(256), 0, c->stream,
             c->velocity + ly.w_off, (int64_t)c->N, cols, c->m_pad, (float*)nullptr, (uint16_t*)nullptr,
             (const DeviceStatus*)c->status, 0.f);
}

// `with_weights`: also the weight segments of the layers that did not take the fused update + average
inline void tc_launch_bias_average(prsgd_ctx* c, float* store, bool with_weights = false) {
  BiasAverageArgs a{};
  a.params = store; a.m_pad = c->m_pad; a.N = c->N; a.L = c->L; a.status = c->status;
  a.divisor = (store == c->params && c->avg_divisor > 0.f) ? c->avg_divisor : (float)c->N;
  int64_t longest = 1;
  for (int l = 1; l <= c->L; ++l) {
    a.b_off[l - 1] = c->layer[l - 1].b_off; a.d_out[l - 1] = c->layer[l - 1].d_out;
    if (a.d_out[l - 1] > longest) longest = a.d_out[l - 1];
    if (with_weights && !tc_layer_fuses_average(c, l)) {
      a.seg_off[a.n_seg] = c->layer[l - 1].w_off;
      a.seg_len[a.n_seg] = (int64_t)c->layer[l - 1].d_out * c->layer[l - 1].d_in;
      if (a.seg_len[a.n_seg] > longest) longest = a.seg_len[a.n_seg];
      ++a.n_seg;
    }
  }
  a.shadow = with_weights ? c->shadow : nullptr;
  int64_t blocks = (longest + 127) / 128;
  if (blocks > 1024) blocks = 1024;                  // (a long segment is walked with a grid stride)
  launch_pdl(bias_average_kernel, dim3((unsigned)blocks, c->L + a.n_seg), dim3(128), 0, c->stream, a);
}

}  // namespace prsgd
