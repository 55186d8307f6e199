// Head of the network in ONE launch (bf16-operand tensor-core path, plain SGD step, class layer L with
// d_L <= 128 and d_{L-1} = 128 * {1, 2, 4, 8}).  Per worker it does what two launches did before:
//   z = W_L a_{L-1} + b_L, the softmax cross-entropy gradient dZ_L and the per-sample loss, the step of b_L,
//   dW_L = dZ_L^T a_{L-1} and the step x <- x - gamma dW_L on the fp32 master and the bf16 copy of W_L,
//   dZ_{L-1} = (dZ_L W_L) .* [a_{L-1} > 0] (from the weights as they were before the step) and the step of b_{L-1}.
// A worker's class layer is tiny (10..128 rows), so as (tile, worker) items of the persistent kernels it is
// pure latency: one CTA walks the whole contraction of 1024 features in eight barrier phases, twice.  Here a
// worker is a thread-block CLUSTER, one CTA per 128-feature slice of a_{L-1}: each CTA forms the slice's share of
// the logits, the shares are summed through the cluster's shared memory in a fixed order (CTA 0, 1, ...), each
// CTA turns B / cluster-size rows of logits into dZ_L rows and writes them into every CTA's operand tile, and
// then every CTA owns the 128 columns of W_L (and the 128 features of dZ_{L-1}) of its slice outright.
// The logits are summed slice by slice, so their last bits differ from the one-accumulator sum of the stream
// kernel; everything is deterministic, and identical for every launch geometry of the other kernels.
//
// Every CTA runs this code exactly once, and the instruction lines of a launch are rarely in any cache (the
// weight stream of the launches in between has pushed them out of L2), so the time of a step is set by how
// many lines it fetches: the loops below are deliberately NOT unrolled, tiles have ceil16(d_L) rows instead of
// 128 padded ones, and the ReLU mask is read from the activation tile that is in shared memory anyway.
#pragma once

namespace prsgd {

struct HeadArgs {
  int B, N;
  int C;                     // d_L
  int Cp;                    // d_L rounded up to 16: rows of a weight tile in shared memory
  float gamma;
  DrawArgs draw;
  const uint8_t* active;     // per-worker flag or nullptr: an inactive worker's cluster does nothing
  DeviceStatus* status;
  int prefetch;              // 1: W_L's tiles may be requested before the previous launch has completed
  float* bias_rw;            // params + b_off of layer L (worker stride bias_stride)
  float* bias_lo_rw;         // params + b_off of layer L - 1
  int64_t bias_stride;
  const int32_t* Y;          // labels [N][P]
  int64_t P;
  float* row_losses;         // [N][B]
  int32_t* draws;            // [N]
  uint16_t* out_bk;          // bf16 dZ_{L-1} [N][B][ld_out]
  int ld_out;
  // Forward GEMM of layer L - 1 in the same launch (`fwd` = 1): CTA s of a worker's cluster forms the 128 features
  // a_{L-1}[:, 128 s ..] = relu(W_{L-1}[128 s .., :] a_{L-2} + b_{L-1}) it needs, streaming its row tile of W_{L-1}
  // through a ring of `fwd_stages` stages like tc_stream_kernel, and writes them straight into the activation
  // tile in shared memory: a_{L-1} never goes to global memory (nothing else reads it).
  int fwd;
  int fwd_ksteps;            // pipeline steps: ceil(d_{L-2} / 128)
  int fwd_stages;
  int fwd_prefetch;          // W_{L-1}'s first tiles may be requested before the previous launch has completed
  int fwd_shared_w;          // every worker's W_{L-1} holds the same bits: read worker 0's (one HBM read serves all)
  WTile wt_lo;               // order of W_{L-1}'s elements
};

constexpr int kHeadThreads = 320;     // warp 0 loads, warp 1 MMAs, warps 2..5 logits / softmax / step of W_L, warps 6..9 dZ_{L-1}

// shared memory: bf16 W_L slice (two {64, Cp} boxes) | a_{L-1} slice (two {64, B} boxes) | fp32 W_L slice (four
// {32, Cp} boxes) | stepped bf16 slice | dZ_L operand tile (two {64, B} boxes, classes contiguous) | this CTA's
// share of the logits [B][Cp + 1] | its rows of summed logits [B][Cp + 1] | b_L | barriers.
// The logits MMA has M = 128: it reads 128 rows (16 KB) from the start of each bf16 box; the rows past Cp are
// whatever lies behind the box (the regions that follow are always longer than that), and their accumulator
// lanes are never read.
__host__ __device__ inline uint32_t head_fixed_bytes(int B, int Cp) {
  const uint32_t op_box = (uint32_t)B * 128u, wbox = (uint32_t)Cp * 128u;
  const uint32_t used = 2u * wbox + 2u * op_box + 4u * wbox + 2u * wbox + 2u * op_box + 2u * (uint32_t)B * (uint32_t)(Cp + 1) * 4u + 512u + 256u;
  return (used + 1023u) & ~1023u;                        // (the forward ring behind it holds swizzled tiles)
}
__host__ __device__ inline uint32_t head_fwd_stage_bytes(int B) { return 2u * (16384u + (uint32_t)B * 128u); }
__host__ __device__ inline uint32_t head_smem_bytes(int B, int Cp, int fwd_stages = 0) {
  return head_fixed_bytes(B, Cp) + (uint32_t)fwd_stages * head_fwd_stage_bytes(B) + 1024u;
}

__global__ void __launch_bounds__(kHeadThreads, 1) tc_head_kernel(const __grid_constant__ CUtensorMap mapShadow,
                                                                  const __grid_constant__ CUtensorMap mapAct,
                                                                  const __grid_constant__ CUtensorMap mapMaster,
                                                                  const __grid_constant__ CUtensorMap mapWlo,
                                                                  const __grid_constant__ CUtensorMap mapActLo,
                                                                  const HeadArgs a) {
  using namespace ptx;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;          // (the same offset in every CTA: peers address each other by it)
  uint8_t* gen = smem_raw + (base - raw);
  const int C = a.C, Cp = a.Cp, ldz = Cp + 1;
  const uint32_t op_box = (uint32_t)a.B * 128u;          // one {64, B} box
  const uint32_t wbox = (uint32_t)Cp * 128u;             // one {64 bf16, Cp} or {32 fp32, Cp} box
  const uint32_t logit_bytes = (uint32_t)(a.B * ldz) * 4u;
  const uint32_t o_act = 2u * wbox, o_mst = o_act + 2u * op_box, o_new = o_mst + 4u * wbox, o_dz = o_new + 2u * wbox;
  const uint32_t o_part = o_dz + 2u * op_box, o_zs = o_part + logit_bytes, o_bias = o_zs + logit_bytes, o_bar = o_bias + 512u;
  const uint32_t g1 = base + o_bar, g2 = g1 + 8u, acc1 = g1 + 16u, acc2 = g1 + 24u, acc3 = g1 + 32u;
  const uint32_t acc0 = g1 + 40u, act_ready = g1 + 48u;  // forward of layer L - 1: product done / a_{L-1} tile written
  auto f_full = [&](int st) { return g1 + 96u + 8u * st; };
  auto f_empty = [&](int st) { return g1 + 160u + 8u * st; };
  const uint32_t o_ring = head_fixed_bytes(a.B, Cp);
  const uint32_t fstage = head_fwd_stage_bytes(a.B);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + o_bar + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + o_bar + 68);
  float* part = reinterpret_cast<float*>(gen + o_part);
  float* zs = reinterpret_cast<float*>(gen + o_zs);
  float* bias_s = reinterpret_cast<float*>(gen + o_bias);
  constexpr uint32_t kColL = 0u, kColW = 64u, kColX = 192u;      // TMEM columns: logits share | dW_L slice | dZ_{L-1} slice

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = blockIdx.y;
  const uint32_t rank = blockIdx.x;                      // the cluster spans the grid's x axis
  const int CL = (int)gridDim.x;
  const int k0 = (int)rank * 128;                        // first feature of this CTA's slice

  if (tid == 0) {
    mbar_init(g1, 1); mbar_init(g2, 1); mbar_init(acc1, 1); mbar_init(acc2, 1); mbar_init(acc3, 1);
    mbar_init(acc0, 1); mbar_init(act_ready, 128);
    for (int st = 0; st < a.fwd_stages; ++st) { mbar_init(f_full(st), 1); mbar_init(f_empty(st), 1); }
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    prefetch_tensormap(&mapShadow); prefetch_tensormap(&mapAct); prefetch_tensormap(&mapMaster);
    if (a.fwd) { prefetch_tensormap(&mapWlo); prefetch_tensormap(&mapActLo); }
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 256u); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  auto load_weights = [&]() {
    mbar_expect_tx(g2, 4u * wbox);
#pragma unroll 1
    for (int q = 0; q < 4; ++q) tma_load_3d(base + o_mst + q * wbox, &mapMaster, g2, k0 + 32 * q, 0, n);
    mbar_expect_tx(g1, 2u * wbox + (a.fwd ? 0u : 2u * op_box));   // (the activation boxes follow after the dependency wait)
    tma_load_3d(base, &mapShadow, g1, k0, 0, n);
    tma_load_3d(base + wbox, &mapShadow, g1, k0 + 64, 0, n);
  };
  // two 64-wide K blocks of this CTA's row tile of W_{L-1} (a block past the end of K is zero-filled by TMA)
  auto load_wlo = [&](int st, int ks) {
    const uint32_t sa = base + o_ring + (uint32_t)st * fstage;
    const int nw = a.fwd_shared_w ? 0 : n;
    tma_load_w(sa, &mapWlo, f_full(st), a.wt_lo, (2 * ks) * 64, k0, nw);
    tma_load_w(sa + 16384u, &mapWlo, f_full(st), a.wt_lo, (2 * ks + 1) * 64, k0, nw);
  };
  // Nothing in flight writes W_L when this launch begins (the launch before it is a forward GEMM of a lower
  // layer or layer 1's update), so its tiles are requested while that launch drains.
  const bool pre = a.prefetch != 0 && *abort_flag == 0;
  int fpre = 0;                                          // forward ring stages whose weight tiles are under way already
  if (warp == 0 && lane == 0) {
    if (a.fwd && a.fwd_prefetch != 0 && *abort_flag == 0) {
      fpre = a.fwd_ksteps < a.fwd_stages ? a.fwd_ksteps : a.fwd_stages;
      for (int ks = 0; ks < fpre; ++ks) {
        mbar_expect_tx(f_full(ks), fstage);
        load_wlo(ks, ks);
      }
    }
    if (pre) load_weights();
  }
  pdl_wait();
  pdl_trigger();
  const uint32_t tmem = *tmem_slot;
  const bool run = *abort_flag == 0 && (a.active == nullptr || a.active[n] != 0);
  const int q4 = warp & 3;
  const int r = q4 * 32 + lane;                          // the TMEM lane this thread reads
  const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
  const int etid = tid - 64;                             // 0..127 among warps 2..5
  float blo_old = 0.f;

  // ---------------- phase 0 (fwd): a_{L-1}[:, slice]; phase 1: this slice's share of the logits
  if (run) {
    if (warp == 0 && lane == 0) {
      if (!pre) load_weights();
      if (a.fwd) {
        bool ok = true;
#pragma unroll 1
        for (int ks = 0; ks < a.fwd_ksteps && ok; ++ks) {
          const int st = ks % a.fwd_stages;
          if (ks >= fpre) {
            ok = mbar_wait(f_empty(st), (((uint32_t)(ks / a.fwd_stages)) & 1u) ^ 1u, abort_flag, a.status, 0x606);
            if (!ok) break;
            mbar_expect_tx(f_full(st), fstage);
            load_wlo(st, ks);
          }
          const uint32_t sb = base + o_ring + (uint32_t)st * fstage + 32768u;
          tma_load_3d(sb, &mapActLo, f_full(st), (2 * ks) * 64, 0, n);
          tma_load_3d(sb + op_box, &mapActLo, f_full(st), (2 * ks + 1) * 64, 0, n);
        }
      } else {
        tma_load_3d(base + o_act, &mapAct, g1, k0, 0, n);
        tma_load_3d(base + o_act + op_box, &mapAct, g1, k0 + 64, 0, n);
      }
    } else if (warp == 1 && lane == 0) {
      bool fok = true;
      if (a.fwd) {
        const uint32_t idesc0 = idesc_bf16(128, a.B, 0, 0);
#pragma unroll 1
        for (int ks = 0; ks < a.fwd_ksteps && fok; ++ks) {
          const int st = ks % a.fwd_stages;
          fok = mbar_wait(f_full(st), ((uint32_t)(ks / a.fwd_stages)) & 1u, abort_flag, a.status, 0x607);
          if (!fok) break;
          tc_fence_after();
          const uint32_t sa = base + o_ring + (uint32_t)st * fstage, sb = sa + 32768u;
#pragma unroll 1
          for (int jk = 0; jk < 8; ++jk) {
            const uint32_t j = (uint32_t)jk >> 2, k = (uint32_t)jk & 3u;
            mma_bf16(tmem + kColX, smem_desc_sw128(sa + j * 16384u + k * 32u, 16u, 1024u),
                     smem_desc_sw128(sb + j * op_box + k * 32u, 16u, 1024u), idesc0, (ks | jk) != 0 ? 1u : 0u);
          }
          mma_commit(f_empty(st));
        }
        if (fok) mma_commit(acc0);
        fok = fok && mbar_wait(act_ready, 0u, abort_flag, a.status, 0x608);
      }
      if (fok && mbar_wait(g1, 0u, abort_flag, a.status, 0x601)) {
        tc_fence_after();
        const uint32_t idesc = idesc_bf16(128, a.B, 0, 0);
#pragma unroll 1
        for (int jk = 0; jk < 8; ++jk) {                  // two 64-feature boxes x four 16-feature steps
          const uint32_t j = (uint32_t)jk >> 2, k = (uint32_t)jk & 3u;
          mma_bf16(tmem + kColL, smem_desc_sw128(base + j * wbox + k * 32u, 16u, 1024u),
                   smem_desc_sw128(base + o_act + j * op_box + k * 32u, 16u, 1024u), idesc, jk != 0 ? 1u : 0u);
        }
        mma_commit(acc1);
      }
    } else if (warp >= 2 && warp < 6) {
      bias_s[r] = r < C ? a.bias_rw[(int64_t)n * a.bias_stride + r] : 0.f;
      // the operand tile's chunks of eight classes that lie wholly beyond C stay zero (their rows of W_L are zero too)
      const int nch = (C + 7) / 8, nz = 16 - nch;
#pragma unroll 1
      for (int task = etid; task < a.B * nz; task += 128) {
        const int b = task / nz, ch = nch + task % nz;
        *reinterpret_cast<uint4*>(gen + o_dz + (uint32_t)(ch >> 3) * op_box + (uint32_t)b * 128u + ((uint32_t)((ch & 7) ^ (b & 7)) << 4)) =
            make_uint4(0u, 0u, 0u, 0u);
      }
      if (a.fwd) {
        // forward epilogue of the slice: bias, ReLU, bf16, written as the two {64, B} activation boxes (row b of a
        // box = 128 bytes, 16-byte chunks swizzled by b) the products below read; thread <-> feature k0 + r
        const float blo = a.bias_lo_rw[(int64_t)n * a.bias_stride + k0 + r];
        const bool ok0 = __all_sync(0xffffffffu, mbar_wait(acc0, 0u, abort_flag, a.status, 0x609));
        if (ok0) {
          tc_fence_after();
          uint8_t* acol = gen + o_act + (uint32_t)(r >> 6) * op_box + (uint32_t)(r & 7) * 2u;
          const uint32_t chunk = (uint32_t)((r & 63) >> 3);
#pragma unroll 1
          for (int b8 = 0; b8 < a.B; b8 += 8) {
            uint32_t v[8];
            tmem_ld8(tmem + lane_off + kColX + (uint32_t)b8, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<uint16_t*>(acol + (uint32_t)(b8 + j) * 128u + ((chunk ^ (uint32_t)j) << 4)) =
                  f32_to_bf16_rn(fmaxf(__uint_as_float(v[j]) + blo, 0.f));
          }
          tc_fence_before();
          fence_proxy_async();
          mbar_arrive(act_ready);
        }
      }
      const bool ok = __all_sync(0xffffffffu, mbar_wait(acc1, 0u, abort_flag, a.status, 0x602));
      if (ok && q4 * 32 < C) {                           // (a warp whose lanes all lie beyond C holds no logits)
        tc_fence_after();
#pragma unroll 1
        for (int b8 = 0; b8 < a.B; b8 += 8) {
          uint32_t v[8];
          tmem_ld8(tmem + lane_off + kColL + (uint32_t)b8, v);
          tmem_ld_wait();
          if (r < C) {
#pragma unroll
            for (int j = 0; j < 8; ++j) part[(b8 + j) * ldz + r] = __uint_as_float(v[j]);
          }
        }
        tc_fence_before();
      }
    } else if (warp >= 6) {
      blo_old = a.bias_lo_rw[(int64_t)n * a.bias_stride + k0 + r];
    }
  }
  __syncwarp();
  cluster_arrive_release();
  cluster_wait_acquire();          // every CTA's share (and its abort flag) is visible to its peers

  // ---------------- phase 2: logits -> dZ_L rows, handed to every CTA of the cluster
  uint32_t bad = run ? 0u : 1u;
  uint32_t peer_part[8], peer_dz[8];
#pragma unroll
  for (int p = 0; p < 8; ++p) {
    if (p < CL) {
      peer_part[p] = cluster_map(base + o_part, (uint32_t)p);
      peer_dz[p] = cluster_map(base + o_dz, (uint32_t)p);
      bad |= ld_cluster_u32(cluster_map(base + o_bar + 68u, (uint32_t)p));
    } else {
      peer_part[p] = 0u; peer_dz[p] = 0u;
    }
  }
  const bool run_all = bad == 0u;
  if (run_all && warp >= 2 && warp < 6) {
    const int rows_per = a.B / CL;                       // minibatch rows whose dZ_L this CTA forms
    int Tr = 128 / rows_per;                             // threads per row (a power of two, one warp at most)
    if (Tr > 32) Tr = 32;
    const int rl = etid / Tr, sub = etid % Tr;
    const bool rowok = rl < rows_per;
    const int bg = (int)rank * rows_per + (rowok ? rl : 0);     // the row's index in the minibatch
    const uint32_t blk = draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks);
    const int label = a.Y[(int64_t)n * a.P + (int64_t)blk * a.B + bg];
#pragma unroll 1
    for (int idx = etid; idx < rows_per * C; idx += 128) {
      const int r2 = idx / C, c = idx - r2 * C;
      const uint32_t off = (uint32_t)(((int)rank * rows_per + r2) * ldz + c) * 4u;
      float s = 0.f;
#pragma unroll
      for (int p = 0; p < 8; ++p)
        if (p < CL) s += ld_cluster_f32(peer_part[p] + off);
      zs[r2 * ldz + c] = s + bias_s[c];
    }
    named_bar_sync(1, 128);
    // dZ_L = (softmax(z) - onehot(y)) / B and the per-sample loss; a row belongs to Tr neighbouring threads
    const int Cc = rowok ? C : 0;
    float* z = zs + (rowok ? rl : 0) * ldz;
    const float invB = 1.f / (float)a.B;
    float mx = -INFINITY;
#pragma unroll 1
    for (int cc = sub; cc < Cc; cc += Tr) mx = fmaxf(mx, z[cc]);
#pragma unroll 1
    for (int o = Tr >> 1; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = 0.f;
#pragma unroll 1
    for (int cc = sub; cc < Cc; cc += Tr) se += __expf(z[cc] - mx);
#pragma unroll 1
    for (int o = Tr >> 1; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const float lse = mx + __logf(se);
    const float zl = rowok ? z[label] : 0.f;
    __syncwarp();
#pragma unroll 1
    for (int cc = sub; cc < Cc; cc += Tr) z[cc] = (__expf(z[cc] - lse) - (cc == label ? 1.f : 0.f)) * invB;
    if (rowok && sub == 0) a.row_losses[(int64_t)n * a.B + bg] = lse - zl;
    if (rank == 0u && etid == 0) a.draws[n] = (int32_t)blk;
    __syncwarp();
    if (rowok) {
      const int nch = (C + 7) / 8;
#pragma unroll 1
      for (int ch = sub; ch < nch; ch += Tr) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = ch * 8 + i < C ? z[ch * 8 + i] : 0.f;
        const uint4 pk = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
        const uint32_t off = (uint32_t)(ch >> 3) * op_box + (uint32_t)bg * 128u + ((uint32_t)((ch & 7) ^ (bg & 7)) << 4);
#pragma unroll
        for (int p = 0; p < 8; ++p)
          if (p < CL) st_cluster_v4(peer_dz[p] + off, pk);
      }
    }
    fence_proxy_async_all();       // the operand tiles (this CTA's and its peers') are read by MMAs next
  }
  __syncwarp();
  cluster_arrive_release();
  cluster_wait_acquire();          // all rows of dZ_L sit in every CTA's operand tile; no CTA touches a peer's memory after this

  // ---------------- phase 3: this slice's columns of W_L and features of dZ_{L-1}
  if (run_all) {
    if (warp == 1 && lane == 0) {
      tc_fence_after();
      // dW_L[:, slice] = dZ_L^T a_{L-1}[:, slice] over K = B (both operands MN-major, as in tc_update_kernel)
      const uint32_t idesc_dw = idesc_bf16(128, 128, 1, 1);
#pragma unroll 1
      for (int k = 0; k < a.B / 16; ++k)
        mma_bf16(tmem + kColW, smem_desc_sw128(base + o_dz + k * 2048u, op_box, 1024u),
                 smem_desc_sw128(base + o_act + k * 2048u, op_box, 1024u), idesc_dw, k != 0 ? 1u : 0u);
      mma_commit(acc2);
      // dZ_{L-1}^T[slice, B] = W_L[:, slice]^T dZ_L^T over K = classes (the slice's bf16 tile read MN-major)
      const uint32_t idesc_dx = idesc_bf16(128, a.B, 1, 0);
#pragma unroll 1
      for (int kk = 0; kk * 16 < C; ++kk)
        mma_bf16(tmem + kColX, smem_desc_sw128(base + (uint32_t)kk * 2048u, wbox, 1024u),
                 smem_desc_sw128(base + o_dz + (uint32_t)(kk >> 2) * op_box + (uint32_t)(kk & 3) * 32u, 16u, 1024u), idesc_dx,
                 kk != 0 ? 1u : 0u);
      mma_commit(acc3);
    } else if (warp >= 2 && warp < 6) {
      // step of b_L by the cluster's first CTA: column sums of dZ_L as the MMAs see it (bf16)
      if (rank == 0u && etid < C) {
        const int m = etid;
        float gsum = 0.f;
        const uint8_t* col = gen + o_dz + (uint32_t)(m >> 6) * op_box + (uint32_t)(m & 7) * 2u;
        const uint32_t chunk = (uint32_t)((m & 63) >> 3);
#pragma unroll 4
        for (int b = 0; b < a.B; ++b) {
          const uint16_t h = *reinterpret_cast<const uint16_t*>(col + (uint32_t)b * 128u + ((chunk ^ (uint32_t)(b & 7)) << 4));
          gsum += __uint_as_float((uint32_t)h << 16);
        }
        a.bias_rw[(int64_t)n * a.bias_stride + m] = fmaf(-a.gamma, gsum, bias_s[m]);
      }
      bool ok = mbar_wait(g2, 0u, abort_flag, a.status, 0x603) && mbar_wait(acc2, 0u, abort_flag, a.status, 0x604);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && q4 * 32 < C) {                           // (a warp whose 32 rows all lie beyond C has nothing to step)
        tc_fence_after();
        uint8_t* mst = gen + o_mst;
        uint8_t* stg = gen + o_new;
        const uint32_t row_off = (uint32_t)r * 128u;
        const uint32_t sw = (uint32_t)(r & 7);
#pragma unroll 1
        for (int it = 0; it < 16; ++it) {                 // eight columns of the slice per step
          const uint32_t c = (uint32_t)it >> 2, jp = (uint32_t)it & 3u;
          uint32_t v[8];
          tmem_ld8(tmem + lane_off + kColW + (uint32_t)(it * 8), v);
          tmem_ld_wait();
          if (r < Cp) {                                   // two 16-byte fp32 chunks = one 16-byte bf16 chunk
            float4* p0 = reinterpret_cast<float4*>(mst + c * wbox + row_off + (((2u * jp) ^ sw) << 4));
            float4* p1 = reinterpret_cast<float4*>(mst + c * wbox + row_off + (((2u * jp + 1u) ^ sw) << 4));
            float4 x = *p0, y = *p1;
            x.x = fmaf(-a.gamma, __uint_as_float(v[0]), x.x); x.y = fmaf(-a.gamma, __uint_as_float(v[1]), x.y);
            x.z = fmaf(-a.gamma, __uint_as_float(v[2]), x.z); x.w = fmaf(-a.gamma, __uint_as_float(v[3]), x.w);
            y.x = fmaf(-a.gamma, __uint_as_float(v[4]), y.x); y.y = fmaf(-a.gamma, __uint_as_float(v[5]), y.y);
            y.z = fmaf(-a.gamma, __uint_as_float(v[6]), y.z); y.w = fmaf(-a.gamma, __uint_as_float(v[7]), y.w);
            *p0 = x; *p1 = y;
            const uint32_t boff = (c >> 1) * wbox + row_off + ((((c & 1u) * 4u + jp) ^ sw) << 4);
            *reinterpret_cast<uint4*>(stg + boff) = make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w),
                                                               pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
          }
        }
        tc_fence_before();
      }
      fence_proxy_async();
      named_bar_sync(1, 128);
      if (ok && etid == 0) {                             // rows beyond C are clipped by the store
#pragma unroll 1
        for (int q = 0; q < 4; ++q) tma_store_3d(&mapMaster, base + o_mst + q * wbox, k0 + 32 * q, 0, n);
        tma_store_3d(&mapShadow, base + o_new, k0, 0, n);
        tma_store_3d(&mapShadow, base + o_new + wbox, k0 + 64, 0, n);
        tma_commit_group();
        tma_wait_group0();
      }
    } else if (warp >= 6) {
      // dX epilogue of the slice: ReLU mask (a_{L-1} > 0, read from the activation tile), bf16 dZ_{L-1}, step of b_{L-1}[k0 + r]
      const int feat = k0 + r;
      const bool ok = __all_sync(0xffffffffu, mbar_wait(acc3, 0u, abort_flag, a.status, 0x605));
      if (ok) {
        tc_fence_after();
        float gsum = 0.f;
        const uint8_t* acol = gen + o_act + (uint32_t)(r >> 6) * op_box + (uint32_t)(r & 7) * 2u;
        const uint32_t chunk = (uint32_t)((r & 63) >> 3);
        uint16_t* out = a.out_bk + (int64_t)n * a.B * a.ld_out + feat;
#pragma unroll 1
        for (int b8 = 0; b8 < a.B; b8 += 8) {
          uint32_t v[8];
          tmem_ld8(tmem + lane_off + kColX + (uint32_t)b8, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) {                   // row b8 + j of the tile: its 16-byte chunks are swizzled by j
            const uint16_t mk = *reinterpret_cast<const uint16_t*>(acol + (uint32_t)(b8 + j) * 128u + ((chunk ^ (uint32_t)j) << 4));
            const float d = (mk & 0x7FFFu) != 0 ? __uint_as_float(v[j]) : 0.f;
            gsum += d;
            out[(int64_t)(b8 + j) * a.ld_out] = f32_to_bf16_rn(d);
          }
        }
        tc_fence_before();
        a.bias_lo_rw[(int64_t)n * a.bias_stride + feat] = fmaf(-a.gamma, gsum, blo_old);
      }
    }
  } else if (run && warp == 0 && lane == 0) {
    // a peer gave up: let this CTA's own copies land before it goes away
    const long long t0 = clock64();
    while (!(mbar_try_wait(g1, 0u) && mbar_try_wait(g2, 0u)) && clock64() - t0 < 200000000ll) {}
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256u);
}

}  // namespace prsgd
