// Fused update + node average from a COMMON starting point (bf16-operand tensor-core path, plain SGD step).
//
// Right after an averaging step every worker holds the same point x (Algorithm 1: all workers restart from the
// node average).  If the very next iteration averages again -- every iteration when I = 1, which the paper
// points out is parallel mini-batch SGD -- the new average is
//     (1/N) sum_i (x - gamma G_i) = x - (gamma / N) sum_i G_i ,     sum_i G_i = sum_i dZ_i^T A_i ,
// i.e. ONE weight-gradient GEMM whose contraction runs over the minibatches of all workers (K = N B).  A CTA
// owns a 128 x 64 tile, accumulates the N workers' products in one TMEM accumulator (no per-worker epilogue, no
// per-worker master tile), applies the step once and stores the result to all N rows.  What bounds the kernel
// is then only the N row stores.  They do not go through TMA: one SM's bulk tensor stores of 128-byte box rows
// top out near 24 GB/s (3.5 TB/s over the GPU, which a kernel that also loads never notices, but a kernel that
// only stores does).  Four warps read the finished tile from shared memory into registers once and write it N
// times with 16-byte stores, a quarter warp per 128-byte row segment; the output buffer is free again as soon
// as it has been read, so the next tile's products and epilogue proceed under the stores.
// One launch serves every layer that takes this form (their tiles form one list, layer by layer: all of them need
// only the dZ and activation buffers, which are complete once the dX launches have run), and the tiles of the
// list's last, partly filled round are cut into row ranges: with 512 tiles on 148 SMs the last round has 68
// tiles, each then formed by two CTAs that store eight rows apiece (forming a tile is hidden under the previous
// tile's stores; storing is what takes time).
// The result equals update-then-average up to fp32 rounding (one rounding of the summed gradient instead of N
// roundings of the stepped models); it is deterministic (fixed worker order inside the accumulator).
#pragma once

namespace prsgd {

constexpr int kCommonMax = 8;     // layers one launch can serve

struct CommonSeg {
  int tiles_n;               // 64-column tiles of d_{l-1}
  int tile0;                 // index of the layer's first tile in the launch's list
  int pool;                  // layer 1: the activation operand is the drawn block of the data pool
  int d_in, d_out;
  float* params;             // fp32 store + offset of W_l (row stride m_pad elements)
  uint16_t* shadow;          // bf16 copy + offset of W_l
  WTile wt;                  // order of the segment's elements
};

struct CommonMaps {
  CUtensorMap delta[kCommonMax];   // bf16 dZ_l, box {64, B, 1}
  CUtensorMap act[kCommonMax];     // bf16 a_{l-1} (the data pool for layer 1), box {64, B, 1}
  CUtensorMap master[kCommonMax];  // fp32 W_l, box {32, 128, 1}
};

struct UpdateCommonArgs {
  int B, N;
  int n_seg, tiles;          // layers and tiles in the list
  int full_tiles;            // the first full_tiles tiles are stored whole (a multiple of the grid size)
  int split;                 // each later tile is shared by `split` CTAs, which store N / split rows each
  float gamma;
  DrawArgs draw;
  DeviceStatus* status;
  int prefetch;              // 1: the first master tile may be requested before the previous launch has completed
  int late;                  // 1: no dependency wait at the start, one before the exit (see UpdateArgs::late)
  float divisor;             // the summed models N x - gamma sum_i G_i are divided by this (N; 1 leaves the row SUM)
  int stages;
  int64_t m_pad;
  CommonSeg seg[kCommonMax];
};

constexpr int kUpdCommonThreads = 320;   // warp 0 loader, 1 MMA, 2..5 epilogue, 6..9 row stores

struct UpdCommonCfg {
  static constexpr uint32_t kMaster = 128u * 64u * 4u;     // fp32 tile, two {32, 128} boxes
  static constexpr uint32_t kOut = 128u * 64u * 2u;        // bf16 tile, one {64, 128} box
  static constexpr uint32_t kBuf = kMaster + kOut;         // the output buffer
  __host__ __device__ static uint32_t stage(int B) { return 3u * (uint32_t)B * 128u; }     // two dZ boxes + one activation box
  static int stages(int B) {
    int s = (int)((227u * 1024u - 2048u - kBuf) / stage(B));
    return s > 8 ? 8 : s;
  }
  static size_t smem(int B) { return (size_t)stages(B) * stage(B) + kBuf + 1024 + 512; }
};

__global__ void __launch_bounds__(kUpdCommonThreads, 1) tc_update_common_kernel(const __grid_constant__ CommonMaps maps,
                                                                                const __grid_constant__ UpdateCommonArgs a) {
  using namespace ptx;
  using Cfg = UpdCommonCfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int S = a.stages;
  const uint32_t op_box = (uint32_t)a.B * 128u;           // one {64, B} box
  const uint32_t stage_bytes = Cfg::stage(a.B);
  const uint32_t buf_u32 = base;                          // the output buffer: fp32 tile, then the bf16 tile
  auto ops_u32 = [&](int s) { return base + Cfg::kBuf + (uint32_t)s * stage_bytes; };
  const uint32_t bar0 = base + Cfg::kBuf + (uint32_t)S * stage_bytes;
  auto full_ops = [&](int s) { return bar0 + 8u * s; };
  auto stage_empty = [&](int s) { return bar0 + 64u + 8u * s; };
  auto acc_full = [&](int q) { return bar0 + 128u + 8u * q; };
  auto acc_empty = [&](int q) { return bar0 + 144u + 8u * q; };
  const uint32_t mst_full = bar0 + 160u, tile_ready = bar0 + 176u, out_free = bar0 + 192u;
  uint8_t* tail = gen + Cfg::kBuf + (size_t)S * stage_bytes;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 260);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The items of this CTA: whole tiles blockIdx.x, + gridDim.x, ... below full_tiles, then (for the first CTAs) one
  // tile of the last round, shared with split - 1 neighbours: item -> (tile, first row, end row).
  const int G = (int)gridDim.x;
  const int n_whole = a.full_tiles / G;
  const int tail_tile = a.full_tiles + (int)blockIdx.x / a.split;
  const int n_items_all = n_whole + (tail_tile < a.tiles ? 1 : 0);
  auto item_tile = [&](int i) { return i < n_whole ? (int)blockIdx.x + i * G : tail_tile; };
  auto item_rows = [&](int i, int& nb, int& ne) {
    if (i < n_whole) { nb = 0; ne = a.N; return; }
    const int part = (int)blockIdx.x % a.split;
    nb = (int)((int64_t)a.N * part / a.split);
    ne = (int)((int64_t)a.N * (part + 1) / a.split);
  };
  auto seg_of = [&](int tile) { int si = 0; while (si + 1 < a.n_seg && tile >= a.seg[si + 1].tile0) ++si; return si; };

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_ops(s), 1); mbar_init(stage_empty(s), 1); }
    for (int q = 0; q < 2; ++q) { mbar_init(acc_full(q), 1); mbar_init(acc_empty(q), 128); }
    mbar_init(mst_full, 1); mbar_init(tile_ready, 128); mbar_init(out_free, 128);
    *abort_flag = *(volatile unsigned int*)&a.status->error != 0u ? 1 : 0;   // an earlier expired wait: no-op (see tc_stream_kernel)
    fence_mbar_init();
    for (int i = 0; i < a.n_seg; ++i) { prefetch_tensormap(&maps.delta[i]); prefetch_tensormap(&maps.act[i]); prefetch_tensormap(&maps.master[i]); }
  }
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 128u); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // the common point is read from worker 0's row (every row holds the same bits)
  auto load_master = [&](int tile) {
    const int si = seg_of(tile);
    const int rel = tile - a.seg[si].tile0;
    const int m0 = (rel / a.seg[si].tiles_n) * 128, n0 = (rel % a.seg[si].tiles_n) * 64;
    mbar_expect_tx(mst_full, Cfg::kMaster);
    tma_load_w(buf_u32, &maps.master[si], mst_full, a.seg[si].wt, n0, m0, 0);
    tma_load_w(buf_u32 + 16384u, &maps.master[si], mst_full, a.seg[si].wt, n0 + 32, m0, 0);
  };
  // The master tiles were last written an iteration ago (the launch before this one only reads bf16 copies), so
  // the first one is requested while that launch drains.
  const bool pre = a.prefetch != 0 && *abort_flag == 0 && n_items_all > 0;
  if (pre && warp == 0 && lane == 0) load_master(item_tile(0));
  if (a.late == 0) {
    pdl_wait();
    pdl_trigger();
  }
  const uint32_t tmem = *tmem_slot;
  const int n_items = *abort_flag != 0 ? 0 : n_items_all;

  // Every role walks the same items; item number ti of this CTA uses accumulator ti % 2; `it` counts (tile, worker)
  // operand stages.  (Dealing out (tile, row) pairs in equal runs for ALL tiles, so that every CTA stores the same
  // number of rows, was slower: every CTA then forms one more tile than it stores, and forming a tile takes a
  // third of the time of storing it; cutting only the tiles of the last round costs nothing, the extra tile is
  // formed while the previous one is stored.)
  if (warp == 0 && lane == 0) {
    // ---------------- loader
    uint32_t it = 0, ti = 0;
    bool ok = true;
    for (; (int)ti < n_items && ok; ++ti) {
      const int w = item_tile((int)ti);
      const int si = seg_of(w);
      const int rel = w - a.seg[si].tile0;
      const int m0 = (rel / a.seg[si].tiles_n) * 128, n0 = (rel % a.seg[si].tiles_n) * 64;
      if (ti >= 1) ok = mbar_wait(out_free, (ti - 1u) & 1u, abort_flag, a.status, 0x701);   // the store warps hold the previous tile in registers
      if (!ok) break;
      if (!(pre && ti == 0)) load_master(w);
      for (int n = 0; n < a.N; ++n, ++it) {
        const int s = it % S;
        ok = mbar_wait(stage_empty(s), ((it / S) & 1u) ^ 1u, abort_flag, a.status, 0x702);
        if (!ok) break;
        const int row0 = a.seg[si].pool ? (int)draw_block(a.draw.seed, a.draw.worker0 + n, draw_t(a.draw), a.draw.n_blocks) * a.B : 0;
        const uint32_t ops = ops_u32(s);
        mbar_expect_tx(full_ops(s), 3u * op_box);
        tma_load_3d(ops, &maps.delta[si], full_ops(s), m0, 0, n);
        tma_load_3d(ops + op_box, &maps.delta[si], full_ops(s), m0 + 64, 0, n);
        tma_load_3d(ops + 2u * op_box, &maps.act[si], full_ops(s), n0, row0, n);
      }
    }
    if (n_items == 0 && pre) {         // the launch turned into a no-op: let the early tile land
      const long long t0 = clock64();
      while (!mbar_try_wait(mst_full, 0u) && clock64() - t0 < 200000000ll) {}
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer: the N workers' products of a tile accumulate in one accumulator
    const uint32_t idesc = idesc_bf16(128, 64, 1, 1);
    const int ksteps = a.B / 16;
    uint32_t it = 0, ti = 0;
    bool ok = true;
    for (; (int)ti < n_items && ok; ++ti) {
      const int q = ti & 1;
      ok = mbar_wait(acc_empty(q), ((ti >> 1) & 1u) ^ 1u, abort_flag, a.status, 0x703);
      if (!ok) break;
      tc_fence_after();
      for (int n = 0; n < a.N; ++n, ++it) {
        const int s = it % S;
        ok = mbar_wait(full_ops(s), (it / S) & 1u, abort_flag, a.status, 0x704);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = ops_u32(s), sb = sa + 2u * op_box;
        for (int k = 0; k < ksteps; ++k)
          mma_bf16(tmem + (uint32_t)(q * 64), smem_desc_sw128(sa + k * 2048u, op_box, 1024u),
                   smem_desc_sw128(sb + k * 2048u, op_box, 1024u), idesc, (n | k) != 0 ? 1u : 0u);
        mma_commit(stage_empty(s));
      }
      if (ok) mma_commit(acc_full(q));
    }
  } else if (warp >= 6) {
    // ---------------- row stores: the finished tile (three boxes of 128 rows x 128 bytes: fp32 columns 0..31,
    // fp32 columns 32..63, bf16 columns 0..63) is read into registers once, 24 sixteen-byte chunks per thread,
    // and written to every worker's row; a quarter warp holds the eight chunks of one box row, so it reads
    // shared memory without bank conflicts and writes one 128-byte line
    const int t = tid - 192;                              // 0..127 among the four store warps
    const int j = t & 7, rsub = t >> 3;                   // chunk within the box row; row = rsub + 16 i
    uint32_t ti = 0;
    bool ok = true;
    for (; (int)ti < n_items && ok; ++ti) {
      const int w = item_tile((int)ti);
      const CommonSeg& sg = a.seg[seg_of(w)];
      const int rel = w - sg.tile0;
      const int m0 = (rel / sg.tiles_n) * 128, n0 = (rel % sg.tiles_n) * 64;
      int nb, ne;
      item_rows((int)ti, nb, ne);
      ok = __all_sync(0xffffffffu, mbar_wait(tile_ready, ti & 1u, abort_flag, a.status, 0x705));
      if (!ok) break;
      const uint8_t* buf = gen;
      uint4 v[24];
#pragma unroll
      for (int i = 0; i < 24; ++i) {
        const int rr = rsub + 16 * (i & 7);
        v[i] = *reinterpret_cast<const uint4*>(buf + (i >> 3) * 16384 + rr * 128 + ((j ^ (rr & 7)) << 4));
      }
      mbar_arrive(out_free);                              // the buffer may take the next tile's master tile
      const int64_t first = wtile_offset(sg.wt, m0 + rsub, n0);       // row rsub of the tile, its first column
      float* prow = sg.params + (int64_t)nb * a.m_pad + first + 4 * j;
      uint16_t* srow = sg.shadow + (int64_t)nb * a.m_pad + first + 8 * j;
      const int64_t step = 16 * (int64_t)(sg.wt.tiled ? 64 : sg.d_in);      // 16 rows further down
      for (int n = nb; n < ne; ++n) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (m0 + rsub + 16 * i < sg.d_out) {            // (rows past the layer's height do not exist)
            *reinterpret_cast<uint4*>(prow + i * step) = v[i];
            *reinterpret_cast<uint4*>(prow + i * step + 32) = v[8 + i];
            *reinterpret_cast<uint4*>(srow + i * step) = v[16 + i];
          }
        }
        prow += a.m_pad;
        srow += a.m_pad;
      }
    }
  } else if (warp >= 2 && warp < 6) {
    // ---------------- epilogue: once per tile, row r of the tile <-> TMEM lane r
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const uint32_t row_off = (uint32_t)r * 128u;
    const uint32_t sw = (uint32_t)(r & 7);
    // (N x - gamma sum_i G_i) / D  =  c1 x - c2 sum_i G_i ;  c1 = 1 exactly when D = N
    const float c1 = __fdiv_rn((float)a.N, a.divisor), c2 = __fdiv_rn(a.gamma, a.divisor);
    uint32_t ti = 0;
    bool ok = true;
    for (; (int)ti < n_items && ok; ++ti) {
      const int ob = ti & 1;                              // the accumulator
      ok = mbar_wait(mst_full, ti & 1u, abort_flag, a.status, 0x706) && mbar_wait(acc_full(ob), (ti >> 1) & 1u, abort_flag, a.status, 0x707);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint8_t* mst = gen;
      uint8_t* stg = mst + Cfg::kMaster;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_off + (uint32_t)(ob * 64 + c * 32), v);
        tmem_ld_wait();
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {                  // two 16-byte fp32 chunks = one 16-byte bf16 chunk
          float4* p0 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp) ^ sw) << 4));
          float4* p1 = reinterpret_cast<float4*>(mst + c * 16384 + row_off + (((uint32_t)(2 * jp + 1) ^ sw) << 4));
          float4 x = *p0, y = *p1;
          x.x = fmaf(-c2, __uint_as_float(v[8 * jp + 0]), c1 * x.x); x.y = fmaf(-c2, __uint_as_float(v[8 * jp + 1]), c1 * x.y);
          x.z = fmaf(-c2, __uint_as_float(v[8 * jp + 2]), c1 * x.z); x.w = fmaf(-c2, __uint_as_float(v[8 * jp + 3]), c1 * x.w);
          y.x = fmaf(-c2, __uint_as_float(v[8 * jp + 4]), c1 * y.x); y.y = fmaf(-c2, __uint_as_float(v[8 * jp + 5]), c1 * y.y);
          y.z = fmaf(-c2, __uint_as_float(v[8 * jp + 6]), c1 * y.z); y.w = fmaf(-c2, __uint_as_float(v[8 * jp + 7]), c1 * y.w);
          *p0 = x; *p1 = y;
          *reinterpret_cast<uint4*>(stg + row_off + (((uint32_t)(c * 4 + jp) ^ sw) << 4)) =
              make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w), pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty(ob));
      mbar_arrive(tile_ready);
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 128u);
  if (a.late != 0) {
    pdl_wait();
    pdl_trigger();
  }
}

}  // namespace prsgd
