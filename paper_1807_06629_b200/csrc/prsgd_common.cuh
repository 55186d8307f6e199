// Shared declarations of the PR-SGD library: the host context, the row layout
// and the minibatch draw.  Internal; the public boundary is include/prsgd.h.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <stddef.h>
#include <string>
#include <vector>

#include "prsgd.h"

namespace prsgd {

// ---------------------------------------------------------------------------
// Minibatch draw zeta_i^t (integer only).  SplitMix64 output function applied
// twice: first to the t-th state of the stream seeded with `seed`, then to that
// word advanced by (i + 1) increments.
// ---------------------------------------------------------------------------
__host__ __device__ inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__host__ __device__ inline uint32_t draw_block(uint64_t seed, int worker, int64_t t, uint32_t n_blocks) {
  const uint64_t inc = 0x9E3779B97F4A7C15ull;
  uint64_t u = mix64(seed + inc * (uint64_t)t);
  uint64_t v = mix64(u + inc * (uint64_t)(worker + 1));
  return (uint32_t)(v % (uint64_t)n_blocks);
}

// ---------------------------------------------------------------------------
// Device status words (first 256 bytes of the scratch area)
// ---------------------------------------------------------------------------
struct DeviceStatus {
  unsigned int error;      // 0 = fine; otherwise a code naming the wait that gave up
  unsigned int where;      // block index that recorded it
  unsigned int nonfinite;      // finite check: number of NaN / infinite words found (saturating)
  unsigned int nonfinite_row;  // finite check: lowest row that holds one
  unsigned int pad[60];
};

// Launch with the programmatic-stream-serialization attribute: the kernel may start while the
// previous kernel of the stream drains; it must call griddepcontrol.wait before touching memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same for a grid of thread-block clusters of `cluster_x` CTAs along x (grid.x a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                      unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

constexpr int kMaxGroups = 4;
constexpr int kSplitMaxCtas = 192;  // CTAs of a launch that may each hold two partial accumulators in global memory
constexpr int64_t kSegAlign = 32;  // every segment of a row starts at a multiple of 32 elements

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

struct Layer {
  int d_in, d_out;
  int64_t w_off, b_off;    // element offsets inside a row
};

// How the d_out x d_in elements of a weight segment (fp32 master, bf16 copy, momentum buffer) are ordered.
// Row-major, or (tensor-core path, hidden layers whose height is a multiple of 128) as 128 x 64 tiles stored
// one after another, tile (row / 128, col / 64) at index (row / 128) * tn + col / 64, row-major inside a tile:
// every tile a kernel loads or stores is then one contiguous 32 KB (fp32) / 16 KB (bf16) piece of a worker's row
// instead of 128 pieces of 256 bytes a whole matrix row apart, which the memory system serves ~7 % faster.
struct WTile {
  int tiled;
  int tn;                  // 64-column tiles per matrix row (d_in / 64)
  int d_in;
};

__host__ __device__ inline int64_t wtile_offset(const WTile& t, int row, int col) {   // element offset of W[row][col] in the segment
  if (!t.tiled) return (int64_t)row * t.d_in + col;
  return (((int64_t)(row >> 7) * t.tn + (col >> 6)) << 13) + ((row & 127) << 6) + (col & 63);
}

// Scratch buffers of one precision path.  Index l = 1..L (index 0 unused);
// act[L] holds the logits on the fp32 path.
struct Buffers {
  float* act_f32[PRSGD_MAX_LAYERS + 1];
  float* delta_f32[PRSGD_MAX_LAYERS + 1];
  // bf16 path: activations and deltas, batch-major rows [N][B][ld] with the leading dimension padded to 64
  uint16_t* act_bk[PRSGD_MAX_LAYERS + 1];
  uint16_t* delta_bk[PRSGD_MAX_LAYERS + 1];
  uint16_t* act1_alt;                       // second buffer for a_1 (same shape as act_bk[1]), see prsgd_ctx::overlap_update
  int ld[PRSGD_MAX_LAYERS + 1];             // padded feature count of layer l's output
};

}  // namespace prsgd

struct prsgd_ctx {
  int N = 0, L = 0, B = 0, precision = 0;
  int dims[PRSGD_MAX_LAYERS + 1] = {0};
  int64_t P = 0;             // pool samples per worker
  uint32_t n_blocks = 0;
  uint64_t seed = 0;
  float gamma = 0.f;
  int I = 0;
  int64_t t = 0;
  int worker0 = 0;               // global index of row 0 when the N workers here are a shard of a larger job
  int N_global = 0;              // workers of the whole job (0: this context is the whole job)
  int check_finite = 0;          // prsgd_sync also runs the finite check
  int fused_average = 1;
  float mu = 0.f;                // momentum of the local step (0 = plain SGD)
  float* velocity = nullptr;     // [N][m_pad] fp32 momentum buffers, caller-owned
  int average_velocity = 0;      // average the buffers together with the models
  int upd_tile = 0;              // column width of the update kernel's tile: 0 = chosen per launch, 64 or 128
  int dx_shared_pair = 1;        // 64-wide update + dX: one pair of bf16 tiles behind the stages (more stages) instead of one per stage
  int split_blocks = 0;          // layer 1's update + next forward: row blocks cut at run boundaries so that every CTA streams the same number of tiles
  float* split_part = nullptr;           // [2 * kSplitMaxCtas][B][128] fp32 partial accumulators
  unsigned int* split_count = nullptr;   // a counter per block, zero between launches
  int tiled_weights = 1;         // tensor-core path: hidden layers' weight segments stored as 128 x 64 tiles (see WTile)
  float* canon_row = nullptr;    // [m_pad] fp32: one row in canonical order (conversions between the two orders)
  int common_point = 1;          // fused update + average from a common starting point: one GEMM over all workers' minibatches
  int merged_small_average = 1;  // fused averaging iteration: weight segments too small for the fused form are averaged by the bias-average launch
  int head_forward = 0;          // the forward GEMM of layer L - 1 runs inside the class layer's cluster launch
  int head_kernel = 1;           // the class layer's forward, softmax-CE gradient, step and dZ below it as one launch of clusters
  int dx_in_update = 1;          // layers >= 2: the update launch also forms dZ of the layer below (tensor-core path)
  int next_forward = 1;          // layer 1's update also forms a_1 of the next iteration (tensor-core path)
  bool a1_ready = false;         // a_1 of the coming iteration has already been formed by the previous update
  // Layer 2's plain update launched AFTER layer 1's update + next forward and without a dependency wait at its
  // start, so that its CTAs fill the SMs that launch leaves idle and take over the others as they drain (tiles are
  // claimed from a device counter).  a_1 of the next iteration then goes to the other one of two buffers, because
  // layer 2's update still reads this iteration's a_1 meanwhile.
  int overlap_update = 1;
  int a1_sel = 0;                        // which of the two a_1 buffers holds (or will receive) the current iteration's a_1
  bool no_early_once = false;            // the next forward launch follows an overlapped update that writes W_2: no early weight loads
  unsigned int* tile_counter = nullptr;  // the overlapped update's next unclaimed item; zeroed by the dX launch before it
  int early_loads = 1;           // tensor-core kernels request tiles nobody is writing before their dependency wait
  int fused_epilogues = 1;       // softmax-CE gradient and bias steps inside the GEMM epilogues (tensor-core path)
  int shared_restart = 1;        // the iteration after a node average reads worker 0's weights for every worker
  int forward_chain = 0;         // the forward GEMMs of consecutive layers run as one launch (tensor-core path)
  // Worker groups (PRSGD_OPT_WORKER_GROUPS): the plain iterations of a period run as G independent launch chains,
  // one per contiguous group of workers, on G streams of the library's own
  int worker_groups = 1;
  uint8_t* group_masks = nullptr;        // [kMaxGroups][N] device: 1 where the worker belongs to the group
  const uint8_t* group_active = nullptr; // mask of the group whose launches are being enqueued (nullptr: none)
  cudaStream_t group_stream[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t group_fork = nullptr, group_join[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t group_stagger[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t record_after_forward = nullptr;   // recorded once after the next forward pass (staggers the groups)
  float avg_divisor = 0.f;               // > 0: an averaging iteration divides the summed rows by this instead of N
  bool upper_weights_quiet = false;      // the launch enqueued last does not write the weights of any layer >= 2
  unsigned int* chain_ready = nullptr;   // [8][N] row-tile counters of the forward chain + one word, zero between launches
  bool rows_identical = false;   // every row of the store (and of the bf16 copy) holds the same bits right now
  int64_t assigned_upto = -1;    // prsgd_assign_rows calls since the last local step have covered columns [0, assigned_upto)
  int64_t launches = 0;
  int64_t m = 0, m_pad = 0;
  prsgd::Layer layer[PRSGD_MAX_LAYERS];
  cudaStream_t stream = nullptr;
  int device = 0;

  float* params = nullptr;       // [N][m_pad] fp32
  uint16_t* shadow = nullptr;    // [N][m_pad] bf16 bits (BF16 precision only)
  unsigned char* scratch = nullptr;
  size_t scratch_bytes = 0;

  prsgd::DeviceStatus* status = nullptr;
  int32_t* draws = nullptr;      // [N]
  float* losses = nullptr;       // [N][B] per-sample losses of the last iteration
  uint8_t* active = nullptr;     // [N] device copy of the Algorithm-3 mask
  bool has_mask = false;
  float* stage_row = nullptr;    // [m_pad] fp32
  prsgd::Buffers buf;

  const void* X = nullptr;       // [N][P][d0] fp32 or bf16
  int x_dtype = -1;
  const int32_t* Y = nullptr;    // [N][P]

  void* tc = nullptr;            // tensor-core path state (tensor maps), owned

  // double-buffered pool upload (prsgd_stage_data / prsgd_swap_data)
  void* staged_X = nullptr;
  int32_t* staged_Y = nullptr;
  cudaEvent_t staged_event = nullptr;   // staged copy complete (recorded on the caller's copy stream)
  cudaEvent_t free_event = nullptr;     // work that read the previous pools complete (recorded at swap)

  // asynchronous read-out of the node average (prsgd_get_average_async)
  cudaEvent_t mean_ready_event = nullptr;   // the mean sits in the staging row (recorded on the compute stream)
  cudaEvent_t readout_event = nullptr;      // its copy to the host has been issued / completed (caller's copy stream)
  bool readout_pending = false;

  // whole averaging periods captured as CUDA graphs (PRSGD_OPT_GRAPH)
  struct PeriodGraph {
    uint64_t key[13];
    cudaGraphExec_t exec;
    int64_t launches;            // kernel launches one replay stands for
  };
  int use_graph = 1;
  bool capturing = false;
  int64_t* t_dev = nullptr;      // device copy of t at the start of the period being replayed
  int64_t t_dev_after = -1;      // what that counter will hold once the enqueued work has run (-1: not known)
  std::vector<PeriodGraph> graphs;

  // optional per-kernel timing (PRSGD_OPT_PROFILE)
  struct Timed { int kind; cudaEvent_t a, b; int launches; };
  bool profile = false;
  int open_kind = -1;
  int open_launches = 0;         // launches enqueued inside the open interval so far
  cudaEvent_t open_a = nullptr, open_b = nullptr;
  std::vector<Timed> pending;
  std::vector<cudaEvent_t> event_pool;
  double prof_ms[PRSGD_KERNEL_FAMILIES] = {0};
  int64_t prof_count[PRSGD_KERNEL_FAMILIES] = {0};
  std::string err;
};
