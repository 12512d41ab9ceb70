// Kernels of libsgdb (sm_100a).
//
//   select_first_n_kernel   which N of the N+b gradients the server keeps
//   stream_rows_kernel      masked mean of the kept rows, fused with the optimizer
//                           rule (or writing the mean), flat or over a segment table
//   update_kernel           optimizer rule from a given mean
//   accumulate_arrival_kernel   one arriving gradient: admit or drop, add, fire at N
//
// The path is a reduction bound by HBM bandwidth (about a quarter of a flop per
// byte), so there are no tensor-core instructions here; what matters is bytes in
// flight per SM, touch-once cache policy and a fixed summation order.
#pragma once

#include "sgdb_device.cuh"

// Programmatic dependent launch for the arrival kernel (one launch per gradient, each
// depending on the one before): measured 52.0 -> 50.3 us per arrival in stream order.
#ifndef SGDB_PDL
#define SGDB_PDL 1
#endif

namespace sgdb {

// ====================================================================== selection
//
// Worker j is valid when tag[j] == t and its arrival time is finite.  The rank of a
// valid worker w is the number of valid workers that arrive before it, where
// "before" compares (arrival time, worker id).  Workers of rank < N are kept;
// order[rank] = w puts them in arrival sequence.
//
// block_select is called by every thread of a block.  Thread i owns workers i,
// i + blockDim.x, ...; keys of valid workers go to shared memory (NaN for the others,
// which never compares as "before"), the valid ones are counted with
// __ballot_sync / __popc, and each thread ranks its own workers with one pass over
// the keys.  A one-warp version that ranked by ballots over register-resident keys
// measured 20 us for W = 100 on a B200 (one warp cannot hide its own latencies);
// this form takes about as long as the load of its inputs.
//
//   s_key   [W] floats of shared memory, s_order [N] ints, s_count one int
//   g_mask / g_order / g_info: global outputs, written only when `writer`
// Time-out rule (keep_all): a worker is valid only if it also arrived by `deadline`,
// and every valid worker is kept; N is then the fewest the caller accepts.
// Returns the number of kept workers (s_order is filled with that many), or 0 when
// fewer than N workers are valid; then nothing but g_info has been written.
__device__ __forceinline__ int block_select(const float* __restrict__ arrival,
                                            const int32_t* __restrict__ tags, int32_t t, int32_t N,
                                            int32_t W, float deadline, bool keep_all, float* s_key,
                                            int* s_order, int* s_count, bool writer,
                                            uint8_t* __restrict__ g_mask, int32_t* __restrict__ g_order,
                                            int32_t* __restrict__ g_info) {
  const int tid = threadIdx.x;
  const int nthreads = blockDim.x;
  if (tid == 0) *s_count = 0;
  __syncthreads();
  const int w_end = (W + 31) & ~31;  // whole warps take part in every ballot
  for (int w = tid; w < w_end; w += nthreads) {
    bool valid = false;
    float a = 0.0f;
    if (w < W) {
      a = arrival[w];
      valid = (tags[w] == t) && isfinite(a) && (a <= deadline);
      s_key[w] = valid ? a : __int_as_float(0x7fc00000);
    }
    const unsigned votes = __ballot_sync(0xffffffffu, valid);
    if ((tid & 31) == 0 && votes != 0) atomicAdd(s_count, __popc(votes));
  }
  __syncthreads();
  const int n_valid = *s_count;
  const bool enough = n_valid >= N;
  if (writer && tid == 0) {
    g_info[0] = n_valid;
    g_info[1] = enough ? SGDB_OK : SGDB_ERR_INSUFFICIENT;
  }
  if (!enough) return 0;
  const int keep = keep_all ? n_valid : N;
  for (int w = tid; w < W; w += nthreads) {
    const float a = s_key[w];
    int rank = 0;
#pragma unroll 8
    for (int j = 0; j < W; ++j) {
      const float aj = s_key[j];
      rank += ((aj < a) || (aj == a && j < w)) ? 1 : 0;
    }
    const bool kept = (a == a) && rank < keep;  // a != a: not valid
    if (kept) s_order[rank] = w;
    if (writer) {
      g_mask[w] = kept ? 1 : 0;
      if (kept) g_order[rank] = w;
    }
  }
  __syncthreads();
  return keep;
}

__global__ void __launch_bounds__(1024) select_first_n_kernel(const float* __restrict__ arrival,
                                                              const int32_t* __restrict__ tags,
                                                              int32_t t, int32_t N, int32_t W,
                                                              float deadline, bool keep_all,
                                                              uint8_t* __restrict__ mask,
                                                              int32_t* __restrict__ order,
                                                              int32_t* __restrict__ info) {
  __shared__ float s_key[SGDB_MAX_WORKERS];
  __shared__ int s_order[SGDB_MAX_WORKERS];
  __shared__ int s_count;
  block_select(arrival, tags, t, N, W, deadline, keep_all, s_key, s_order, &s_count, true, mask, order, info);
}

// ---------------------------------------------------------------------- two-level selection
//
// Workers share machines: group[w] in [0, M).  A machine's message counts when the machine
// has at least one worker and every one of its workers is valid (tag == t, finite arrival); it
// arrives when its slowest worker does.  Machines are ranked like workers above, by (message
// arrival, machine id); the first N are kept.  The rows that will be added are the workers of
// the kept machines, machine by machine in message order and, within a machine, in (arrival,
// id) order: s_order[gend[r] .. gend[r + 1]) are the rows of the machine of rank r.
//
// Finite floats are mapped to unsigned integers of the same order so that the latest arrival
// of a machine is one shared-memory atomicMax per worker; 0 is below every mapped value.
__device__ __forceinline__ unsigned ordered_bits(float a) {
  const unsigned u = __float_as_uint(a);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(unsigned u) {
  return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}

// Inclusive scan of a[1..n] in place by the first warp (a[0] stays): a[i] <- a[1] + ... + a[i].
__device__ __forceinline__ void warp_scan_in_place(int* a, int n) {
  const int lane = threadIdx.x & 31;
  int carry = 0;
  for (int base = 1; base <= n; base += 32) {
    const int idx = base + lane;
    int v = idx <= n ? a[idx] : 0;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, v, d);
      if (lane >= d) v += up;
    }
    v += carry;
    if (idx <= n) a[idx] = v;
    carry = __shfl_sync(0xffffffffu, v, 31);
  }
}

//   s_key [W] floats, s_order [W] ints, s_gkey [M] words, s_gcnt / s_gbad / s_grank [M] ints,
//   s_gend [N + 1] ints, s_count [2] ints; global outputs are written only when `writer`.
// Returns the number of rows to add (s_order holds that many, s_gend their split by machine), or
// 0 when fewer than N machines count or a machine id is out of range; then only g_info is written:
// {machines that count, status, rows used}.
__device__ __forceinline__ int block_select_grouped(const float* __restrict__ arrival, const int32_t* __restrict__ tags,
                                                    const int32_t* __restrict__ group, int32_t t, int32_t N, int32_t W,
                                                    int32_t M, float* s_key, int* s_order, unsigned* s_gkey,
                                                    int* s_gcnt, int* s_gbad, int* s_grank, int* s_gend, int* s_count,
                                                    bool writer, uint8_t* __restrict__ g_mask,
                                                    int32_t* __restrict__ g_group_order, int32_t* __restrict__ g_order,
                                                    int32_t* __restrict__ g_info) {
  const int tid = threadIdx.x;
  const int nthreads = blockDim.x;
  for (int g = tid; g < M; g += nthreads) {
    s_gkey[g] = 0u;
    s_gcnt[g] = 0;
    s_gbad[g] = 0;
  }
  if (tid == 0) {
    s_count[0] = 0;  // machines that count
    s_count[1] = 0;  // a machine id out of range was seen
  }
  __syncthreads();
  for (int w = tid; w < W; w += nthreads) {
    const int g = group[w];
    const float a = arrival[w];
    s_key[w] = a;
    if (g < 0 || g >= M) {
      s_count[1] = 1;
    } else if (tags[w] == t && isfinite(a)) {
      atomicMax(&s_gkey[g], ordered_bits(a));
      atomicAdd(&s_gcnt[g], 1);
    } else {
      s_gbad[g] = 1;
    }
  }
  __syncthreads();
  if (s_count[1] != 0) {
    if (writer && tid == 0) {
      g_info[0] = 0;
      g_info[1] = SGDB_ERR_INVALID_ARG;
      g_info[2] = 0;
    }
    return 0;
  }
  float* s_gtime = reinterpret_cast<float*>(s_gkey);  // same words, now the message's arrival time
  const int m_end = (M + 31) & ~31;
  for (int g = tid; g < m_end; g += nthreads) {
    bool counts = false;
    if (g < M) {
      counts = s_gcnt[g] > 0 && s_gbad[g] == 0;
      s_gtime[g] = counts ? from_ordered_bits(s_gkey[g]) : __int_as_float(0x7fc00000);
    }
    const unsigned votes = __ballot_sync(0xffffffffu, counts);
    if ((tid & 31) == 0 && votes != 0) atomicAdd(&s_count[0], __popc(votes));
  }
  __syncthreads();
  const int n_valid = s_count[0];
  const bool enough = n_valid >= N;
  if (!enough) {
    if (writer && tid == 0) {
      g_info[0] = n_valid;
      g_info[1] = SGDB_ERR_INSUFFICIENT;
      g_info[2] = 0;
    }
    return 0;
  }
  for (int g = tid; g < M; g += nthreads) {
    const float a = s_gtime[g];
    int rank = 0;
#pragma unroll 8
    for (int j = 0; j < M; ++j) {
      const float aj = s_gtime[j];
      rank += ((aj < a) || (aj == a && j < g)) ? 1 : 0;
    }
    const bool kept = (a == a) && rank < N;
    s_grank[g] = kept ? rank : -1;
    if (kept) {
      s_gend[rank + 1] = s_gcnt[g];
      if (writer) g_group_order[rank] = g;
    }
  }
  if (tid == 0) s_gend[0] = 0;
  __syncthreads();
  if (tid < 32) warp_scan_in_place(s_gend, N);
  __syncthreads();
  for (int w = tid; w < W; w += nthreads) {
    const int g = group[w];
    const int r = s_grank[g];
    if (r >= 0) {
      const float a = s_key[w];
      int before = 0;
      for (int j = 0; j < W; ++j) {
        const float aj = s_key[j];
        before += (group[j] == g && ((aj < a) || (aj == a && j < w))) ? 1 : 0;
      }
      const int pos = s_gend[r] + before;
      s_order[pos] = w;
      if (writer) g_order[pos] = w;
    }
    if (writer) g_mask[w] = r >= 0 ? 1 : 0;
  }
  __syncthreads();
  const int n_rows = s_gend[N];
  if (writer && tid == 0) {
    g_info[0] = n_valid;
    g_info[1] = SGDB_OK;
    g_info[2] = n_rows;
  }
  return n_rows;
}

__global__ void __launch_bounds__(1024) select_grouped_kernel(const float* __restrict__ arrival,
                                                              const int32_t* __restrict__ tags,
                                                              const int32_t* __restrict__ group, int32_t t, int32_t N,
                                                              int32_t W, int32_t M, uint8_t* __restrict__ mask,
                                                              int32_t* __restrict__ group_order,
                                                              int32_t* __restrict__ order, int32_t* __restrict__ info) {
  __shared__ float s_key[SGDB_MAX_WORKERS];
  __shared__ int s_order[SGDB_MAX_WORKERS];
  __shared__ unsigned s_gkey[SGDB_MAX_WORKERS];
  __shared__ int s_gcnt[SGDB_MAX_WORKERS], s_gbad[SGDB_MAX_WORKERS], s_grank[SGDB_MAX_WORKERS];
  __shared__ int s_gend[SGDB_MAX_WORKERS + 1];
  __shared__ int s_count[2];
  block_select_grouped(arrival, tags, group, t, N, W, M, s_key, s_order, s_gkey, s_gcnt, s_gbad, s_grank, s_gend, s_count,
                       true, mask, group_order, order, info);
}

// ====================================================================== row streaming
//
// Persistent blocks walk over column tiles of TILE = NT*CH*V columns.  For a tile,
// the N kept rows are added in order[] sequence into fp32 registers; then the tile's
// slice of theta and optimizer state is updated (or the mean is stored).
//
// Row slices reach shared memory through a ring of `stages` buffers filled by 1-D
// bulk async copies issued by one producer thread; each buffer has a "full"
// mbarrier (armed with the byte count, completed by the copy engine) and an "empty"
// mbarrier (one arrival per consumer warp).  The ring keeps running across tiles, so
// the next tile's rows are already in flight while this tile's epilogue runs.
//
// Bulk copies need 16-byte aligned addresses and sizes.  A segment whose gradient
// base or row pitch is not 16-byte aligned is read with ordinary element loads by
// the consumers instead; the additions happen in the same order either way.  With
// an aligned pitch the last 16-byte chunk of a ragged tile is copied whole: the
// columns between len and the next multiple of 16 bytes are padding inside the row
// pitch (or at least inside the same 16-byte block as the last valid element), they
// are read and never used.

struct StreamParams {
  const sgdb_segment_t* table;  // device segment table, or nullptr: use `flat`
  sgdb_segment_t flat;          // with EP_MEAN, flat.theta is where the mean goes
  int S;                        // entries in `table`
  int total_tiles;              // flat case: number of TILE-wide tiles (tables: counted in the kernel)
  int N;                        // rows to add
  int stages;                   // ring depth
  const int32_t* order;         // [N] row ids in summation order (when the selection is given)
  const int32_t* info;          // optional [2]; info[1] != SGDB_OK: do nothing
  int32_t* status_out;          // optional: receives SGDB_ERR_TIMEOUT if a wait runs out, or
                                // SGDB_ERR_INVALID_ARG for an incomplete segment table entry
  // When `arrival` is not null the kernel takes the selection itself: every block
  // ranks the W workers in its prologue (the same deterministic result in each) and
  // block 0 writes mask_out, order_out and info_out.
  const float* arrival;
  const int32_t* tags;
  int32_t t;
  int32_t W;
  float deadline;   // time-out rule: arrival <= deadline (first-N rule: +infinity)
  bool keep_all;    // time-out rule: keep every valid worker, N is the fewest accepted
  int order_cap;    // ints of shared memory reserved for order[]: N, or W with keep_all
  uint8_t* mask_out;
  int32_t* order_out;
  int32_t* info_out;
  // Two-level aggregation (GROUPED kernels): worker w runs on machine group[w] in [0, M); N counts
  // machines, W workers; the kept machines go to group_order_out [N], info_out has 3 words.
  const int32_t* group;
  int32_t M;
  int32_t* group_order_out;
  // Optional: exponential moving average of the parameters, updated in the same pass from the
  // value theta had BEFORE this step's update.  Flat case: `ema`; with a segment table:
  // `ema_table` [S] device pointers, one per tensor (a null entry: that tensor keeps no average).
  float* ema;
  float* const* ema_table;
  float ema_alpha, ema_one_minus_alpha;
  // Rows by address (ROWS kernels): the gradient of worker w starts at rows[w] (W_rows entries, this GPU's
  // memory or a peer's, mapped into this process) instead of at flat.grad + w * ld; column i of this server's
  // shard is element i of every row, of flat.theta and of the state.  The new parameters are also stored to
  // replicas[0 .. R): the copies of this shard that the workers read (this GPU's or a peer's memory).
  const void* const* rows;
  int32_t W_rows;
  float* const* replicas;
  int32_t R;
  unsigned long long wait_limit_ns;  // patience of every wait on a ring barrier (see mbar_wait_for)
  // Tiles are walked from the last to the first instead of from the first to the last.  Callers alternate it
  // from one iteration to the next (the parity of t), so that a launch starts with the parameters and state
  // its predecessor wrote last, which are still in L2.  The order of tiles never changes a result.
  int reverse;
  Hyper h;
};

template <typename GT>
struct TileDesc {
  const GT* grad;  // row 0 of this tile's columns
  float* theta;    // this tile's slice (mean output for EP_MEAN)
  float* ema;      // this tile's slice of the averaged parameters, or nullptr
  float* s0;
  float* s1;
  long long ld;
  int ncols;      // valid columns in the tile
  int bulk_cols;  // leading columns delivered by bulk copy (0: none); may exceed ncols by the row's padding
  bool vec_ok;    // theta/state slices may be accessed 16 bytes at a time
  bool bad;       // a pointer this rule needs is null in the segment table: the tile is skipped
};

// A table entry the kernel may use: the pointers its rule needs are there and aligned to their
// element type, and the rows do not overlap (ld >= len).  The table lives in device memory, so the
// host cannot check it; an entry that fails is left alone and reported instead of being dereferenced.
template <typename GT, int EP>
__device__ __forceinline__ bool segment_usable(const sgdb_segment_t& seg, const float* ema) {
  using Rule = RuleTraits<EP>;
  if (seg.theta == nullptr || seg.grad == nullptr || (Rule::kState0 && seg.state0 == nullptr) ||
      (Rule::kState1 && seg.state1 == nullptr))
    return false;
  const uintptr_t fp32_ptrs = reinterpret_cast<uintptr_t>(seg.theta) | reinterpret_cast<uintptr_t>(seg.state0) |
                              reinterpret_cast<uintptr_t>(seg.state1) | reinterpret_cast<uintptr_t>(ema);
  if ((fp32_ptrs & 3u) != 0 || (reinterpret_cast<uintptr_t>(seg.grad) & (sizeof(GT) - 1)) != 0) return false;
  return seg.ld >= seg.len;
}

template <typename GT, int TILE, int EP>
__device__ __forceinline__ TileDesc<GT> locate_tile(const StreamParams& p, const int* prefix_s,
                                                    int tile) {
  constexpr int V = GradTraits<GT>::kVec;
  sgdb_segment_t seg;
  long long col0;
  float* ema = p.ema;
  if (p.table == nullptr) {
    seg = p.flat;
    col0 = static_cast<long long>(tile) * TILE;
  } else {
    int lo = 0, hi = p.S;  // first index whose prefix exceeds `tile`, minus one
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (prefix_s[mid + 1] > tile) hi = mid; else lo = mid + 1;
    }
    seg = p.table[lo];
    col0 = static_cast<long long>(tile - prefix_s[lo]) * TILE;
    ema = p.ema_table != nullptr ? p.ema_table[lo] : nullptr;
  }
  TileDesc<GT> td;
  td.grad = static_cast<const GT*>(seg.grad) + col0;
  td.theta = static_cast<float*>(seg.theta) + col0;
  td.s0 = seg.state0 ? static_cast<float*>(seg.state0) + col0 : nullptr;
  td.s1 = seg.state1 ? static_cast<float*>(seg.state1) + col0 : nullptr;
  td.ld = seg.ld;
  const long long rest = seg.len - col0;
  td.ncols = rest < TILE ? static_cast<int>(rest) : TILE;
  const bool bulk_ok = ((reinterpret_cast<uintptr_t>(seg.grad) & 15u) == 0) &&
                       (((seg.ld * static_cast<long long>(sizeof(GT))) & 15) == 0);
  // A 16-byte aligned row pitch leaves room for the whole last 16-byte chunk of a ragged tile (ld is a multiple
  // of V and ld >= len): the copy takes it along, padding included; lanes beyond ncols are never stored.
  td.bulk_cols = bulk_ok ? ((td.ncols + V - 1) / V) * V : 0;
  td.bad = false;
  td.ema = ema != nullptr ? ema + col0 : nullptr;
  td.vec_ok = (((reinterpret_cast<uintptr_t>(seg.theta) | reinterpret_cast<uintptr_t>(seg.state0) |
                 reinterpret_cast<uintptr_t>(seg.state1) | reinterpret_cast<uintptr_t>(ema)) & 15u) == 0);
  if (p.table != nullptr && !segment_usable<GT, EP>(seg, ema)) {
    td.bad = true;
    td.ncols = 0;
    td.bulk_cols = 0;
  }
  return td;
}

// GROUPED: the kept rows fall into runs (one per kept machine); every run is summed on its own,
// divided by its length, and the runs' means are added in sequence and divided by their number.
// ROWS: every row has an address of its own (a table of pointers, peers' memory allowed) and the new
// parameters are also stored to a list of replicas; this is the form a parameter server takes when the
// workers' gradients live in other GPUs' memory: it pulls its columns of the kept rows with the same
// bulk copies (never multicast) and pushes its shard of theta back with ordinary stores.  No block
// waits for another GPU: the caller orders the launches of different GPUs (gradients complete before,
// replicas complete after).
template <typename GT, int EP, int NT, int CH, bool GROUPED = false, bool ROWS = false>
__global__ void __launch_bounds__(NT + 32, 2) stream_rows_kernel(const StreamParams p) {
  using Tr = GradTraits<GT>;
  using Rule = RuleTraits<EP>;
  constexpr int V = Tr::kVec;
  constexpr int TILE = NT * CH * V;
  constexpr uint32_t STAGE_BYTES = TILE * sizeof(GT);
  constexpr int NW = NT / 32;

  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_abort;
  __shared__ int s_count;
  __shared__ unsigned s_issued;      // copies the producer has issued so far (read only after a wait ran out)
  __shared__ int s_producer_done;    // the producer has left its loop and issues nothing more

  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int stages = p.stages;
  int N = p.N;  // rows to add; with the time-out rule the selection below decides it
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + static_cast<size_t>(stages) * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + stages;
  // ROWS: the kept rows' addresses in summation order, then the replicas' addresses
  uint64_t* after_bars = empty_bar + stages;
  const GT** rowptr_s = reinterpret_cast<const GT**>(after_bars);
  float** repl_s = reinterpret_cast<float**>(after_bars + (ROWS ? p.order_cap : 0));
  int* order_s = reinterpret_cast<int*>(after_bars + (ROWS ? p.order_cap + p.R : 0));
  int* prefix_s = order_s + ((p.order_cap + 3) & ~3);
  float* key_s = reinterpret_cast<float*>(prefix_s + (p.table != nullptr ? p.S + 1 : 0));
  int* gend_s = nullptr;  // GROUPED: rows of the machine of rank r are order_s[gend_s[r] .. gend_s[r + 1])
  int n_div = N;          // what the sum is divided by in the end

  if constexpr (GROUPED) {
    unsigned* gkey_s = reinterpret_cast<unsigned*>(key_s + p.W);
    int* gcnt_s = reinterpret_cast<int*>(gkey_s + p.M);
    int* gbad_s = gcnt_s + p.M;
    int* grank_s = gbad_s + p.M;
    gend_s = grank_s + p.M;
    __shared__ int s_gcount[2];
    N = block_select_grouped(p.arrival, p.tags, p.group, p.t, p.N, p.W, p.M, key_s, order_s, gkey_s, gcnt_s, gbad_s,
                             grank_s, gend_s, s_gcount, blockIdx.x == 0, p.mask_out, p.group_order_out, p.order_out,
                             p.info_out);
    if (N == 0) return;
    n_div = p.N;
  } else if (p.arrival != nullptr) {
    // fewer than N current gradients: the iteration cannot complete, nothing is touched
    N = block_select(p.arrival, p.tags, p.t, N, p.W, p.deadline, p.keep_all, key_s, order_s, &s_count,
                     blockIdx.x == 0, p.mask_out, p.order_out, p.info_out);
    if (N == 0) return;
    n_div = N;
  } else {
    if (p.info != nullptr && p.info[1] != SGDB_OK) return;
    for (int i = tid; i < N; i += NT + 32) order_s[i] = p.order[i];
  }
  bool rows_bulk = false;   // ROWS: every kept row starts on a 16-byte boundary
  bool repl_vec = true;     // ROWS: every replica starts on a 16-byte boundary
  if constexpr (ROWS) {
    __syncthreads();  // order_s is complete
    // bit 0: an address or a row id the kernel must not use; bit 1: a row off the 16-byte grid;
    // bit 2: a replica off the 16-byte grid
    int flags = 0;
    for (int k = tid; k < N; k += NT + 32) {
      const int w = order_s[k];
      const GT* row = nullptr;
      if (w >= 0 && w < p.W_rows) row = static_cast<const GT*>(p.rows[w]);
      rowptr_s[k] = row;
      const uintptr_t a = reinterpret_cast<uintptr_t>(row);
      if (row == nullptr || (a & (sizeof(GT) - 1)) != 0) flags |= 1;
      if ((a & 15u) != 0) flags |= 2;
    }
    for (int r = tid; r < p.R; r += NT + 32) {
      float* dst = p.replicas[r];
      repl_s[r] = dst;
      const uintptr_t a = reinterpret_cast<uintptr_t>(dst);
      if (dst == nullptr || (a & 3u) != 0) flags |= 1;
      if ((a & 15u) != 0) flags |= 4;
    }
    const bool unusable = __syncthreads_or(flags & 1) != 0;  // (the call returns a truth value, not the bits)
    rows_bulk = __syncthreads_or(flags & 2) == 0;
    repl_vec = __syncthreads_or(flags & 4) == 0;
    if (unusable) {  // nothing is touched; every block takes the same decision
      if (blockIdx.x == 0 && tid == 0 && p.status_out != nullptr) *p.status_out = SGDB_ERR_INVALID_ARG;
      return;
    }
  }
  if (tid == 0) {
    s_abort = 0;
    s_issued = 0u;
    s_producer_done = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_addr(full_bar + s), 1);
      mbar_init(smem_addr(empty_bar + s), NW);
    }
    fence_barrier_init();
  }
  if (p.table != nullptr) {
    // tiles per segment, then an inclusive scan: prefix_s[i] = tiles in segments < i
    // The same pass looks for entries the kernel must not use (a missing or misaligned pointer,
    // rows that overlap); their tiles are skipped below and block 0 reports them once.
    int incomplete = 0;
    for (int i = tid; i < p.S; i += NT + 32) {
      const sgdb_segment_t seg = p.table[i];
      prefix_s[i + 1] = seg.len > 0 ? static_cast<int>((seg.len + TILE - 1) / TILE) : 0;
      if (seg.len > 0 && !segment_usable<GT, EP>(seg, p.ema_table != nullptr ? p.ema_table[i] : nullptr)) incomplete = 1;
    }
    if (tid == 0) prefix_s[0] = 0;
    incomplete = __syncthreads_or(incomplete);
    if (incomplete && blockIdx.x == 0 && tid == 0 && p.status_out != nullptr) *p.status_out = SGDB_ERR_INVALID_ARG;
    if (tid < 32) {
      int carry = 0;
      for (int base = 1; base <= p.S; base += 32) {
        const int idx = base + lane;
        int v = idx <= p.S ? prefix_s[idx] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int up = __shfl_up_sync(0xffffffffu, v, d);
          if (lane >= d) v += up;
        }
        v += carry;
        if (idx <= p.S) prefix_s[idx] = v;
        carry = __shfl_sync(0xffffffffu, v, 31);
      }
    }
  }
  __syncthreads();
  const int total_tiles = p.table != nullptr ? prefix_s[p.S] : p.total_tiles;
  const uint32_t ring_addr = smem_addr(smem);
  const uint32_t full_addr = smem_addr(full_bar);
  const uint32_t empty_addr = smem_addr(empty_bar);
  bool timed_out = false;

  if (tid >= NT) {
    // ------------------------------------------------------------ producer (one thread)
    if (tid == NT) {
      const uint64_t policy = l2_policy_evict_first();  // rows are read exactly once
      int s = 0;
      uint32_t phase = 0;
      unsigned issued = 0u;
      for (int slot_tile = blockIdx.x; slot_tile < total_tiles && !timed_out; slot_tile += gridDim.x) {
        const int tile = p.reverse ? total_tiles - 1 - slot_tile : slot_tile;
        TileDesc<GT> td = locate_tile<GT, TILE, EP>(p, prefix_s, tile);
        if constexpr (ROWS) td.bulk_cols = rows_bulk ? (td.ncols / V) * V : 0;  // whole 16-byte chunks only
        if (td.bulk_cols == 0) continue;
        const uint32_t bytes = static_cast<uint32_t>(td.bulk_cols) * sizeof(GT);
        for (int k = 0; k < N; ++k) {
          if (!mbar_wait_for(empty_addr + 8u * s, phase ^ 1u, &s_abort, p.wait_limit_ns)) {
            timed_out = true;
            break;
          }
          const GT* src = ROWS ? rowptr_s[k] + static_cast<long long>(tile) * TILE
                               : td.grad + static_cast<long long>(order_s[k]) * td.ld;
          mbar_arrive_expect_tx(full_addr + 8u * s, bytes);
          bulk_copy_g2s(ring_addr + static_cast<uint32_t>(s) * STAGE_BYTES, src, bytes,
                        full_addr + 8u * s, policy);
          ++issued;
          if (++s == stages) {
            s = 0;
            phase ^= 1u;
          }
        }
      }
      // what a consumer needs to know if it has to wait for copies still in flight after a wait ran out
      *reinterpret_cast<volatile unsigned*>(&s_issued) = issued;
      __threadfence_block();
      *reinterpret_cast<volatile int*>(&s_producer_done) = 1;
    }
  } else {
    // ------------------------------------------------------------ consumers
    const float n_as_float = static_cast<float>(n_div);
    constexpr bool kKeepState = sizeof(GT) == 4 && EP != EP_MEAN;
    const uint64_t pol_keep = kKeepState ? l2_policy_evict_last() : 0ull;
    int s = 0;
    uint32_t phase = 0;
    for (int slot_tile = blockIdx.x; slot_tile < total_tiles && !timed_out; slot_tile += gridDim.x) {
      const int tile = p.reverse ? total_tiles - 1 - slot_tile : slot_tile;
      TileDesc<GT> td = locate_tile<GT, TILE, EP>(p, prefix_s, tile);
      if constexpr (ROWS) {
        td.bulk_cols = rows_bulk ? (td.ncols / V) * V : 0;
        td.vec_ok = td.vec_ok && repl_vec;
      }

      float acc[CH][V];
#pragma unroll
      for (int c = 0; c < CH; ++c)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[c][e] = 0.0f;

      // columns of this thread that the bulk copy did not deliver (ragged end, unaligned
      // segment) are read straight from global memory, row by row, in the same order
      auto add_row_tail = [&](int k) {
        const GT* row = ROWS ? rowptr_s[k] + static_cast<long long>(tile) * TILE
                             : td.grad + static_cast<long long>(order_s[k]) * td.ld;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const int o = (tid + c * NT) * V;
          if (o + V > td.bulk_cols && o < td.ncols) {
#pragma unroll
            for (int e = 0; e < V; ++e)
              if (o + e < td.ncols) acc[c][e] = __fadd_rn(acc[c][e], Tr::widen(row[o + e]));
          }
        }
      };
      const bool has_tail = td.bulk_cols < td.ncols;

      if (td.bad) continue;  // reported by block 0 in the prologue

      // adds rows order_s[k .. k_end) into acc, in that sequence; false when a wait ran out
      auto add_rows = [&](int k, const int k_end) -> bool {
        if (td.bulk_cols == 0) {
          for (; k < k_end; ++k) add_row_tail(k);
          return true;
        }
        // two rows per pass: both slots are waited for and read before the dependent adds
        for (; k + 1 < k_end; k += 2) {
          const int sa = s;
          const uint32_t pa = phase;
          if (++s == stages) {
            s = 0;
            phase ^= 1u;
          }
          const int sb = s;
          const uint32_t pb = phase;
          if (++s == stages) {
            s = 0;
            phase ^= 1u;
          }
          if (!mbar_wait_for(full_addr + 8u * sa, pa, &s_abort, p.wait_limit_ns) ||
              !mbar_wait_for(full_addr + 8u * sb, pb, &s_abort, p.wait_limit_ns))
            return false;
          const unsigned char* stage_a = smem + static_cast<size_t>(sa) * STAGE_BYTES;
          const unsigned char* stage_b = smem + static_cast<size_t>(sb) * STAGE_BYTES;
          uint4 va[CH], vb[CH];
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            const int o = (tid + c * NT) * V;
            if (o + V <= td.bulk_cols) {
              va[c] = *reinterpret_cast<const uint4*>(stage_a + static_cast<size_t>(o) * sizeof(GT));
              vb[c] = *reinterpret_cast<const uint4*>(stage_b + static_cast<size_t>(o) * sizeof(GT));
            }
          }
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            const int o = (tid + c * NT) * V;
            if (o + V <= td.bulk_cols) {
              float x[V];
              Tr::unpack(va[c], x);
#pragma unroll
              for (int e = 0; e < V; ++e) acc[c][e] = __fadd_rn(acc[c][e], x[e]);
              Tr::unpack(vb[c], x);
#pragma unroll
              for (int e = 0; e < V; ++e) acc[c][e] = __fadd_rn(acc[c][e], x[e]);
            }
          }
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(empty_addr + 8u * sa);
            mbar_arrive(empty_addr + 8u * sb);
          }
          if (has_tail) {
            add_row_tail(k);
            add_row_tail(k + 1);
          }
        }
        if (k < k_end) {  // an odd count: the last row on its own
          if (!mbar_wait_for(full_addr + 8u * s, phase, &s_abort, p.wait_limit_ns)) return false;
          const unsigned char* stage = smem + static_cast<size_t>(s) * STAGE_BYTES;
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            const int o = (tid + c * NT) * V;
            if (o + V <= td.bulk_cols) {
              const uint4 v = *reinterpret_cast<const uint4*>(stage + static_cast<size_t>(o) * sizeof(GT));
              float x[V];
              Tr::unpack(v, x);
#pragma unroll
              for (int e = 0; e < V; ++e) acc[c][e] = __fadd_rn(acc[c][e], x[e]);
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_addr + 8u * s);
          if (++s == stages) {
            s = 0;
            phase ^= 1u;
          }
          if (has_tail) add_row_tail(k);
        }
        return true;
      };

      if constexpr (GROUPED) {
        float total[CH][V];
#pragma unroll
        for (int c = 0; c < CH; ++c)
#pragma unroll
          for (int e = 0; e < V; ++e) total[c][e] = 0.0f;
        for (int r = 0; r < n_div; ++r) {
          const int k0 = gend_s[r], k1 = gend_s[r + 1];
          if (!add_rows(k0, k1)) {
            timed_out = true;
            break;
          }
          const float members = static_cast<float>(k1 - k0);
#pragma unroll
          for (int c = 0; c < CH; ++c)
#pragma unroll
            for (int e = 0; e < V; ++e) {
              total[c][e] = __fadd_rn(total[c][e], __fdiv_rn(acc[c][e], members));  // this machine's message
              acc[c][e] = 0.0f;
            }
        }
#pragma unroll
        for (int c = 0; c < CH; ++c)
#pragma unroll
          for (int e = 0; e < V; ++e) acc[c][e] = total[c][e];
      } else {
        if (!add_rows(0, N)) timed_out = true;
      }
      if (timed_out) break;

#pragma unroll
      for (int c = 0; c < CH; ++c) {
        const int o = (tid + c * NT) * V;
        const int n = td.ncols - o;
        if (n > 0) {
          const bool vec = td.vec_ok && n >= V;
          float g[V];
#pragma unroll
          for (int e = 0; e < V; ++e) g[e] = __fdiv_rn(acc[c][e], n_as_float);
          if (EP == EP_MEAN) {
            store_floats<V>(td.theta + o, vec, n, g);
          } else {
            // theta and state are loaded here, not ahead of the row loop: holding them in
            // registers through the loop measured no faster for fp32 rows and slower for bf16
            // rows (spills at two resident blocks); the other block on the SM and the ring,
            // which keeps filling, cover this latency
            // With fp32 rows the parameters and state are loaded and stored evict-last: together with the
            // alternating tile order, the slices written at the end of one iteration are found in L2 at the
            // start of the next (C1: 1.414 -> 1.396 ms; either measure alone gains a third of that or loses).
            // With bf16 rows the same policy costs 1 % (the kernel is short of registers): streaming accesses.
            float th[V], s0[V], s1[V];
            if constexpr (kKeepState) {
              if (Rule::kTheta) load_floats_hint<V>(td.theta + o, vec, n, th, pol_keep);
              if (Rule::kState0) load_floats_hint<V>(td.s0 + o, vec, n, s0, pol_keep);
              if (Rule::kState1) load_floats_hint<V>(td.s1 + o, vec, n, s1, pol_keep);
            } else {
              if (Rule::kTheta) load_floats<V>(td.theta + o, vec, n, th);
              if (Rule::kState0) load_floats<V>(td.s0 + o, vec, n, s0);
              if (Rule::kState1) load_floats<V>(td.s1 + o, vec, n, s1);
            }
            if (td.ema != nullptr) {
              float avg[V];
              load_floats<V>(td.ema + o, vec, n, avg);
#pragma unroll
              for (int e = 0; e < V; ++e) avg[e] = ema_rule(p.ema_alpha, p.ema_one_minus_alpha, avg[e], th[e]);
              store_floats<V>(td.ema + o, vec, n, avg);
            }
#pragma unroll
            for (int e = 0; e < V; ++e) apply_rule<EP>(p.h, g[e], th[e], s0[e], s1[e]);
            if constexpr (kKeepState) {
              store_floats_hint<V>(td.theta + o, vec, n, th, pol_keep);
              if (Rule::kState0) store_floats_hint<V>(td.s0 + o, vec, n, s0, pol_keep);
              if (Rule::kState1) store_floats_hint<V>(td.s1 + o, vec, n, s1, pol_keep);
            } else {
              store_floats<V>(td.theta + o, vec, n, th);
              if (Rule::kState0) store_floats<V>(td.s0 + o, vec, n, s0);
              if (Rule::kState1) store_floats<V>(td.s1 + o, vec, n, s1);
            }
            if constexpr (ROWS) {  // the workers' copies of this shard
              for (int r = 0; r < p.R; ++r)
                store_floats<V>(repl_s[r] + static_cast<long long>(tile) * TILE + o, vec, n, th);
            }
          }
        }
      }
    }
  }
  if (timed_out && p.status_out != nullptr) *p.status_out = SGDB_ERR_TIMEOUT;
  // A wait ran out somewhere in this block.  Copies the producer has issued may still be on their way into this
  // block's shared memory, which the next block on this SM will own: thread 0 stays until they have landed.  The
  // producer stops at its next wait (it sees the abort flag) and then publishes how many copies it issued; the
  // most recent copy into each ring slot is the one whose barrier phase may still be open.  These waits have a
  // patience of their own: the copies were issued to valid addresses and land within microseconds.
  if (tid == 0 && *reinterpret_cast<volatile int*>(&s_abort) != 0) {
    const unsigned long long give_up = global_timer_ns() + kWaitLimitNs;
    while (*reinterpret_cast<volatile int*>(&s_producer_done) == 0 && global_timer_ns() < give_up) {
    }
    __threadfence_block();
    const unsigned issued = *reinterpret_cast<volatile unsigned*>(&s_issued);
    const unsigned first = issued > static_cast<unsigned>(stages) ? issued - static_cast<unsigned>(stages) : 0u;
    for (unsigned i = first; i < issued; ++i) {
      const uint32_t bar = full_addr + 8u * (i % static_cast<unsigned>(stages));
      const uint32_t parity = (i / static_cast<unsigned>(stages)) & 1u;
      while (!mbar_try_wait(bar, parity) && global_timer_ns() < give_up) {
      }
    }
  }
}

// ====================================================================== update from a mean

struct UpdateParams {
  float* theta;
  float* s0;
  float* s1;
  const float* mean;
  long long P;
  const int32_t* info;
  Hyper h;
};

template <int EP>
__global__ void __launch_bounds__(256) update_kernel(const UpdateParams p) {
  using Rule = RuleTraits<EP>;
  if (p.info != nullptr && p.info[1] != SGDB_OK) return;
  const long long chunks = (p.P + 3) / 4;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  constexpr int U = 2;  // two chunks per thread and pass, all loads issued before the arithmetic
  for (long long q0 = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; q0 < chunks; q0 += stride * U) {
    float g[U][4], th[U][4], s0[U][4], s1[U][4];
    int n[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long q = q0 + u * stride;
      const long long i = q * 4;
      const long long rest = p.P - i;
      n[u] = q < chunks ? (rest < 4 ? static_cast<int>(rest) : 4) : 0;
      if (n[u] > 0) {
        const bool vec = n[u] == 4;
        load_floats<4>(p.mean + i, vec, n[u], g[u]);
        load_floats<4>(p.theta + i, vec, n[u], th[u]);
        if (Rule::kState0) load_floats<4>(p.s0 + i, vec, n[u], s0[u]);
        if (Rule::kState1) load_floats<4>(p.s1 + i, vec, n[u], s1[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (n[u] > 0) {
        const long long i = (q0 + u * stride) * 4;
        const bool vec = n[u] == 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) apply_rule<EP>(p.h, g[u][e], th[u][e], s0[u][e], s1[u][e]);
        store_floats<4>(p.theta + i, vec, n[u], th[u]);
        if (Rule::kState0) store_floats<4>(p.s0 + i, vec, n[u], s0[u]);
        if (Rule::kState1) store_floats<4>(p.s1 + i, vec, n[u], s1[u]);
      }
    }
  }
}

// ====================================================================== parameter average alone

struct EmaParams {
  float* ema;
  const float* theta;
  long long P;
  float alpha, one_minus_alpha;
  const int32_t* info;
};

__global__ void __launch_bounds__(256) ema_kernel(const EmaParams p) {
  if (p.info != nullptr && p.info[1] != SGDB_OK) return;
  const long long chunks = (p.P + 3) / 4;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long q = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; q < chunks; q += stride) {
    const long long i = q * 4;
    const long long rest = p.P - i;
    const int n = rest < 4 ? static_cast<int>(rest) : 4;
    const bool vec = n == 4;
    float avg[4], th[4];
    load_floats<4>(p.ema + i, vec, n, avg);
    load_floats<4>(p.theta + i, vec, n, th);
#pragma unroll
    for (int e = 0; e < 4; ++e) avg[e] = ema_rule(p.alpha, p.one_minus_alpha, avg[e], th[e]);
    store_floats<4>(p.ema + i, vec, n, avg);
  }
}

// ====================================================================== one arrival
//
// Every block reads the server state {accepted, seen, ticket, lowest open iteration}
// before doing anything and takes the same decision from it.  The state is only
// changed by the block that finishes last (it holds the last ticket), i.e. after
// every block has read it, so one launch needs neither a grid-wide barrier nor a
// wait.  The next arrival's launch is ordered after this one by the stream.

struct ArrivalParams {
  const void* row;
  int32_t row_tag, t, N;
  long long P;
  float* acc;
  int32_t* counter;  // [4]
  float* theta;
  float* s0;
  float* s1;
  int32_t* info;  // [2]
  float* ema;     // optional: average of the parameters, moved when the update fires
  float ema_alpha, ema_one_minus_alpha;
  long long acc_resident;  // leading elements of acc that are asked to stay in L2 between launches
  int32_t admissible;      // 0: the host already knows this gradient is dropped (it arrived after the deadline)
  Hyper h;
};

// The running sum is written by one launch and read by the next.  Where it fits, it is kept in
// L2 across launches, by two means.  (1) Consecutive launches walk through the vector in opposite
// directions (forward when an even number of gradients has been accepted, backward when odd), so a
// launch starts with the part of the sum its predecessor wrote last, which is still in L2 whatever
// the policy.  (2) The leading `acc_resident` elements of the sum are loaded and stored with an
// evict-last policy, while the gradient row (read once) and the rest of the sum stream through
// evict-first.  Measured on a B200 at 23.8 M columns, per iteration of 96 gradients: everything
// streaming in one direction 4.80 ms; evict-last loads with streaming stores, one direction 3.70 ms
// (evict-last stores were slower then); alternating directions with streaming accesses 3.44 ms,
// with evict-last loads 3.33 ms, with evict-last loads and stores 3.23 ms.  The launch that
// completes the set reads the sum for the last time and releases it (evict-first).  Direction and
// policies change where the bytes live, never the arithmetic: every element still sees the same
// additions in the same order.
template <typename GT, int EP>
__global__ void __launch_bounds__(256, 4) accumulate_arrival_kernel(const ArrivalParams p) {
  using Tr = GradTraits<GT>;
  using Rule = RuleTraits<EP>;
  constexpr int V = Tr::kVec;
  __shared__ int s_accepted, s_open;
#if SGDB_PDL
  // Launched with programmatic stream serialization: the next arrival's launch may be
  // set up while this one runs, and nothing of the previous launch is read before it
  // has completed and its writes are visible.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
  if (threadIdx.x == 0) {
    s_accepted = *reinterpret_cast<volatile int32_t*>(p.counter + 0);
    s_open = *reinterpret_cast<volatile int32_t*>(p.counter + 3);
  }
  __syncthreads();
  const int accepted = s_accepted;
  const bool admit = p.admissible != 0 && (p.row_tag == p.t) && (p.t >= s_open) && (accepted < p.N);
  const bool first = accepted == 0;          // the set was empty: start the sum from +0
  const bool last = accepted + 1 == p.N;     // this gradient completes the set

  if (admit) {
    const GT* row = static_cast<const GT*>(p.row);
    const bool row_vec = (reinterpret_cast<uintptr_t>(p.row) & 15u) == 0;
    const float n_as_float = static_cast<float>(p.N);
    const long long chunks = (p.P + V - 1) / V;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const long long first_chunk = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const uint64_t pol_keep = l2_policy_evict_last();
    const uint64_t pol_stream = l2_policy_evict_first();
    if (!last) {
      const bool reverse = (accepted & 1) != 0;  // start with the part of the sum the previous launch wrote last
      // U chunks per thread and pass, all loads issued before the first use: enough bytes
      // in flight per SM for a stream that reads two arrays and writes one.
      constexpr int U = 16 / V;  // 64 bytes of the row per thread and pass
      for (long long q0 = first_chunk; q0 < chunks; q0 += stride * U) {
        float x[U][V], a[U][V];
        int n[U];
        long long idx[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const long long q_fwd = q0 + u * stride;
          const long long q = reverse ? chunks - 1 - q_fwd : q_fwd;
          const long long i = q * V;
          const long long rest = p.P - i;
          n[u] = q_fwd < chunks ? (rest < V ? static_cast<int>(rest) : V) : 0;
          idx[u] = i;
          if (n[u] > 0) {
            if (n[u] == V && row_vec) {
              const uint4 v = __ldcs(reinterpret_cast<const uint4*>(row + i));
              Tr::unpack(v, x[u]);
            } else {
#pragma unroll
              for (int e = 0; e < V; ++e) x[u][e] = e < n[u] ? Tr::widen(row[i + e]) : 0.0f;
            }
            if (first) {
#pragma unroll
              for (int e = 0; e < V; ++e) a[u][e] = 0.0f;
            } else {
              load_floats_hint<V>(p.acc + i, n[u] == V, n[u], a[u], i < p.acc_resident ? pol_keep : pol_stream);
            }
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (n[u] > 0) {
#pragma unroll
            for (int e = 0; e < V; ++e) a[u][e] = __fadd_rn(a[u][e], x[u][e]);
            store_floats_hint<V>(p.acc + idx[u], n[u] == V, n[u], a[u], idx[u] < p.acc_resident ? pol_keep : pol_stream);
          }
        }
      }
    } else {
      // the gradient that completes the set: mean and optimizer rule in the same pass
      const bool reverse = (accepted & 1) != 0;  // as above: start where the previous launch stopped writing
      for (long long q_fwd = first_chunk; q_fwd < chunks; q_fwd += stride) {
        const long long q = reverse ? chunks - 1 - q_fwd : q_fwd;
        const long long i = q * V;
        const long long rest = p.P - i;
        const int n = rest < V ? static_cast<int>(rest) : V;
        const bool vec = n == V;
        float x[V], a[V], th[V], s0[V], s1[V];
        if (vec && row_vec) {
          const uint4 v = __ldcs(reinterpret_cast<const uint4*>(row + i));
          Tr::unpack(v, x);
        } else {
#pragma unroll
          for (int e = 0; e < V; ++e) x[e] = e < n ? Tr::widen(row[i + e]) : 0.0f;
        }
        if (first) {
#pragma unroll
          for (int e = 0; e < V; ++e) a[e] = 0.0f;
        } else {
          load_floats_hint<V>(p.acc + i, vec, n, a, pol_stream);  // last use of the sum: let it go
        }
        load_floats<V>(p.theta + i, vec, n, th);
        if (Rule::kState0) load_floats<V>(p.s0 + i, vec, n, s0);
        if (Rule::kState1) load_floats<V>(p.s1 + i, vec, n, s1);
        if (p.ema != nullptr) {  // the average takes in theta as it is before this update
          float avg[V];
          load_floats<V>(p.ema + i, vec, n, avg);
#pragma unroll
          for (int e = 0; e < V; ++e) avg[e] = ema_rule(p.ema_alpha, p.ema_one_minus_alpha, avg[e], th[e]);
          store_floats<V>(p.ema + i, vec, n, avg);
        }
#pragma unroll
        for (int e = 0; e < V; ++e) {
          a[e] = __fadd_rn(a[e], x[e]);
          apply_rule<EP>(p.h, __fdiv_rn(a[e], n_as_float), th[e], s0[e], s1[e]);
        }
        store_floats<V>(p.theta + i, vec, n, th);
        if (Rule::kState0) store_floats<V>(p.s0 + i, vec, n, s0);
        if (Rule::kState1) store_floats<V>(p.s1 + i, vec, n, s1);
      }
    }
  }

  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned ticket = atomicAdd(reinterpret_cast<unsigned*>(p.counter + 2), 1u);
    if (ticket == gridDim.x - 1) {  // every block has read the state: now it may change
      p.counter[2] = 0;
      p.counter[1] += 1;
      int outcome = 0, after = accepted;
      if (admit) {
        after = accepted + 1;
        outcome = 1;
        if (last) {
          outcome = 2;
          p.counter[0] = 0;
          p.counter[3] = p.t + 1;
        } else {
          p.counter[0] = after;
        }
      }
      p.info[0] = outcome;
      p.info[1] = after;
    }
  }
}

// ====================================================================== closing an iteration
//
// Time-out rule, arrival by arrival: the deadline of iteration t has passed.  With at least n_min
// gradients in the running sum the parameters move by their mean (divisor: the number accepted),
// the set is emptied and t + 1 opens; otherwise nothing changes.  Same protocol on the server
// state as the arrival kernel: every block reads it first, the last ticket changes it.

struct CloseParams {
  int32_t t, n_min;
  long long P;
  const float* acc;
  int32_t* counter;  // [4]
  float* theta;
  float* s0;
  float* s1;
  int32_t* info;  // [2]: {2 updated | 0 nothing done, gradients in the set}
  float* ema;     // optional
  float ema_alpha, ema_one_minus_alpha;
  Hyper h;
};

template <int EP>
__global__ void __launch_bounds__(256, 4) close_iteration_kernel(const CloseParams p) {
  using Rule = RuleTraits<EP>;
  __shared__ int s_accepted, s_open;
#if SGDB_PDL
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
  if (threadIdx.x == 0) {
    s_accepted = *reinterpret_cast<volatile int32_t*>(p.counter + 0);
    s_open = *reinterpret_cast<volatile int32_t*>(p.counter + 3);
  }
  __syncthreads();
  const int accepted = s_accepted;
  const bool fire = (p.t >= s_open) && (accepted >= p.n_min);
  if (fire) {
    const float n_as_float = static_cast<float>(accepted);
    const uint64_t pol_stream = l2_policy_evict_first();
    const long long chunks = (p.P + 3) / 4;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const bool reverse = (accepted & 1) != 0;  // opposite to the launch that added the last gradient (see the arrival kernel)
    for (long long q_fwd = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; q_fwd < chunks; q_fwd += stride) {
      const long long q = reverse ? chunks - 1 - q_fwd : q_fwd;
      const long long i = q * 4;
      const long long rest = p.P - i;
      const int n = rest < 4 ? static_cast<int>(rest) : 4;
      const bool vec = n == 4;
      float a[4], th[4], s0[4], s1[4];
      load_floats_hint<4>(p.acc + i, vec, n, a, pol_stream);  // last use of the sum
      load_floats<4>(p.theta + i, vec, n, th);
      if (Rule::kState0) load_floats<4>(p.s0 + i, vec, n, s0);
      if (Rule::kState1) load_floats<4>(p.s1 + i, vec, n, s1);
      if (p.ema != nullptr) {
        float avg[4];
        load_floats<4>(p.ema + i, vec, n, avg);
#pragma unroll
        for (int e = 0; e < 4; ++e) avg[e] = ema_rule(p.ema_alpha, p.ema_one_minus_alpha, avg[e], th[e]);
        store_floats<4>(p.ema + i, vec, n, avg);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) apply_rule<EP>(p.h, __fdiv_rn(a[e], n_as_float), th[e], s0[e], s1[e]);
      store_floats<4>(p.theta + i, vec, n, th);
      if (Rule::kState0) store_floats<4>(p.s0 + i, vec, n, s0);
      if (Rule::kState1) store_floats<4>(p.s1 + i, vec, n, s1);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned ticket = atomicAdd(reinterpret_cast<unsigned*>(p.counter + 2), 1u);
    if (ticket == gridDim.x - 1) {
      p.counter[2] = 0;
      if (fire) {
        p.counter[0] = 0;
        p.counter[3] = p.t + 1;
      }
      p.info[0] = fire ? 2 : 0;
      p.info[1] = accepted;
    }
  }
}

// ====================================================================== bounded wait, on its own
//
// One block arms nothing and waits, with the same routine the row-streaming kernel uses, for a barrier
// phase that nobody will ever complete.  The wait must give up after `limit_ns`, raise the block's abort
// flag and let the kernel end normally; the second warp, which watches only the flag, must see it.
//   out[0] = SGDB_ERR_TIMEOUT when the wait gave up (SGDB_OK if it claims the phase completed)
//   out[1] = nanoseconds the waiting thread spent, clamped to int32
//   out[2] = 1 when the watching warp left through the abort flag
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(unsigned long long limit_ns, int32_t* out) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(smem_addr(&bar), 1);
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned long long t0 = global_timer_ns();
    const bool done = mbar_wait_for(smem_addr(&bar), 0u, &s_abort, limit_ns);
    const unsigned long long waited = global_timer_ns() - t0;
    out[0] = done ? SGDB_OK : SGDB_ERR_TIMEOUT;
    out[1] = waited > 0x7fffffffull ? 0x7fffffff : static_cast<int32_t>(waited);
  } else if (threadIdx.x == 32) {
    // a second waiter with a limit it cannot reach first: it leaves because the first raised the flag
    const bool done = mbar_wait_for(smem_addr(&bar), 0u, &s_abort, limit_ns + kWaitLimitNs);
    out[2] = (!done && s_abort != 0) ? 1 : 0;
  }
}

}  // namespace sgdb
