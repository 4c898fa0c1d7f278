// hpctopk: exact Top-K over ragged FP32 score rows, hand-written for sm_100a.
//
// Two launch forms over the same device functions.  A single persistent kernel (hpctopk_kernel):
// CTAs claim tasks (a whole row, or one contiguous segment of a long row) from a device counter;
// used for calls of few rows, where long rows are split over CTAs.  And a three-kernel pipeline
// (pipe_boundary_kernel, pipe_pass_kernel, pipe_refine_kernel) for all other calls, which keeps
// the kernel that reads every score streaming all the time.  Everything that
// depends on row lengths is decided on the device, so the launch geometry is a function of
// (num_rows, K, device) only.
//
// Per row (notation of Sections 4.2-4.4 of the paper):
//   Phase 1  stride-s view -> 2048-bin coarse histogram (11 leading bits of the fp16 key) ->
//            tau_0, nested tau_1 (plus a bracket bin and a wider tau_2 of the same histogram) ->
//            inclusive FP32 cutoffs (as ordered keys)
//   Phase 2  one complete-row pass: key <= cutoff(tau_1) ? append (key, index); C(tau_0) is
//            counted from the stored tail, so the band extension costs no second pass
//   Phase 3  one pass over a row-adaptive 2048-bin digit and a ranking of the boundary bin; the
//            general radix refinement 11+11+10, continued over the index bits when the final
//            equal-key group is larger than the remaining quota, behind it
//   recovery one band pass for (tau_1, tau_2]; storage-free full-radix select over the whole row
//            otherwise
//
// Keys: kd(x) is the descending sortable key (smaller key = larger score), kd = u for a set
// sign bit and u ^ 0x7FFFFFFF otherwise, u the raw bits.
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <type_traits>
#include <mutex>

#include "../../include/hpctopk.h"

// Per-phase cycle counters (hpctopk_stats::cycles_*) are a tuning aid: reading the SM clock
// pins the instruction schedule around it and costs measurable throughput, so the counters
// are compiled in only with -DHPCTOPK_TIMERS=1 and read as zero otherwise.
#ifndef HPCTOPK_TIMERS
#define HPCTOPK_TIMERS 0
#endif

namespace {

__device__ __forceinline__ long long tick() {
#if HPCTOPK_TIMERS
  return clock64();
#else
  return 0;
#endif
}

constexpr int kBins = 2048;            // B_c and the widest refinement digit
constexpr int kSplitRowsMax = 512;     // rows beyond this are never split (enough row parallelism)
constexpr int kSegMinElems = 16384;    // shortest segment worth a CTA
constexpr int kTasksPerCta = 1;        // split target: tasks >= kTasksPerCta * grid
constexpr int kSmallMax = kBins / 2;   // boundary group resolved by direct ranking (pairs held in the histogram's memory)

// workspace layout (bytes)
constexpr size_t kOffCtrl = 0;                       // uint32 task_counter
constexpr size_t kOffStats = 256;                    // hpctopk_stats (176 B)
constexpr size_t kOffSplit = 512;                    // arrive[512], count[512], count of A(tau_0)[512]
constexpr size_t kZeroBytes = kOffSplit + 3 * kSplitRowsMax * sizeof(uint32_t);
constexpr size_t kOffRowInfo = 8192;
constexpr int kPrefetchAheadBytes = 65536;   // L2 prefetch distance inside a row's scan (warp-specialised kernels)
constexpr int kPrefetchHeadBytes = 131072;   // bytes of the next task's range warmed in L2 ahead of time
constexpr int kMaxGrid = 1024;         // upper bound on resident CTAs (sizes the spill region)

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// Candidate capacity: `capacity_for` entries in total, the first `smem_capacity_for` of them in
// shared memory and the rest in the CTA's global overflow slice (Section 5.3).
__host__ __device__ inline int capacity_for(int K) { return 4 * K > 4096 ? 4 * K : 4096; }
#ifndef HPCTOPK_CAPS3
__host__ __device__ inline int smem_capacity_for(int K) { return 2 * K > 2048 ? 2 * K : 2048; }
#else
// 3K entries up to K = 2048 (the nested tail A(tau_1) holds about 1.75K, rarely more than 2.5K),
// 2K above, where three CTAs of 3K entries would no longer fit one SM.
__host__ __device__ inline int smem_capacity_for(int K) { return K <= 2048 ? (3 * K > 3072 ? 3 * K : 3072) : 2 * K; }
#endif
__host__ __device__ inline int stride_for(int K) {
  int s = 1;
  while (s * 2 <= 128 && s * 2 * 16 <= K) s *= 2;
  return s;
}

struct Params {
  const float* scores;
  const int32_t* row_starts;    // NULL: padded matrix, row r starts at element r * pitch
  int64_t pitch;
  const int32_t* row_lengths;
  int32_t num_rows;
  int32_t K;
  int32_t* out_idx;
  float* out_val;
  unsigned char* ws;
  int32_t cap;          // total candidate capacity (entries)
  int32_t cap_s;        // entries held in shared memory; the rest spill to the CTA's global slice
  int32_t stride;
  int32_t q0, q1;
  int32_t split_enabled;
  // Three-kernel pipeline only (zero otherwise): workspace offsets of the per-row boundary
  // records, the per-row admitted counts, the per-row candidate ranges and the overflow slices.
  int64_t pipe_rec_off, pipe_cnt_off, pipe_cand_off, pipe_spill_off;
  int32_t row_begin, row_end;   // the rows this launch of a pipeline kernel covers
};

// What the boundary kernel leaves for a row and the other two kernels read.
struct RowRec {
  uint32_t cutd[4];          // cutoffs of tau_0, tau_1, tau_hi, tau_2
  int32_t tau_pack;          // tau_0 | tau_1 << 16, or -1
  uint32_t usable;           // 1: sampled row with a usable view
  uint32_t pad[2];
};
static_assert(sizeof(RowRec) == 32, "RowRec is read as two 16-byte vectors");

// Element offset of row r in `scores`.
__device__ __forceinline__ int64_t row_start(const Params& P, int row) {
  return P.row_starts ? (int64_t)P.row_starts[row] : (int64_t)row * P.pitch;
}

struct Shared {
  hpctopk_stats acc;         // this CTA's counters (first member of every kernel's shared state)
  alignas(16) uint32_t hist[kBins];   // read and cleared as 16-byte vectors
  uint32_t warp_sums[32];
  uint32_t cand_count;
  uint32_t out_count;
  uint32_t small_count;
  uint32_t count0;           // C(tau_0) within the stored nested tail
  uint32_t min_bin;          // Phase 1: smallest occupied coarse bin of the view
  int32_t loc_bin[4];
  uint32_t loc_below[4];
  uint32_t loc_at[4];
  uint32_t cutd[4];          // cutoffs of tau_0, tau_1, of the bracket bin tau_hi, and of tau_2
  int32_t task;
  int32_t claim;
  uint32_t bcast0;
  uint32_t bcast1;
  uint32_t seg_len_vec;     // vectors per segment unit (split table)
  uint32_t total_tasks;
  unsigned long long* detail;   // hpctopk_stats::cycles_detail of this call's workspace (tuning aid)
};

// Dynamic shared memory: [Shared][cand: cap x (kd, idx) pairs][seg_base: kSplitRowsMax + 1 u32].
// Device functions re-derive these pointers from the extern array (instead of receiving
// generic pointers) so that loads, stores and atomics compile to shared-space instructions.
extern __shared__ __align__(16) unsigned char smem_raw[];
__device__ __forceinline__ Shared& SH() { return *reinterpret_cast<Shared*>(smem_raw); }
__device__ __forceinline__ uint2* CAND() {
  return reinterpret_cast<uint2*>(smem_raw + ((sizeof(Shared) + 15) / 16 * 16));
}

// ---------------------------------------------------------------- keys and the coarse map
__device__ __forceinline__ uint32_t kd_of_bits(uint32_t u) {
  return u ^ (~(uint32_t)((int32_t)u >> 31) & 0x7FFFFFFFu);
}
__device__ __forceinline__ uint32_t bits_of_kd(uint32_t kd) {
  return (kd & 0x80000000u) ? kd : (kd ^ 0x7FFFFFFFu);
}
// c(x) of Eq. "coarse-map", evaluated from the descending key.  NaN patterns (outside the
// contract) are placed by sign so that the map stays monotone in the key.
__device__ __forceinline__ int coarse_bin_of_kd(uint32_t kd) {
  const uint32_t u = bits_of_kd(kd);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 31) ? (kBins - 1) : 0;
  const uint32_t h = __half_as_ushort(__float2half_rn(__uint_as_float(u)));
  const uint32_t asc = (h & 0x8000u) ? (h ^ 0xFFFFu) : (h | 0x8000u);
  return (int)((0xFFFFu - asc) >> 5);
}
// Largest descending key whose coarse bin is <= tau: the inclusive FP32 endpoint of the
// admitted prefix.  Searched with the same map the histogram used, so the two cannot disagree.
// One warp, 32 probes per step (c is non-decreasing in kd, so the probes that pass form a
// prefix); every lane of the calling warp must take part and receives the result.
__device__ __noinline__ uint32_t cutoff_of_bin(int tau) {
  const uint32_t lane = threadIdx.x & 31;
  uint32_t lo = 0u;                         // invariant: c(lo) <= tau  (c(0) = 0)
#pragma unroll 1
  for (int b = 27; b >= -3; b -= 5) {
    const int sh = b < 0 ? 0 : b;
    const uint32_t nprobe = b < 0 ? 3u : 31u;            // last step resolves the two low bits
    const uint64_t probe = (uint64_t)lo + ((uint64_t)(lane + 1) << sh);
    const bool ok = lane < nprobe && probe <= 0xFFFFFFFFull && coarse_bin_of_kd((uint32_t)probe) <= tau;
    lo += (uint32_t)__popc(__ballot_sync(0xFFFFFFFFu, ok)) << sh;
  }
  return lo;
}

// Bin -> cutoff table: g_cut_table[tau] is the largest descending key whose coarse bin is <= tau
// (the inclusive FP32 endpoint of Section 5.2).  It depends on the coarse map only, so it is
// filled once per device by init_cut_table_kernel and read from then on.
__device__ uint32_t g_cut_table[kBins];
__global__ void init_cut_table_kernel() {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (warp < kBins) {
    const uint32_t c = cutoff_of_bin(warp);
    if ((threadIdx.x & 31) == 0) g_cut_table[warp] = c;
  }
}

#if !HPCTOPK_TIMERS
#define DSTAMP(k, t_prev) do { (void)(t_prev); } while (0)
#else
#define DSTAMP(k, t_prev) do { if (threadIdx.x == 0) { const long long t_now = tick(); atomicAdd(reinterpret_cast<unsigned long long*>(&stats_of(nullptr)->cycles_detail[k]), (unsigned long long)(t_now - (t_prev))); (t_prev) = t_now; } } while (0)
#endif

#if HPCTOPK_TIMERS == 2      // finer stamps inside Phase 1, in slots the refinement stamps otherwise use
#define DSTAMP1(k, t_prev) DSTAMP(k, t_prev)
#else
#define DSTAMP1(k, t_prev) do { (void)(t_prev); } while (0)
#endif

// ---------------------------------------------------------------- warp-level primitives
// min{b : H(b) >= quota} over the 2048-bin histogram, by one warp: lane sums of 64 bins, warp
// prefix, then the 64 bins of the lane that holds the quota are scanned two per lane.
// Returns the bin (or -1), with H(b - 1) in `below` and h(b) in `at`; uniform across the warp.
struct LaneSums { uint32_t sum, incl; };
__device__ __forceinline__ LaneSums w_lane_sums(const uint32_t* hist, int lane) {
  // lane l owns bins [64 l, 64 l + 64); its sixteen 16-byte chunks are read in an order rotated
  // by l, so that the lanes of a quarter warp touch different banks
  const uint4* hv = reinterpret_cast<const uint4*>(hist + lane * 64);
  uint32_t sum = 0;
#pragma unroll
  for (int b = 0; b < 16; ++b) { const uint4 v = hv[(b + lane) & 15]; sum += v.x + v.y + v.z + v.w; }
  uint32_t incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += n;
  }
  return LaneSums{sum, incl};
}
__device__ __forceinline__ int w_locate(const uint32_t* hist, const LaneSums ls, uint32_t quota, int lane,
                                        uint32_t& below, uint32_t& at) {
  const uint32_t excl = ls.incl - ls.sum;
  const uint32_t hit = __ballot_sync(0xFFFFFFFFu, excl < quota && quota <= ls.incl);
  if (hit == 0u) { below = 0; at = 0; return -1; }
  const int L = __ffs(hit) - 1;
  const uint32_t base = __shfl_sync(0xFFFFFFFFu, excl, L);
  const uint2 pr = *reinterpret_cast<const uint2*>(hist + L * 64 + 2 * lane);
  const uint32_t s2 = pr.x + pr.y;
  uint32_t incl2 = s2;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl2, d);
    if (lane >= d) incl2 += n;
  }
  const uint32_t excl2 = base + incl2 - s2;
  const uint32_t hit2 = __ballot_sync(0xFFFFFFFFu, excl2 < quota && quota <= excl2 + s2);
  const int M = __ffs(hit2) - 1;               // exists: the quota lies inside lane L's bins
  const bool first = excl2 + pr.x >= quota;
  const int bin_m = L * 64 + 2 * lane + (first ? 0 : 1);
  const uint32_t below_m = first ? excl2 : excl2 + pr.x;
  const uint32_t at_m = first ? pr.x : pr.y;
  below = __shfl_sync(0xFFFFFFFFu, below_m, M);
  at = __shfl_sync(0xFFFFFFFFu, at_m, M);
  return __shfl_sync(0xFFFFFFFFu, bin_m, M);
}
// Several quotas located together: the three dependent chains of shuffles and loads advance in
// lockstep, so their latencies overlap instead of adding up (a warp issues in order).
template <int N>
__device__ __forceinline__ void w_locate_n(const uint32_t* hist, const LaneSums ls, const uint32_t (&quota)[N], int lane,
                                           int (&bin)[N]) {
  const uint32_t excl = ls.incl - ls.sum;
  uint32_t hit[N];
#pragma unroll
  for (int k = 0; k < N; ++k) hit[k] = __ballot_sync(0xFFFFFFFFu, excl < quota[k] && quota[k] <= ls.incl);
  int L[N];
  uint32_t base[N];
  uint2 pr[N];
#pragma unroll
  for (int k = 0; k < N; ++k) { L[k] = hit[k] ? __ffs(hit[k]) - 1 : 0; base[k] = __shfl_sync(0xFFFFFFFFu, excl, L[k]); }
#pragma unroll
  for (int k = 0; k < N; ++k) pr[k] = *reinterpret_cast<const uint2*>(hist + L[k] * 64 + 2 * lane);
  uint32_t s2[N], incl2[N];
#pragma unroll
  for (int k = 0; k < N; ++k) { s2[k] = pr[k].x + pr[k].y; incl2[k] = s2[k]; }
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t n[N];
#pragma unroll
    for (int k = 0; k < N; ++k) n[k] = __shfl_up_sync(0xFFFFFFFFu, incl2[k], d);
#pragma unroll
    for (int k = 0; k < N; ++k) if (lane >= d) incl2[k] += n[k];
  }
#pragma unroll
  for (int k = 0; k < N; ++k) {
    const uint32_t excl2 = base[k] + incl2[k] - s2[k];
    const uint32_t hit2 = __ballot_sync(0xFFFFFFFFu, excl2 < quota[k] && quota[k] <= excl2 + s2[k]);
    const int M = hit2 ? __ffs(hit2) - 1 : 0;
    const int bin_m = L[k] * 64 + 2 * lane + ((excl2 + pr[k].x >= quota[k]) ? 0 : 1);
    bin[k] = (hit[k] && hit2) ? __shfl_sync(0xFFFFFFFFu, bin_m, M) : -1;
  }
}
__device__ __forceinline__ void w_locate3(const uint32_t* hist, const LaneSums ls, const uint32_t (&quota)[3], int lane,
                                          int (&bin)[3]) {
  w_locate_n<3>(hist, ls, quota, lane, bin);
}
__device__ __forceinline__ void w_clear_hist(uint32_t* hist, int lane) {
  uint4* hv = reinterpret_cast<uint4*>(hist);
#pragma unroll
  for (int b = 0; b < 16; ++b) hv[b * 32 + lane] = make_uint4(0u, 0u, 0u, 0u);
}

// ---------------------------------------------------------------- block primitives
template <int THREADS>
__device__ __forceinline__ uint32_t warp_inclusive_scan(uint32_t v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, v, d);
    if (lane >= d) v += n;
  }
  return v;
}

// For up to two quotas: min{b : H(b) >= quota} over the inclusive prefix of sh.hist, with
// H(b-1) ("below") and h(b) ("at").  loc_bin stays -1 when the histogram total is short.
// Contains block barriers; every thread must call it.  Leaves sh.hist unchanged.
template <int THREADS>
__device__ void locate(Shared& sh, uint32_t quota0, uint32_t quota1, int nq) {
  constexpr int BPT = (kBins + THREADS - 1) / THREADS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t h[BPT];
  uint32_t sum = 0;
#pragma unroll
  for (int b = 0; b < BPT; ++b) { h[b] = tid * BPT + b < kBins ? sh.hist[tid * BPT + b] : 0u; sum += h[b]; }
  const uint32_t incl = warp_inclusive_scan<THREADS>(sum);
  if (lane == 31) sh.warp_sums[warp] = incl;
  if (tid < 2) sh.loc_bin[tid] = -1;
  __syncthreads();
  uint32_t woff = 0;
  for (int w = 0; w < warp; ++w) woff += sh.warp_sums[w];
  const uint32_t excl = woff + incl - sum;
  for (int qi = 0; qi < nq; ++qi) {
    const uint32_t quota = qi ? quota1 : quota0;
    if (excl < quota && quota <= excl + sum) {
      uint32_t run = excl;
#pragma unroll
      for (int b = 0; b < BPT; ++b) {
        if (run < quota && run + h[b] >= quota) {
          sh.loc_bin[qi] = tid * BPT + b; sh.loc_below[qi] = run; sh.loc_at[qi] = h[b];
        }
        run += h[b];
      }
    }
  }
  __syncthreads();
}

// The same for N <= 4 quotas with every warp taking part: a thread owns 4 (8 below 512 threads)
// consecutive bins read as 16-byte vectors, so the critical path is one vector load, one warp
// scan, one barrier and a look at the warp totals, whatever the other CTAs of the SM are doing.
// (A single warp walking the histogram takes 13 K to 18 K cycles per row next to streaming CTAs,
// against about 6 K here, yet the whole call ran 3 % slower with this form: the idle warps of the
// single-warp search cost nothing, the fifteen extra warps here take issue slots from the CTAs
// that are streaming.  The boundary and refinement kernels of the pipeline, which share the SM
// with no streaming CTA, use this form: BLOCK_SEARCH = true.)
template <int THREADS, int N>
__device__ __forceinline__ void locate_n(const uint32_t (&quota)[N]) {
  Shared& sh = SH();
  constexpr int BPT = THREADS >= 512 ? 4 : (THREADS >= 256 ? 8 : 16);
  constexpr int NT = kBins / BPT, NW = NT / 32;
  static_assert(NT <= THREADS, "locate_n needs at least 128 threads");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t h[BPT];
  uint32_t sum = 0;
  if (tid < NT) {
    const uint4* hv = reinterpret_cast<const uint4*>(sh.hist) + tid * (BPT / 4);
#pragma unroll
    for (int v = 0; v < BPT / 4; ++v) {
      const uint4 x = hv[v];
      h[4 * v] = x.x; h[4 * v + 1] = x.y; h[4 * v + 2] = x.z; h[4 * v + 3] = x.w;
      sum += x.x + x.y + x.z + x.w;
    }
  }
  uint32_t incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += up;
  }
  if (lane == 31 && warp < NW) sh.warp_sums[warp] = incl;
  if (tid < N) sh.loc_bin[tid] = -1;
  __syncthreads();
  if (tid < NT) {
    uint32_t woff = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) { const uint32_t ws = sh.warp_sums[w]; woff += w < warp ? ws : 0u; }
    const uint32_t excl = woff + incl - sum;
#pragma unroll
    for (int k = 0; k < N; ++k) {
      if (excl < quota[k] && quota[k] <= excl + sum) {
        uint32_t run = excl;
#pragma unroll
        for (int b = 0; b < BPT; ++b) {
          if (run < quota[k] && run + h[b] >= quota[k]) {
            sh.loc_bin[k] = tid * BPT + b; sh.loc_below[k] = run; sh.loc_at[k] = h[b];
          }
          run += h[b];
        }
      }
    }
  }
  __syncthreads();
}

template <int THREADS>
__device__ __forceinline__ void clear_hist(Shared& sh) {
  uint4* hv = reinterpret_cast<uint4*>(sh.hist);
  for (int b = threadIdx.x; b < kBins / 4; b += THREADS) hv[b] = make_uint4(0u, 0u, 0u, 0u);
}

// Admission test on raw bits, one integer compare per score (Section 5.3 compares the FP32
// score with the cutoff directly).  With cu the bit pattern of the cutoff score:
//   cu >= 0 as int32 (cutoff positive):  admitted  <=>  (int32)u >= (int32)cu
//   cu <  0          (cutoff negative):  admitted  <=>  u <= cu   (unsigned)
// Both are (int32)(u ^ flip) >= bound with flip = 0 / 0x7FFFFFFF and bound = cu ^ flip, and
// both agree with kd(u) <= kd(cu), including signed zeros, infinities and NaN patterns.
struct Admit {
  uint32_t flip;
  int32_t bound;
  __device__ __forceinline__ explicit Admit(uint32_t cut_kd) {
    const uint32_t cu = bits_of_kd(cut_kd);
    flip = (cu & 0x80000000u) ? 0x7FFFFFFFu : 0u;
    bound = (int32_t)(cu ^ flip);
  }
  __device__ __forceinline__ bool operator()(uint32_t u) const { return (int32_t)(u ^ flip) >= bound; }
};

// Where admitted scores go: shared memory first, then this CTA's global overflow slice.
struct CandCtx {
  uint32_t cap_s, cap;
  uint2* spill;
};
__device__ __forceinline__ CandCtx cand_ctx(const Params& P) {
  const size_t cand_off = align_up(kOffRowInfo + (size_t)P.num_rows * sizeof(hpctopk_row_info), 256);
  const size_t split_rows = P.num_rows < kSplitRowsMax ? P.num_rows : kSplitRowsMax;
  const size_t spill_off = P.pipe_spill_off ? (size_t)P.pipe_spill_off : cand_off + split_rows * (size_t)P.cap * 8;
  CandCtx c;
  c.cap_s = (uint32_t)P.cap_s;
  c.cap = (uint32_t)P.cap;
  c.spill = reinterpret_cast<uint2*>(P.ws + spill_off) + (size_t)blockIdx.x * (size_t)(P.cap - P.cap_s);
  return c;
}
__device__ __forceinline__ uint2 cand_load(const CandCtx& c, uint32_t i) {   // (kd, idx)
  return i < c.cap_s ? CAND()[i] : __ldcg(c.spill + (i - c.cap_s));
}
__device__ __forceinline__ void cand_store(const CandCtx& c, uint32_t i, uint2 v) {
  if (i < c.cap_s) CAND()[i] = v; else c.spill[i - c.cap_s] = v;
}

// Append one admitted score: reserve a slot, store (kd, idx).  Entries beyond the capacity are
// counted, not stored.  (The histogram of the refinement digit is built from the compacted
// on-chip tail right after the pass, see select_adaptive; no second row pass is involved.)
// Measured on this path, and left out because the whole call got slower although fewer
// instructions ran: storing the raw bits and forming the key when an entry is read; loops
// specialised on the sign of the cutoff (one compare instead of xor + compare); one atomic per
// lane and register tile; one atomic per warp and tile after a shuffle scan of the lane counts;
// one vote per element position with converged stores; one gating branch per vector or tile.
// (Diverged lanes on this short path run in the shadow of the converged ones; every converged
// form makes the whole warp wait at its votes and shuffles.)
__device__ __forceinline__ void append_candidate(uint32_t u, uint32_t idx, const CandCtx& c) {
  Shared& sh = SH();
  const uint32_t kd = kd_of_bits(u);
  const uint32_t pos = atomicAdd(&sh.cand_count, 1u);
  if (pos < c.cap_s) CAND()[pos] = make_uint2(kd, idx);
  else if (pos < c.cap) c.spill[pos - c.cap_s] = make_uint2(kd, idx);
}

// ---------------------------------------------------------------- Phase 2: the complete-row pass
// Scans global elements [e0, e1) of `scores`; row-local index = e - g0.
//   BAND = false: admit kd <= cut_hi.            (A(tau_0), Eq. "candidate-set")
//   BAND = true : admit cut_lo < kd <= cut_hi.   (the band of Eq. "rescue-band")
// Admitted scores are rare (about 1.5 K / L of the row), so the loop spends one compare and one
// branch per score and leaves everything else to the taken branch.
template <int THREADS, int U, bool BAND>
__device__ __noinline__ void scan_range(const float* __restrict__ scores, int64_t g0, int64_t e0, int64_t e1,
                                             uint32_t cut_lo, uint32_t cut_hi, const CandCtx cc) {
  const int tid = threadIdx.x;
  if (e1 <= e0) return;
  const Admit in_hi(cut_hi);
  const Admit in_lo(cut_lo);                 // BAND: scores admitted by tau_0 are already held
  auto admit = [&](uint32_t u) -> bool { return BAND ? (in_hi(u) && !in_lo(u)) : in_hi(u); };
  int64_t b0 = (e0 + 3) & ~(int64_t)3;       // first 16-byte aligned element
  int64_t b1 = e1 & ~(int64_t)3;             // end of the last whole vector
  if (b0 > b1) { b0 = e1; b1 = e1; }         // range holds no whole vector
  // ragged edges: at most 3 + 3 scalar elements
  if (tid < 16) {
    const int64_t head_end = b0 < e1 ? b0 : e1;
    const int nhead = (int)(head_end - e0);
    const int ntail = (int)(e1 - (b1 > head_end ? b1 : head_end));
    int64_t e = -1;
    if (tid < nhead) e = e0 + tid;
    else if (tid >= 8 && tid - 8 < ntail) e = e1 - ntail + (tid - 8);
    if (e >= 0) {
      const uint32_t u = __float_as_uint(__ldg(scores + e));
      if (admit(u)) append_candidate(u, (uint32_t)(e - g0), cc);
    }
  }
  const int64_t nvec = (b1 - b0) >> 2;
  if (nvec <= 0) return;
  const float4* __restrict__ vp = reinterpret_cast<const float4*>(scores + b0);
  const uint32_t idx0 = (uint32_t)(b0 - g0);
  constexpr int TILE = THREADS * U;
  const int64_t nfull = nvec / TILE;

  auto classify = [&](const float4& f, uint32_t i) {
    const uint32_t u0 = __float_as_uint(f.x), u1 = __float_as_uint(f.y);
    const uint32_t u2 = __float_as_uint(f.z), u3 = __float_as_uint(f.w);
    if (admit(u0)) append_candidate(u0, i + 0, cc);
    if (admit(u1)) append_candidate(u1, i + 1, cc);
    if (admit(u2)) append_candidate(u2, i + 2, cc);
    if (admit(u3)) append_candidate(u3, i + 3, cc);
  };
  // (Asking the L2 for lines further ahead with prefetch.global.L2 was measured: no gain.)
  auto load_tile = [&](float4 (&buf)[U], const float4* p) {
#pragma unroll
    for (int j = 0; j < U; ++j) buf[j] = __ldcs(p + j * THREADS);
  };
  auto process_tile = [&](const float4 (&buf)[U], uint32_t ibase) {
#pragma unroll
    for (int j = 0; j < U; ++j) classify(buf[j], ibase + (uint32_t)(j * THREADS * 4));
  };

  // Two register tiles: the loads of one are in flight while the other is classified.
  float4 A[U], B[U];
  const float4* p = vp + tid;
  uint32_t ib = idx0 + (uint32_t)(tid << 2);
  uint32_t left = (uint32_t)nfull;
  if (left > 0) load_tile(A, p);
  while (left >= 2) {
    load_tile(B, p + TILE);
    process_tile(A, ib);
    if (left > 2) load_tile(A, p + 2 * TILE);
    process_tile(B, ib + TILE * 4);
    p += 2 * TILE;
    ib += 2 * TILE * 4;
    left -= 2;
  }
  if (left == 1) process_tile(A, ib);
  // remainder: fewer than TILE vectors
  for (int64_t v = nfull * TILE + tid; v < nvec; v += THREADS)
    classify(__ldcs(vp + v), idx0 + (uint32_t)(v << 2));
}

// ---------------------------------------------------------------- element sources for selection
// A source visits every element once per pass, calling f(valid, kd, idx) with a block-uniform
// trip count (so f may use warp collectives).
struct CandidateSource {          // the admitted tail: shared memory, then the overflow slice
  CandCtx cc;
  uint32_t n;
  uint32_t kd_max = 0xFFFFFFFFu;  // entries with a larger key are skipped (split rows hold A(tau_1))
  template <int THREADS, typename F>
  __device__ __forceinline__ void for_each(F f) const {
    for (uint32_t b = 0; b < n; b += THREADS) {
      const uint32_t i = b + threadIdx.x;
      const bool v = i < n;
      const uint2 c = v ? cand_load(cc, i) : make_uint2(0u, 0u);
      f(v && c.x <= kd_max, c.x, c.y);
    }
  }
};

struct RowSource {                // the complete row in global memory (recovery)
  const float* scores;
  int64_t g0, g1;
  template <int THREADS, typename F>
  __device__ __forceinline__ void for_each(F f) const {
    const int64_t va = g0 >> 2, vb = (g1 + 3) >> 2;
    constexpr int R = 1;       // vectors per thread in flight; 2 spills under the 40-register budget and measured slower
    for (int64_t base = va + threadIdx.x; base < vb + threadIdx.x; base += R * THREADS) {
      float4 x[R];
#pragma unroll
      for (int k = 0; k < R; ++k) {
        const int64_t e = (base + k * THREADS) << 2;
        const bool full = e >= g0 && e + 4 <= g1;
        x[k] = full ? __ldg(reinterpret_cast<const float4*>(scores + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < R; ++k) {
        const int64_t e = (base + k * THREADS) << 2;
        const bool full = e >= g0 && e + 4 <= g1;
        float xs[4] = {x[k].x, x[k].y, x[k].z, x[k].w};
        bool ok[4] = {full, full, full, full};
        if (!full && e < g1) {                                       // a ragged first or last vector
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            ok[j] = (e + j >= g0) && (e + j < g1);
            if (ok[j]) xs[j] = __ldg(scores + e + j);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) f(ok[j], kd_of_bits(__float_as_uint(xs[j])), (uint32_t)(e + j - g0));
      }
    }
  }
};

// ---------------------------------------------------------------- Phase 3 and the output commit
// Radix selection of the `K` best elements of a source under the composite order
// (kd ascending, index ascending): digits 11+11+10 of kd (Section 4.4), then, only if the final
// equal-key group exceeds the remaining quota, 11+11+10 of the index.  Each round is
// prefix -> boundary digit -> k_{j+1} = k_j - |R_j| (Eqs. "digit-boundary", "refine-recurrence");
// the frontier Q_j is the set of elements matching the prefix chosen so far.  Selected elements
// are committed in one final pass: composite >> shift <= prefix.
// When `hist_ready`, sh.hist already holds the leading-digit histogram of the source.
template <int THREADS, typename Source>
__device__ __noinline__ void select_and_emit(const Source src, uint32_t K, bool hist_ready,
                                             int32_t* out_idx, float* out_val) {
  Shared& sh = SH();
  const int shifts[6] = {53, 42, 32, 21, 10, 0};
  const int widths[6] = {11, 11, 10, 11, 11, 10};
  uint64_t prefix = 0;
  int prev_shift = 64;
  uint32_t k_rem = K;
#pragma unroll 1
  for (int j = 0; j < 6; ++j) {
    const int shift = shifts[j];
    const uint32_t mask = (1u << widths[j]) - 1u;
    if (!(j == 0 && hist_ready)) {
      __syncthreads();
      clear_hist<THREADS>(sh);
      __syncthreads();
      src.template for_each<THREADS>([&](bool valid, uint32_t kd, uint32_t idx) {
        if (valid) {
          const uint64_t comp = ((uint64_t)kd << 32) | idx;
          if (j == 0 || (comp >> prev_shift) == prefix)
            atomicAdd(&sh.hist[(uint32_t)(comp >> shift) & mask], 1u);
        }
      });
    }
    __syncthreads();
    locate<THREADS>(sh, k_rem, 0, 1);
    const int b = sh.loc_bin[0];
    const uint32_t below = sh.loc_below[0], at = sh.loc_at[0];
    if (b < 0) break;                       // cannot happen for a certified state; keeps the loop finite
    k_rem -= below;
    prefix = (prefix << widths[j]) | (uint32_t)b;
    prev_shift = shift;
    if (at == k_rem) break;                 // the whole boundary group is taken
  }
  __syncthreads();
  if (threadIdx.x == 0) sh.out_count = 0;
  __syncthreads();
  src.template for_each<THREADS>([&](bool valid, uint32_t kd, uint32_t idx) {
    const uint64_t comp = ((uint64_t)kd << 32) | idx;
    const bool pred = valid && (prev_shift < 64) && ((comp >> prev_shift) <= prefix);
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, pred);
    if (m) {
      const int lane = threadIdx.x & 31;
      const int leader = __ffs(m) - 1;
      uint32_t base = 0;
      if (lane == leader) base = atomicAdd(&sh.out_count, (uint32_t)__popc(m));
      base = __shfl_sync(0xFFFFFFFFu, base, leader);
      if (pred) {
        const uint32_t slot = base + __popc(m & ((1u << lane) - 1u));
        if (slot < K) {
          out_idx[slot] = (int32_t)idx;
          if (out_val) out_val[slot] = __uint_as_float(bits_of_kd(kd));
        }
      }
    }
  });
  __syncthreads();
}

// ---------------------------------------------------------------- per-row bookkeeping
// Counters are accumulated per CTA in shared memory (the first bytes of the dynamic shared
// segment) and added to the workspace once, when the CTA leaves: per-row global atomics on a
// handful of addresses were a measurable serial cost.
__device__ __forceinline__ hpctopk_stats* stats_of(unsigned char*) {
  return reinterpret_cast<hpctopk_stats*>(smem_raw);
}
__device__ __forceinline__ void stats_clear() {
  unsigned long long* a = reinterpret_cast<unsigned long long*>(smem_raw);
  for (int i = threadIdx.x; i < (int)(sizeof(hpctopk_stats) / 8); i += blockDim.x) a[i] = 0ull;
}
// One thread, after every contributor of the CTA is done.
__device__ __forceinline__ void stats_flush(unsigned char* ws) {
  const unsigned long long* a = reinterpret_cast<const unsigned long long*>(smem_raw);
  unsigned long long* g = reinterpret_cast<unsigned long long*>(ws + kOffStats);
  constexpr int kMaxIdx = (int)(offsetof(hpctopk_stats, candidates_max) / 8);
  for (int i = 0; i < (int)(sizeof(hpctopk_stats) / 8); ++i) {
    const unsigned long long v = a[i];
    if (v == 0ull) continue;
    if (i == kMaxIdx) atomicMax(&g[i], v); else atomicAdd(&g[i], v);
  }
}
__device__ __forceinline__ void add64(uint64_t* p, uint64_t v) {
  atomicAdd(reinterpret_cast<unsigned long long*>(p), (unsigned long long)v);
}
__device__ __forceinline__ void max64(uint64_t* p, uint64_t v) {
  atomicMax(reinterpret_cast<unsigned long long*>(p), (unsigned long long)v);
}
__device__ void record_row(const Params& P, int row, int route, int tau, uint32_t c0, uint32_t cfin,
                           uint64_t scanned, uint64_t sampled, uint64_t L) {
  if (threadIdx.x != 0) return;
  hpctopk_stats* st = stats_of(P.ws);
  if (route == HPCTOPK_ROUTE_BAND2) add64(&st->rows_band2, 1);
  else add64(&st->rows_by_route[route], 1);
  if (route == HPCTOPK_ROUTE_PRIMARY || route == HPCTOPK_ROUTE_BAND || route == HPCTOPK_ROUTE_BAND2) {
    add64(&st->candidates_sum, cfin);
    max64(&st->candidates_max, cfin);
  }
  if (scanned) add64(&st->elements_scanned, scanned);
  if (sampled) add64(&st->elements_sampled, sampled);
  add64(&st->elements_valid, L);
  int4 info = make_int4(route, tau, (int)c0, (int)cfin);
  reinterpret_cast<int4*>(P.ws + kOffRowInfo)[row] = info;
}

// Phase 1 (Section 4.2): sample view -> coarse histogram -> tau_0, tau_1 -> cutoffs in sh.cutd.
// A third, tighter bin tau_hi at a quarter of the rank K (sample rank ceil(K / 4s)) brackets the K-th
// score from above; its cutoff sizes the refinement digit of select_adaptive.
// Returns false when the view cannot support the requested sample ranks.
template <int THREADS, bool BLOCK_SEARCH = false>
__device__ __noinline__ bool phase1(const Params& P, int row, int64_t g0, int64_t L, int& tau_pack) {
  Shared& sh = SH();
  const int s = P.stride;
  const int bits = 31 - __clz(s);
  const int a = bits ? (int)(__brev((uint32_t)(row & (s - 1))) >> (32 - bits)) : 0;   // pi_s: bit reversal
  const int64_t n_view = L > a ? ((L - a + s - 1) >> bits) : 0;
  tau_pack = -1;
  if (n_view < P.q1) return false;
  long long ts = tick();
  __syncthreads();
  clear_hist<THREADS>(sh);
  if (threadIdx.x == 0) sh.min_bin = kBins - 1;
  __syncthreads();
  DSTAMP(5, ts);
  uint32_t my_min = kBins - 1;
  const float* __restrict__ rowp = P.scores + g0 + a;
  for (int64_t t0 = 0; t0 < n_view; t0 += 4 * THREADS) {
    uint32_t u[4];
    bool v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int64_t t = t0 + k * THREADS + threadIdx.x;
      v[k] = t < n_view;
      // no L1 line, 64-byte L2 fetch: the default 128-byte fetch doubles the DRAM traffic of the view
      u[k] = 0u;
      if (v[k]) asm volatile("ld.global.nc.L1::no_allocate.L2::64B.b32 %0, [%1];" : "=r"(u[k]) : "l"(rowp + t * s));
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (v[k]) {
        const uint32_t bin = (uint32_t)coarse_bin_of_kd(kd_of_bits(u[k]));
        atomicAdd(&sh.hist[bin], 1u);
        my_min = bin < my_min ? bin : my_min;
      }
  }
  my_min = __reduce_min_sync(0xFFFFFFFFu, my_min);
  if ((threadIdx.x & 31) == 0 && my_min < kBins - 1) atomicMin(&sh.min_bin, my_min);
  __syncthreads();
  DSTAMP(6, ts);
  {
    int q_hi = (P.K + 4 * s - 1) / (4 * s);                           // bracket: sample rank ceil(K/4s)
    if (q_hi < 1) q_hi = 1;
    uint32_t q2 = (uint32_t)((3 * P.K + s - 1) / s);                   // second band: sample rank ceil(3K/s)
    if (q2 <= (uint32_t)P.q1) q2 = (uint32_t)P.q1 + 1u;
    const uint32_t quota[4] = {(uint32_t)P.q0, (uint32_t)P.q1, (uint32_t)q_hi, q2};
    // The four sample ranks are all small (at most 3K/s of the n_view samples), so their bins lie
    // within a few dozen bins of the best occupied one: one warp walks the histogram upwards from
    // there, 32 bins per step, instead of forming the prefix of all 2048 bins.
    if (threadIdx.x < 32) {
      const int lane = threadIdx.x;
      int tau[4] = {-1, -1, -1, -1};
      uint32_t carry = 0;
      for (int base = (int)(sh.min_bin & ~31u); base < kBins; base += 32) {
        const uint32_t h = sh.hist[base + lane];
        uint32_t incl = h;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
          if (lane >= d) incl += up;
        }
        const uint32_t cum = carry + incl;
        bool all = true;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (tau[k] < 0) {
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, cum >= quota[k]);
            if (m) tau[k] = base + __ffs(m) - 1;
          }
          all = all && tau[k] >= 0;
        }
        if (all) break;
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
      }
      if (lane < 4) sh.loc_bin[lane] = lane == 0 ? tau[0] : (lane == 1 ? tau[1] : (lane == 2 ? tau[2] : tau[3]));
      __syncwarp();
    }
    DSTAMP1(0, ts);
    if (threadIdx.x < 4) {
      int tau = sh.loc_bin[threadIdx.x];
      if (tau < 0) tau = sh.loc_bin[1];                                // view shorter than q2: no second band
      sh.cutd[threadIdx.x] = g_cut_table[tau];
    }
  }
  __syncthreads();
  DSTAMP(7, ts);
  tau_pack = sh.loc_bin[0] | (sh.loc_bin[1] << 16);
  return true;
}

// The row's boundary: read from the record a boundary kernel left (when the call ran one), else
// computed here.  Leaves the cutoffs in sh.cutd like phase1; contains block barriers.
// The per-row regions of the pipeline's workspace are indexed from the first row of the launch
// (a call of very many rows runs as several launches that reuse them).
__device__ __forceinline__ RowRec* pipe_rec(const Params& P) { return reinterpret_cast<RowRec*>(P.ws + P.pipe_rec_off) - P.row_begin; }
template <int THREADS>
__device__ __forceinline__ bool row_boundary(const Params& P, int row, int64_t g0, int64_t L, int& tau_pack) {
  if (P.pipe_rec_off == 0) return phase1<THREADS>(P, row, g0, L, tau_pack);
  Shared& sh = SH();
  const RowRec* rec = pipe_rec(P) + row;
  __syncthreads();
  if (threadIdx.x < 4) sh.cutd[threadIdx.x] = __ldg(&rec->cutd[threadIdx.x]);
  tau_pack = __ldg(&rec->tau_pack);
  const bool usable = __ldg(&rec->usable) != 0u;
  __syncthreads();
  return usable;
}

// Phase 3 with a row-adaptive first digit (any monotone digit of the key is a valid refinement
// digit, Section 4.4): d = min((cut_base - kd) >> sh, 2047) measures the distance from the
// admitted cutoff in units of 2^sh ulps, with sh chosen so that the bracket [cut_hi, cut_base]
// spans the 2048 bins; only a handful of scores then share the boundary bin.  One histogram pass,
// one boundary search (every warp for itself), one commit pass; the boundary bin is resolved by
// ranking its members against each other under (kd, idx).  Returns false, with nothing written,
// when the K-th score falls outside the bracket or the boundary bin is too large: the caller
// then runs the general 11+11+10 refinement.
// STAGE_OUT: the K results are collected in the shared memory behind the kernel's Shared block
// (2 x K words, which the launch must provide) and written out as whole lines at the end; the
// commit pass otherwise scatters 4-byte stores over the output row, which cost the refinement
// kernel a third of its time.
template <int THREADS, bool BLOCK_SEARCH = false, bool COUNT0 = false, bool STAGE_OUT = false>
__device__ __noinline__ bool select_adaptive(const CandCtx cc, uint32_t C, uint32_t K, uint32_t cut_base, uint32_t cut_hi,
                                             int32_t* out_idx, float* out_val, uint32_t cut_count = 0u) {
  int32_t* const w_idx = STAGE_OUT ? reinterpret_cast<int32_t*>(CAND()) : out_idx;
  float* const w_val = STAGE_OUT ? reinterpret_cast<float*>(CAND()) + K : out_val;
  Shared& sh = SH();
  constexpr int W = THREADS <= 128 ? 8 : 4;      // entries per thread and batch (independent loads in flight)
  const int tid = threadIdx.x, lane = tid & 31;
  const uint32_t span = cut_base > cut_hi ? cut_base - cut_hi : 0u;
  int shv = 0;
  while (shv < 31 && (span >> shv) >= 2047u) ++shv;
  // digit: 0 = the clamped group far above the bracket, 2047 = next to the cutoff
  auto digit = [&](uint32_t kd) -> uint32_t {
    const uint32_t d = (cut_base - kd) >> shv;
    return 2047u - (d < 2047u ? d : 2047u);
  };
  long long ts = tick();
  __syncthreads();
  clear_hist<THREADS>(sh);
  if (tid == 0) { sh.out_count = 0; sh.small_count = 0; }
  __syncthreads();
  DSTAMP(0, ts);
  uint32_t n0 = 0;                               // COUNT0: entries with kd <= cut_count, added to sh.count0
  for (uint32_t i0 = 0; i0 < C; i0 += W * THREADS) {
    uint2 c[W];
    bool v[W];
#pragma unroll
    for (int k = 0; k < W; ++k) {
      const uint32_t i = i0 + k * THREADS + tid;
      c[k] = i < C ? cand_load(cc, i) : make_uint2(0xFFFFFFFFu, 0u);
      v[k] = i < C && c[k].x <= cut_base;       // a split row's buffer also holds the band beyond tau_0
      if (COUNT0) n0 += (i < C && c[k].x <= cut_count) ? 1u : 0u;
    }
#pragma unroll
    for (int k = 0; k < W; ++k) if (v[k]) atomicAdd(&sh.hist[digit(c[k].x)], 1u);
  }
  if (COUNT0) {
    n0 = __reduce_add_sync(0xFFFFFFFFu, n0);
    if (lane == 0 && n0) atomicAdd(&sh.count0, n0);
  }
  __syncthreads();
  DSTAMP(1, ts);
  if (!BLOCK_SEARCH) {
  if (tid < 32) {
    const LaneSums ls = w_lane_sums(sh.hist, lane);
    uint32_t below0, at0;
    const int b0 = w_locate(sh.hist, ls, K, lane, below0, at0);
    if (lane == 0) { sh.loc_bin[0] = b0; sh.loc_below[0] = below0; sh.loc_at[0] = at0; }
  }
  __syncthreads();
  } else {
    const uint32_t quota[1] = {K};
    locate_n<THREADS, 1>(quota);
  }
  const int b = sh.loc_bin[0];
  const uint32_t below = sh.loc_below[0], at = sh.loc_at[0];
  DSTAMP(2, ts);
  if (b <= 0 || at > (uint32_t)kSmallMax) return false;
  const uint32_t k_rem = K - below;             // to take from the boundary bin
  uint2* const list = reinterpret_cast<uint2*>(sh.hist);
  __syncthreads();                              // the histogram's memory becomes the boundary list
  for (uint32_t i0 = 0; i0 < C; i0 += W * THREADS) {
    uint2 c[W];
    uint32_t dg[W];
    uint32_t cnt = 0;
#pragma unroll
    for (int k = 0; k < W; ++k) {
      const uint32_t i = i0 + k * THREADS + tid;
      c[k] = i < C ? cand_load(cc, i) : make_uint2(0xFFFFFFFFu, 0u);
      dg[k] = (i < C && c[k].x <= cut_base) ? digit(c[k].x) : 0xFFFFFFFFu;
      cnt += dg[k] < (uint32_t)b ? 1u : 0u;
    }
    const uint32_t incl = warp_inclusive_scan<THREADS>(cnt);
    const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    uint32_t base = 0;                          // one reservation of output slots per warp and batch
    if (lane == 31 && tot) base = atomicAdd(&sh.out_count, tot);
    base = __shfl_sync(0xFFFFFFFFu, base, 31);
    uint32_t pos = base + incl - cnt;
#pragma unroll
    for (int k = 0; k < W; ++k) {
      if (dg[k] < (uint32_t)b) {
        if (pos < K) { w_idx[pos] = (int32_t)c[k].y; if (w_val) w_val[pos] = __uint_as_float(bits_of_kd(c[k].x)); }
        ++pos;
      } else if (dg[k] == (uint32_t)b) {
        const uint32_t lp = atomicAdd(&sh.small_count, 1u);
        if (lp < (uint32_t)kSmallMax) list[lp] = c[k];
      }
    }
  }
  __syncthreads();
  DSTAMP(3, ts);
  for (uint32_t i = tid; i < at; i += THREADS) {
    const uint2 me = list[i];
    const uint64_t mine = ((uint64_t)me.x << 32) | me.y;
    uint32_t rank = 0;
    for (uint32_t t = 0; t < at; ++t) {
      const uint2 o = list[t];
      rank += ((((uint64_t)o.x << 32) | o.y) < mine) ? 1u : 0u;
    }
    if (rank < k_rem) {
      w_idx[below + rank] = (int32_t)me.y;
      if (w_val) w_val[below + rank] = __uint_as_float(bits_of_kd(me.x));
    }
  }
  __syncthreads();
  if (STAGE_OUT) {
    const bool vec = (K & 3u) == 0u && ((reinterpret_cast<uintptr_t>(out_idx) | reinterpret_cast<uintptr_t>(out_val)) & 15u) == 0u;
    if (vec) {                                   // whole 16-byte vectors (K words each of indices and values)
      const uint4* si = reinterpret_cast<const uint4*>(w_idx);
      const uint4* sv = reinterpret_cast<const uint4*>(w_val);
      for (uint32_t i = tid; i < (K >> 2); i += THREADS) reinterpret_cast<uint4*>(out_idx)[i] = si[i];
      if (out_val) for (uint32_t i = tid; i < (K >> 2); i += THREADS) reinterpret_cast<uint4*>(out_val)[i] = sv[i];
    } else {
      for (uint32_t i = tid; i < K; i += THREADS) out_idx[i] = w_idx[i];
      if (out_val) for (uint32_t i = tid; i < K; i += THREADS) out_val[i] = w_val[i];
    }
  }
  DSTAMP(4, ts);
  return true;
}

template <int THREADS>
__device__ void emit_short_row(const Params& P, int row, int64_t g0, int64_t L) {
  int32_t* oi = P.out_idx + (int64_t)row * P.K;
  float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
  for (int i = threadIdx.x; i < P.K; i += THREADS) {
    const bool v = i < L;
    oi[i] = v ? i : -1;
    if (ov) ov[i] = v ? __ldg(P.scores + g0 + i) : __uint_as_float(0xFF800000u);
  }
}

// C(tau_0) of the stored part of the nested tail: entries whose key passes the tau_0 cutoff.
// Adds into sh.count0 (cleared by the caller before the pass).
template <int THREADS>
__device__ __forceinline__ void count_primary(const CandCtx& cc, uint32_t n, uint32_t cut0) {
  Shared& sh = SH();
  uint32_t c = 0;
  for (uint32_t i = threadIdx.x; i < n; i += THREADS) c += cand_load(cc, i).x <= cut0 ? 1u : 0u;
  c = __reduce_add_sync(0xFFFFFFFFu, c);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(&sh.count0, c);
  __syncthreads();
}

// Everything after the complete-row pass of a sampled row: certification branch (Section 4.3),
// refinement or exact recovery, output commit.  The pass admitted the nested tail A(tau_1) and
// counted A(tau_0) inside it, so the band extension of an underfilled primary boundary costs no
// second pass: C(tau_0) >= K refines the entries with kd <= cut(tau_0), C(tau_0) < K <= C(tau_1)
// all of them.  A row that is still underfilled appends one wider band (tau_1, tau_2] in a
// second pass before it falls back to the storage-free recovery.  On entry the candidate arrays
// hold min(C1, cap) entries and sh.cand_count == C1.
template <int THREADS, int U, bool BLOCK_SEARCH = false>
__device__ void finish_sampled_row(const Params& P, const CandCtx cc, int row, int64_t g0, int64_t L, uint32_t C0,
                                   uint32_t C1, int tau_pack, uint64_t scanned, uint64_t sampled) {
  Shared& sh = SH();
  int32_t* oi = P.out_idx + (int64_t)row * P.K;
  float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
  const uint32_t K = (uint32_t)P.K, cap = (uint32_t)P.cap;
  int route;
  uint32_t cfin = 0, C = C1, cut_base = 0;
  if (C1 > cap) {
    route = HPCTOPK_ROUTE_OVERFLOW;
  } else if (C0 >= K) {
    route = HPCTOPK_ROUTE_PRIMARY; cfin = C0; cut_base = sh.cutd[0];
  } else if (C1 >= K) {
    route = HPCTOPK_ROUTE_BAND; cfin = C1; cut_base = sh.cutd[1];
  } else {
    route = HPCTOPK_ROUTE_RECOVERY;
    if (sh.cutd[3] > sh.cutd[1]) {
      __syncthreads();
      scan_range<THREADS, U, true>(P.scores, g0, g0, g0 + L, sh.cutd[1], sh.cutd[3], cc);
      __syncthreads();
      scanned += (uint64_t)L;
      const uint32_t C2 = sh.cand_count;
      if (C2 >= K && C2 <= cap) { route = HPCTOPK_ROUTE_BAND2; cfin = C2; C = C2; cut_base = sh.cutd[3]; }
    }
  }
  if (cfin) {
    if (!select_adaptive<THREADS, BLOCK_SEARCH>(cc, C, K, cut_base, sh.cutd[2], oi, ov)) {
      if (threadIdx.x == 0) add64(&stats_of(P.ws)->general_refinements, 1);
      __syncthreads();
      CandidateSource cs{cc, C, cut_base};
      select_and_emit<THREADS>(cs, K, false, oi, ov);
    }
  } else {
    RowSource rs{P.scores, g0, g0 + L};
    select_and_emit<THREADS>(rs, K, false, oi, ov);
    scanned += 4ull * (uint64_t)L;          // three digit passes and the commit pass, at least
  }
  record_row(P, row, route, tau_pack, C0, cfin, scanned, sampled, (uint64_t)L);
}

// A row owned by one CTA from Phase 1 to the output commit.
template <int THREADS, int U>
__device__ void process_row(const Params& P, int row, const CandCtx cc) {
  Shared& sh = SH();
  const int64_t g0 = row_start(P, row);
  int64_t L = P.row_lengths[row];
  if (L < 0) L = 0;
  const uint32_t K = (uint32_t)P.K, cap = (uint32_t)P.cap;
  int32_t* oi = P.out_idx + (int64_t)row * P.K;
  float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
  if (L <= (int64_t)K) {
    emit_short_row<THREADS>(P, row, g0, L);
    record_row(P, row, HPCTOPK_ROUTE_SHORT, -1, 0, 0, (uint64_t)L, 0, (uint64_t)L);
    return;
  }
  __syncthreads();
  if (L <= (int64_t)cap) {
    // direct route: the whole row is the admitted tail (C = L), refined on chip
    clear_hist<THREADS>(sh);
    if (threadIdx.x == 0) sh.cand_count = 0;
    __syncthreads();
    scan_range<THREADS, U, false>(P.scores, g0, g0, g0 + L, 0u, 0xFFFFFFFFu, cc);
    __syncthreads();
    CandidateSource cs{cc, (uint32_t)L};
    select_and_emit<THREADS>(cs, K, false, oi, ov);
    record_row(P, row, HPCTOPK_ROUTE_DIRECT, -1, (uint32_t)L, (uint32_t)L, (uint64_t)L, 0, (uint64_t)L);
    return;
  }
  int tau_pack;
  const long long t0 = tick();
  if (!row_boundary<THREADS>(P, row, g0, L, tau_pack)) {
    RowSource rs{P.scores, g0, g0 + L};
    select_and_emit<THREADS>(rs, K, false, oi, ov);
    record_row(P, row, HPCTOPK_ROUTE_RECOVERY, -1, 0, 0, 4ull * (uint64_t)L, 0, (uint64_t)L);
    return;
  }
  const long long t1 = tick();
  const uint64_t sampled = (uint64_t)((L + P.stride - 1) / P.stride);
  if (threadIdx.x == 0) { sh.cand_count = 0; sh.count0 = 0; }
  __syncthreads();
  scan_range<THREADS, U, false>(P.scores, g0, g0, g0 + L, 0u, sh.cutd[1], cc);
  __syncthreads();
  count_primary<THREADS>(cc, sh.cand_count < cap ? sh.cand_count : cap, sh.cutd[0]);
  const long long t2 = tick();
  finish_sampled_row<THREADS, U>(P, cc, row, g0, L, sh.count0, sh.cand_count, tau_pack, (uint64_t)L, sampled);
  if (threadIdx.x == 0) {
    hpctopk_stats* st = stats_of(P.ws);
    add64(&st->cycles_phase1, (uint64_t)(t1 - t0));
    add64(&st->cycles_scan, (uint64_t)(t2 - t1));
    add64(&st->cycles_finish, (uint64_t)(tick() - t2));
  }
}

// One segment of a KV-split row (Section 4.5): same boundary as every other segment of the row,
// private scan, publication into the row's global candidate range, last arriver finishes.
template <int THREADS, int U>
__device__ void process_segment(const Params& P, int row, int seg, int nseg) {
  Shared& sh = SH();
  const CandCtx cc = cand_ctx(P);
  const int64_t g0 = row_start(P, row);
  const int64_t L = P.row_lengths[row];       // > cap, checked when the table was built
  const int64_t g1 = g0 + L;
  const uint32_t cap = (uint32_t)P.cap;
  uint32_t* arrive = reinterpret_cast<uint32_t*>(P.ws + kOffSplit);
  uint32_t* rowcnt = arrive + kSplitRowsMax;
  const size_t cand_off = align_up(kOffRowInfo + (size_t)P.num_rows * sizeof(hpctopk_row_info), 256);
  uint2* gcand = reinterpret_cast<uint2*>(P.ws + cand_off) + (size_t)row * cap;

  int tau_pack;
  const long long t0 = tick();
  const bool usable = row_boundary<THREADS>(P, row, g0, L, tau_pack);
  const long long t1 = tick();
  // the view is read once per row when a boundary kernel ran, once per segment otherwise
  const uint64_t sampled = usable && (P.pipe_rec_off == 0 || seg == 0) ? (uint64_t)((L + P.stride - 1) / P.stride) : 0;
  // contiguous, 16-byte aligned partition of the row's vectors
  const int64_t va = g0 >> 2, vb = (g1 + 3) >> 2;
  const int64_t per = (vb - va + nseg - 1) / nseg;
  int64_t e0 = (va + (int64_t)seg * per) << 2, e1 = (va + (int64_t)(seg + 1) * per) << 2;
  if (e0 < g0) e0 = g0;
  if (e1 > g1) e1 = g1;
  if (e1 < e0) e1 = e0;
  // A split row admits the nested tail A(tau_1) in its one pass (and counts A(tau_0) inside it),
  // so that an underfilled primary boundary never costs the finisher a second, single-CTA pass.
  uint32_t* rowcnt0 = rowcnt + kSplitRowsMax;
  __syncthreads();
  if (threadIdx.x == 0) { sh.cand_count = 0; sh.count0 = 0; }
  __syncthreads();
  if (usable) scan_range<THREADS, U, false>(P.scores, g0, e0, e1, 0u, sh.cutd[1], cc);
  __syncthreads();
  if (usable) count_primary<THREADS>(cc, sh.cand_count < cap ? sh.cand_count : cap, sh.cutd[0]);
  const uint32_t Cp = sh.cand_count;
  const long long t2 = tick();
  if (threadIdx.x == 0) {
    sh.bcast0 = atomicAdd(&rowcnt[row], Cp);
    atomicAdd(&rowcnt0[row], sh.count0);
    hpctopk_stats* st = stats_of(P.ws);
    add64(&st->cycles_phase1, (uint64_t)(t1 - t0));
    add64(&st->cycles_scan, (uint64_t)(t2 - t1));
    add64(&st->elements_scanned, (uint64_t)(e1 - e0));
    if (sampled) add64(&st->elements_sampled, sampled);
  }
  __syncthreads();
  const uint32_t base = sh.bcast0;
  if (base + Cp <= cap) {
    for (uint32_t i = threadIdx.x; i < Cp; i += THREADS) gcand[base + i] = cand_load(cc, i);
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) sh.bcast1 = atomicAdd(&arrive[row], 1u);
  __syncthreads();
  if (sh.bcast1 != (uint32_t)(nseg - 1)) return;      // not the last arriver
  // ---- finisher: C(tau_0) = sum_p C_p, A(tau_0) = union of the published ranges (Eq. "split-reduce")
  __threadfence();
  const uint32_t C1 = *reinterpret_cast<volatile uint32_t*>(&rowcnt[row]);      // C(tau_1)
  const uint32_t C0 = *reinterpret_cast<volatile uint32_t*>(&rowcnt0[row]);     // C(tau_0)
  if (threadIdx.x == 0) add64(&stats_of(P.ws)->rows_split, 1);
  if (!usable) {
    RowSource rs{P.scores, g0, g1};
    select_and_emit<THREADS>(rs, (uint32_t)P.K, false, P.out_idx + (int64_t)row * P.K,
                             P.out_val ? P.out_val + (int64_t)row * P.K : nullptr);
    record_row(P, row, HPCTOPK_ROUTE_RECOVERY, -1, 0, 0, 4ull * (uint64_t)L, 0, (uint64_t)L);
    return;
  }
  __syncthreads();
  if (C1 <= cap) {
    for (uint32_t i = threadIdx.x; i < C1; i += THREADS) cand_store(cc, i, __ldcg(gcand + i));
  }
  if (threadIdx.x == 0) sh.cand_count = C1;
  __syncthreads();
  finish_sampled_row<THREADS, U>(P, cc, row, g0, L, C0, C1, tau_pack, 0, 0);
  if (threadIdx.x == 0) add64(&stats_of(P.ws)->cycles_finish, (uint64_t)(tick() - t2));
}

// ---------------------------------------------------------------- the persistent kernel
// Warm the L2 with the stride-s view of a row this CTA will own next, so that its Phase 1 does
// not start with a DRAM round trip.
template <int THREADS>
__device__ __forceinline__ void prefetch_view(const Params& P, int row) {
  const int64_t g0 = row_start(P, row);
  const int64_t L = P.row_lengths[row];
  if (L <= P.cap) return;
  const int s = P.stride;
  const int bits = 31 - __clz(s);
  const int a = bits ? (int)(__brev((uint32_t)(row & (s - 1))) >> (32 - bits)) : 0;
  const int64_t n_view = (L - a + s - 1) / s;
  const float* rowp = P.scores + g0 + a;
  for (int64_t t = threadIdx.x; t < n_view; t += THREADS)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + t * s));
}

// Warm the L2 with the first kPrefetchHeadBytes of the element range [e0, e1) a later task scans.
template <int THREADS>
__device__ __forceinline__ void prefetch_head(const Params& P, int64_t e0, int64_t e1) {
  const char* base = reinterpret_cast<const char*>(P.scores + e0);
  int64_t bytes = (e1 - e0) * 4;
  if (bytes > kPrefetchHeadBytes) bytes = kPrefetchHeadBytes;
  for (int64_t off = (int64_t)threadIdx.x * 128; off < bytes; off += (int64_t)THREADS * 128)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
}

// Unsplit calls hand rows out from the end of the batch: causal prefill lists rows by growing
// length, so this runs the longest rows first and leaves short ones to fill the tail of the grid.
__device__ __forceinline__ int row_of_task(const Params& P, uint32_t task) {
  return P.num_rows - 1 - (int)task;
}

// Device-side ragged dispatch (Section 4.5): every CTA derives the same task table from
// row_lengths.  seg_base[r] is the first task of row r, seg_base[num_rows] the task count; a long
// row gets ceil(L / S) segment tasks with S = max(16384, total / (grid' * kTasksPerCta)) rounded
// up to 4096 elements (grid' = grid minus the number of long rows), every other row one task.
// Contains block barriers.
template <int THREADS>
__device__ uint32_t build_task_table(const Params& P, uint32_t* seg_base) {
  Shared& sh = SH();
  const int tid = threadIdx.x;
  constexpr int RPT = (kSplitRowsMax + THREADS - 1) / THREADS;
  unsigned long long mine = 0;
  for (int j = 0; j < RPT; ++j) {
    const int r = tid * RPT + j;
    if (r < P.num_rows) { const int64_t L = P.row_lengths[r]; if (L > P.cap) mine += (unsigned long long)L + (1ull << 50); }   // length sum, row count above bit 50
  }
  for (int d = 16; d > 0; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);
  if ((tid & 31) == 0) { sh.hist[2 * (tid >> 5)] = (uint32_t)mine; sh.hist[2 * (tid >> 5) + 1] = (uint32_t)(mine >> 32); }
  __syncthreads();
  unsigned long long total = 0;
  for (int w = 0; w < THREADS / 32; ++w) total += (unsigned long long)sh.hist[2 * w] | ((unsigned long long)sh.hist[2 * w + 1] << 32);
  // one task per CTA, so that a row's boundary (recomputed by every segment's CTA) is on the
  // critical path once; every long row may add one partial segment, hence the correction
  const unsigned long long nlong = total >> 50;
  total &= (1ull << 50) - 1ull;
  unsigned long long target = (unsigned long long)gridDim.x * kTasksPerCta;
  if (target > 2ull * nlong) target -= nlong;
  unsigned long long S = (total + target - 1) / target;
  if (S < (unsigned long long)kSegMinElems) S = kSegMinElems;
  S = (S + 4095ull) / 4096ull * 4096ull;
  __syncthreads();
  uint32_t cnt[RPT];
  uint32_t sum = 0;
  for (int j = 0; j < RPT; ++j) {
    const int r = tid * RPT + j;
    cnt[j] = 0;
    if (r < P.num_rows) {
      const int64_t L = P.row_lengths[r];
      cnt[j] = (L > P.cap) ? (uint32_t)((L + (int64_t)S - 1) / (int64_t)S) : 1u;
    }
    sum += cnt[j];
  }
  const uint32_t incl = warp_inclusive_scan<THREADS>(sum);
  if ((tid & 31) == 31) sh.warp_sums[tid >> 5] = incl;
  __syncthreads();
  uint32_t woff = 0;
  for (int w = 0; w < (tid >> 5); ++w) woff += sh.warp_sums[w];
  uint32_t run = woff + incl - sum;
  for (int j = 0; j < RPT; ++j) {
    const int r = tid * RPT + j;
    if (r < P.num_rows) seg_base[r] = run;
    run += cnt[j];
    if (r == P.num_rows - 1) { seg_base[P.num_rows] = run; sh.total_tasks = run; }
  }
  __syncthreads();
  return sh.total_tasks;
}

template <int THREADS, int U, int MINB>
__global__ void __launch_bounds__(THREADS, MINB) hpctopk_kernel(const Params P) {
  Shared& sh = SH();
  uint32_t* const seg_base = reinterpret_cast<uint32_t*>(CAND() + P.cap_s);   // [kSplitRowsMax + 1], only when splitting
  uint32_t* task_counter = reinterpret_cast<uint32_t*>(P.ws + kOffCtrl);
  const int tid = threadIdx.x;

  stats_clear();
  __syncthreads();
  uint32_t total_tasks = (uint32_t)P.num_rows;
  if (P.split_enabled) total_tasks = build_task_table<THREADS>(P, seg_base);

  // Two statically assigned waves, then completion-order claiming from the device counter.
  // The claim for the task after next is issued at the top of each task, so its latency and the
  // L2 warm-up of the next row's view overlap the current row.
  uint32_t task = blockIdx.x;
  uint32_t next = blockIdx.x + gridDim.x;
  while (task < total_tasks) {
    const long long task_t0 = tick();
    if (tid == 0) sh.claim = (int32_t)(2u * gridDim.x + atomicAdd(task_counter, 1u));
    if (!P.split_enabled && next < total_tasks) {
      const int nrow = row_of_task(P, next);
      prefetch_view<THREADS>(P, nrow);
      const int64_t ng0 = row_start(P, nrow), nL = P.row_lengths[nrow];
      if (nL > P.K) prefetch_head<THREADS>(P, ng0, ng0 + nL);
    }
    if (P.split_enabled) {
      // largest r with seg_base[r] <= task
      int lo = 0, hi = P.num_rows - 1;
      while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (seg_base[mid] <= task) lo = mid; else hi = mid - 1; }
      const int row = lo;
      const int nseg = (int)(seg_base[row + 1] - seg_base[row]);
      if (nseg <= 1) process_row<THREADS, U>(P, row, cand_ctx(P));
      else process_segment<THREADS, U>(P, row, (int)(task - seg_base[row]), nseg);
    } else {
      process_row<THREADS, U>(P, row_of_task(P, task), cand_ctx(P));
    }
    __syncthreads();
    const uint32_t claimed = (uint32_t)sh.claim;
    if (tid == 0) {
      add64(&stats_of(P.ws)->tasks, 1);
      add64(&stats_of(P.ws)->cycles_total, (uint64_t)(tick() - task_t0));
    }
    __syncthreads();
    task = next;
    next = claimed;
  }
  __syncthreads();
  if (tid == 0) stats_flush(P.ws);
}


// ---------------------------------------------------------------- the three-kernel pipeline
// The same steps as hpctopk_kernel, cut at the two points where a row's CTA would otherwise stop
// streaming: (1) boundary kernel, Phase 1 of every sampled row; (2) pass kernel, nothing but
// complete-row passes, each leaving its admitted tail in the row's global candidate range;
// (3) refinement kernel, certification branch, Phase 3 and the output commit of every row.
// In the single kernel a CTA streams for about half of its time (Phase 1 and Phase 3 hold its
// registers and shared memory while its loads are stopped); here the pass kernel streams all the
// time and the short phases run at their own, higher occupancy.  Cost: the admitted tails cross
// HBM once each way (about 57 KB per row at K = 2048, 11 % of a 129 K-score row).
constexpr uint32_t kBand2Flag = 0x80000000u;    // in a row's admitted count: the tail includes the second band
__device__ __forceinline__ uint32_t* pipe_cnt(const Params& P) { return reinterpret_cast<uint32_t*>(P.ws + P.pipe_cnt_off) - P.row_begin; }
__device__ __forceinline__ uint2* pipe_cand(const Params& P, int row) {
  return reinterpret_cast<uint2*>(P.ws + P.pipe_cand_off) + (size_t)(row - P.row_begin) * (size_t)P.cap;
}

template <int THREADS>
__global__ void __launch_bounds__(THREADS) pipe_boundary_kernel(const Params P) {
  Shared& sh = SH();
  stats_clear();
  __syncthreads();
  for (int row = P.row_begin + blockIdx.x; row < P.row_end; row += gridDim.x) {
    const int64_t g0 = row_start(P, row);
    const int64_t L = P.row_lengths[row];
    int tau_pack = -1;
    bool usable = false;
    if (L > (int64_t)P.cap) usable = phase1<THREADS, true>(P, row, g0, L, tau_pack);
    __syncthreads();
    RowRec* rec = pipe_rec(P) + row;
    if (threadIdx.x < 4) rec->cutd[threadIdx.x] = usable ? sh.cutd[threadIdx.x] : 0u;
    if (threadIdx.x == 0) {
      rec->tau_pack = tau_pack;
      rec->usable = usable ? 1u : 0u;
      pipe_cnt(P)[row] = 0u;
    }
    __syncthreads();
  }
}

// The pass kernel's work on one row.
template <int THREADS, int U>
__device__ void pipe_pass_task(const Params& P, int row) {
  Shared& sh = SH();
  // entries beyond the on-chip part go straight to their place in the row's global range
  CandCtx cc;
  cc.cap_s = (uint32_t)P.cap_s; cc.cap = (uint32_t)P.cap; cc.spill = pipe_cand(P, row) + P.cap_s;
  const int64_t g0 = row_start(P, row);
  const int64_t L = P.row_lengths[row];
  if (L <= (int64_t)P.cap) return;                       // short and direct rows: refinement kernel
  const RowRec* rec = pipe_rec(P) + row;
  const uint4 r0 = __ldg(reinterpret_cast<const uint4*>(rec));
  const uint4 r1 = __ldg(reinterpret_cast<const uint4*>(rec) + 1);
  if (r1.y == 0u) return;                                // unusable view: refinement kernel recovers
  const uint32_t cut1 = r0.y, cap = (uint32_t)P.cap;
  const int64_t g1 = g0 + L;
  __syncthreads();
  if (threadIdx.x == 0) sh.cand_count = 0;
  __syncthreads();
  scan_range<THREADS, U, false>(P.scores, g0, g0, g1, 0u, cut1, cc);
  __syncthreads();
  uint32_t Cp = sh.cand_count;
  uint32_t flag = 0u;
  uint64_t scanned = (uint64_t)L;
  if (Cp < (uint32_t)P.K && r0.w > cut1) {
    // Underfilled row owned by this CTA: append the second band (tau_1, tau_2] here, where the
    // row has just passed through the L2 and 16 warps stream it, and tell the refinement kernel.
    __syncthreads();
    scan_range<THREADS, U, true>(P.scores, g0, g0, g1, cut1, r0.w, cc);
    __syncthreads();
    Cp = sh.cand_count;
    flag = kBand2Flag;
    scanned += (uint64_t)L;
  }
  if (threadIdx.x == 0) {
    pipe_cnt(P)[row] = Cp | flag;
    add64(&stats_of(P.ws)->elements_scanned, scanned);
  }
  if (Cp <= cap) {                                       // otherwise the refinement kernel recovers the row
    uint2* gc = pipe_cand(P, row);
    const uint32_t on_chip = Cp < cc.cap_s ? Cp : cc.cap_s;
    for (uint32_t i = threadIdx.x; i < on_chip; i += THREADS) gc[i] = CAND()[i];
  }
}

// One CTA per row, longest rows (highest row numbers of a causal batch) first; the hardware
// hands out CTAs as SM resources free up.  (4096 rows on 444 CTA slots take 10 row times where 9.2
// would do; handing out the rows of the last wave in quarter-row segments was measured and
// changed nothing - 467 against 468 us for boundary + pass - because the kernel is bound by DRAM
// bandwidth while all slots are busy and the few CTAs of a last wave run faster.)
template <int THREADS, int U, int MINB>
__global__ void __launch_bounds__(THREADS, MINB) pipe_pass_kernel(const Params P) {
  stats_clear();
  __syncthreads();
  pipe_pass_task<THREADS, U>(P, P.row_end - 1 - (int)blockIdx.x);
  __syncthreads();
  if (threadIdx.x == 0) {
    add64(&stats_of(P.ws)->tasks, 1);
    stats_flush(P.ws);
  }
}

// The refinement kernel keeps no candidates on chip: it reads a row's admitted tail from its
// global range (L2 for the most part, the pass kernel has just written it), so a CTA needs only
// the 8 KB histogram and many rows are in flight per SM; the refinement is a chain of short
// dependent steps and is bound by latency, not by bandwidth.  P.cap_s is 0 in this launch: the
// rare rows that need a staging area (direct rows, second band) use the CTA's global slice.
template <int THREADS, int U, int MINB>
__global__ void __launch_bounds__(THREADS, MINB) pipe_refine_kernel(const Params P) {
  Shared& sh = SH();
  const int tid = threadIdx.x;
  const uint32_t cap = (uint32_t)P.cap, K = (uint32_t)P.K;
  stats_clear();
  __syncthreads();
  {
    const int row = P.row_end - 1 - (int)blockIdx.x;
    // everything the row needs from global memory, requested together
    const RowRec* rec = pipe_rec(P) + row;
    const uint4 rq0 = __ldg(reinterpret_cast<const uint4*>(rec));
    const uint4 rq1 = __ldg(reinterpret_cast<const uint4*>(rec) + 1);
    const uint32_t cnt = __ldcg(&pipe_cnt(P)[row]);
    const int64_t g0 = row_start(P, row);
    const int64_t L = P.row_lengths[row];
    const bool sampled = L > (int64_t)cap && rq1.y != 0u;
    if (!sampled) {
      CandCtx rc;                                        // staging area: the row's own global range
      rc.cap_s = 0u; rc.cap = cap; rc.spill = pipe_cand(P, row);
      process_row<THREADS, U>(P, row, rc);               // short, direct, or recovery of an unusable view
    } else {
      __syncthreads();
      if (tid == 0) { sh.cutd[0] = rq0.x; sh.cutd[1] = rq0.y; sh.cutd[2] = rq0.z; sh.cutd[3] = rq0.w; }
      const int tau_pack = (int)rq1.x;
      const bool band2 = (cnt & kBand2Flag) != 0u;
      const uint32_t C1 = cnt & ~kBand2Flag;             // entries of A(tau_1), or of A(tau_2) with the flag
      if (tid == 0) { sh.cand_count = C1; sh.count0 = 0; }
      __syncthreads();
      CandCtx rc;                                        // the row's global candidate range
      rc.cap_s = 0u; rc.cap = cap; rc.spill = pipe_cand(P, row);
      const uint64_t sampled_n = (uint64_t)((L + P.stride - 1) / P.stride);
      int32_t* oi = P.out_idx + (int64_t)row * P.K;
      float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
      if (C1 >= K && C1 <= cap) {
        // The K best of a larger nested tail are the K best of every smaller one that holds K
        // entries, so the whole stored tail is refined against its own cutoff and C(tau_0) is
        // only counted (for the route the row reports).
        const uint32_t cut_base = band2 ? sh.cutd[3] : sh.cutd[1];
        if (!select_adaptive<THREADS, true, true, true>(rc, C1, K, cut_base, sh.cutd[2], oi, ov, sh.cutd[0])) {
          if (tid == 0) add64(&stats_of(P.ws)->general_refinements, 1);
          __syncthreads();
          CandidateSource cs{rc, C1, cut_base};
          select_and_emit<THREADS>(cs, K, false, oi, ov);
        }
        const uint32_t C0 = sh.count0;
        const int route = band2 ? HPCTOPK_ROUTE_BAND2 : (C0 >= K ? HPCTOPK_ROUTE_PRIMARY : HPCTOPK_ROUTE_BAND);
        record_row(P, row, route, tau_pack, C0, route == HPCTOPK_ROUTE_PRIMARY ? C0 : C1, 0, sampled_n, (uint64_t)L);
      } else if (!band2) {
        // a split row that is still short, or a tail beyond the capacity: the general branch
        count_primary<THREADS>(rc, C1 <= cap ? C1 : 0u, sh.cutd[0]);
        finish_sampled_row<THREADS, U, true>(P, rc, row, g0, L, sh.count0, C1, tau_pack, 0, sampled_n);
      } else {
        // the second band was tried by the pass kernel and did not certify the row
        count_primary<THREADS>(rc, C1 <= cap ? C1 : 0u, sh.cutd[0]);
        RowSource rs{P.scores, g0, g0 + L};
        select_and_emit<THREADS>(rs, K, false, oi, ov);
        record_row(P, row, C1 > cap ? HPCTOPK_ROUTE_OVERFLOW : HPCTOPK_ROUTE_RECOVERY, tau_pack, sh.count0, 0,
                   4ull * (uint64_t)L, sampled_n, (uint64_t)L);
      }
    }
  }
  __syncthreads();
  if (tid == 0) stats_flush(P.ws);
}


// ---------------------------------------------------------------- ordered output (optional)
// Sorts the K slots of every row in place by (score descending under the key, index ascending);
// sentinel slots stay last.  One CTA per row, bitonic sort of 64-bit composites (kd << 32 | idx)
// in shared memory (N = smallest power of two >= K, at most 4096 entries = 32 KB).
template <int THREADS>
__global__ void __launch_bounds__(THREADS) sort_rows_kernel(const Params P) {
  extern __shared__ __align__(16) unsigned char sort_smem[];
  unsigned long long* a = reinterpret_cast<unsigned long long*>(sort_smem);
  const int row = blockIdx.x;
  const uint32_t K = (uint32_t)P.K;
  uint32_t N = 1;
  while (N < K) N <<= 1;
  const int64_t g0 = row_start(P, row);
  int32_t* oi = P.out_idx + (int64_t)row * P.K;
  float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
  for (uint32_t i = threadIdx.x; i < N; i += THREADS) {
    unsigned long long v = ~0ull;                                  // sentinel and padding slots sort last
    if (i < K) {
      const int32_t idx = oi[i];
      if (idx >= 0) {
        const uint32_t u = __float_as_uint(ov ? ov[i] : __ldg(P.scores + g0 + idx));
        v = ((unsigned long long)kd_of_bits(u) << 32) | (uint32_t)idx;
      }
    }
    a[i] = v;
  }
  __syncthreads();
  for (uint32_t k = 2; k <= N; k <<= 1) {
    for (uint32_t j = k >> 1; j > 0; j >>= 1) {
      for (uint32_t p = threadIdx.x; p < (N >> 1); p += THREADS) {     // one compare-exchange per pair
        const uint32_t i = ((p & ~(j - 1u)) << 1) | (p & (j - 1u));       // j is a power of two
        const uint32_t l = i | j;
        const unsigned long long x = a[i], y = a[l];
        const bool up = (i & k) == 0;
        if ((x > y) == up) { a[i] = y; a[l] = x; }
      }
      __syncthreads();
    }
  }
  for (uint32_t i = threadIdx.x; i < K; i += THREADS) {
    const unsigned long long v = a[i];
    const bool valid = v != ~0ull;
    oi[i] = valid ? (int32_t)(uint32_t)v : -1;
    if (ov) ov[i] = valid ? __uint_as_float(bits_of_kd((uint32_t)(v >> 32))) : __uint_as_float(0xFF800000u);
  }
}

}  // namespace
#include "hpctopk_ws.cuh"            // namespace wsk: scanner warps + helper groups
#define HPCTOPK_WS_NAMESPACE wsf     // namespace wsf: single-role variant, warp-synchronous compaction
#define HPCTOPK_WS_FUSED 1
#define HPCTOPK_NS 16
#ifndef HPCTOPK_FUSED_MINB
#define HPCTOPK_FUSED_MINB 2
#endif
#ifndef HPCTOPK_FUSED_U
#define HPCTOPK_FUSED_U 2
#endif
#define HPCTOPK_WS_U HPCTOPK_FUSED_U
#define HPCTOPK_WS_MINB HPCTOPK_FUSED_MINB
#include "hpctopk_ws.cuh"
namespace {

// ---------------------------------------------------------------- host side
using KernelFn = void (*)(const Params);
struct Variant {
  KernelFn fn;
  int threads;
};
// Launch shapes (threads per CTA, register tiles per thread, minimum CTAs per SM).  Index 0 is
// the default; the others exist for tuning runs (environment variable HPCTOPK_VARIANT).
const Variant kVariants[] = {
    {hpctopk_kernel<512, 2, 2>, 512},
    {hpctopk_kernel<256, 2, 4>, 256},
    {hpctopk_kernel<256, 4, 3>, 256},
    {hpctopk_kernel<512, 2, 3>, 512},
    {hpctopk_kernel<384, 2, 4>, 384},
    {hpctopk_kernel<640, 2, 2>, 640},
    {hpctopk_kernel<512, 1, 3>, 512},
    {hpctopk_kernel<1024, 1, 1>, 1024},
    {hpctopk_kernel<1024, 2, 1>, 1024},
    {hpctopk_kernel<448, 2, 3>, 448},
    {hpctopk_kernel<384, 2, 3>, 384},
};
constexpr int kNumVariants = sizeof(kVariants) / sizeof(kVariants[0]);
// 0 selects the warp-specialised kernel, v >= 1 the single-role kernel kVariants[v - 1].
// kPipeVariant selects the three-kernel pipeline for calls beyond the split-mode row count, one
// launch of the three per kPipeRowsMax rows (the per-row workspace regions are sized for that many).
constexpr int kPipeVariant = 200;
constexpr int kDefaultVariant = kPipeVariant;
constexpr int kMonoVariant = 4;
constexpr int kSplitVariant = 1;
constexpr int kPipeRowsMax = 8192;
constexpr int kTimingSlots = 1024;
constexpr int kBoundaryThreads = 128;
#ifndef HPCTOPK_REFINE_T
#define HPCTOPK_REFINE_T 128
#define HPCTOPK_REFINE_MINB 8
#endif
constexpr int kRefineThreads = HPCTOPK_REFINE_T;
constexpr int kFusedVariant = 100;     // single-role kernel with warp-synchronous compaction (namespace wsf)

struct DeviceInfo {
  bool ready = false;
  int sm_count = 0;
  int variant = 0;      // 0: warp-specialised kernel; v >= 1: single-role kernel kVariants[v - 1]
  int ctas_per_sm[2][3] = {{0, 0, 0}, {0, 0, 0}};   // [split][capacity class]
  int boundary_per_sm = 0;                          // pipeline: boundary kernel
  bool timing = false;                              // hpctopk_stage_timing
  int timed = 0;                                    // event pairs recorded since the last read
  int timed_calls = 0;                              // calls they belong to (a call of many rows records several)
  cudaEvent_t ev0[kTimingSlots] = {}, ev1[kTimingSlots] = {};
  int pipe_stages = 3;                              // tuning: run only the first n kernels (HPCTOPK_PIPE_STAGES)
};
DeviceInfo g_dev[64];
std::mutex g_setup_mutex;

size_t smem_bytes_for(int cap_s, bool split) {
  size_t b = align_up(sizeof(Shared), 16) + (size_t)cap_s * 8;
  if (split) b += (kSplitRowsMax + 1) * sizeof(uint32_t);
  return align_up(b, 16);
}

// Index into kVariants for a call: calls with few rows (split mode) are latency-bound and
// prefer fewer, fatter CTAs per SM than the streaming default.
int variant_index(int variant, bool split) {
  if (variant == kPipeVariant) variant = kMonoVariant;
  const int v = (variant == kMonoVariant && split) ? kSplitVariant : variant;
  return (v > 0 && v <= kNumVariants) ? v - 1 : 0;
}

// Shared memory is sized by capacity class so that occupancy (and the grid) depends on K only.
int cap_class(int K) { return K <= 1024 ? 0 : (K <= 2048 ? 1 : 2); }
int class_cap_s(int cls) { return smem_capacity_for(cls == 0 ? 1024 : (cls == 1 ? 2048 : HPCTOPK_MAX_K)); }

// Workspace layout of the pipeline: the common head (control block, counters, row records of
// hpctopk_read_row_info), then boundary records, admitted counts and one candidate range of
// `capacity` entries per row (a pass CTA writes what exceeds its shared memory straight into
// that range, and the refinement kernel stages nothing on chip, so there are no overflow slices).
struct PipeLayout { size_t rec, cnt, cand, total; };
PipeLayout pipe_layout(int all_rows, int K) {
  const size_t cap = (size_t)capacity_for(K);
  const int rows = all_rows < kPipeRowsMax ? all_rows : kPipeRowsMax;      // rows of one launch
  PipeLayout l;
  l.rec = align_up(kOffRowInfo + (size_t)all_rows * sizeof(hpctopk_row_info), 256);
  l.cnt = align_up(l.rec + (size_t)rows * sizeof(RowRec), 256);
  l.cand = align_up(l.cnt + (size_t)rows * sizeof(uint32_t), 256);
  l.total = align_up(l.cand + (size_t)rows * cap * 8, 256);
  return l;
}

#ifndef HPCTOPK_PASS_T
#define HPCTOPK_PASS_T 512
#define HPCTOPK_PASS_MINB 3
#endif
#ifndef HPCTOPK_PASS_U
#define HPCTOPK_PASS_U 2
#endif
const auto kPassKernel = pipe_pass_kernel<HPCTOPK_PASS_T, HPCTOPK_PASS_U, HPCTOPK_PASS_MINB>;
constexpr int kPassThreads = HPCTOPK_PASS_T;
const auto kRefineKernel = pipe_refine_kernel<kRefineThreads, 2, HPCTOPK_REFINE_MINB>;
const auto kBoundaryKernel = pipe_boundary_kernel<kBoundaryThreads>;

// Policy override for ablation runs (hpctopk_set_policy); all zero: the built-in policy.
struct PolicyOverride { int32_t stride = 0, rho = 0, rho1 = 0; };
PolicyOverride g_policy;

// Event pair for this call, or -1 when stage timing is off, full, or the stream is being captured.
int timing_slot(DeviceInfo& di, cudaStream_t st) {
  if (!di.timing || di.timed >= kTimingSlots) return -1;
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) { cudaGetLastError(); return -1; }
  return di.timed++;
}

}  // namespace

extern "C" {

int hpctopk_set_policy(int32_t stride, int32_t rho_permille, int32_t rho1_permille) {
  if (stride == 0 && rho_permille == 0 && rho1_permille == 0) { g_policy = PolicyOverride(); return HPCTOPK_OK; }
  if (stride < 1 || stride > 1024 || (stride & (stride - 1)) != 0) return HPCTOPK_ERR_INVALID_ARG;
  if (rho_permille < 1000 || rho1_permille < rho_permille || rho1_permille > 2500) return HPCTOPK_ERR_INVALID_ARG;
  g_policy.stride = stride; g_policy.rho = rho_permille; g_policy.rho1 = rho1_permille;
  return HPCTOPK_OK;
}

int hpctopk_stage_timing(int enable) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HPCTOPK_ERR_CUDA;
  DeviceInfo& di = g_dev[dev];
  if (enable && !di.ev0[0]) {
    for (int i = 0; i < kTimingSlots; ++i)
      if (cudaEventCreate(&di.ev0[i]) != cudaSuccess || cudaEventCreate(&di.ev1[i]) != cudaSuccess) {
        cudaGetLastError();
        return HPCTOPK_ERR_CUDA;
      }
  }
  di.timing = enable != 0;
  return HPCTOPK_OK;
}

int hpctopk_read_stage_timing(float* total_ms, int32_t* calls) {
  if (!total_ms || !calls) return HPCTOPK_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HPCTOPK_ERR_CUDA;
  DeviceInfo& di = g_dev[dev];
  float sum = 0.f;
  for (int i = 0; i < di.timed; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(di.ev1[i]) != cudaSuccess || cudaEventElapsedTime(&ms, di.ev0[i], di.ev1[i]) != cudaSuccess) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    sum += ms;
  }
  *total_ms = sum;
  *calls = di.timed_calls;
  di.timed = 0;
  di.timed_calls = 0;
  return HPCTOPK_OK;
}

int hpctopk_version(void) { return 1000 * 0 + 1; }

const char* hpctopk_status_string(int status) {
  switch (status) {
    case HPCTOPK_OK: return "ok";
    case HPCTOPK_ERR_INVALID_ARG: return "invalid argument";
    case HPCTOPK_ERR_UNSUPPORTED_K: return "K exceeds HPCTOPK_MAX_K";
    case HPCTOPK_ERR_MISALIGNED: return "misaligned scores or workspace pointer";
    case HPCTOPK_ERR_WORKSPACE: return "workspace error";
    case HPCTOPK_ERR_CUDA: return "CUDA runtime error";
    case HPCTOPK_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

size_t hpctopk_workspace_bytes(int32_t max_num_rows, int32_t K) {
  if (max_num_rows < 0 || K < 1 || K > HPCTOPK_MAX_K) return 0;
  const size_t cap = (size_t)capacity_for(K);
  const int cap_s_cls = class_cap_s(cap_class(K));
  const size_t cap_s = (size_t)cap_s_cls < cap ? (size_t)cap_s_cls : cap;
  const size_t split_rows = max_num_rows < kSplitRowsMax ? (size_t)max_num_rows : (size_t)kSplitRowsMax;
  size_t b = align_up(kOffRowInfo + (size_t)max_num_rows * sizeof(hpctopk_row_info), 256);
  b += split_rows * cap * 8;                       // published candidate ranges of split rows
  size_t spill = (size_t)kMaxGrid * (cap - cap_s) * 8;       // one overflow slice per resident CTA
  const size_t spill_ws = wsk::ws_spill_bytes(K, wsk::kWsMaxGrid);
  if (spill_ws > spill) spill = spill_ws;
  const size_t spill_wf = wsf::ws_spill_bytes(K, kMaxGrid);
  if (spill_wf > spill) spill = spill_wf;
  b += spill;
  b = align_up(b, 256);
  {
    const size_t p = pipe_layout(max_num_rows, K).total;
    if (p > b) b = p;
  }
  return b;
}

int hpctopk_kernels_per_call(int32_t num_rows) {
  if (num_rows <= 0) return 0;
  const char* env = getenv("HPCTOPK_VARIANT");
  const int variant = env ? atoi(env) : kDefaultVariant;
  if (variant != kPipeVariant || num_rows <= kSplitRowsMax) return 1;
  return 3 * ((num_rows + kPipeRowsMax - 1) / kPipeRowsMax);
}

int hpctopk_query_policy(int32_t K, int64_t L, int32_t* stride, int32_t* capacity, int32_t* route) {
  if (K < 1) return HPCTOPK_ERR_INVALID_ARG;
  if (K > HPCTOPK_MAX_K) return HPCTOPK_ERR_UNSUPPORTED_K;
  if (stride) *stride = g_policy.stride ? g_policy.stride : stride_for(K);
  if (capacity) *capacity = capacity_for(K);
  if (route) *route = L <= K ? HPCTOPK_ROUTE_SHORT : (L <= capacity_for(K) ? HPCTOPK_ROUTE_DIRECT : HPCTOPK_ROUTE_PRIMARY);
  return HPCTOPK_OK;
}

static int select_impl(const float* scores, const int32_t* row_starts, int64_t pitch, const int32_t* row_lengths,
                       int32_t num_rows, int32_t K, int32_t* out_idx, float* out_val,
                       void* workspace, hpctopk_stream_t stream);

int hpctopk_select(const float* scores, const int32_t* row_starts, const int32_t* row_lengths,
                   int32_t num_rows, int32_t K, int32_t* out_idx, float* out_val,
                   void* workspace, hpctopk_stream_t stream) {
  if (num_rows > 0 && !row_starts) return HPCTOPK_ERR_INVALID_ARG;
  return select_impl(scores, row_starts, 0, row_lengths, num_rows, K, out_idx, out_val, workspace, stream);
}

int hpctopk_select_padded(const float* scores, int64_t pitch, const int32_t* row_lengths,
                          int32_t num_rows, int32_t K, int32_t* out_idx, float* out_val,
                          void* workspace, hpctopk_stream_t stream) {
  if (pitch < 0) return HPCTOPK_ERR_INVALID_ARG;
  return select_impl(scores, nullptr, pitch, row_lengths, num_rows, K, out_idx, out_val, workspace, stream);
}

static int select_impl(const float* scores, const int32_t* row_starts, int64_t pitch, const int32_t* row_lengths,
                       int32_t num_rows, int32_t K, int32_t* out_idx, float* out_val,
                       void* workspace, hpctopk_stream_t stream) {
  if (num_rows < 0 || K < 1) return HPCTOPK_ERR_INVALID_ARG;
  if (K > HPCTOPK_MAX_K) return HPCTOPK_ERR_UNSUPPORTED_K;
  if (num_rows == 0) return HPCTOPK_OK;
  if (!scores || !row_lengths || !out_idx || !workspace) return HPCTOPK_ERR_INVALID_ARG;
  if (((uintptr_t)scores & 15u) || ((uintptr_t)workspace & 255u)) return HPCTOPK_ERR_MISALIGNED;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HPCTOPK_ERR_CUDA;
  DeviceInfo& di = g_dev[dev];
  const bool split = num_rows <= kSplitRowsMax;
  std::unique_lock<std::mutex> setup_lock(g_setup_mutex);      // first call per device: one thread sets up
  if (!di.ready) {
    if (cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return HPCTOPK_ERR_CUDA;
    init_cut_table_kernel<<<kBins * 32 / 256, 256>>>();
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return HPCTOPK_ERR_CUDA; }
    if (const char* stg = getenv("HPCTOPK_PIPE_STAGES")) di.pipe_stages = atoi(stg);
    const char* env = getenv("HPCTOPK_VARIANT");
    di.variant = env ? atoi(env) : kDefaultVariant;
    if (di.variant != kFusedVariant && di.variant != kPipeVariant && (di.variant < 0 || di.variant > kNumVariants)) di.variant = kDefaultVariant;
    if (cudaFuncSetAttribute(wsk::hpctopk_ws_kernel<wsk::kWsU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)wsk::ws_smem_bytes(HPCTOPK_MAX_K, true)) != cudaSuccess) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    if (cudaFuncSetAttribute(wsf::hpctopk_ws_kernel<wsf::kWsU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)wsf::ws_smem_bytes(HPCTOPK_MAX_K, true)) != cudaSuccess) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    const size_t max_smem = smem_bytes_for(class_cap_s(2), true);
    for (int sp = 0; sp < 2; ++sp) {
      const Variant& v = kVariants[variant_index(di.variant, sp != 0)];
      if (cudaFuncSetAttribute(v.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem) != cudaSuccess) {
        cudaGetLastError();
        return HPCTOPK_ERR_CUDA;
      }
      for (int c = 0; c < 3; ++c) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, v.fn, v.threads, smem_bytes_for(class_cap_s(c), sp != 0)) != cudaSuccess || n < 1) {
          cudaGetLastError();
          return HPCTOPK_ERR_CUDA;
        }
        di.ctas_per_sm[sp][c] = n;
      }
    }
    if (cudaFuncSetAttribute(kPassKernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(kRefineKernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem) != cudaSuccess) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&di.boundary_per_sm, kBoundaryKernel, kBoundaryThreads,
                                                      align_up(sizeof(Shared), 16)) != cudaSuccess || di.boundary_per_sm < 1) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    di.ready = true;
  }
  setup_lock.unlock();
  const Variant& v = kVariants[variant_index(di.variant, split)];
  const int cls = cap_class(K);
  Params P;
  P.scores = scores; P.row_starts = row_starts; P.pitch = pitch; P.row_lengths = row_lengths;
  P.num_rows = num_rows; P.K = K; P.out_idx = out_idx; P.out_val = out_val;
  P.ws = static_cast<unsigned char*>(workspace);
  P.cap = capacity_for(K);
  P.cap_s = class_cap_s(cls) < P.cap ? class_cap_s(cls) : P.cap;
  P.stride = g_policy.stride ? g_policy.stride : stride_for(K);
  if (g_policy.stride) {                                   // ablation runs: margins in permille
    P.q0 = (int32_t)(((int64_t)g_policy.rho * K + 1000ll * P.stride - 1) / (1000ll * P.stride));
    P.q1 = (int32_t)(((int64_t)g_policy.rho1 * K + 1000ll * P.stride - 1) / (1000ll * P.stride));
  } else {
    P.q0 = (3 * K + 2 * P.stride - 1) / (2 * P.stride);    // ceil(1.5 K / s)
    P.q1 = (7 * K + 4 * P.stride - 1) / (4 * P.stride);    // ceil(1.75 K / s)
  }
  P.split_enabled = split ? 1 : 0;
  P.pipe_rec_off = P.pipe_cnt_off = P.pipe_cand_off = P.pipe_spill_off = 0;
  const size_t smem = smem_bytes_for(class_cap_s(cls), split);
  int grid = di.sm_count * di.ctas_per_sm[split ? 1 : 0][cls];
  if (grid > kMaxGrid) grid = kMaxGrid;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(workspace, 0, kZeroBytes, st) != cudaSuccess) { cudaGetLastError(); return HPCTOPK_ERR_CUDA; }
  // Calls of few rows (split mode) are latency-bound: one launch and on-chip tails serve them better.
  if (di.variant == kPipeVariant && !split) {
    const PipeLayout l = pipe_layout(num_rows, K);
    P.pipe_rec_off = (int64_t)l.rec; P.pipe_cnt_off = (int64_t)l.cnt;
    P.pipe_cand_off = (int64_t)l.cand;
    // Three launches on the caller's stream.  (Cutting the rows into chunks and overlapping the
    // boundary and refinement kernels of neighbouring chunks with the pass kernel on extra streams
    // was measured: no gain, the streaming CTAs leave no room on the SMs until they exit, and
    // limiting them to two per SM costs the pass kernel more than the overlap returns.  Letting
    // the refinement kernel of one chunk share the SMs with the boundary kernel of the next,
    // between two pass kernels, was measured too: every extra chunk costs about 85 us, because
    // each pass kernel then drains and the next one ramps up.)
    const size_t smem_pass = smem_bytes_for(class_cap_s(cls), false);
    const size_t smem_small = smem_bytes_for(0, false);
    // calls of more than kPipeRowsMax rows run as consecutive launches over row chunks, longest
    // rows first, which reuse the per-row regions of the workspace
    bool counted = false;
    for (int hi = num_rows; hi > 0; hi -= kPipeRowsMax) {
      P.row_end = hi;
      P.row_begin = hi > kPipeRowsMax ? hi - kPipeRowsMax : 0;
      const int rows = P.row_end - P.row_begin;
      int g1 = di.sm_count * di.boundary_per_sm;
      if (g1 > rows) g1 = rows;
      kBoundaryKernel<<<g1, kBoundaryThreads, smem_small, st>>>(P);
      const int slot = timing_slot(di, st);
      if (slot >= 0) {
        cudaEventRecord(di.ev0[slot], st);
        if (!counted) { ++di.timed_calls; counted = true; }
      }
      if (di.pipe_stages >= 2) kPassKernel<<<rows, kPassThreads, smem_pass, st>>>(P);
      if (slot >= 0) cudaEventRecord(di.ev1[slot], st);
      Params R = P;
      R.cap_s = 0;
      if (di.pipe_stages >= 3) kRefineKernel<<<rows, kRefineThreads, smem_bytes_for(K, false), st>>>(R);   // + 2K words of output staging
    }
  } else if (di.variant == kFusedVariant) {
    const size_t fsmem = wsf::ws_smem_bytes(K, split);
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, wsf::hpctopk_ws_kernel<wsf::kWsU>, wsf::THREADS, fsmem) != cudaSuccess || per_sm < 1) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    int fgrid = di.sm_count * per_sm;
    if (fgrid > kMaxGrid) fgrid = kMaxGrid;
    wsf::hpctopk_ws_kernel<wsf::kWsU><<<fgrid, wsf::THREADS, fsmem, st>>>(P);
  } else if (di.variant == 0) {
    int ws_grid = di.sm_count < wsk::kWsMaxGrid ? di.sm_count : wsk::kWsMaxGrid;
    wsk::hpctopk_ws_kernel<wsk::kWsU><<<ws_grid, wsk::THREADS, wsk::ws_smem_bytes(K, split), st>>>(P);
  } else {
    // (A boundary kernel in front of a split call, so that Phase 1 runs once per row instead of
    // once per segment, was measured: the segments' Phase 1 run side by side anyway and the extra
    // launch is serial - config 2 went from 58 to 71 us, config 4 from 75 to 69 us.  Left out.)
    const int slot = timing_slot(di, st);
    if (slot >= 0) { cudaEventRecord(di.ev0[slot], st); ++di.timed_calls; }
    v.fn<<<grid, v.threads, smem, st>>>(P);
    if (slot >= 0) cudaEventRecord(di.ev1[slot], st);
  }
  if (cudaGetLastError() != cudaSuccess) return HPCTOPK_ERR_CUDA;
  return HPCTOPK_OK;
}

int hpctopk_sort_output(const float* scores, const int32_t* row_starts, int64_t pitch, int32_t num_rows, int32_t K,
                        int32_t* out_idx, float* out_val, hpctopk_stream_t stream) {
  if (num_rows < 0 || K < 1 || pitch < 0) return HPCTOPK_ERR_INVALID_ARG;
  if (K > HPCTOPK_MAX_K) return HPCTOPK_ERR_UNSUPPORTED_K;
  if (num_rows == 0) return HPCTOPK_OK;
  if (!out_idx || (!out_val && !scores)) return HPCTOPK_ERR_INVALID_ARG;
  Params P;
  P.scores = scores; P.row_starts = row_starts; P.pitch = pitch; P.row_lengths = nullptr;
  P.num_rows = num_rows; P.K = K; P.out_idx = out_idx; P.out_val = out_val; P.ws = nullptr;
  P.cap = P.cap_s = 0; P.stride = 1; P.q0 = P.q1 = 0; P.split_enabled = 0;
  P.pipe_rec_off = P.pipe_cnt_off = P.pipe_cand_off = P.pipe_spill_off = 0;
  P.row_begin = 0; P.row_end = num_rows;
  size_t n = 1;
  while (n < (size_t)K) n <<= 1;
  sort_rows_kernel<512><<<num_rows, 512, n * sizeof(unsigned long long), reinterpret_cast<cudaStream_t>(stream)>>>(P);
  if (cudaGetLastError() != cudaSuccess) return HPCTOPK_ERR_CUDA;
  return HPCTOPK_OK;
}

int hpctopk_read_stats(const void* workspace, hpctopk_stats* host_out, hpctopk_stream_t stream) {
  if (!workspace || !host_out) return HPCTOPK_ERR_INVALID_ARG;
  if (cudaMemcpyAsync(host_out, static_cast<const unsigned char*>(workspace) + kOffStats, sizeof(hpctopk_stats),
                      cudaMemcpyDeviceToHost, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return HPCTOPK_ERR_CUDA;
  }
  return HPCTOPK_OK;
}

int hpctopk_read_row_info(const void* workspace, int32_t num_rows, hpctopk_row_info* host_out,
                          hpctopk_stream_t stream) {
  if (!workspace || !host_out || num_rows < 0) return HPCTOPK_ERR_INVALID_ARG;
  if (num_rows == 0) return HPCTOPK_OK;
  if (cudaMemcpyAsync(host_out, static_cast<const unsigned char*>(workspace) + kOffRowInfo,
                      (size_t)num_rows * sizeof(hpctopk_row_info), cudaMemcpyDeviceToHost,
                      reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return HPCTOPK_ERR_CUDA;
  }
  return HPCTOPK_OK;
}

}  // extern "C"

// ---------------------------------------------------------------- selection without a caller workspace
// Scratch for hpctopk_select_static: one fixed array per GPU that loads the library, held until
// the process exits.  In host code `g_static_scratch` is only a handle for the runtime; the
// device address is obtained once per device with cudaGetSymbolAddress and cached below.
namespace {
constexpr int kStaticMaxRows = HPCTOPK_STATIC_MAX_ROWS;
constexpr int kStaticMaxK = HPCTOPK_STATIC_MAX_K;
constexpr int kStaticMaxGrid = 160;
constexpr size_t static_layout_bytes(size_t rows, size_t cap, size_t cap_s, size_t grid) {
  return ((kOffRowInfo + rows * sizeof(hpctopk_row_info) + 255) / 256 * 256)   // control block, counters, row records
         + (rows < (size_t)kSplitRowsMax ? rows : (size_t)kSplitRowsMax) * cap * 8   // published ranges of split rows
         + grid * (cap - cap_s) * 8;                                           // overflow slice per CTA
}
constexpr size_t kStaticScratchBytes =
    (static_layout_bytes(kStaticMaxRows, 4 * kStaticMaxK, 2 * kStaticMaxK, kStaticMaxGrid) + 255) / 256 * 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void* g_static_scratch_addr[64] = {nullptr};
}  // namespace

extern "C" int hpctopk_select_static(const float* scores, const int32_t* row_starts, const int32_t* row_lengths,
                                     int32_t num_rows, int32_t K, int32_t* out_idx, float* out_val,
                                     hpctopk_stream_t stream) {
  if (num_rows < 0 || K < 1) return HPCTOPK_ERR_INVALID_ARG;
  if (K > kStaticMaxK || num_rows > kStaticMaxRows) return HPCTOPK_ERR_WORKSPACE;   // beyond the fixed scratch
  if (num_rows == 0) return HPCTOPK_OK;
  if (!scores || !row_starts || !row_lengths || !out_idx) return HPCTOPK_ERR_INVALID_ARG;
  if ((uintptr_t)scores & 15u) return HPCTOPK_ERR_MISALIGNED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HPCTOPK_ERR_CUDA;
  const Variant& v = kVariants[0];
  static int sm_count[64] = {0};
  static int ctas_per_sm[64][3] = {{0}};
  if (!g_static_scratch_addr[dev]) {
    // one-time set-up on this device (the device is current): resolve the array's device address
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) { cudaGetLastError(); return HPCTOPK_ERR_CUDA; }
    init_cut_table_kernel<<<kBins * 32 / 256, 256>>>();      // bin -> cutoff table used by Phase 1
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return HPCTOPK_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return HPCTOPK_ERR_CUDA;
    if (cudaFuncSetAttribute(v.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes_for(class_cap_s(2), true)) != cudaSuccess) {
      cudaGetLastError();
      return HPCTOPK_ERR_CUDA;
    }
    for (int c = 0; c < 3; ++c) {
      int n = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, v.fn, v.threads, smem_bytes_for(class_cap_s(c), true)) != cudaSuccess || n < 1) {
        cudaGetLastError();
        return HPCTOPK_ERR_CUDA;
      }
      ctas_per_sm[dev][c] = n;
    }
    g_static_scratch_addr[dev] = addr;
  }
  const int cls = cap_class(K);
  Params P;
  P.scores = scores; P.row_starts = row_starts; P.pitch = 0; P.row_lengths = row_lengths;
  P.num_rows = num_rows; P.K = K; P.out_idx = out_idx; P.out_val = out_val;
  P.ws = static_cast<unsigned char*>(g_static_scratch_addr[dev]);
  P.cap = capacity_for(K);
  P.cap_s = class_cap_s(cls) < P.cap ? class_cap_s(cls) : P.cap;
  P.stride = stride_for(K);
  P.q0 = (3 * K + 2 * P.stride - 1) / (2 * P.stride);
  P.q1 = (7 * K + 4 * P.stride - 1) / (4 * P.stride);
  P.split_enabled = 1;                                   // num_rows <= kStaticMaxRows <= kSplitRowsMax
  P.pipe_rec_off = P.pipe_cnt_off = P.pipe_cand_off = P.pipe_spill_off = 0;
  int grid = sm_count[dev] * ctas_per_sm[dev][cls];
  if (grid > kStaticMaxGrid) grid = kStaticMaxGrid;
  if (static_layout_bytes((size_t)num_rows, (size_t)P.cap, (size_t)P.cap_s, (size_t)grid) > kStaticScratchBytes) return HPCTOPK_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the control block must start at zero
  if (cudaMemsetAsync(P.ws, 0, kZeroBytes, st) != cudaSuccess) { cudaGetLastError(); return HPCTOPK_ERR_CUDA; }
  v.fn<<<grid, v.threads, smem_bytes_for(class_cap_s(cls), true), st>>>(P);
  if (cudaGetLastError() != cudaSuccess) return HPCTOPK_ERR_CUDA;
  return HPCTOPK_OK;
}
