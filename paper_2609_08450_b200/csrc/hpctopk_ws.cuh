// Warp-specialised persistent kernel (included by hpctopk.cu after the common definitions).
//
// One CTA per SM.  Its warps have two roles that run concurrently:
//   * scanner warps stream score rows (Phase 2, Section 4.3) back to back and never wait for a
//     refinement: each scanner warp compacts the admitted scores of its share of the row into
//     its own region of a candidate buffer, with no atomics;
//   * helper warps prepare the next row (Phase 1, Section 4.2: sample, coarse histogram, tau_0,
//     tau_1, cutoffs) and retire the previous one (certification branch, Phase 3 of Section 4.4,
//     output commit) while the scanners are busy.
// Two task slots, each with its own candidate buffer, alternate strictly: step i uses slot
// i & 1.  The helpers post a descriptor into a slot (mbarrier `posted`), the scanners execute
// it (mbarrier `scanned`), the helpers retire it and post the slot's next task.  A band
// extension (Eq. "rescue-band") is just another task on the same slot that appends to the
// same buffer.  Every wait is bounded: on a timeout the CTA raises an error flag and leaves.
// The header can be included more than once with different settings (macros below) and a
// different namespace: HPCTOPK_WS_FUSED = 1 builds the single-role variant in which all warps
// of the CTA scan a row together and then act as one helper group for the same row.
#ifndef HPCTOPK_WS_NAMESPACE
#define HPCTOPK_WS_NAMESPACE wsk
#endif
#ifndef HPCTOPK_WS_FUSED
#define HPCTOPK_WS_FUSED 0
#endif
#ifndef HPCTOPK_WS_MINB
#define HPCTOPK_WS_MINB 1
#endif

namespace HPCTOPK_WS_NAMESPACE {

#ifndef HPCTOPK_NS
#define HPCTOPK_NS 24
#endif
#ifndef HPCTOPK_GROUPS
#define HPCTOPK_GROUPS 4
#endif
#ifndef HPCTOPK_GW
#define HPCTOPK_GW 2
#endif
#ifndef HPCTOPK_WS_U
#define HPCTOPK_WS_U 4
#endif
constexpr bool kFused = HPCTOPK_WS_FUSED != 0;
constexpr int NS = HPCTOPK_NS;         // scanner warps (= candidate regions per buffer)
constexpr int kSlots = kFused ? 1 : HPCTOPK_GROUPS;   // task slots = helper groups (group g owns slot g)
constexpr int kGW = kFused ? NS : HPCTOPK_GW;         // warps per helper group
constexpr int NH = kFused ? 0 : kSlots * kGW;         // dedicated helper warps
constexpr int kWsU = HPCTOPK_WS_U;     // float4 loads per thread per register tile
constexpr int ST = NS * 32;            // scanner threads
constexpr int HT = kGW * 32;           // threads per helper group
constexpr int THREADS = ST + NH * 32;
constexpr int kMinBlocks = HPCTOPK_WS_MINB;
constexpr int kSmallMax = kBins / 2;   // frontier size resolved by direct ranking (pairs held in the histogram's memory)
constexpr int kWsTasksPerCta = 8;      // split target: tasks >= kWsTasksPerCta * grid
constexpr int kWsMaxGrid = 160;        // CTAs (one per SM) the overflow region is sized for

struct __align__(16) HelperShared {   // private to one helper group
  uint32_t hist[kBins];      // histograms; later the small-frontier list
  uint32_t warp_sums[32];
  uint32_t out_count;
  uint32_t small_count;
  int32_t loc_bin[2];
  uint32_t loc_below[2];
  uint32_t loc_at[2];
  uint32_t cutd[4];
  uint32_t bcast0, bcast1;
  int32_t claim;
  int32_t pad;
};

// A helper group: HT threads that synchronise on their own named barrier.
struct Grp {
  static constexpr int N = HT;
  int g, t;
  __device__ __forceinline__ int tid() const { return t; }
  __device__ __forceinline__ void sync() const {
    if (kFused) __syncthreads();
    else if (HT == 32) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(HT) : "memory");
  }
};

enum { MODE_DONE = 0, MODE_SCAN = 1, MODE_BAND = 2 };

struct Desc {
  int64_t g0;              // global element index of the row's first score
  int64_t e0, e1;          // global element range to scan
  uint32_t cut_lo, cut_hi; // descending-key cutoffs (band: cut_lo < kd <= cut_hi)
  int32_t mode;
  int32_t pad;
};

static_assert(sizeof(hpctopk_stats) % 16 == 0, "counters must keep 16-byte alignment of what follows");
static_assert(sizeof(HelperShared) % 16 == 0, "helper state must keep 16-byte alignment");
struct WsShared {
  hpctopk_stats acc;         // this CTA's counters (first member of every kernel's shared state)
  HelperShared h[kSlots];
  uint32_t cnt[kSlots][32];  // admitted scores per region of each slot's buffer
  Desc desc[kSlots];
  unsigned long long posted[kSlots];   // mbarrier: helper group -> scanners, 1 arrival
  unsigned long long scanned[kSlots];  // mbarrier: scanners -> helper group, NS arrivals
  uint32_t warp_sums[32];    // prologue only
  uint32_t total_tasks;
  int32_t abort;
  uint32_t groups_done;      // helper groups that have finished (the last one flushes the counters)
  unsigned long long* detail;
};

__device__ __forceinline__ WsShared& WSH() { return *reinterpret_cast<WsShared*>(smem_raw); }
__device__ __forceinline__ uint2* WCAND(int slot, uint32_t region_entries) {
  return reinterpret_cast<uint2*>(smem_raw + ((sizeof(WsShared) + 15) / 16 * 16)) + (size_t)slot * NS * region_entries;
}

#if HPCTOPK_TIMERS
#define WSTAMP(k, t_prev) do { if (G.tid() == 0) { const long long t_now = tick(); atomicAdd(&WSH().detail[k], (unsigned long long)(t_now - (t_prev))); (t_prev) = t_now; } } while (0)
#else
#define WSTAMP(k, t_prev) do { (void)(t_prev); } while (0)
#endif

// ---------------------------------------------------------------- mbarrier helpers (bounded waits)
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_addr(bar)) : "memory");
}
// Waits for the completion of the phase with the given parity.  Gives up after about two
// seconds (or as soon as another thread gave up), sets the abort flag and returns false.
__device__ __noinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity) {
  WsShared& sh = WSH();
  const uint32_t addr = smem_addr(bar);
  unsigned long long t_start = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    // the suspend-time hint lets the hardware park the thread instead of spinning on the pipe
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(addr), "r"(parity), "r"(2000u) : "memory");
    if (ok) return true;
    __nanosleep(400);                      // a poller must not compete with the working warps for issue slots
    if (*reinterpret_cast<volatile int32_t*>(&sh.abort)) return false;
    if ((it & 255u) == 255u) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t_start == 0) t_start = now;
      else if (now - t_start > 2000000000ull) { *reinterpret_cast<volatile int32_t*>(&sh.abort) = 1; return false; }
    }
  }
}

// ---------------------------------------------------------------- candidate buffers
struct Buf {
  uint2* region0;      // shared memory: NS regions of `rw` entries
  uint2* spill;        // global overflow: NS regions of `sw` entries (this CTA, this slot)
  uint32_t* cnt;       // [NS] admitted per region
  uint32_t rw, sw, sw_log2;   // rw: any multiple of 16; sw: a power of two
};
__device__ __forceinline__ uint2 buf_load(const Buf& b, uint32_t w, uint32_t j) {
  return j < b.rw ? b.region0[w * b.rw + j] : __ldcg(b.spill + ((w << b.sw_log2) + (j - b.rw)));
}
__device__ __forceinline__ void buf_store(const Buf& b, uint32_t w, uint32_t j, uint2 v) {
  if (j < b.rw) b.region0[w * b.rw + j] = v;
  else if (j < b.rw + b.sw) b.spill[(w << b.sw_log2) + (j - b.rw)] = v;
}
struct Tally { uint32_t total; bool spilled; bool overflow; };
__device__ __forceinline__ Tally buf_tally(const Buf& b) {
  Tally t{0u, false, false};
  for (int w = 0; w < NS; ++w) {
    const uint32_t n = b.cnt[w];
    t.total += n;
    t.spilled |= n > b.rw;
    t.overflow |= n > b.rw + b.sw;
  }
  return t;
}
// Region geometry per K: shared entries per region (a power of two holding 1.5x the expected
// share of a 1.5 K tail) and the total per-region capacity (1.5x an even share of the capacity).
__host__ __device__ inline int ws_region_entries(int K) {
  int r = ((22 * K / 10 + NS - 1) / NS + 15) / 16 * 16;      // an even share of a 2.2 K tail (1.5 K expected)
  const int r_max = (160 * 1024 / (kSlots * NS * 8)) / 16 * 16;   // kSlots buffers must fit in shared memory
  if (r < 64) r = 64;
  if (r > r_max) r = r_max;
  return r;
}
__host__ __device__ inline int ws_region_total(int K) {
  int need = (capacity_for(K) + NS - 1) / NS;    // with the shared part: 1.5x an even share of the capacity
  int r = 64;
  while (r < need) r *= 2;
  return r;
}

// ---------------------------------------------------------------- the complete-row pass (scanner side)
// Scans global elements [e0, e1); NT threads take part, `t` is this thread's index among them
// and `region` the buffer region this warp appends to.  BAND selects the band predicate.
// Compaction is warp-synchronous: per-lane counts of admitted scores in the register tile, a
// warp prefix sum, positions inside the warp's region; the running count stays in a register.
template <int NT, int U, bool BAND>
__device__ __noinline__ uint32_t scan_share(const float* __restrict__ scores, int64_t g0, int64_t e0, int64_t e1,
                                            uint32_t cut_lo, uint32_t cut_hi, const Buf buf, int t, uint32_t region,
                                            uint32_t wbase) {
  const int lane = t & 31;
  if (e1 <= e0) return wbase;
  const Admit in_hi(cut_hi);
  const Admit in_lo(cut_lo);
  auto admit = [&](uint32_t u) -> bool { return BAND ? (in_hi(u) && !in_lo(u)) : in_hi(u); };
  uint2* const reg = buf.region0 + region * buf.rw;

  auto append_group = [&](auto N_tag, const uint32_t* u, const bool* p, auto idx_of) {
    constexpr int N = decltype(N_tag)::value;
    uint32_t c = 0;
#pragma unroll
    for (int e = 0; e < N; ++e) c += p[e] ? 1u : 0u;
    uint32_t incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += n;
    }
    const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    if (total) {
      uint32_t pos = wbase + incl - c;
      if (wbase + total <= buf.rw) {
#pragma unroll
        for (int e = 0; e < N; ++e)
          if (p[e]) { reg[pos] = make_uint2(u[e], idx_of(e)); ++pos; }
      } else {
#pragma unroll
        for (int e = 0; e < N; ++e)
          if (p[e]) { buf_store(buf, region, pos, make_uint2(u[e], idx_of(e))); ++pos; }
      }
      wbase += total;
    }
  };

  int64_t b0 = (e0 + 3) & ~(int64_t)3;
  int64_t b1 = e1 & ~(int64_t)3;
  if (b0 > b1) { b0 = e1; b1 = e1; }
  if (t < 32) {                                  // ragged edges: at most 3 + 3 scalars, first warp
    const int64_t head_end = b0 < e1 ? b0 : e1;
    const int nhead = (int)(head_end - e0);
    const int ntail = (int)(e1 - (b1 > head_end ? b1 : head_end));
    int64_t e = -1;
    if (lane < nhead) e = e0 + lane;
    else if (lane >= 8 && lane - 8 < ntail) e = e1 - ntail + (lane - 8);
    uint32_t u1[1] = {0u};
    bool p1[1] = {false};
    if (e >= 0) { u1[0] = __float_as_uint(__ldg(scores + e)); p1[0] = admit(u1[0]); }
    const uint32_t i1 = (uint32_t)(e - g0);
    append_group(std::integral_constant<int, 1>{}, u1, p1, [&](int) { return i1; });
  }
  const int64_t nvec = (b1 - b0) >> 2;
  if (nvec <= 0) return wbase;
  const float4* __restrict__ vp = reinterpret_cast<const float4*>(scores + b0);
  const uint32_t idx0 = (uint32_t)(b0 - g0);
  constexpr int TILE = NT * U;
  const int64_t nfull = nvec / TILE;
  constexpr int PF_VEC = kPrefetchAheadBytes / 16;
  const float4* const pf_end = vp + nvec;
  auto load_tile = [&](float4 (&b)[U], const float4* p) {
#pragma unroll
    for (int j = 0; j < U; ++j) {
      b[j] = __ldcs(p + j * NT);
      if (!BAND) {
        const float4* q = p + j * NT + PF_VEC;
        if (q < pf_end) asm volatile("prefetch.global.L2 [%0];" ::"l"(q));
      }
    }
  };
  auto process_tile = [&](const float4 (&b)[U], uint32_t ibase) {
    uint32_t u[U * 4];
    bool p[U * 4];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      u[j * 4 + 0] = __float_as_uint(b[j].x); u[j * 4 + 1] = __float_as_uint(b[j].y);
      u[j * 4 + 2] = __float_as_uint(b[j].z); u[j * 4 + 3] = __float_as_uint(b[j].w);
    }
#pragma unroll
    for (int e = 0; e < U * 4; ++e) p[e] = admit(u[e]);
    append_group(std::integral_constant<int, U * 4>{}, u, p,
                 [&](int e) { return ibase + (uint32_t)((e >> 2) * NT * 4 + (e & 3)); });
  };
  // One register tile per thread: with wide tiles the warps of the SM cover each other's load
  // latency, and the whole register budget goes into the width of the tile.
  float4 A[U];
  const float4* p = vp + t;
  uint32_t ib = idx0 + (uint32_t)(t << 2);
  for (uint32_t left = (uint32_t)nfull; left > 0; --left) {
    load_tile(A, p);
    process_tile(A, ib);
    p += TILE;
    ib += TILE * 4;
  }
  for (int64_t vb = nfull * TILE; vb < nvec; vb += NT) {       // remainder, uniform trip count
    const int64_t v = vb + t;
    const bool in = v < nvec;
    float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
    if (in) f = __ldcs(vp + v);
    const uint32_t i = idx0 + (uint32_t)(v << 2);
    uint32_t u[4] = {__float_as_uint(f.x), __float_as_uint(f.y), __float_as_uint(f.z), __float_as_uint(f.w)};
    bool pp[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) pp[e] = in && admit(u[e]);
    append_group(std::integral_constant<int, 4>{}, u, pp, [&](int e) { return i + (uint32_t)e; });
  }
  return wbase;
}

// ---------------------------------------------------------------- helper-side primitives
__device__ __forceinline__ void g_clear_hist(const Grp& G, HelperShared& sh) {
  for (int b = G.tid(); b < kBins; b += Grp::N) sh.hist[b] = 0;
}

// min{b : H(b) >= quota} for up to two quotas (Eqs. "primary-threshold", "digit-boundary").
__device__ void g_locate(const Grp& G, HelperShared& sh, uint32_t quota0, uint32_t quota1, int nq) {
  if (Grp::N == 32) {
    // one warp: every lane owns 64 consecutive bins
    constexpr int BPL = kBins / 32;
    const int lane = G.tid();
    const uint4* hv = reinterpret_cast<const uint4*>(sh.hist + lane * BPL);
    uint32_t sum = 0;
#pragma unroll 4
    for (int b = 0; b < BPL / 4; ++b) { const uint4 v = hv[b]; sum += v.x + v.y + v.z + v.w; }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += n;
    }
    const uint32_t excl = incl - sum;
    if (lane < 2) sh.loc_bin[lane] = -1;
    __syncwarp();
    for (int qi = 0; qi < nq; ++qi) {
      const uint32_t quota = qi ? quota1 : quota0;
      if (excl < quota && quota <= incl) {
        uint32_t run = excl;
        for (int b = 0; b < BPL; ++b) {
          const uint32_t hb = sh.hist[lane * BPL + b];
          if (run + hb >= quota) { sh.loc_bin[qi] = lane * BPL + b; sh.loc_below[qi] = run; sh.loc_at[qi] = hb; break; }
          run += hb;
        }
      }
    }
    __syncwarp();
    return;
  }
  constexpr int BPT = kBins / (Grp::N == 32 ? 64 : Grp::N);
  const int tid = G.tid(), lane = tid & 31, warp = tid >> 5;
  uint32_t h[BPT];
  uint32_t sum = 0;
#pragma unroll
  for (int b = 0; b < BPT; ++b) { h[b] = sh.hist[tid * BPT + b]; sum += h[b]; }
  uint32_t incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += n;
  }
  if (lane == 31) sh.warp_sums[warp] = incl;
  if (tid < 2) sh.loc_bin[tid] = -1;
  G.sync();
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
  G.sync();
}

struct BufSource {                // the admitted tail held in a slot's buffer
  Buf b;
  bool spilled;
  // Visits the filled part of every region: entries j < jmax of each region, four entries per
  // thread and iteration so that the shared-memory loads of a batch overlap.
  template <typename F>
  __device__ __forceinline__ void for_each(const Grp& G, F f) const {
    uint32_t jmax = 0;
    for (int w = 0; w < NS; ++w) jmax = max(jmax, min(b.cnt[w], b.rw));
    const uint32_t jr = (jmax + 31u) & ~31u;                  // entries visited per region
    const uint32_t total = jr * NS;
    const uint32_t inv = jr ? (0xFFFFFFFFu / jr + 1u) : 0u;   // w = i / jr for i < 2^16
    for (uint32_t i0 = 0; i0 < total; i0 += 4 * Grp::N) {
      uint2 c[4];
      bool v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t i = i0 + k * Grp::N + G.tid();
        const uint32_t w = __umulhi(i, inv), j = i - w * jr;
        v[k] = i < total && j < min(b.cnt[w], b.rw);
        c[k] = v[k] ? b.region0[w * b.rw + j] : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) f(v[k], kd_of_bits(c[k].x), c[k].y);
    }
    if (spilled) {
      const uint32_t n_g = (uint32_t)NS << b.sw_log2;
      for (uint32_t i0 = 0; i0 < n_g; i0 += Grp::N) {
        const uint32_t i = i0 + G.tid();
        const uint32_t w = i >> b.sw_log2, j = i & (b.sw - 1);
        const bool v = i < n_g && b.rw + j < b.cnt[w];
        const uint2 c = v ? __ldcg(b.spill + i) : make_uint2(0u, 0u);
        f(v, kd_of_bits(c.x), c.y);
      }
    }
  }
};

struct RowSrc {                   // the complete row in global memory (recovery)
  const float* scores;
  int64_t g0, g1;
  template <typename F>
  __device__ __forceinline__ void for_each(const Grp& G, F f) const {
    const int64_t va = g0 >> 2, vb = (g1 + 3) >> 2;
    for (int64_t base = va; base < vb; base += Grp::N) {
      const int64_t v = base + G.tid();
      const int64_t e = v << 2;
      const bool in = v < vb;
      const bool full = in && e >= g0 && e + 4 <= g1;
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      bool ok[4] = {false, false, false, false};
      if (full) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(scores + e));
        x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
        ok[0] = ok[1] = ok[2] = ok[3] = true;
      } else if (in) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          ok[j] = (e + j >= g0) && (e + j < g1);
          if (ok[j]) x[j] = __ldg(scores + e + j);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) f(ok[j], kd_of_bits(__float_as_uint(x[j])), (uint32_t)(e + j - g0));
    }
  }
};

// Phase 3 and the output commit (Section 4.4): radix rounds 11+11+10 over kd, then over the
// index bits if the last equal-key group is still larger than the remaining quota; a frontier
// of at most kSmallMax members left after the second digit is resolved by ranking its members
// against each other.  Everything strictly ahead of the boundary is committed in one pass.
template <typename Source>
__device__ __noinline__ void g_select_and_emit(const Grp G, const Source src, uint32_t K, int32_t* out_idx, float* out_val) {
  HelperShared& sh = WSH().h[G.g];
  long long ts = tick();
  const int shifts[6] = {53, 42, 32, 21, 10, 0};
  const int widths[6] = {11, 11, 10, 11, 11, 10};
  uint64_t prefix = 0;
  int prev_shift = 64;
  uint32_t k_rem = K;
  bool small = false;
  uint32_t small_n = 0;
  auto emit = [&](uint32_t kd, uint32_t idx) {
    const uint32_t slot = atomicAdd(&sh.out_count, 1u);
    if (slot < K) {
      out_idx[slot] = (int32_t)idx;
      if (out_val) out_val[slot] = __uint_as_float(bits_of_kd(kd));
    }
  };
  G.sync();
  if (G.tid() == 0) { sh.out_count = 0; sh.small_count = 0; }
#pragma unroll 1
  for (int j = 0; j < 6; ++j) {
    const int shift = shifts[j];
    const uint32_t mask = (1u << widths[j]) - 1u;
    g_clear_hist(G, sh);
    G.sync();
    src.for_each(G, [&](bool valid, uint32_t kd, uint32_t idx) {
      if (valid) {
        const uint64_t comp = ((uint64_t)kd << 32) | idx;
        if (j == 0 || (comp >> prev_shift) == prefix)
          atomicAdd(&sh.hist[(uint32_t)(comp >> shift) & mask], 1u);
      }
    });
    G.sync();
    g_locate(G, sh, k_rem, 0, 1);
    const int b = sh.loc_bin[0];
    const uint32_t below = sh.loc_below[0], at = sh.loc_at[0];
    if (b < 0) { prev_shift = 64; break; }
    k_rem -= below;
    prefix = (prefix << widths[j]) | (uint32_t)b;
    prev_shift = shift;
    if (at == k_rem) break;
    if (j >= 1 && at <= (uint32_t)kSmallMax) { small = true; small_n = at; break; }
    G.sync();
  }
  G.sync();
  WSTAMP(4, ts);
  uint2* const list = reinterpret_cast<uint2*>(sh.hist);
  src.for_each(G, [&](bool valid, uint32_t kd, uint32_t idx) {
    if (valid && prev_shift < 64) {
      const uint64_t q = (((uint64_t)kd << 32) | idx) >> prev_shift;
      if (small ? (q < prefix) : (q <= prefix)) emit(kd, idx);
      else if (small && q == prefix) {
        const uint32_t pos = atomicAdd(&sh.small_count, 1u);
        if (pos < (uint32_t)kSmallMax) list[pos] = make_uint2(kd, idx);
      }
    }
  });
  G.sync();
  if (small) {
    for (uint32_t i = G.tid(); i < small_n; i += Grp::N) {
      const uint2 me = list[i];
      const uint64_t mine = ((uint64_t)me.x << 32) | me.y;
      uint32_t rank = 0;
      for (uint32_t t = 0; t < small_n; ++t) {
        const uint2 o = list[t];
        rank += ((((uint64_t)o.x << 32) | o.y) < mine) ? 1u : 0u;
      }
      if (rank < k_rem) emit(me.x, me.y);
    }
    G.sync();
  }
  WSTAMP(5, ts);
}

// Phase 1 (Section 4.2) by the helper group; cutoffs land in sh.cutd.
__device__ __noinline__ bool g_phase1(const Grp G, const Params& P, int row, int64_t g0, int64_t L, int& tau_pack) {
  HelperShared& sh = WSH().h[G.g];
  const int s = P.stride;
  const int bits = 31 - __clz(s);
  const int a = bits ? (int)(__brev((uint32_t)(row & (s - 1))) >> (32 - bits)) : 0;
  const int64_t n_view = L > a ? ((L - a + s - 1) >> bits) : 0;
  tau_pack = -1;
  if (n_view < P.q1) return false;
  long long ts = tick();
  G.sync();
  g_clear_hist(G, sh);
  G.sync();
  WSTAMP(0, ts);
  const float* __restrict__ rowp = P.scores + g0 + a;
  for (int64_t t = G.tid(); t < n_view; t += Grp::N) {
    const uint32_t kd = kd_of_bits(__float_as_uint(__ldg(rowp + t * s)));
    atomicAdd(&sh.hist[coarse_bin_of_kd(kd)], 1u);
  }
  G.sync();
  WSTAMP(1, ts);
  g_locate(G, sh, (uint32_t)P.q0, (uint32_t)P.q1, 2);
  WSTAMP(2, ts);
  const int tau0 = sh.loc_bin[0], tau1 = sh.loc_bin[1];
  if (Grp::N == 32) {                       // a single warp converts both bins
    const uint32_t c0 = cutoff_of_bin(tau0);
    const uint32_t c1 = cutoff_of_bin(tau1);
    if (G.tid() == 0) { sh.cutd[0] = c0; sh.cutd[1] = c1; }
  } else if (G.tid() < 32) {
    const uint32_t c0 = cutoff_of_bin(tau0);
    if (G.tid() == 0) sh.cutd[0] = c0;
  } else if (G.tid() < 64) {
    const uint32_t c1 = cutoff_of_bin(tau1);
    if (G.tid() == 32) sh.cutd[1] = c1;
  }
  G.sync();
  WSTAMP(3, ts);
  tau_pack = tau0 | (tau1 << 16);
  return true;
}

__device__ void g_emit_short_row(const Grp& G, const Params& P, int row, int64_t g0, int64_t L) {
  int32_t* oi = P.out_idx + (int64_t)row * P.K;
  float* ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
  for (int i = G.tid(); i < P.K; i += Grp::N) {
    const bool v = i < L;
    oi[i] = v ? i : -1;
    if (ov) ov[i] = v ? __ldg(P.scores + g0 + i) : __uint_as_float(0xFF800000u);
  }
}

__device__ __forceinline__ void g_record_row(const Grp& G, const Params& P, int row, int route, int tau, uint32_t c0, uint32_t cfin,
                                             uint64_t scanned, uint64_t sampled, uint64_t L) {
  if (G.tid() != 0) return;
  hpctopk_stats* st = stats_of(P.ws);
  add64(&st->rows_by_route[route], 1);
  if (route == HPCTOPK_ROUTE_PRIMARY || route == HPCTOPK_ROUTE_BAND) {
    add64(&st->candidates_sum, cfin);
    max64(&st->candidates_max, cfin);
  }
  if (scanned) add64(&st->elements_scanned, scanned);
  if (sampled) add64(&st->elements_sampled, sampled);
  add64(&st->elements_valid, L);
  reinterpret_cast<int4*>(P.ws + kOffRowInfo)[row] = make_int4(route, tau, (int)c0, (int)cfin);
}

// Warm the L2 with the stride-s view and the head of a row that will be scanned soon.
__device__ __forceinline__ void g_prefetch_row(const Grp& G, const Params& P, int row, int64_t g0, int64_t L, int64_t e0, int64_t e1) {
  if (L <= P.K) return;
  if (L > P.cap) {
    const int s = P.stride;
    const int bits = 31 - __clz(s);
    const int a = bits ? (int)(__brev((uint32_t)(row & (s - 1))) >> (32 - bits)) : 0;
    const int64_t n_view = (L - a + s - 1) >> bits;
    const float* rowp = P.scores + g0 + a;
    for (int64_t t = G.tid(); t < n_view; t += Grp::N)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp + t * s));
  }
  const char* base = reinterpret_cast<const char*>(P.scores + e0);
  int64_t bytes = (e1 - e0) * 4;
  if (bytes > kPrefetchHeadBytes) bytes = kPrefetchHeadBytes;
  for (int64_t off = (int64_t)G.tid() * 128; off < bytes; off += (int64_t)Grp::N * 128)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
}


// ---------------------------------------------------------------- single-warp helper routines
// A helper warp works alone, so its routines are warp-synchronous: no block barriers, results
// passed through shuffles, loads issued in batches so that their latencies overlap.

// Phase 1 (Section 4.2) by one warp.  Besides tau_0 and tau_1 it locates a tighter bin tau_hi
// at half the rank K (sample rank ceil(K / 2s)); its cutoff brackets the K-th score from above
// and sizes the refinement digit of w_select_adaptive.  Results are uniform across the warp.
struct Phase1Out { bool usable; int tau_pack; uint32_t cut0, cut1, cut_hi; };
__device__ __noinline__ Phase1Out w_phase1(const Grp G, const Params& P, int row, int64_t g0, int64_t L) {
  HelperShared& sh = WSH().h[G.g];
  const int lane = G.tid() & 31, wi = G.tid() >> 5;     // lane and warp index inside the group
  Phase1Out o{false, -1, 0u, 0u, 0u};
  const int s = P.stride;
  const int bits = 31 - __clz(s);
  const int a = bits ? (int)(__brev((uint32_t)(row & (s - 1))) >> (32 - bits)) : 0;
  const int64_t n_view = L > a ? ((L - a + s - 1) >> bits) : 0;
  if (n_view < P.q1) return o;
  long long ts = tick();
  G.sync();
  if (wi == 0) w_clear_hist(sh.hist, lane);
  G.sync();
  const float* __restrict__ rowp = P.scores + g0 + a;
  // wide batches: while the scanner warps keep the load/store queues full, every dependent
  // round trip through them is expensive, so as many loads as possible share one trip
  for (int64_t t0 = (int64_t)wi * 512; t0 < n_view; t0 += 512 * kGW) {
    uint32_t u[16];
    bool v[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const int64_t t = t0 + k * 32 + lane;
      v[k] = t < n_view;
      u[k] = v[k] ? __float_as_uint(__ldg(rowp + t * s)) : 0u;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k)
      if (v[k]) atomicAdd(&sh.hist[coarse_bin_of_kd(kd_of_bits(u[k]))], 1u);
  }
  G.sync();
  WSTAMP(1, ts);
  if (wi == 0) {                                // one warp locates the bins and looks the cutoffs up
    const LaneSums ls = w_lane_sums(sh.hist, lane);
    uint32_t below, at;
    int q_hi = (P.K + 2 * s - 1) / (2 * s);
    if (q_hi < 1) q_hi = 1;
    const uint32_t quota[3] = {(uint32_t)P.q0, (uint32_t)P.q1, (uint32_t)q_hi};
    int tau[3];
    w_locate3(sh.hist, ls, quota, lane, tau);
    (void)below; (void)at;
    if (lane < 3) sh.cutd[lane] = g_cut_table[lane == 0 ? tau[0] : (lane == 1 ? tau[1] : tau[2])];
    if (lane == 0) { sh.loc_bin[0] = tau[0]; sh.loc_bin[1] = tau[1]; }
  }
  G.sync();
  WSTAMP(3, ts);
  o.usable = true;
  o.tau_pack = sh.loc_bin[0] | (sh.loc_bin[1] << 16);
  o.cut0 = sh.cutd[0]; o.cut1 = sh.cutd[1]; o.cut_hi = sh.cutd[2];
  G.sync();                                     // values are in registers before the next row overwrites them
  return o;
}

// Phase 3 by one warp over a slot's buffer, with a row-adaptive first digit (any monotone digit
// of the key is a valid refinement digit, Section 4.4): d = min((cut_base - kd) >> sh, 2047)
// measures the distance from the admitted cutoff in units of 2^sh ulps; `sh` is chosen so that
// the bracket [cut_hi, cut_base] spans the 2048 bins, which leaves only a handful of scores
// in the boundary bin.  One histogram pass, one boundary search, one commit pass; the boundary
// bin is resolved by ranking its members against each other under (kd, idx).  Returns false
// (nothing written) when the K-th score falls outside the bracket or the boundary bin is too
// large; the caller then runs the general 11+11+10 refinement.
__device__ __noinline__ bool w_select_adaptive(const Grp G, const Buf buf, bool spilled, uint32_t K, uint32_t cut_base,
                                               uint32_t cut_hi, int32_t* out_idx, float* out_val) {
  HelperShared& sh = WSH().h[G.g];
  const int lane = G.tid() & 31, wi = G.tid() >> 5;     // lane and warp index inside the group
  long long ts = tick();
  const uint32_t span = cut_base > cut_hi ? cut_base - cut_hi : 0u;
  int shv = 0;
  while (shv < 31 && (span >> shv) >= 2047u) ++shv;
  G.sync();
  if (wi == 0) w_clear_hist(sh.hist, lane);
  if (G.tid() == 0) { sh.small_count = 0; sh.out_count = 0; }
  G.sync();
  // digit: 0 = the clamped group far above the bracket, 2047 = next to the cutoff
  auto digit = [&](uint32_t kd) -> uint32_t {
    const uint32_t d = (cut_base - kd) >> shv;
    return 2047u - (d < 2047u ? d : 2047u);
  };
  // The filled parts of the NS regions are visited as one flat index space, sixteen entries
  // per lane and batch (one trip through the shared-memory queue per batch).  Lane w keeps
  // the fill count of region w; the others obtain it by shuffle.
  const uint32_t cnt_l = lane < NS ? min(buf.cnt[lane], buf.rw) : 0u;
  uint32_t jmax = cnt_l;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) jmax = max(jmax, __shfl_xor_sync(0xFFFFFFFFu, jmax, d));
  const uint32_t jr = (jmax + 31u) & ~31u;
  const uint32_t total = jr * NS;
  const uint32_t inv = jr ? (0xFFFFFFFFu / jr + 1u) : 0u;   // w = i / jr for i < 2^16
  auto fetch = [&](uint32_t i, uint2& c) -> bool {
    const uint32_t w = min(__umulhi(i, inv), (uint32_t)(NS - 1)), j = i - w * jr;
    const uint32_t n_w = __shfl_sync(0xFFFFFFFFu, cnt_l, (int)w);
    const bool v = i < total && j < n_w;
    c = v ? buf.region0[w * buf.rw + j] : make_uint2(0u, 0u);
    return v;
  };
  // pass A: histogram of the digit (batches dealt to the warps of the group)
  for (uint32_t i0 = (uint32_t)wi * 512u; i0 < total; i0 += 512u * kGW) {
    uint2 c[16];
    bool v[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = fetch(i0 + k * 32 + lane, c[k]);
#pragma unroll
    for (int k = 0; k < 16; ++k) if (v[k]) atomicAdd(&sh.hist[digit(kd_of_bits(c[k].x))], 1u);
  }
  if (spilled) {                                // entries in the overflow slice (uncommon)
    const uint32_t n_g = (uint32_t)NS << buf.sw_log2;
    for (uint32_t i = G.tid(); i < n_g; i += Grp::N) {
      const uint32_t w = i >> buf.sw_log2, j = i & (buf.sw - 1);
      if (buf.rw + j < buf.cnt[w]) atomicAdd(&sh.hist[digit(kd_of_bits(__ldcg(buf.spill + i).x))], 1u);
    }
  }
  G.sync();
  if (wi == 0) {                                // one warp locates the boundary bin
    const LaneSums ls = w_lane_sums(sh.hist, lane);
    uint32_t below0, at0;
    const int b0 = w_locate(sh.hist, ls, K, lane, below0, at0);
    if (lane == 0) { sh.loc_bin[0] = b0; sh.loc_below[0] = below0; sh.loc_at[0] = at0; }
  }
  G.sync();
  const int b = sh.loc_bin[0];
  const uint32_t below = sh.loc_below[0], at = sh.loc_at[0];
  WSTAMP(4, ts);
  if (b <= 0 || at > (uint32_t)kSmallMax) return false;
  const uint32_t k_rem = K - below;             // to take from the boundary bin
  uint2* const list = reinterpret_cast<uint2*>(sh.hist);
  G.sync();                                     // the histogram's memory becomes the boundary list
  // pass B: commit everything ahead of the boundary bin, collect the boundary bin
  for (uint32_t i0 = (uint32_t)wi * 512u; i0 < total; i0 += 512u * kGW) {
    uint2 c[16];
    uint32_t sel = 0, bnd = 0, cnt = 0;         // bit k: entry k is committed / lies in the boundary bin
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const bool v = fetch(i0 + k * 32 + lane, c[k]);
      const uint32_t dg = v ? digit(kd_of_bits(c[k].x)) : 0xFFFFFFFFu;
      if (dg < (uint32_t)b) { sel |= 1u << k; ++cnt; }
      else if (dg == (uint32_t)b) bnd |= 1u << k;
    }
    uint32_t incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t m = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += m;
    }
    const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    uint32_t out_base = 0;                      // one reservation of output slots per warp and batch
    if (lane == 31 && tot) out_base = atomicAdd(&sh.out_count, tot);
    out_base = __shfl_sync(0xFFFFFFFFu, out_base, 31);
    uint32_t pos = out_base + incl - cnt;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((sel >> k) & 1u) {
        if (pos < K) { out_idx[pos] = (int32_t)c[k].y; if (out_val) out_val[pos] = __uint_as_float(c[k].x); }
        ++pos;
      } else if ((bnd >> k) & 1u) {
        const uint32_t lp = atomicAdd(&sh.small_count, 1u);
        if (lp < (uint32_t)kSmallMax) list[lp] = make_uint2(kd_of_bits(c[k].x), c[k].y);
      }
    }
  }
  if (spilled) {
    const uint32_t n_g = (uint32_t)NS << buf.sw_log2;
    for (uint32_t i = G.tid(); i < n_g; i += Grp::N) {
      const uint32_t w = i >> buf.sw_log2, j = i & (buf.sw - 1);
      if (buf.rw + j < buf.cnt[w]) {
        const uint2 c = __ldcg(buf.spill + i);
        const uint32_t dg = digit(kd_of_bits(c.x));
        if (dg < (uint32_t)b) {
          const uint32_t pos = atomicAdd(&sh.out_count, 1u);
          if (pos < K) { out_idx[pos] = (int32_t)c.y; if (out_val) out_val[pos] = __uint_as_float(c.x); }
        } else if (dg == (uint32_t)b) {
          const uint32_t lp = atomicAdd(&sh.small_count, 1u);
          if (lp < (uint32_t)kSmallMax) list[lp] = make_uint2(kd_of_bits(c.x), c.y);
        }
      }
    }
  }
  G.sync();
  // boundary bin: rank under (kd, idx); the k_rem best are committed
  for (uint32_t i = G.tid(); i < at; i += Grp::N) {
    const uint2 me = list[i];
    const uint64_t mine = ((uint64_t)me.x << 32) | me.y;
    uint32_t rank = 0;
    for (uint32_t t = 0; t < at; ++t) {
      const uint2 o = list[t];
      rank += ((((uint64_t)o.x << 32) | o.y) < mine) ? 1u : 0u;
    }
    if (rank < k_rem) {
      const uint32_t pos = below + rank;
      out_idx[pos] = (int32_t)me.y;
      if (out_val) out_val[pos] = __uint_as_float(bits_of_kd(me.x));
    }
  }
  G.sync();
  WSTAMP(5, ts);
  return true;
}

// ---------------------------------------------------------------- per-slot task state (helper registers)
struct Task {
  int32_t row, seg, nseg;
  int64_t g0, L;
  int64_t e0, e1;        // range given to the scanners
  int32_t tau_pack;
  int32_t banded;        // the band extension has been appended already
  uint32_t cut0, cut1;   // cutoffs of tau_0 and tau_1 (descending keys)
  uint32_t cut_hi;       // cutoff of the bracket bin at half the rank (sizes the refinement digit)
  uint32_t c0;           // C(tau_0)
  uint64_t scanned, sampled;
  long long t_post;
};

__device__ __forceinline__ Buf make_slot_buf(const Params& P, int slot, uint32_t rw, uint32_t sw) {
  WsShared& sh = WSH();
  const size_t cand_off = align_up(kOffRowInfo + (size_t)P.num_rows * sizeof(hpctopk_row_info), 256);
  const size_t split_rows = P.num_rows < kSplitRowsMax ? P.num_rows : kSplitRowsMax;
  const size_t spill_off = cand_off + split_rows * (size_t)P.cap * 8;
  Buf b;
  b.region0 = WCAND(slot, rw);
  b.spill = reinterpret_cast<uint2*>(P.ws + spill_off) + ((size_t)blockIdx.x * kSlots + slot) * (size_t)NS * sw;
  b.cnt = sh.cnt[slot];
  b.rw = rw; b.sw = sw;
  b.sw_log2 = 31 - __clz(sw);
  return b;
}

// Scanner warps: execute the posted descriptors, rotating over the slots, until every slot has
// posted DONE.
template <int U>
__device__ __noinline__ void scanner_main(const Params& P, uint32_t rw, uint32_t sw) {
  WsShared& sh = WSH();
  const int tid = (int)threadIdx.x - NH * 32, warp = tid >> 5, lane = tid & 31;   // helpers hold the lowest warp ids
  uint32_t parity = 0;                    // bit s: parity of the next descriptor of slot s
  uint32_t done = 0;                      // bit s: slot s has posted DONE
  int live = kSlots;
  while (live > 0) {
#pragma unroll 1
    for (int s = 0; s < kSlots; ++s) {
      if ((done >> s) & 1u) continue;
      int ok = 0;
      const long long tw0 = tick();
      if (lane == 0) ok = mbar_wait(&sh.posted[s], (parity >> s) & 1u) ? 1 : 0;   // one poller per warp
      ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
      if (!ok) return;
      const long long tw1 = tick();
      if (tid == 0) atomicAdd(&sh.detail[6], (unsigned long long)(tw1 - tw0));
      parity ^= 1u << s;
      const Desc d = sh.desc[s];
      if (d.mode == MODE_DONE) { done |= 1u << s; --live; continue; }
      const Buf buf = make_slot_buf(P, s, rw, sw);
      uint32_t wbase = (d.mode == MODE_SCAN) ? 0u : sh.cnt[s][warp];
      if (d.mode == MODE_SCAN) wbase = scan_share<ST, U, false>(P.scores, d.g0, d.e0, d.e1, d.cut_lo, d.cut_hi, buf, tid, (uint32_t)warp, wbase);
      else wbase = scan_share<ST, U, true>(P.scores, d.g0, d.e0, d.e1, d.cut_lo, d.cut_hi, buf, tid, (uint32_t)warp, wbase);
      if (lane == 0) sh.cnt[s][warp] = wbase;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.scanned[s]);
      if (tid == 0) atomicAdd(&sh.detail[7], (unsigned long long)(tick() - tw1));
    }
  }
}

// One helper group: owns slot G.g.  Claims tasks, prepares them (Phase 1), hands the scan to the
// scanner warps, and retires the result (certification branch, Phase 3, output commit).
__device__ __noinline__ void helper_main(const Grp G, const Params& P, uint32_t rw, uint32_t sw, uint32_t total_tasks,
                                         const uint32_t* seg_base) {
  WsShared& wsh = WSH();
  HelperShared& sh = wsh.h[G.g];
  const int ht = G.tid();
  const int s = G.g;
  const uint32_t K = (uint32_t)P.K;
  uint32_t* task_counter = reinterpret_cast<uint32_t*>(P.ws + kOffCtrl);
  uint32_t* arrive = reinterpret_cast<uint32_t*>(P.ws + kOffSplit);
  uint32_t* rowcnt = arrive + kSplitRowsMax;
  const size_t cand_off = align_up(kOffRowInfo + (size_t)P.num_rows * sizeof(hpctopk_row_info), 256);
  const Buf buf = make_slot_buf(P, s, rw, sw);
  Task t{};
  uint32_t uses = 0;                      // descriptors posted so far (mbarrier phase bookkeeping)
  // task claiming: one statically assigned task per group, then the device counter, one claim in flight
  const uint32_t n_static = gridDim.x * kSlots;
  uint32_t next_task = blockIdx.x * kSlots + (uint32_t)s;
  if (ht == 0) sh.claim = (int32_t)(n_static + atomicAdd(task_counter, 1u));
  G.sync();
  uint32_t after_next = (uint32_t)sh.claim;
  G.sync();

  auto post = [&](int mode, int64_t g0, int64_t e0, int64_t e1, uint32_t cut_lo, uint32_t cut_hi) {
    if (kFused) {
      // single-role variant: the group scans the range itself, right now
      if (mode == MODE_DONE) return;
      const int warp = ht >> 5;
      G.sync();
      if (mode == MODE_SCAN && ht < 32) wsh.cnt[s][ht] = 0;
      G.sync();
      uint32_t wbase = wsh.cnt[s][warp];
      if (mode == MODE_SCAN) wbase = scan_share<ST, kWsU, false>(P.scores, g0, e0, e1, cut_lo, cut_hi, buf, ht, (uint32_t)warp, wbase);
      else wbase = scan_share<ST, kWsU, true>(P.scores, g0, e0, e1, cut_lo, cut_hi, buf, ht, (uint32_t)warp, wbase);
      if ((ht & 31) == 0) wsh.cnt[s][warp] = wbase;
      G.sync();
      return;
    }
    if (ht == 0) {
      Desc& d = wsh.desc[s];
      d.g0 = g0; d.e0 = e0; d.e1 = e1; d.cut_lo = cut_lo; d.cut_hi = cut_hi; d.mode = mode;
    }
    G.sync();                             // descriptor (and any buffer writes by the group) are in place
    if (ht == 0) mbar_arrive(&wsh.posted[s]);
    ++uses;
  };
  int32_t* oi = nullptr;
  float* ov = nullptr;
  // Exact recovery and every other rare continuation runs on the helper warps themselves.
  auto recover_row = [&](int route, uint32_t c0, uint64_t scanned) {
    RowSrc rs{P.scores, t.g0, t.g0 + t.L};
    g_select_and_emit(G, rs, K, oi, ov);
    g_record_row(G, P, t.row, route, t.tau_pack, c0, 0, scanned + 4ull * (uint64_t)t.L, t.sampled, (uint64_t)t.L);
  };

  // Claims tasks until one needs the scanners (posts it) or none is left (returns false).
  auto start_next = [&]() -> bool {
    for (;;) {
      const uint32_t task = next_task;
      if (task >= total_tasks) return false;
      next_task = after_next;             // the claim issued one task ago
      if (ht == 0) sh.claim = (int32_t)(n_static + atomicAdd(task_counter, 1u));
      G.sync();
      after_next = (uint32_t)sh.claim;
      G.sync();
      int row = (int)task, seg = 0, nseg = 1;
      if (P.split_enabled) {
        int lo = 0, hi = P.num_rows - 1;
        while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (seg_base[mid] <= task) lo = mid; else hi = mid - 1; }
        row = lo;
        nseg = (int)(seg_base[row + 1] - seg_base[row]);
        seg = (int)(task - seg_base[row]);
      }
      const int64_t g0 = row_start(P, row);
      int64_t L = P.row_lengths[row];
      if (L < 0) L = 0;
      t.row = row; t.seg = seg; t.nseg = nseg; t.g0 = g0; t.L = L;
      t.banded = 0; t.tau_pack = -1; t.c0 = 0; t.scanned = 0; t.sampled = 0; t.cut0 = 0; t.cut1 = 0; t.cut_hi = 0;
      oi = P.out_idx + (int64_t)row * P.K;
      ov = P.out_val ? P.out_val + (int64_t)row * P.K : nullptr;
      if (ht == 0) add64(&stats_of(P.ws)->tasks, 1);
      if (L <= (int64_t)K) {                       // every valid index, then sentinels
        g_emit_short_row(G, P, row, g0, L);
        g_record_row(G, P, row, HPCTOPK_ROUTE_SHORT, -1, 0, 0, (uint64_t)L, 0, (uint64_t)L);
        continue;
      }
      if (L <= (int64_t)P.cap) {                   // direct route: the whole row is admitted
        t.e0 = g0; t.e1 = g0 + L; t.t_post = tick();
        post(MODE_SCAN, g0, t.e0, t.e1, 0u, 0xFFFFFFFFu);
        return true;
      }
      const long long t0 = tick();
      const Phase1Out p1 = w_phase1(G, P, row, g0, L);
      const bool usable = p1.usable;
      t.tau_pack = p1.tau_pack;
      if (ht == 0) add64(&stats_of(P.ws)->cycles_phase1, (uint64_t)(tick() - t0));
      t.sampled = usable ? (uint64_t)((L + P.stride - 1) / P.stride) : 0;
      if (!usable && nseg == 1) { recover_row(HPCTOPK_ROUTE_RECOVERY, 0, 0); continue; }
      int64_t e0 = g0, e1 = g0 + L;
      if (nseg > 1) {                              // contiguous, 16-byte aligned partition of the row
        const int64_t va = g0 >> 2, vb = (g0 + L + 3) >> 2;
        const int64_t per = (vb - va + nseg - 1) / nseg;
        e0 = (va + (int64_t)seg * per) << 2; e1 = (va + (int64_t)(seg + 1) * per) << 2;
        if (e0 < g0) e0 = g0;
        if (e1 > g0 + L) e1 = g0 + L;
        if (e1 < e0) e1 = e0;
        if (!usable) e1 = e0;                      // nothing to scan; the finisher recovers the row
      }
      t.cut0 = p1.cut0;
      t.cut1 = p1.cut1;
      t.cut_hi = p1.cut_hi;
      t.e0 = e0; t.e1 = e1; t.t_post = tick();
      t.scanned = (uint64_t)(e1 - e0);
      post(MODE_SCAN, g0, e0, e1, 0u, t.cut0);
      return true;
    }
  };

  // Retires the posted task after the scanners are done with it.  Returns false when the same
  // row went back to the scanners (band extension), true when the slot is free again.
  auto complete = [&]() -> bool {
    const long long tc0 = tick();
    if (ht == 0) add64(&stats_of(P.ws)->cycles_scan, (uint64_t)(tc0 - t.t_post));
    const bool direct = t.L <= (int64_t)P.cap;
    Tally ty = buf_tally(buf);
    if (t.nseg > 1 && !t.banded) {
      // ---- KV-split: publish this segment's tail, last arriver gathers (Eq. "split-reduce")
      uint2* gcand = reinterpret_cast<uint2*>(P.ws + cand_off) + (size_t)t.row * P.cap;
      const uint32_t Cp = ty.total;
      if (ht == 0) {
        sh.bcast0 = atomicAdd(&rowcnt[t.row], Cp);
        add64(&stats_of(P.ws)->elements_scanned, t.scanned);
        if (t.sampled) add64(&stats_of(P.ws)->elements_sampled, t.sampled);
      }
      G.sync();
      const uint32_t base = sh.bcast0;
      if (!ty.overflow && base + Cp <= (uint32_t)P.cap) {
        const int hw = ht >> 5, hl = ht & 31;
        for (int w = hw; w < NS; w += kGW) {       // each helper warp copies a share of the regions
          uint32_t pre = 0;
          for (int w2 = 0; w2 < w; ++w2) pre += buf.cnt[w2];
          const uint32_t n = buf.cnt[w];
          for (uint32_t j = hl; j < n; j += 32) gcand[base + pre + j] = buf_load(buf, (uint32_t)w, j);
        }
      }
      __threadfence();
      G.sync();
      if (ht == 0) sh.bcast1 = atomicAdd(&arrive[t.row], 1u + (ty.overflow ? 0x10000u : 0u)) + (ty.overflow ? 0x10000u : 0u);
      G.sync();
      const uint32_t arrived = sh.bcast1;
      G.sync();
      if ((arrived & 0xFFFFu) != (uint32_t)(t.nseg - 1)) return true;      // not the last arriver: slot is free
      __threadfence();
      const uint32_t C0 = *reinterpret_cast<volatile uint32_t*>(&rowcnt[t.row]);
      if (ht == 0) add64(&stats_of(P.ws)->rows_split, 1);
      t.scanned = 0; t.sampled = 0;                // already accounted by the segments
      if (t.tau_pack < 0) { recover_row(HPCTOPK_ROUTE_RECOVERY, 0, 0); return true; }
      if ((arrived >> 16) != 0 || C0 > (uint32_t)P.cap) { recover_row(HPCTOPK_ROUTE_OVERFLOW, C0, 0); return true; }
      for (uint32_t i = ht; i < C0; i += HT) buf_store(buf, i % NS, i / NS, __ldcg(gcand + i));
      if (ht < NS) buf.cnt[ht] = (C0 + NS - 1 - (uint32_t)ht) / NS;
      G.sync();
      ty = buf_tally(buf);
      t.e0 = t.g0; t.e1 = t.g0 + t.L;              // any further pass covers the whole row
    }
    if (!t.banded) t.c0 = ty.total;
    if (direct) {
      if (!ty.overflow) { BufSource bs{buf, ty.spilled}; g_select_and_emit(G, bs, K, oi, ov); }
      else { RowSrc rs{P.scores, t.g0, t.g0 + t.L}; g_select_and_emit(G, rs, K, oi, ov); }
      g_record_row(G, P, t.row, HPCTOPK_ROUTE_DIRECT, -1, (uint32_t)t.L, (uint32_t)t.L, (uint64_t)t.L, 0, (uint64_t)t.L);
    } else if (ty.overflow || ty.total > (uint32_t)P.cap) {
      recover_row(HPCTOPK_ROUTE_OVERFLOW, t.c0, t.scanned);
    } else if (ty.total >= K) {
      bool done = false;
      done = w_select_adaptive(G, buf, ty.spilled, K, t.banded ? t.cut1 : t.cut0, t.cut_hi, oi, ov);
      if (!done) {
        if (ht == 0) add64(&stats_of(P.ws)->general_refinements, 1);      // general refinement taken
        BufSource bs{buf, ty.spilled};
        g_select_and_emit(G, bs, K, oi, ov);
      }
      g_record_row(G, P, t.row, t.banded ? HPCTOPK_ROUTE_BAND : HPCTOPK_ROUTE_PRIMARY, t.tau_pack, t.c0, ty.total,
                   t.scanned, t.sampled, (uint64_t)t.L);
    } else if (!t.banded) {
      // band extension (Eq. "rescue-band"): same slot, same buffer, appended by the scanners
      t.banded = 1;
      t.scanned += (uint64_t)t.L;
      t.t_post = tick();
      post(MODE_BAND, t.g0, t.g0, t.g0 + t.L, t.cut0, t.cut1);
      return false;
    } else {
      recover_row(HPCTOPK_ROUTE_RECOVERY, t.c0, t.scanned);
    }
    if (ht == 0) add64(&stats_of(P.ws)->cycles_finish, (uint64_t)(tick() - tc0));
    return true;
  };

  bool busy = start_next();
  while (busy) {
    if (!kFused) {
      if (ht == 0) sh.bcast0 = mbar_wait(&wsh.scanned[s], (uses - 1) & 1u) ? 1u : 0u;
      G.sync();
      const bool ok = sh.bcast0 != 0u;
      G.sync();
      if (!ok) break;
    }
    if (complete()) busy = start_next();
  }
  post(MODE_DONE, 0, 0, 0, 0u, 0u);       // releases the scanners from this slot
  G.sync();
  if (ht == 0) {
    if (*reinterpret_cast<volatile int32_t*>(&wsh.abort)) add64(&stats_of(P.ws)->error_flags, 1);
    __threadfence_block();
    if (atomicAdd(&wsh.groups_done, 1u) == (uint32_t)(kSlots - 1)) { __threadfence_block(); stats_flush(P.ws); }
  }
}

template <int U>
__global__ void __launch_bounds__(THREADS, kMinBlocks) hpctopk_ws_kernel(const Params P) {
  WsShared& sh = WSH();
  const int tid = threadIdx.x;
  const uint32_t rw = (uint32_t)ws_region_entries(P.K);
  const uint32_t sw = (uint32_t)ws_region_total(P.K);     // overflow entries per region (a power of two)
  uint32_t* const seg_base = reinterpret_cast<uint32_t*>(WCAND(kSlots, rw));   // after the buffers

  stats_clear();
  if (tid == 0) {
    sh.detail = reinterpret_cast<unsigned long long*>(stats_of(P.ws)->cycles_detail);
    sh.abort = 0;
    sh.groups_done = 0;
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sh.posted[s], 1); mbar_init(&sh.scanned[s], NS); }
  }
  __syncthreads();

  uint32_t total_tasks = (uint32_t)P.num_rows;
  if (P.split_enabled) {
    // Device-side ragged dispatch: every CTA derives the same task table from row_lengths.
    // (kSplitRowsMax <= THREADS: one row per thread.)
    uint32_t* scratch = sh.h[0].hist;
    unsigned long long mine = 0;
    const int r = tid;
    int64_t Lr = 0;
    if (r < P.num_rows) { Lr = P.row_lengths[r]; if (Lr > P.cap) mine = (unsigned long long)Lr; }
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);
    if ((tid & 31) == 0) { scratch[2 * (tid >> 5)] = (uint32_t)mine; scratch[2 * (tid >> 5) + 1] = (uint32_t)(mine >> 32); }
    __syncthreads();
    unsigned long long total = 0;
    for (int w = 0; w < THREADS / 32; ++w) total += (unsigned long long)scratch[2 * w] | ((unsigned long long)scratch[2 * w + 1] << 32);
    const unsigned long long target = (unsigned long long)gridDim.x * kWsTasksPerCta;
    unsigned long long S = (total + target - 1) / target;
    if (S < (unsigned long long)kSegMinElems) S = kSegMinElems;
    S = (S + 4095ull) / 4096ull * 4096ull;
    __syncthreads();
    uint32_t mycnt = 0;
    if (r < P.num_rows) mycnt = (Lr > P.cap) ? (uint32_t)((Lr + (int64_t)S - 1) / (int64_t)S) : 1u;
    uint32_t incl = mycnt;
    for (int d = 1; d < 32; d <<= 1) { const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, d); if ((tid & 31) >= d) incl += n; }
    if ((tid & 31) == 31) sh.warp_sums[tid >> 5] = incl;
    __syncthreads();
    uint32_t woff = 0;
    for (int w = 0; w < (tid >> 5); ++w) woff += sh.warp_sums[w];
    const uint32_t excl = woff + incl - mycnt;
    if (r < P.num_rows) seg_base[r] = excl;
    if (r == P.num_rows - 1) { seg_base[P.num_rows] = excl + mycnt; sh.total_tasks = excl + mycnt; }
    __syncthreads();
    total_tasks = sh.total_tasks;
  }

  // The helper groups take the lowest warp ids: the warp schedulers favour older warps, and the
  // helpers' short, latency-bound phases must not queue behind the streaming warps.
  if (kFused) {
    Grp G;
    G.g = 0;
    G.t = tid;
    helper_main(G, P, rw, sw, total_tasks, seg_base);
  } else if (tid >= NH * 32) {
    scanner_main<U>(P, rw, sw);
  } else {
    Grp G;
    G.g = tid / HT;
    G.t = tid % HT;
    helper_main(G, P, rw, sw, total_tasks, seg_base);
  }
}

// ---- host-side geometry
inline size_t ws_smem_bytes(int K, bool split) {
  size_t b = (sizeof(WsShared) + 15) / 16 * 16 + (size_t)kSlots * NS * ws_region_entries(K) * 8;
  if (split) b += (kSplitRowsMax + 1) * sizeof(uint32_t);
  return (b + 15) / 16 * 16;
}
inline size_t ws_spill_bytes(int K, int grid) {
  return (size_t)grid * kSlots * NS * ws_region_total(K) * 8;
}

}  // namespace HPCTOPK_WS_NAMESPACE

#undef HPCTOPK_WS_NAMESPACE
#undef HPCTOPK_WS_FUSED
#undef HPCTOPK_WS_MINB
#undef HPCTOPK_NS
#undef HPCTOPK_GROUPS
#undef HPCTOPK_GW
#undef HPCTOPK_WS_U
#undef WSTAMP
