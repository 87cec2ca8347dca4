// grass_select: compute_P of the GRASS paper (Section 3.2) -- Top-r; sampling
// with replacement from q ~ norm, norm^2 or uniform with rho_j = 1/sqrt(r q_sigma_j);
// and the same three distributions without replacement with rho = 1.
//
// m is at most a few tens of thousands and r at most a few thousand, so this
// is a latency-bound single-CTA kernel (1024 threads); everything it needs to
// agree on is agreed on through shared memory and block-wide scans, and the
// output order (ascending row) is produced by scans in row order, so the
// result does not depend on thread scheduling.
//
//   Top-r: the fp32 bit pattern of a non-negative float orders like the float,
//   so the r-th largest norm is found by a 4-pass, 8-bit-digit radix select.
//   Rows above the threshold are taken; rows equal to it are taken lowest row
//   first until r are chosen.
//
//   Without replacement: every row gets an exponential-race score (one Philox
//   word per row), and the Top-r machinery ranks the fp32 scores.
//
//   With replacement: fp64 inclusive running sum of the weights (block scan in
//   row order), then one thread per draw: Philox4x32-10 word -> u -> binary
//   search for min{k : c_k > u S}; hits are counted per row with integer
//   atomics (order-independent), and a last scan over the counts writes the
//   rows in ascending order with their rho.
#include "common.cuh"

namespace grass {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kStreamTag = 0x47524153u;

// ---- Philox4x32-10 (Salmon et al., SC'11) ----
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// Inclusive block scan over kThreads values; returns this thread's inclusive
// prefix and sets `total` for all threads.  `scratch` holds kWarps + 1 values.
template <typename T>
__device__ __forceinline__ T block_inclusive_scan(T v, T* scratch, T& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T up = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += up;
  }
  __syncthreads();  // scratch may still be read from a previous call
  if (lane == 31) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    T w = lane < kWarps ? scratch[lane] : T(0);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      T up = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += up;
    }
    if (lane < kWarps) scratch[lane] = w;
  }
  __syncthreads();
  total = scratch[kWarps - 1];
  return warp == 0 ? v : v + scratch[warp - 1];
}

__device__ __forceinline__ uint32_t norm_key(float v) {
  return v == 0.f ? 0u : __float_as_uint(v);  // folds -0 into +0
}

__device__ __forceinline__ bool is_nr(int method) {
  return method == GRASS_SEL_MULTINOMIAL_NORM_NR || method == GRASS_SEL_MULTINOMIAL_NORM2_NR ||
         method == GRASS_SEL_UNIFORM_NR;
}
// Unnormalised q of the three sampling distributions (Section 3.2 A), in fp64.
__device__ __forceinline__ double sampling_weight(int method, float lambda) {
  const double l = static_cast<double>(lambda);
  if (method == GRASS_SEL_MULTINOMIAL_NORM2 || method == GRASS_SEL_MULTINOMIAL_NORM2_NR) return l * l;
  if (method == GRASS_SEL_UNIFORM || method == GRASS_SEL_UNIFORM_NR) return 1.0;
  return l;
}

struct SelectArgs {
  const float* norms;
  int m, r, method;
  uint32_t seed_lo, seed_hi, layer_id, epoch;
  int32_t* idx;
  float* rho;
  double* cdf;    // [m]   (sampling methods)
  int* counts;    // [m]   (sampling methods)
  int* status;
  int stage_norms;   // dynamic shared memory holds a copy of the norms (m floats) ...
  int stage_counts;  // ... followed by the hit counters (m ints)
  int stage_cdf;     // ... followed by the running sum (m doubles)
};

__global__ void __launch_bounds__(kThreads) select_kernel(SelectArgs a) {
  extern __shared__ __align__(16) float s_dyn[];   // staged norms / scores, then hit counters
  __shared__ int s_hist[256];
  __shared__ int s_int[kWarps + 1];
  __shared__ int s_flag;
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  const int tid = threadIdx.x;
  const int m = a.m, r = a.r;

  // ---- validate: every norm finite and >= 0 ----
  if (tid == 0) s_flag = 0;
  __syncthreads();
  {
    // the one pass that reads global memory: 8 loads in flight per thread, not one at a time
    int bad = 0;
    for (int k0 = tid; k0 < m; k0 += 8 * kThreads) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int k = k0 + u * kThreads;
        v[u] = k < m ? __ldg(a.norms + k) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int k = k0 + u * kThreads;
        if (k < m) {
          if (a.stage_norms) s_dyn[k] = v[u];   // every later pass reads shared memory, not L2
          if (!(v[u] >= 0.f) || isinf(v[u])) bad = k + 1;
        }
      }
    }
    if (bad) atomicMax(&s_flag, bad);
  }
  __syncthreads();
  if (s_flag != 0) {
    if (tid == 0) record_status(a.status, GRASS_ERR_DEGENERATE, s_flag - 1);
    return;
  }

  const float* nrm = a.stage_norms ? s_dyn : a.norms;
  int* counts = a.stage_counts ? reinterpret_cast<int*>(s_dyn + ((m + 3) & ~3)) : a.counts;
  double* cdf = a.stage_cdf ? reinterpret_cast<double*>(s_dyn + 2 * ((m + 3) & ~3)) : a.cdf;
  const float* keys = nrm;   // what the r largest are taken of
  if (is_nr(a.method)) {
    // ---- without replacement: exponential race (Efraimidis & Spirakis).  Row k scores
    // w_k / (-log u_k), u_k = (word_k + 1/2) 2^-32; the r largest scores are distributed as r
    // successive draws without replacement.  Scores are rounded to fp32 and ranked as such. ----
    float* scores = a.stage_norms ? s_dyn : reinterpret_cast<float*>(a.cdf);   // in place if staged
    int positive = 0;
    for (int k = tid; k < m; k += kThreads) {
      const uint4 blk = philox4x32_10(make_uint4(static_cast<uint32_t>(k >> 2), a.layer_id, a.epoch,
                                                 kStreamTag),
                                      make_uint2(a.seed_lo, a.seed_hi));
      const uint32_t sel = k & 3;
      const uint32_t word = sel == 0 ? blk.x : sel == 1 ? blk.y : sel == 2 ? blk.z : blk.w;
      const double u = (static_cast<double>(word) + 0.5) * 0x1p-32;
      const double w = sampling_weight(a.method, nrm[k]);
      scores[k] = static_cast<float>(w / -log(u));
      positive += w > 0.0;
    }
    int total_positive;
    block_inclusive_scan<int>(positive, s_int, total_positive);
    if (total_positive < r) {
      if (tid == 0) record_status(a.status, GRASS_ERR_DEGENERATE, total_positive);
      return;
    }
    __syncthreads();
    keys = scores;
  }
  if (a.method == GRASS_SEL_TOPR || is_nr(a.method)) {
    // ---- radix select of the r-th largest key ----
    if (tid == 0) { s_prefix = 0u; s_need = r; }
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = pass * 8;
      if (tid < 256) s_hist[tid] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      const uint32_t himask = pass == 3 ? 0u : (0xffffffffu << (shift + 8));
      for (int k = tid; k < m; k += kThreads) {
        const uint32_t key = norm_key(keys[k]);
        // norms share their leading bytes, so most of a warp lands in one bin: one atomic per
        // distinct bin per warp instead of one per row
        const bool in = (key & himask) == prefix;
        const uint32_t voters = __ballot_sync(__activemask(), in);
        if (in) {
          const uint32_t bin = (key >> shift) & 0xff;
          const uint32_t peers = __match_any_sync(voters, bin);
          if ((tid & 31) == __ffs(peers) - 1) atomicAdd(&s_hist[bin], __popc(peers));
        }
      }
      __syncthreads();
      if (tid < 32) {
        // digit d with (keys above d) < need <= (keys at or above d), found by one warp: lane l
        // owns bins 8l..8l+7; a suffix scan over the lanes, then a look inside one lane's bins
        int h[8], mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { h[i] = s_hist[8 * tid + i]; mine += h[i]; }
        int incl = mine;                     // keys in this lane's bins and all higher lanes'
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int dn = __shfl_down_sync(0xffffffffu, incl, o);
          if (tid + o < 32) incl += dn;
        }
        const int need = s_need;
        const int above = incl - mine;       // keys in higher lanes' bins
        const bool here = above < need && need <= incl;   // true in exactly one lane
        if (here) {
          int rem = need - above, d = 7;
          for (; d > 0; --d) {
            if (h[d] >= rem) break;
            rem -= h[d];
          }
          s_need = rem;                      // how many to take among keys with this digit
          s_prefix = prefix | (static_cast<uint32_t>(8 * tid + d) << shift);
        }
      }
      __syncthreads();
    }
    const uint32_t tau = s_prefix;           // key of the r-th largest norm
    const int need_eq = s_need;              // rows equal to tau to take, lowest row first
    // ---- emit in ascending row order.  Each warp owns a contiguous segment of rows; one
    // counting pass, one scan over the 32 warp totals, one writing pass: three block barriers
    // in all, instead of a block-wide scan for every 1024 rows. ----
    const int lane = tid & 31, warp = tid >> 5;
    const int seg = ((m + kWarps - 1) / kWarps + 31) & ~31;   // rows per warp, multiple of 32
    const int k_begin = warp * seg, k_end = k_begin + seg < m ? k_begin + seg : m;
    int n_eq = 0, n_gt = 0;
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
      const int k = k0 + lane;
      const uint32_t key = k < k_end ? norm_key(keys[k]) : 0u;
      n_eq += __popc(__ballot_sync(0xffffffffu, k < k_end && key == tau));
      n_gt += __popc(__ballot_sync(0xffffffffu, k < k_end && key > tau));
    }
    __shared__ int s_eq_base[kWarps], s_out_base[kWarps];
    if (lane == 0) { s_eq_base[warp] = n_eq; s_out_base[warp] = n_gt; }
    __syncthreads();
    if (warp == 0) {
      // exclusive prefix of the eq counts, then of the selected counts, over the 32 warps
      const int eq = s_eq_base[lane], gt = s_out_base[lane];
      int eq_incl = eq;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, eq_incl, o);
        if (lane >= o) eq_incl += up;
      }
      const int eq_excl = eq_incl - eq;
      int take = need_eq - eq_excl;                    // equal rows this warp may still take
      take = take < 0 ? 0 : (take > eq ? eq : take);
      const int sel = gt + take;
      int sel_incl = sel;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, sel_incl, o);
        if (lane >= o) sel_incl += up;
      }
      s_eq_base[lane] = eq_excl;
      s_out_base[lane] = sel_incl - sel;
    }
    __syncthreads();
    int eq_base = s_eq_base[warp], out_base = s_out_base[warp];
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
      const int k = k0 + lane;
      const uint32_t key = k < k_end ? norm_key(keys[k]) : 0u;
      const bool is_eq = k < k_end && key == tau, is_gt = k < k_end && key > tau;
      const uint32_t eq_bits = __ballot_sync(0xffffffffu, is_eq);
      const bool sel = is_gt || (is_eq && eq_base + __popc(eq_bits & lt_mask) < need_eq);
      const uint32_t sel_bits = __ballot_sync(0xffffffffu, sel);
      if (sel) {
        const int pos = out_base + __popc(sel_bits & lt_mask);
        a.idx[pos] = k;
        a.rho[pos] = 1.f;
      }
      eq_base += __popc(eq_bits);
      out_base += __popc(sel_bits);
    }
    return;
  }

  // ---- with replacement: inverse CDF of the sampling weights.  Same two-pass scheme as the
  // emit above: a warp owns a contiguous segment of rows, sums it, one scan over the 32 warp
  // totals gives every segment its base, and a second pass writes the running sum. ----
  const int lane = tid & 31, warp = tid >> 5;
  const int seg = ((m + kWarps - 1) / kWarps + 31) & ~31;
  const int k_begin = warp * seg, k_end = k_begin + seg < m ? k_begin + seg : m;
  __shared__ double s_wbase[kWarps];
  __shared__ double s_total;
  __shared__ int s_cbase[kWarps];
  // local[k] = running sum inside the segment (warp scan per 32 rows, carried across the
  // segment); cdf[k] = base[warp] + local[k] with base[w + 1] = base[w] + local total of w added
  // by one thread in order.  A shuffle scan adds the same terms in a different order in every
  // lane, so neighbouring entries can disagree in the last bit; what a draw must never do is
  // land on a row of zero weight (rho would be infinite).  Therefore a zero-weight row takes
  // the entry of the nearest row of positive weight before it, bit for bit (0 if the slice has
  // none, which makes it equal to the previous slice's last entry): cdf[k] > target can then
  // first become true only at a row of positive weight.
  auto slice_scan = [&](int k0) {
    const int k = k0 + lane;
    const double w = k < k_end ? sampling_weight(a.method, nrm[k]) : 0.0;
    double v = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += up;
    }
    const uint32_t positive = __ballot_sync(0xffffffffu, w > 0.0);
    const uint32_t at_or_before = positive & (0xffffffffu >> (31 - lane));
    const int src = at_or_before != 0u ? 31 - __clz(at_or_before) : 0;
    const double taken = __shfl_sync(0xffffffffu, v, src);
    return at_or_before != 0u ? taken : 0.0;
  };
  {
    double run = 0.0;
    for (int k0 = k_begin; k0 < k_end; k0 += 32)
      run = run + __shfl_sync(0xffffffffu, slice_scan(k0), 31);
    if (lane == 0) s_wbase[warp] = run;
  }
  __syncthreads();
  if (tid == 0) {
    double base = 0.0;
    for (int w = 0; w < kWarps; ++w) {
      const double t = s_wbase[w];
      s_wbase[w] = base;
      base = base + t;
    }
    s_total = base;
  }
  __syncthreads();
  const double S = s_total;
  if (!(S > 0.0)) {
    if (tid == 0) record_status(a.status, GRASS_ERR_DEGENERATE, -1);
    return;
  }
  {
    const double base = s_wbase[warp];
    double run = 0.0;
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
      const int k = k0 + lane;
      const double v = slice_scan(k0);
      if (k < k_end) {
        cdf[k] = base + (run + v);
        counts[k] = 0;
      }
      run = run + __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();  // cdf and counts visible block-wide (same CTA: global writes + barrier)
  for (int j = tid; j < r; j += kThreads) {
    const uint4 blk = philox4x32_10(make_uint4(static_cast<uint32_t>(j >> 2), a.layer_id, a.epoch,
                                               kStreamTag),
                                    make_uint2(a.seed_lo, a.seed_hi));
    const uint32_t sel = j & 3;
    const uint32_t word = sel == 0 ? blk.x : sel == 1 ? blk.y : sel == 2 ? blk.z : blk.w;
    const double target = (static_cast<double>(word) * 0x1p-32) * S;
    int lo = 0, hi = m - 1;                  // first k with cdf[k] > target
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (cdf[mid] > target) hi = mid; else lo = mid + 1;
    }
    // (the entries of zero-weight rows repeat their predecessor's, so lo has positive weight;
    // the loop below only guards the very last rows when the target rounds up to the total)
    while (lo > 0 && !(sampling_weight(a.method, nrm[lo]) > 0.0)) --lo;
    atomicAdd(&counts[lo], 1);
  }
  __syncthreads();
  // expand the hit counts in row order: per-warp totals, one scan, one writing pass
  {
    int run = 0;
    for (int k0 = k_begin; k0 < k_end; k0 += 32) {
      const int k = k0 + lane;
      int c = k < k_end ? counts[k] : 0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
      run += c;
    }
    if (lane == 0) s_cbase[warp] = run;
  }
  __syncthreads();
  if (warp == 0) {
    const int mine = s_cbase[lane];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    s_cbase[lane] = incl - mine;
  }
  __syncthreads();
  int out_base = s_cbase[warp];
  for (int k0 = k_begin; k0 < k_end; k0 += 32) {
    const int k = k0 + lane;
    const int cnt = k < k_end ? counts[k] : 0;
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (cnt > 0) {
      const double q = sampling_weight(a.method, nrm[k]) / S;
      const float rho = static_cast<float>(1.0 / sqrt(static_cast<double>(r) * q));
      const int pos = out_base + incl - cnt;
      for (int i = 0; i < cnt; ++i) {
        a.idx[pos + i] = k;
        a.rho[pos + i] = rho;
      }
    }
    out_base += __shfl_sync(0xffffffffu, incl, 31);
  }
}

// Stage the norms (and, if they still fit, the hit counters) in shared memory: the kernel is a
// chain of short passes over m values, each of which would otherwise wait on an L2 round trip.
int launch_select(SelectArgs& a, cudaStream_t s) {
  constexpr size_t kBudget = 200 * 1024;
  const size_t m4 = (static_cast<size_t>(a.m) + 3) / 4 * 4 * sizeof(float);
  a.stage_norms = m4 <= kBudget;
  a.stage_counts = a.stage_norms && a.method != GRASS_SEL_TOPR && 2 * m4 <= kBudget;
  a.stage_cdf = a.stage_counts && 4 * m4 <= kBudget;
  const size_t smem = a.stage_norms ? (a.stage_cdf ? 4 * m4 : a.stage_counts ? 2 * m4 : m4) : 0;
  static bool attr_set[64] = {false};
  int dev = 0;
  GRASS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    GRASS_CUDA_TRY(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kBudget)));
    attr_set[dev] = true;
  }
  {
    ProfileScope prof(GRASS_K_SELECT, s);
    select_kernel<<<1, kThreads, smem, s>>>(a);
  }
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

size_t cdf_bytes(int64_t m) { return round_up(static_cast<size_t>(m) * sizeof(double), 256); }

}  // namespace
}  // namespace grass

extern "C" size_t grass_select_workspace_bytes(int64_t m, int32_t r, int method) {
  (void)r;
  if (m < 1) return 0;
  if (method == GRASS_SEL_TOPR) return 256;  // unused, but never zero so callers can allocate
  return grass::cdf_bytes(m) + grass::round_up(static_cast<size_t>(m) * sizeof(int), 256);
}

extern "C" int grass_select(const float* norms, int64_t m, int32_t r, int method, uint64_t seed,
                            uint32_t layer_id, uint32_t epoch, int32_t* idx, float* rho, void* ws,
                            size_t ws_bytes, void* stream) {
  using namespace grass;
  if (norms == nullptr || idx == nullptr || rho == nullptr || m < 1 || m > 0x7fffffffLL ||
      r < 1 || r > m)
    return GRASS_ERR_INVALID_ARG;
  if (method < GRASS_SEL_TOPR || method > GRASS_SEL_UNIFORM_NR) return GRASS_ERR_UNSUPPORTED;
  SelectArgs a;
  a.cdf = nullptr;
  a.counts = nullptr;
  if (method != GRASS_SEL_TOPR) {
    if (ws == nullptr || !aligned_to(ws, 256) ||
        ws_bytes < grass_select_workspace_bytes(m, r, method))
      return GRASS_ERR_WORKSPACE;
    a.cdf = static_cast<double*>(ws);
    a.counts = reinterpret_cast<int*>(static_cast<char*>(ws) + cdf_bytes(m));
  }
  cudaError_t err;
  a.status = status_word(&err);
  if (a.status == nullptr) GRASS_CUDA_TRY(err);
  a.norms = norms;
  a.m = static_cast<int>(m);
  a.r = r;
  a.method = method;
  a.seed_lo = static_cast<uint32_t>(seed & 0xffffffffu);
  a.seed_hi = static_cast<uint32_t>(seed >> 32);
  a.layer_id = layer_id;
  a.epoch = epoch;
  a.idx = idx;
  a.rho = rho;
  return launch_select(a, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------
// grass_select_static: the same selection with its scratch in a fixed device
// array that is part of the library image, for callers that cannot allocate.
// ---------------------------------------------------------------------------
namespace grass {
namespace {

constexpr int kStaticMaxM = GRASS_SELECT_STATIC_MAX_M;

// Running sum (fp64) followed by the per-row hit counts (int32) for up to
// kStaticMaxM rows: 192 KiB, resident on every GPU that loads the library.
static __device__ __align__(256) unsigned char g_select_scratch[kStaticMaxM * (sizeof(double) + sizeof(int))];

// Device address of g_select_scratch on the current device, resolved once per
// device.  In host code the symbol name is only a handle; a kernel must be
// given the address the runtime reports for it.
int static_scratch(unsigned char** out) {
  static unsigned char* cached[64] = {nullptr};
  int dev = 0;
  GRASS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return GRASS_ERR_INVALID_ARG;
  if (cached[dev] == nullptr) {
    unsigned char* p = nullptr;
    GRASS_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_select_scratch));
    cached[dev] = p;
  }
  *out = cached[dev];
  return GRASS_OK;
}

}  // namespace
}  // namespace grass

extern "C" int grass_select_static(const float* norms, int64_t m, int32_t r, int method,
                                   uint64_t seed, uint32_t layer_id, uint32_t epoch, int32_t* idx,
                                   float* rho, void* stream) {
  using namespace grass;
  if (norms == nullptr || idx == nullptr || rho == nullptr || m < 1 || r < 1 || r > m)
    return GRASS_ERR_INVALID_ARG;
  if (m > kStaticMaxM) {
    fprintf(stderr, "grass_select_static: m = %lld exceeds the built-in scratch (%d rows); "
                    "use grass_select with a caller-provided workspace\n",
            static_cast<long long>(m), kStaticMaxM);
    return GRASS_ERR_WORKSPACE;
  }
  if (method < GRASS_SEL_TOPR || method > GRASS_SEL_UNIFORM_NR) return GRASS_ERR_UNSUPPORTED;
  unsigned char* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != GRASS_OK) return rc;
  cudaError_t err;
  SelectArgs a;
  a.status = status_word(&err);
  if (a.status == nullptr) GRASS_CUDA_TRY(err);
  a.cdf = reinterpret_cast<double*>(scratch);
  a.counts = reinterpret_cast<int*>(scratch + static_cast<size_t>(kStaticMaxM) * sizeof(double));
  a.norms = norms;
  a.m = static_cast<int>(m);
  a.r = r;
  a.method = method;
  a.seed_lo = static_cast<uint32_t>(seed & 0xffffffffu);
  a.seed_hi = static_cast<uint32_t>(seed >> 32);
  a.layer_id = layer_id;
  a.epoch = epoch;
  a.idx = idx;
  a.rho = rho;
  // Of the array the kernel can reach only the running sum, and only for m > 12800 with a
  // with-replacement method (everything else is staged in shared memory); it writes every
  // running-sum entry before reading it, so whatever an earlier call left there is never
  // observed.
  return launch_select(a, static_cast<cudaStream_t>(stream));
}
