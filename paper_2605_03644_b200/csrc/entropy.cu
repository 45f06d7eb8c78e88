// Softmax entropy of last-token logits (paper Eq. 2, over the whole vocabulary)
// and the threshold rule stated after it.
//
// One pass: every thread keeps (m, s, t) with s = sum e^{x-m}, t = sum e^{x-m}(x-m)
// for a running maximum m; states merge exactly (up to rounding) under a change of
// maximum, and H = ln s - t / s at the end.  Rows are split over several CTAs so a
// handful of 128K-entry rows still fills the machine; the per-split states go
// through the caller's workspace and a second, tiny kernel merges them.
#include <float.h>

#include "common.cuh"

namespace {

struct EntState {
  float m, s, t;
};

__device__ __forceinline__ EntState ent_merge(EntState a, EntState b) {
  float M = fmaxf(a.m, b.m);
  float ea = __expf(a.m - M), eb = __expf(b.m - M);
  // a state with s == 0 has seen nothing (or only -inf): it adds nothing
  float ta = a.s > 0.f ? (a.t + a.s * (a.m - M)) * ea : 0.f;
  float tb = b.s > 0.f ? (b.t + b.s * (b.m - M)) * eb : 0.f;
  EntState r;
  r.m = M;
  r.s = a.s * ea + b.s * eb;
  r.t = ta + tb;
  return r;
}

__device__ __forceinline__ float ent_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ent_max3(float a, float b, float c) {   // one instruction on sm_100
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Logits at or below this value count as -inf: the loaders raise every logit to it (an exact
// operation), so that x - m stays finite and e * (x - m) is -0, not NaN, where e underflows to 0.
// -2^97 is exact in bf16 and in fp32.  A row that holds nothing above it has entropy 0 by
// convention (entropy_finish_kernel).
constexpr float kEntFloor = -1.5845632502852868e29f;
constexpr uint32_t kEntFloorBf16x2 = 0xF000F000u;

// Adds N logits (already raised to kEntFloor) to a state.  d = x - m is formed exactly (the row
// maximum itself gives d = 0 and e = 1), e = 2^(d log2 e) is one multiply and one MUFU operation,
// t accumulates e * d.  Pairs of logits go through the two-wide fp32 add / multiply / FMA forms,
// which halves the instructions around the exponential.
template <int N>
__device__ __forceinline__ void ent_accumulate(EntState& st, const float (&x)[N]) {
  constexpr float kLog2e = 1.4426950408889634f;
  float vm = x[0];
  {
    int i = 1;
#pragma unroll
    for (; i + 1 < N; i += 2) vm = ent_max3(vm, x[i], x[i + 1]);
    if (i < N) vm = fmaxf(vm, x[i]);
  }
  if (vm > st.m) {
    float e = __expf(st.m - vm);
    st.t = st.s > 0.f ? (st.t + st.s * (st.m - vm)) * e : 0.f;
    st.s *= e;
    st.m = vm;
  }
  if constexpr (N % 2 == 0) {
    const float2 neg_m = make_float2(-st.m, -st.m);
    const float2 l2e = make_float2(kLog2e, kLog2e);
    float2 s2 = make_float2(0.f, 0.f), t2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < N; i += 2) {
      const float2 d = __fadd2_rn(make_float2(x[i], x[i + 1]), neg_m);
      const float2 a = __fmul2_rn(d, l2e);
      const float2 e = make_float2(ent_ex2(a.x), ent_ex2(a.y));
      s2 = __fadd2_rn(s2, e);
      t2 = __ffma2_rn(e, d, t2);
    }
    st.s += s2.x + s2.y;
    st.t += t2.x + t2.y;
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float d = x[i] - st.m;
      const float e = ent_ex2(d * kLog2e);
      st.s += e;
      st.t = fmaf(e, d, st.t);
    }
  }
}

__device__ __forceinline__ EntState ent_warp_reduce(EntState st) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    EntState other;
    other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
    other.s = __shfl_xor_sync(0xffffffffu, st.s, o);
    other.t = __shfl_xor_sync(0xffffffffu, st.t, o);
    st = ent_merge(st, other);
  }
  return st;
}

constexpr int kEntThreads = 256;

// One-dimensional grid of R * n_split blocks (block = r * n_split + s, so the row count is not
// bound by the 65535 limit of the other grid dimensions).
// partial[(r * n_split + s)] = state of slice s of row r.
template <typename T>
__global__ void __launch_bounds__(kEntThreads, 6)
entropy_partial_kernel(const T* __restrict__ logits, int V, long long row_stride, int slice, int n_split,
                       float* __restrict__ partial) {
  constexpr int kVec = 16 / sizeof(T);
  constexpr float kLog2e = 1.4426950408889634f;
  const int r = blockIdx.x / n_split, sp = blockIdx.x % n_split;
  const T* row = logits + (long long)r * row_stride;
  const int begin = sp * slice;
  const int end = V - begin <= slice ? V : begin + slice;      // (begin + slice may not fit an int)
  EntState st{kEntFloor, 0.f, 0.f};    // every logit is at least the floor, so m starts there

  const int n_vec = (end - begin) / kVec;                        // slice is a multiple of kVec
  auto widen = [](const uint4& raw, float (&x)[kVec]) {
    if constexpr (sizeof(T) == 4) {
      x[0] = fmaxf(__uint_as_float(raw.x), kEntFloor); x[1] = fmaxf(__uint_as_float(raw.y), kEntFloor);
      x[2] = fmaxf(__uint_as_float(raw.z), kEntFloor); x[3] = fmaxf(__uint_as_float(raw.w), kEntFloor);
    } else {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {   // the floor on both halves at once; bf16 -> fp32 is a 16-bit shift
        uint32_t c;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(c) : "r"(w[j]), "r"(kEntFloorBf16x2));
        x[2 * j] = __uint_as_float(c << 16);
        x[2 * j + 1] = __uint_as_float(c & 0xffff0000u);
      }
    }
  };
  // Four 16-byte loads per thread are kept in flight: a vector is copied out of its register,
  // the load of the vector four steps ahead goes into that register at once, and only then is
  // the copy worked on, so the memory system is never idle while a warp computes.  The host cuts
  // rows into slices that are multiples of kEntSliceUnit, so that all but a row's last slice run
  // in this loop alone.
  constexpr int kUnroll = 4;
  const uint4* vp = reinterpret_cast<const uint4*>(row + begin) + threadIdx.x;
  const uint4* const vp_end = reinterpret_cast<const uint4*>(row + begin) + n_vec;
  const int trips = n_vec / (kUnroll * kEntThreads);
  if (trips > 0) {
    uint4 raw[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) raw[u] = __ldcs(vp + u * kEntThreads);
    for (int t = 1; t < trips; ++t) {
      vp += kUnroll * kEntThreads;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        float x[kVec];
        widen(raw[u], x);
        raw[u] = __ldcs(vp + u * kEntThreads);
        ent_accumulate(st, x);
      }
    }
    vp += kUnroll * kEntThreads;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float x[kVec];
      widen(raw[u], x);
      ent_accumulate(st, x);
    }
  }
  for (; vp < vp_end; vp += kEntThreads) {
    float x[kVec];
    widen(__ldcs(vp), x);
    ent_accumulate(st, x);
  }
  for (int i = begin + n_vec * kVec + threadIdx.x; i < end; i += kEntThreads) {   // ragged tail of the row
    float x[1];
    if constexpr (sizeof(T) == 4) x[0] = fmaxf(row[i], kEntFloor);
    else x[0] = fmaxf(__bfloat162float(row[i]), kEntFloor);
    ent_accumulate(st, x);
  }

  // CTA-wide merge: the maximum first; every thread then moves its (s, t) to it once, and what is
  // left are plain sums (a butterfly of whole states would pay two exponentials per level)
  __shared__ float sh_m[kEntThreads / 32], sh_s[kEntThreads / 32], sh_t[kEntThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float M = st.m;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  if (lane == 0) sh_m[warp] = M;
  __syncthreads();
  M = sh_m[0];
#pragma unroll
  for (int w = 1; w < kEntThreads / 32; ++w) M = fmaxf(M, sh_m[w]);
  const float d = fmaxf(st.m - M, -1.0e30f);          // <= 0; the clamp keeps s * d finite
  const float e = ent_ex2(d * kLog2e);
  float ss = st.s * e, tt = fmaf(st.s, d, st.t) * e;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
    tt += __shfl_xor_sync(0xffffffffu, tt, o);
  }
  if (lane == 0) { sh_s[warp] = ss; sh_t[warp] = tt; }
  __syncthreads();
  if (threadIdx.x == 0) {
    ss = 0.f; tt = 0.f;
#pragma unroll
    for (int w = 0; w < kEntThreads / 32; ++w) { ss += sh_s[w]; tt += sh_t[w]; }
    float* o = partial + 3ll * ((long long)r * n_split + sp);
    o[0] = M; o[1] = ss; o[2] = tt;
  }
}

// One CTA per group of `rows_per_group` rows; warp w merges the splits of rows
// w, w + n_warps, ...; thread 0 then applies the threshold rule to the group.
__global__ void __launch_bounds__(256)
entropy_finish_kernel(const float* __restrict__ partial, int n_split, int R, int rows_per_group,
                      float tau, float* __restrict__ H, int32_t* __restrict__ first_ok) {
  extern __shared__ float sh_h[];
  const int g = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int j = warp; j < rows_per_group; j += n_warps) {
    const int r = g * rows_per_group + j;
    if (r >= R) break;
    EntState st{-FLT_MAX, 0.f, 0.f};
    for (int s = lane; s < n_split; s += 32) {
      const float* p = partial + 3ll * ((long long)r * n_split + s);
      st = ent_merge(st, EntState{p[0], p[1], p[2]});
    }
    st = ent_warp_reduce(st);
    if (lane == 0) {
      // a maximum at the floor: the row holds nothing but -inf (or values that count as it)
      float h = (st.s > 0.f && st.m > kEntFloor) ? logf(st.s) - st.t / st.s : 0.f;
      h = fmaxf(h, 0.f);
      H[r] = h;
      sh_h[j] = h;
    }
  }
  __syncthreads();
  if (first_ok != nullptr && threadIdx.x == 0) {
    int ok = -1;
    for (int j = 0; j < rows_per_group && g * rows_per_group + j < R; ++j) {
      if (sh_h[j] <= tau) { ok = j; break; }
    }
    first_ok[g] = ok;
  }
}

// Two-token form of Eq. 2 (the paper takes the entropy over the answer tokens {Yes, No}): like
// entropy_finish_kernel, but the sum runs over the `n_subset` listed token ids only.
//   renorm == 0: p_v from the softmax over the whole vocabulary, H = -sum_{v in S} p_v ln p_v
//   renorm == 1: q_v = p_v / sum_{S} p, H = -sum q_v ln q_v
template <typename T>
__global__ void __launch_bounds__(256)
entropy_subset_finish_kernel(const float* __restrict__ partial, int n_split, int R, int rows_per_group,
                             const T* __restrict__ logits, long long row_stride, int V,
                             const int32_t* __restrict__ subset_ids, int n_subset, int renorm,
                             float tau, float* __restrict__ H, int32_t* __restrict__ first_ok,
                             int32_t* __restrict__ status) {
  extern __shared__ float sh_h[];
  const int g = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int j = warp; j < rows_per_group; j += n_warps) {
    const int r = g * rows_per_group + j;
    if (r >= R) break;
    EntState st{-FLT_MAX, 0.f, 0.f};
    for (int s = lane; s < n_split; s += 32) {
      const float* p = partial + 3ll * ((long long)r * n_split + s);
      st = ent_merge(st, EntState{p[0], p[1], p[2]});
    }
    st = ent_warp_reduce(st);
    const float m = __shfl_sync(0xffffffffu, st.m, 0);
    const float ln_s = logf(__shfl_sync(0xffffffffu, st.s, 0));
    const T* row = logits + (long long)r * row_stride;
    float z = 0.f, u = 0.f, h = 0.f;           // sum e^{x-m}, sum e^{x-m}(x-m), -sum p ln p
    for (int i = lane; i < n_subset; i += 32) {
      const int id = subset_ids[i];
      if (id < 0 || id >= V) {
        ads_set_status(status, ADAPSHOT_EINDEX);
        continue;
      }
      float x;
      if constexpr (sizeof(T) == 4) x = row[id]; else x = __bfloat162float(row[id]);
      const float d = x - m;
      const float e = __expf(d);
      z += e;
      u += e > 0.f ? e * d : 0.f;
      const float lp = d - ln_s;                // ln p_v
      const float pv = __expf(lp);
      h -= pv > 0.f ? pv * lp : 0.f;
    }
    z = warp_sum(z); u = warp_sum(u); h = warp_sum(h);
    if (lane == 0) {
      float out = renorm ? (z > 0.f ? logf(z) - u / z : 0.f) : h;
      out = fmaxf(out, 0.f);
      H[r] = out;
      sh_h[j] = out;
    }
  }
  __syncthreads();
  if (first_ok != nullptr && threadIdx.x == 0) {
    int ok = -1;
    for (int j = 0; j < rows_per_group && g * rows_per_group + j < R; ++j) {
      if (sh_h[j] <= tau) { ok = j; break; }
    }
    first_ok[g] = ok;
  }
}

// A fixed figure rather than the SM count of the current device, so that the workspace size
// can be asked for without a device and does not change from one GPU to another: one resident
// wave of 256-thread CTAs at 40 registers (six per SM) on 148 SMs.
constexpr int kEntTargetCtas = 888;
constexpr int kEntSliceUnit = 8192;      // entries: what a CTA's unrolled loop takes per trip (bf16)
constexpr int kEntCtaOverhead = 2048;    // fixed cost of a CTA (start, state merge, store) in entries

// Rows are cut into slices of j * kEntSliceUnit entries (the last one shorter).  A call's CTAs run
// in ceil(R * n / kEntTargetCtas) waves of about equal length (slice + overhead), so the j that
// minimises waves * (slice + overhead) is taken: 2048 rows of 128 256 run as 2 slices each (4.6
// waves) rather than whole (2.3 waves, the third one a third full), 224 rows as 3 slices (one wave).  `max_states` bounds R * n (the fixed scratch of the static entry point).
struct EntSplit { int slice, n; };
EntSplit ent_split(int R, int V, long long max_states = 0x7fffffffll) {
  const long long unit = kEntSliceUnit;
  const long long kMaxSlice = 0x7fffe000ll;                             // the largest multiple of the unit an int holds
  EntSplit best{(int)((long long)V <= kMaxSlice ? ((long long)V + unit - 1) / unit * unit : kMaxSlice),
                (long long)V <= kMaxSlice ? 1 : 2};                      // the row in one piece (two beyond 2^31 - 8192)
  double best_cost = 0.0;
  for (int want = 1; want <= 64; ++want) {
    // the shortest slice (a multiple of the unit) that cuts the row into at most `want` pieces
    const long long per = ((long long)V + want - 1) / want;
    long long slice = (per + unit - 1) / unit * unit;
    if (slice > kMaxSlice) slice = kMaxSlice;
    const int n = (int)(((long long)V + slice - 1) / slice);
    if ((long long)R * n > max_states) break;                            // n only grows with `want`
    const long long waves = ((long long)R * n + kEntTargetCtas - 1) / kEntTargetCtas;
    const double cost = (double)waves * (double)(slice + kEntCtaOverhead);
    if (want == 1 || cost < best_cost) {
      best = EntSplit{(int)slice, n};
      best_cost = cost;
    }
  }
  return best;
}
int ent_splits(int R, int V) { return ent_split(R, V).n; }

}  // namespace

extern "C" size_t adapshot_entropy_workspace_bytes(int32_t R, int32_t V) {
  if (R <= 0 || V <= 0) return 0;
  return ads_round_up((size_t)R * ent_splits(R, V) * 3 * sizeof(float), 256);
}

extern "C" int adapshot_entropy(const void* logits, int32_t dtype, int32_t R, int32_t V,
                                int64_t row_stride, float* H, float tau, int32_t rows_per_group,
                                int32_t* first_ok, void* ws, size_t ws_bytes, int32_t* status,
                                void* stream) {
  (void)status;
  if (logits == nullptr || H == nullptr || ws == nullptr) return ADAPSHOT_EINVAL;
  if (R <= 0 || V <= 0 || row_stride < V) return ADAPSHOT_EINVAL;
  if (dtype != ADAPSHOT_F32 && dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (rows_per_group <= 0) rows_per_group = 1;
  if (R % rows_per_group != 0 || rows_per_group > 8192) return ADAPSHOT_ESHAPE;
  if ((long long)R * ent_splits(R, V) > 0x7fffffffll) return ADAPSHOT_ESHAPE;
  const size_t es = dtype == ADAPSHOT_F32 ? 4 : 2;
  if (!ads_aligned16(logits) || !ads_aligned16(ws) || (row_stride * es) % 16 != 0) return ADAPSHOT_EALIGN;
  if (ws_bytes < adapshot_entropy_workspace_bytes(R, V)) return ADAPSHOT_ECAPACITY;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const EntSplit cut = ent_split(R, V);
  const int n_split = cut.n, slice = cut.slice;
  const unsigned grid = (unsigned)((long long)R * n_split);
  float* partial = static_cast<float*>(ws);
  if (dtype == ADAPSHOT_F32)
    entropy_partial_kernel<float><<<grid, kEntThreads, 0, st>>>(
        static_cast<const float*>(logits), V, row_stride, slice, n_split, partial);
  else
    entropy_partial_kernel<__nv_bfloat16><<<grid, kEntThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(logits), V, row_stride, slice, n_split, partial);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  entropy_finish_kernel<<<R / rows_per_group, 256, rows_per_group * sizeof(float), st>>>(
      partial, n_split, R, rows_per_group, tau, H, first_ok);
  return ads_launch_status();
}


extern "C" int adapshot_entropy_subset(const void* logits, int32_t dtype, int32_t R, int32_t V,
                                       int64_t row_stride, const int32_t* subset_ids, int32_t n_subset,
                                       uint32_t flags, float* H, float tau, int32_t rows_per_group,
                                       int32_t* first_ok, void* ws, size_t ws_bytes, int32_t* status,
                                       void* stream) {
  if (logits == nullptr || H == nullptr || ws == nullptr || subset_ids == nullptr) return ADAPSHOT_EINVAL;
  if (R <= 0 || V <= 0 || row_stride < V || n_subset <= 0 || n_subset > V || (flags & ~1u) != 0)
    return ADAPSHOT_EINVAL;
  if (dtype != ADAPSHOT_F32 && dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (rows_per_group <= 0) rows_per_group = 1;
  if (R % rows_per_group != 0 || rows_per_group > 8192) return ADAPSHOT_ESHAPE;
  if ((long long)R * ent_splits(R, V) > 0x7fffffffll) return ADAPSHOT_ESHAPE;
  const size_t es = dtype == ADAPSHOT_F32 ? 4 : 2;
  if (!ads_aligned16(logits) || !ads_aligned16(ws) || (row_stride * es) % 16 != 0 ||
      ((uintptr_t)subset_ids & 3u))
    return ADAPSHOT_EALIGN;
  if (ws_bytes < adapshot_entropy_workspace_bytes(R, V)) return ADAPSHOT_ECAPACITY;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const EntSplit cut = ent_split(R, V);
  const int n_split = cut.n, slice = cut.slice;
  const unsigned grid = (unsigned)((long long)R * n_split);
  float* partial = static_cast<float*>(ws);
  const int renorm = (int)(flags & 1u);
  const size_t sh = rows_per_group * sizeof(float);
  if (dtype == ADAPSHOT_F32) {
    const float* lg = static_cast<const float*>(logits);
    entropy_partial_kernel<float><<<grid, kEntThreads, 0, st>>>(lg, V, row_stride, slice, n_split, partial);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
    entropy_subset_finish_kernel<float><<<R / rows_per_group, 256, sh, st>>>(
        partial, n_split, R, rows_per_group, lg, row_stride, V, subset_ids, n_subset, renorm, tau, H, first_ok,
        status);
  } else {
    const __nv_bfloat16* lg = static_cast<const __nv_bfloat16*>(logits);
    entropy_partial_kernel<__nv_bfloat16><<<grid, kEntThreads, 0, st>>>(lg, V, row_stride, slice, n_split, partial);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
    entropy_subset_finish_kernel<__nv_bfloat16><<<R / rows_per_group, 256, sh, st>>>(
        partial, n_split, R, rows_per_group, lg, row_stride, V, subset_ids, n_subset, renorm, tau, H, first_ok,
        status);
  }
  return ads_launch_status();
}


// --------------------------------------------------------------------------
// Entropy without any caller-provided or allocated scratch.
//
// Some callers may not allocate device memory at all: code running inside a
// memory-pool-managed serving process whose allocator must not be bypassed, a
// plugin loaded into a host that forbids cudaMalloc after start-up, or a
// latency-critical path where an allocation could synchronise the device.  For
// them the per-split states live in the fixed array below, which every GPU that
// loads this library keeps until the process exits (192 KiB per device).
constexpr int kStaticEntStates = 16384;   // most (row, split) states one call may need
static __device__ __align__(256) float g_entropy_static_scratch[kStaticEntStates * 3];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_ptr[kMaxDevices] = {nullptr};

// In host code the array's name is only a handle for the runtime; the device
// address has to be asked for, once per device, with that device current.
int static_scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ADAPSHOT_ECUDA;
  if (g_static_scratch_ptr[dev] == nullptr) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_entropy_static_scratch) != cudaSuccess ||
        ptr == nullptr)
      return ADAPSHOT_ECUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = g_static_scratch_ptr[dev];
  return ADAPSHOT_OK;
}
}  // namespace

extern "C" int adapshot_entropy_static(const void* logits, int32_t dtype, int32_t R, int32_t V,
                                       int64_t row_stride, float* H, float tau, int32_t rows_per_group,
                                       int32_t* first_ok, int32_t* status, void* stream) {
  (void)status;
  if (logits == nullptr || H == nullptr) return ADAPSHOT_EINVAL;
  if (R <= 0 || V <= 0 || row_stride < V) return ADAPSHOT_EINVAL;
  if (dtype != ADAPSHOT_F32 && dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (rows_per_group <= 0) rows_per_group = 1;
  if (R % rows_per_group != 0 || rows_per_group > 8192) return ADAPSHOT_ESHAPE;
  if ((long long)R * ent_splits(R, V) > 0x7fffffffll) return ADAPSHOT_ESHAPE;
  const size_t es = dtype == ADAPSHOT_F32 ? 4 : 2;
  if (!ads_aligned16(logits) || (row_stride * es) % 16 != 0) return ADAPSHOT_EALIGN;
  if (R > kStaticEntStates) return ADAPSHOT_ECAPACITY;   // beyond the fixed array
  const EntSplit cut = ent_split(R, V, kStaticEntStates);
  const int n_split = cut.n, slice = cut.slice;

  float* partial = nullptr;
  const int rc = static_scratch_for_current_device(&partial);
  if (rc != ADAPSHOT_OK) return rc;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const unsigned grid = (unsigned)((long long)R * n_split);
  // every (row, split) state this call reads is written by the first kernel, so
  // nothing in the shared array has to start at zero
  if (dtype == ADAPSHOT_F32)
    entropy_partial_kernel<float><<<grid, kEntThreads, 0, st>>>(
        static_cast<const float*>(logits), V, row_stride, slice, n_split, partial);
  else
    entropy_partial_kernel<__nv_bfloat16><<<grid, kEntThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(logits), V, row_stride, slice, n_split, partial);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  entropy_finish_kernel<<<R / rows_per_group, 256, rows_per_group * sizeof(float), st>>>(
      partial, n_split, R, rows_per_group, tau, H, first_ok);
  return ads_launch_status();
}
