// KV-level concatenation of the selected shots with position re-encoding of K
// (paper Sec. 4.3: Eq. 6 rotary form, Eq. 7 correction by Delta; offsets as in the
// two-shot example, where a shot's Delta is the total length placed before it).
//
// Kernel 1 (plan): ctx_off[b][r] = exclusive prefix sum of the selected lengths.
// Kernel 2 (gather): one warp moves one destination token of one query for every
// layer of the call: V rows are copied with 16-byte vectors, K rows are rotated in
// registers between the 16-byte load and store.  The rotation angles of a token do
// not depend on layer or head, so each lane forms its few (sin, cos) pairs once per
// token, in fp64 before the fp32 sincos, and reuses them over heads and layers.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int kPlanThreads = 256;
constexpr int kTile = 128;   // the attention kernel reads the cache in 128-token tiles
constexpr int kRunMax = 4;   // consecutive destination tokens per warp (fewer when the launch is small)

// One CTA per query: lengths of the selected shots, block-wide exclusive scan.
__global__ void __launch_bounds__(kPlanThreads)
plan_offsets_kernel(const int32_t* __restrict__ sel_idx, const long long* __restrict__ shot_off,
                    int n_shots, int k, long long ctx_cap, bool check_cap,
                    long long* __restrict__ ctx_off, int32_t* __restrict__ status) {
  __shared__ long long warp_tot[kPlanThreads / 32];
  __shared__ long long carry_sh;
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_sh = 0;
  __syncthreads();
  for (int base = 0; base < k; base += kPlanThreads) {
    const int r = base + threadIdx.x;
    long long len = 0;
    if (r < k) {
      const int s = sel_idx[(long long)b * k + r];
      if (s < 0 || s >= n_shots) ads_set_status(status, ADAPSHOT_EINDEX);
      else len = shot_off[s + 1] - shot_off[s];
    }
    long long incl = len;   // inclusive scan inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      long long up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    long long before = carry_sh;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (r < k) ctx_off[(long long)b * (k + 1) + r] = before + incl - len;
    __syncthreads();
    if (threadIdx.x == kPlanThreads - 1) carry_sh = before + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const long long L = carry_sh;
    ctx_off[(long long)b * (k + 1) + k] = L;
    if (check_cap && L > ctx_cap) ads_set_status(status, ADAPSHOT_ECAPACITY);
  }
}

template <typename T> struct Vec16;   // one 16-byte vector of T as fp32 lanes
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4& r, float* x) {
    x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
  }
  __device__ static uint4 pack(const float* x) {
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]),
                      __float_as_uint(x[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4& r, float* x) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      x[2 * j] = __uint_as_float(w[j] << 16);
      x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
  __device__ static uint4 pack(const float* x) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * j], x[2 * j + 1]);   // round to nearest even
      w[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

struct GatherArgs {
  const void* k_pool;
  const void* v_pool;
  void* k_ctx;
  void* v_ctx;
  const long long* shot_off;
  const int32_t* sel_idx;
  const long long* ctx_off;
  long long pool_tokens;
  long long ctx_cap;
  int n_shots, B, k, n_kv_heads;
  int layer_begin, n_layers_call;
  int shot_begin;              // first selected shot to gather (earlier positions of the cache are kept)
  int k_pos_mode;
  double rope_base;
  int32_t* status;
  double theta[64];            // theta_i = rope_base^(-2i/D), i < D/2, formed on the host
  int run;                     // destination tokens per warp and plan lookup
};

// D = head_dim.  A "pair unit" is the 16-byte vector j of the low half of one head
// together with vector j of the high half (elements i and i + D/2 rotate together).
// 128-thread CTAs of at most 88 registers: small enough to be co-resident with a persistent
// attention CTA (which leaves about 11.7 K registers and 1.5 KB of shared memory per SM), so
// that the gather of the next layer chunk can run under the attention of the current one.
// WITH_V = false: the K-only form (V is taken from the pool by its consumer); it keeps two layers'
// loads in flight and takes the registers for that (five CTAs per SM instead of six).
template <typename T, int D, bool WITH_V>
__global__ void __launch_bounds__(128, WITH_V ? 6 : 5)
gather_rope_kernel(const GatherArgs a) {
  constexpr int EPV = Vec16<T>::N;                 // elements per 16-byte vector
  constexpr int VPH = D / EPV;                     // vectors per head row
  constexpr int HALF_V = VPH / 2;                  // pair units per head
  static_assert(32 % HALF_V == 0, "a lane must keep the same vector column over its units");
  const int lane = threadIdx.x & 31;
  const long long warp_global = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * (blockDim.x >> 5);
  const int row_vecs = a.n_kv_heads * VPH;         // 16-byte vectors in one token row
  const int pair_units = a.n_kv_heads * HALF_V;
  const long long layer_stride_pool = a.pool_tokens * row_vecs;   // in uint4
  const long long layer_stride_ctx = a.ctx_cap * row_vecs;

  // the EPV values of theta of this lane's column
  const int jcol = lane % HALF_V;
  double theta[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e) theta[e] = a.theta[jcol * EPV + e];

  const uint4* kp = static_cast<const uint4*>(a.k_pool);
  const uint4* vp = static_cast<const uint4*>(a.v_pool);
  uint4* kc = static_cast<uint4*>(a.k_ctx);
  uint4* vc = static_cast<uint4*>(a.v_ctx);
  constexpr bool with_v = WITH_V;

  // A warp takes a run of kRun consecutive destination tokens of one query.  The plan lookup
  // (which selected shot covers the position) is a dependent chain of global loads, so it is
  // done once per run by the whole warp (a 32-ary search: two rounds of parallel probes of the
  // offsets instead of log2(k) serial ones) and then walked forward token by token.
  const int kRun = a.run;
  const long long runs_per_query = (a.ctx_cap + kRun - 1) / kRun;
  const long long n_runs = (long long)a.B * runs_per_query;
  for (long long run = warp_global; run < n_runs; run += n_warps) {
    const int b = (int)(run / runs_per_query);
    const long long p0 = (run % runs_per_query) * kRun;
    const long long* off = a.ctx_off + (long long)b * (a.k + 1);
    const long long L = off[a.k];
    const long long pad_end = (L + kTile - 1) / kTile * kTile;
    const long long first_pos = off[a.shot_begin];                // positions before it stay as they are
    if (p0 >= pad_end || p0 + kRun <= first_pos) continue;
    int lo = 0;
    long long o = 0, o_next = 0, src0 = 0;
    int s = -1;
    if (p0 < L) {
      // largest lo in [0, k) with off[lo] <= p0 (zero-length slots are skipped by the search)
      int seg_lo = 0, seg_n = a.k;
      while (seg_n > 1) {
        const int stride = (seg_n + 31) / 32;
        const int idx = seg_lo + lane * stride;
        const bool le = idx < seg_lo + seg_n && off[idx] <= p0;
        const int cnt = __popc(__ballot_sync(0xffffffffu, le));      // probes are ascending: a prefix is true
        const int first = seg_lo + (cnt - 1) * stride;                // cnt >= 1: off[seg_lo] <= p0
        seg_n = min(stride, seg_lo + seg_n - first);
        seg_lo = first;
      }
      lo = seg_lo;
      o = off[lo];
      o_next = off[lo + 1];
      s = a.sel_idx[(long long)b * a.k + lo];
      if (s >= 0 && s < a.n_shots) src0 = a.shot_off[s];
    }
#pragma unroll 1
    for (int tt = 0; tt < kRun; ++tt) {
    const long long p = p0 + tt;
    if (p >= a.ctx_cap) break;
    if (p < first_pos) continue;
    if (p >= L) {
      // zero the rest of the last 128-token tile so whole tiles can be read later
      if (p < pad_end) {
        for (int l = 0; l < a.n_layers_call; ++l) {
          const long long dst = ((long long)b * a.n_layers_call + l) * layer_stride_ctx + p * row_vecs;
          for (int i = lane; i < row_vecs; i += 32) {
            kc[dst + i] = make_uint4(0, 0, 0, 0);
            if (with_v) vc[dst + i] = make_uint4(0, 0, 0, 0);
          }
        }
      }
      continue;
    }
    if (p >= o_next) {               // next selected shot (skipping zero-length slots); warp-uniform
      do {
        ++lo;
        o = o_next;
        o_next = off[lo + 1];
      } while (p >= o_next);
      s = a.sel_idx[(long long)b * a.k + lo];
      src0 = (s >= 0 && s < a.n_shots) ? a.shot_off[s] : 0;
    }
    if (s < 0 || s >= a.n_shots) continue;           // reported by the plan kernel
    const long long src_tok = src0 + (p - o);
    const double delta = a.k_pos_mode == 0 ? (double)p : (double)o;

    float sn[EPV], cs[EPV];
#pragma unroll
    for (int e = 0; e < EPV; ++e) {
      // bf16 storage rounds at 2^-9: the hardware sin/cos of the reduced angle is ample there
      if constexpr (sizeof(T) == 2) rope_sincos_fast(delta, theta[e], &sn[e], &cs[e]);
      else rope_sincos(delta, theta[e], &sn[e], &cs[e]);
    }

    // rotates one pair unit (vector j of the low half of a head with vector j of the high half) and stores it
    auto rot_store = [&](const uint4& lo_v, const uint4& hi_v, long long d0) {
      float x[EPV], y[EPV], xr[EPV], yr[EPV];
      Vec16<T>::unpack(lo_v, x); Vec16<T>::unpack(hi_v, y);
#pragma unroll
      for (int e = 0; e < EPV; ++e) {
        xr[e] = x[e] * cs[e] - y[e] * sn[e];
        yr[e] = y[e] * cs[e] + x[e] * sn[e];
      }
      kc[d0] = Vec16<T>::pack(xr);
      kc[d0 + HALF_V] = Vec16<T>::pack(yr);
    };
    int l_first = 0;
    if (!with_v) {
      // K alone: the loads of two layers are issued before either is rotated, so that a warp keeps as
      // many bytes on their way as it does when it also copies V
      for (; l_first + 1 < a.n_layers_call; l_first += 2) {
        const long long srcA = (long long)(a.layer_begin + l_first) * layer_stride_pool + src_tok * row_vecs;
        const long long srcB = srcA + layer_stride_pool;
        const long long dstA = ((long long)b * a.n_layers_call + l_first) * layer_stride_ctx + p * row_vecs;
        const long long dstB = dstA + layer_stride_ctx;
        for (int unit = lane; unit < pair_units; unit += 64) {
          const int unit2 = unit + 32;
          const bool two = unit2 < pair_units;
          const int o0 = (unit / HALF_V) * VPH + jcol, o1 = (unit2 / HALF_V) * VPH + jcol;
          const uint4 z = make_uint4(0, 0, 0, 0);
          const uint4 aLo0 = kp[srcA + o0], aHi0 = kp[srcA + o0 + HALF_V];
          const uint4 bLo0 = kp[srcB + o0], bHi0 = kp[srcB + o0 + HALF_V];
          const uint4 aLo1 = two ? kp[srcA + o1] : z, aHi1 = two ? kp[srcA + o1 + HALF_V] : z;
          const uint4 bLo1 = two ? kp[srcB + o1] : z, bHi1 = two ? kp[srcB + o1 + HALF_V] : z;
          rot_store(aLo0, aHi0, dstA + o0);
          rot_store(bLo0, bHi0, dstB + o0);
          if (two) {
            rot_store(aLo1, aHi1, dstA + o1);
            rot_store(bLo1, bHi1, dstB + o1);
          }
        }
      }
    }
    for (int l = l_first; l < a.n_layers_call; ++l) {
      const long long src = (long long)(a.layer_begin + l) * layer_stride_pool + src_tok * row_vecs;
      const long long dst = ((long long)b * a.n_layers_call + l) * layer_stride_ctx + p * row_vecs;
      // K: rotate pairs.  unit = head * HALF_V + column; lane stride 32 keeps the column.
      for (int unit = lane; unit < pair_units; unit += 64) {
        const int unit2 = unit + 32;
        const bool two = unit2 < pair_units;
        const int o0 = (unit / HALF_V) * VPH + jcol, o1 = (unit2 / HALF_V) * VPH + jcol;
        const uint4 lo0 = kp[src + o0], hi0 = kp[src + o0 + HALF_V];
        uint4 lo1 = make_uint4(0, 0, 0, 0), hi1 = lo1;
        if (two) { lo1 = kp[src + o1]; hi1 = kp[src + o1 + HALF_V]; }
        rot_store(lo0, hi0, dst + o0);
        if (two) rot_store(lo1, hi1, dst + o1);
      }
      // V: plain copy, four vectors in flight per lane
      for (int i = lane; with_v && i < row_vecs; i += 128) {
        uint4 r0 = vp[src + i];
        uint4 r1 = i + 32 < row_vecs ? vp[src + i + 32] : make_uint4(0, 0, 0, 0);
        uint4 r2 = i + 64 < row_vecs ? vp[src + i + 64] : make_uint4(0, 0, 0, 0);
        uint4 r3 = i + 96 < row_vecs ? vp[src + i + 96] : make_uint4(0, 0, 0, 0);
        vc[dst + i] = r0;
        if (i + 32 < row_vecs) vc[dst + i + 32] = r1;
        if (i + 64 < row_vecs) vc[dst + i + 64] = r2;
        if (i + 96 < row_vecs) vc[dst + i + 96] = r3;
      }
    }
    }
  }
}

template <typename T, int D>
int launch_gather(GatherArgs a, cudaStream_t st) {
  const int warps_per_block = 4;
  // Resident warps: about six 128-thread CTAs per SM.  Long runs amortise the plan lookup; a
  // small launch takes shorter runs so that every resident warp gets several and the tail
  // wave stays short.
  const long long n_sm = ads_sm_count();
  if (n_sm <= 0) return ADAPSHOT_ECUDA;
  const long long resident_warps = n_sm * 6 * warps_per_block;
  const long long tokens = (long long)a.B * a.ctx_cap;
  // a call of one or two layers has little work per token to spread the plan lookup over: longer runs
  a.run = a.n_layers_call <= 2 ? 4 * kRunMax : kRunMax;
  while (a.run > 1 && tokens / a.run < 4 * resident_warps) a.run >>= 1;
  const long long units = (long long)a.B * ((a.ctx_cap + a.run - 1) / a.run);
  long long blocks = (units + warps_per_block - 1) / warps_per_block;
  // measured: one resident wave with a grid-stride loop is best when a run is short (one
  // layer per call), several waves when every run walks several layers
  const long long max_blocks = a.n_layers_call == 1 ? n_sm * 6 : n_sm * 16 * 4;
  if (blocks > max_blocks) blocks = max_blocks;
  if (a.v_ctx != nullptr) gather_rope_kernel<T, D, true><<<(unsigned)blocks, warps_per_block * 32, 0, st>>>(a);
  else gather_rope_kernel<T, D, false><<<(unsigned)blocks, warps_per_block * 32, 0, st>>>(a);
  return ads_launch_status();
}

}  // namespace

extern "C" int adapshot_assemble_kv(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                    const int32_t* sel_idx, int32_t B, int32_t k,
                                    int32_t layer_begin, int32_t layer_end, void* k_ctx, void* v_ctx,
                                    int64_t ctx_cap, int64_t* ctx_off, uint32_t flags,
                                    int32_t* status, void* stream) {
  return adapshot_assemble_kv_from(model, pool, sel_idx, B, k, 0, layer_begin, layer_end, k_ctx, v_ctx, ctx_cap,
                                   ctx_off, flags, status, stream);
}

extern "C" int adapshot_assemble_kv_from(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                         const int32_t* sel_idx, int32_t B, int32_t k, int32_t shot_begin,
                                         int32_t layer_begin, int32_t layer_end, void* k_ctx, void* v_ctx,
                                         int64_t ctx_cap, int64_t* ctx_off, uint32_t flags,
                                         int32_t* status, void* stream) {
  if (model == nullptr || pool == nullptr || sel_idx == nullptr || ctx_off == nullptr) return ADAPSHOT_EINVAL;
  if (shot_begin < 0 || shot_begin >= k) return ADAPSHOT_ESHAPE;
  if (B <= 0 || (flags & ~(ADAPSHOT_ASSEMBLE_KEEP_PLAN | ADAPSHOT_ASSEMBLE_K_ONLY)) != 0 ||
      pool->shot_off == nullptr || pool->n_shots <= 0)
    return ADAPSHOT_EINVAL;
  const bool k_only = (flags & ADAPSHOT_ASSEMBLE_K_ONLY) != 0;
  if (k_only) v_ctx = nullptr;
  if (k < 1 || k > pool->n_shots) return ADAPSHOT_ESHAPE;
  const bool plan_only = k_ctx == nullptr && v_ctx == nullptr;
  const bool keep_plan = (flags & ADAPSHOT_ASSEMBLE_KEEP_PLAN) != 0;
  if (plan_only && keep_plan) return ADAPSHOT_EINVAL;
  if (!plan_only && (k_ctx == nullptr || (v_ctx == nullptr && !k_only))) return ADAPSHOT_EINVAL;
  if (((uintptr_t)sel_idx & 3u) || ((uintptr_t)ctx_off & 7u)) return ADAPSHOT_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  if (!plan_only) {
    if (pool->k == nullptr || (pool->v == nullptr && !k_only)) return ADAPSHOT_EINVAL;
    if (model->head_dim != 64 && model->head_dim != 128) return ADAPSHOT_ESHAPE;
    if (model->n_kv_heads <= 0 || model->n_q_heads % model->n_kv_heads != 0) return ADAPSHOT_ESHAPE;
    if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
    if (ctx_cap <= 0 || pool->pool_tokens <= 0) return ADAPSHOT_EINVAL;
    if (model->dtype != ADAPSHOT_F32 && model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
    if (model->k_pos_mode != 0 && model->k_pos_mode != 1) return ADAPSHOT_EUNSUPPORTED;
    if (!(model->rope_base > 1.0)) return ADAPSHOT_EINVAL;
    if (!ads_aligned16(pool->k) || (!k_only && !ads_aligned16(pool->v)) || !ads_aligned16(k_ctx) ||
        !ads_aligned16(v_ctx))
      return ADAPSHOT_EALIGN;
  }

  if (!keep_plan) {
    plan_offsets_kernel<<<B, kPlanThreads, 0, st>>>(
        sel_idx, reinterpret_cast<const long long*>(pool->shot_off), pool->n_shots, k, ctx_cap, ctx_cap > 0,
        reinterpret_cast<long long*>(ctx_off), status);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  }
  if (plan_only) return ADAPSHOT_OK;

  GatherArgs a;
  a.k_pool = pool->k; a.v_pool = pool->v; a.k_ctx = k_ctx; a.v_ctx = v_ctx;
  a.shot_off = reinterpret_cast<const long long*>(pool->shot_off);
  a.sel_idx = sel_idx;
  a.ctx_off = reinterpret_cast<const long long*>(ctx_off);
  a.pool_tokens = pool->pool_tokens; a.ctx_cap = ctx_cap;
  a.n_shots = pool->n_shots; a.B = B; a.k = k; a.n_kv_heads = model->n_kv_heads;
  a.layer_begin = layer_begin; a.n_layers_call = layer_end - layer_begin;
  a.shot_begin = shot_begin;
  a.k_pos_mode = model->k_pos_mode; a.rope_base = model->rope_base; a.status = status;
  for (int i = 0; i < model->head_dim / 2; ++i)
    a.theta[i] = pow(model->rope_base, -2.0 * (double)i / (double)model->head_dim);

  const bool f32 = model->dtype == ADAPSHOT_F32;
  if (model->head_dim == 128)
    return f32 ? launch_gather<float, 128>(a, st) : launch_gather<__nv_bfloat16, 128>(a, st);
  return f32 ? launch_gather<float, 64>(a, st) : launch_gather<__nv_bfloat16, 64>(a, st);
}
