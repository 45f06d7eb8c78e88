// Attention-based relevance ranking (paper Sec. 4.2, Eq. 5 and the ranking sentence after it): the
// query's Q at a representative layer against the cached K of every shot of the pool.  Eq. 5 as
// printed normalises over one shot's own tokens, which makes every shot's mean score 1 / T_i; the
// reading taken here is ONE softmax per query token and head over the keys of the whole pool, a
// shot's relevance being the attention mass that falls on its tokens, averaged over query tokens
// and heads (optionally divided by T_i).  Q and K enter as stored; 1/sqrt(d) scaling as in Eq. 5.
//
// Two passes over the pool's K of that layer, both on the tensor cores (tcgen05, S in TMEM, tiles
// staged by TMA), because the normaliser of a row is only known after all keys have been seen:
//   pass 1  S = Q K^T, one thread per query row (TMEM lane): running maximum and sum of exponentials
//           over the CTA's range of key tiles; a small kernel merges the ranges into log2-sum-exp;
//   pass 2  S^T = K Q^T (the same two shared-memory tiles with their roles swapped), one thread per
//           KEY: p = 2^(s c - lse(row)) summed over the query rows of the tile is the key's mass
//           from these rows; keys are folded into their shots by a segmented warp sum and one fp64
//           atomic per (warp, shot).
// The scores then go through the same top-k as the embedding selector (ties -> lower shot id).
#include <float.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace {

using namespace sm100;

constexpr int kTile = 128;            // query rows per M tile, keys per tile
constexpr int kRelThreads = 192;      // warp 0 TMA, warp 1 MMA, warps 2-5 consumers (one thread per TMEM lane)
// K tiles in flight per CTA: two CTAs share an SM (96 KB each at d = 128), so that one's consumers
// work while the other's wait for a score tile
template <int D> constexpr int kKStages = D == 128 ? 2 : 4;

// 2^x by the hardware approximation (one MUFU operation, relative error about 2^-22; 2^-inf = 0)
__device__ __forceinline__ float rel_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair of scores on the FMA pipe (for x <= 0 or thereabouts; x below -125, -inf included, gives
// about 2^-125 instead of 0, which no sum here can see):
// x = n + f with n = round(x) taken from the low mantissa bits of x + 1.5 * 2^23, 2^f by a cubic on
// [-0.5, 0.5] (relative error 7.5e-5, fitted for this build), n added to the exponent field.  The
// passes send every fourth pair here: the exponential unit (16 results per clock and SM) is what
// bounds them, the FMA pipe is nine tenths idle (measured: 4 % faster at 8 queries, 13 % at one;
// every second pair is slower again).
__device__ __forceinline__ float2 rel_ex2_poly2(float2 x) {
  const float kMagic = 12582912.f;
  x.x = fmaxf(x.x, -125.f);      // keeps the exponent field of the result positive
  x.y = fmaxf(x.y, -125.f);
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
  float2 p = __ffma2_rn(make_float2(0.0551716685f, 0.0551716685f), f, make_float2(0.2426111251f, 0.2426111251f));
  p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
  return make_float2(__uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23)),
                     __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23)));
}

struct RelParams {
  float* ml_part;               // pass 1 out: [unit][split][128][2] (max in log2 units, sum)
  const float* lse2;            // pass 2 in:  [unit][128] log2-sum-exp of every query row
  double* mass;                 // pass 2 out: [B][n_shots], zeroed before the pass
  const int* tok_shot;          // [pool_tokens] shot of every pool token
  int32_t* status;
  long long pool_tokens;
  int B, Hkv, n_mt, rows, n_shots, layer;   // rows = T_q * G query rows per (query, kv head)
  int n_tiles, splits, tiles_per_split;
  float scale_log2;
};

// q [B][Tq][Hq][D] -> q_pack [B][Hkv][n_mt * 128][D]: row m = t * G + hh of kv head g holds query
// head g * G + hh of token t; rows beyond T_q * G are zero.
template <int D>
__global__ void __launch_bounds__(256) rel_pack_q_kernel(const __nv_bfloat16* __restrict__ q,
                                                         __nv_bfloat16* __restrict__ q_pack, int B, int Tq, int Hq,
                                                         int Hkv, int rows_pad) {
  constexpr int VPR = D / 8;                         // 16-byte vectors per row
  const int G = Hq / Hkv;
  const long long n = (long long)B * Hkv * rows_pad * VPR;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int v = (int)(i % VPR);
  const long long row_g = i / VPR;
  const int m = (int)(row_g % rows_pad);
  const int g = (int)((row_g / rows_pad) % Hkv);
  const int b = (int)(row_g / ((long long)rows_pad * Hkv));
  uint4 val = make_uint4(0, 0, 0, 0);
  if (m < Tq * G) {
    const int t = m / G, hh = m % G;
    val = reinterpret_cast<const uint4*>(q)[(((long long)b * Tq + t) * Hq + g * G + hh) * VPR + v];
  }
  reinterpret_cast<uint4*>(q_pack)[i] = val;
}

// tok_shot[t] = shot that owns pool token t (one thread per token, binary search of the offsets).
__global__ void __launch_bounds__(256) rel_token_shot_kernel(const long long* __restrict__ shot_off, int n_shots,
                                                             long long pool_tokens, int* __restrict__ tok_shot) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= pool_tokens) return;
  int lo = 0, hi = n_shots;                          // shot with shot_off[lo] <= t < shot_off[lo + 1]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (shot_off[mid] <= t) lo = mid; else hi = mid;
  }
  tok_shot[t] = lo;
}

enum RelBar { kRQFull = 0, kRKFull = 1, kRKEmpty = 5, kRSFull = 9, kRSEmpty = 11, kRDrain = 13, kRNumBars = 14 };

template <int D>
struct RelSmem {
  static constexpr uint32_t kTileBytes = (D / 64) * 16384u;
  static constexpr uint32_t kOffQ = 0;
  static constexpr uint32_t kOffK = kTileBytes;
  static constexpr uint32_t kOffBar = kOffK + kKStages<D> * kTileBytes;
  static constexpr uint32_t kOffLse = kOffBar + 128;
  static constexpr uint32_t kTotal = kOffLse + 512 + 1024;      // + alignment slack
};

// grid (B * n_mt, splits, Hkv): the CTAs that differ only in (query, M tile) walk the same key tiles
// at the same time, so the pool's K layer is read from DRAM about once and from L2 otherwise.
template <int D, int PASS>
__global__ void __launch_bounds__(kRelThreads, 2)
rel_pass_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const RelParams p) {
  using SM = RelSmem<D>;
  constexpr int SUB = D / 64;
  constexpr int kStages = kKStages<D>;
  constexpr uint32_t kTileBytes = SM::kTileBytes;
  constexpr uint32_t kIdesc = idesc_bf16_f32(kTile, kTile, 0);
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - raw_addr);
  const uint32_t bar0 = base + SM::kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + SM::kOffBar + 8 * kRNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + SM::kOffBar + 8 * kRNumBars + 8);
  float* lse_s = reinterpret_cast<float*>(base_ptr + SM::kOffLse);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / p.n_mt, mt = blockIdx.x % p.n_mt;
  const int split = blockIdx.y, g = blockIdx.z;
  const int unit = (b * p.Hkv + g) * p.n_mt + mt;
  const int t0 = split * p.tiles_per_split;
  const int t1 = min(p.n_tiles, t0 + p.tiles_per_split);
  const int n_it = max(0, t1 - t0);

  if (threadIdx.x == 32) {
    mbar_init(bar(kRQFull), 1);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar(kRKFull + i), 1);
      mbar_init(bar(kRKEmpty + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kRSFull + i), 1);
      mbar_init(bar(kRSEmpty + i), 128);
    }
    mbar_init(bar(kRDrain), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 256);
    tmem_relinquish();
  }
  if (PASS == 2 && threadIdx.x >= 64) {
    // -lse per query row; rows of the M tile that do not exist get -inf: their 2^(s c - lse) is exactly zero
    const int c = threadIdx.x - 64;
    lse_s[c] = c < min(kTile, p.rows - mt * kTile) ? -p.lse2[(long long)unit * kTile + c] : -INFINITY;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && n_it > 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k);
      mbar_arrive_expect_tx(bar(kRQFull), kTileBytes);
#pragma unroll
      for (int s = 0; s < SUB; ++s)
        tma_load_3d(base + SM::kOffQ + s * 16384u, &tm_q, bar(kRQFull), s * 64, mt * kTile, b * p.Hkv + g);
      bool ok = true;
      int i = 0;
      for (; i < n_it && ok; ++i) {
        const int st = i % kStages;
        ok = mbar_wait(bar(kRKEmpty + st), ((i / kStages) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar(kRKFull + st), kTileBytes);
#pragma unroll
        for (int s = 0; s < SUB; ++s)
          tma_load_4d(base + SM::kOffK + st * kTileBytes + s * 16384u, &tm_k, bar(kRKFull + st), s * 64, g,
                      (t0 + i) * kTile, p.layer);
      }
      if (!ok) {      // gave up: let the copies in flight land before the CTA retires
        mbar_wait(bar(kRQFull), 0, abort_flag + 1);
        for (int t = max(0, i - kStages); t < i; ++t)
          mbar_wait(bar(kRKFull + t % kStages), (t / kStages) & 1, abort_flag + 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0 && n_it > 0) {
      constexpr uint32_t kHi = smem_desc_hi_sw128(1024);
      const uint32_t q_lo = smem_desc_lo(base + SM::kOffQ, 16);
      bool ok = mbar_wait(bar(kRQFull), 0, abort_flag);
      for (int i = 0; i < n_it && ok; ++i) {
        const int st = i % kStages, sb = i & 1;
        ok = mbar_wait(bar(kRKFull + st), (i / kStages) & 1, abort_flag) &&
             mbar_wait(bar(kRSEmpty + sb), ((i >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t k_lo = smem_desc_lo(base + SM::kOffK + st * kTileBytes, 16);
        const uint32_t d = tmem_base + sb * kTile;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t o = ((ks / 4) * 16384u + (ks % 4) * 32u) >> 4;
          if (PASS == 1) umma_ss_lohi(d, q_lo + o, kHi, k_lo + o, kHi, kIdesc, ks > 0 ? 1u : 0u);   // rows = queries
          else umma_ss_lohi(d, k_lo + o, kHi, q_lo + o, kHi, kIdesc, ks > 0 ? 1u : 0u);             // rows = keys
        }
        umma_commit(bar(kRSFull + sb));
        umma_commit(bar(kRKEmpty + st));
      }
      if (!ok) {      // gave up: the UMMAs already issued must be done before the tensor memory is freed
        umma_commit(bar(kRDrain));
        mbar_wait(bar(kRDrain), 0, abort_flag + 1);
      }
    }
    __syncwarp();
  } else {
    // --------------------------------------------------------------- consumers
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;                      // TMEM lane: query row (pass 1) or key of the tile (pass 2)
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    float m_run = -1.0e30f, l_run = 0.f;
    bool ok = true;
    for (int i = 0; i < n_it; ++i) {
      const int sb = i & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kRSFull + sb), (i >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      float s[kTile];
      tmem_ld128(tmem_base + lane_addr + sb * kTile, reinterpret_cast<uint32_t*>(s));
      tc_fence_before();
      mbar_arrive(bar(kRSEmpty + sb));                      // the scores are in registers: the buffer is free
      const long long key0 = (long long)(t0 + i) * kTile;
      if (PASS == 1) {
        const int limit = (int)min((long long)kTile, p.pool_tokens - key0);   // keys of this tile that exist
        if (limit < kTile) {                       // only the pool's last tile: keys beyond it count as -inf
#pragma unroll
          for (int c = 0; c < kTile; ++c) s[c] = c < limit ? s[c] : -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < kTile; c += 8) {
#pragma unroll
          for (int u = 0; u < 4; ++u) mx4[u] = fmax3(mx4[u], s[c + 2 * u], s[c + 2 * u + 1]);
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
        if (mx > m_run) {
          l_run *= rel_ex2(m_run - mx);
          m_run = mx;
        }
        // two scores per FMA / add instruction; the exponentials themselves are one MUFU operation each
        const float2 scale2 = make_float2(p.scale_log2, p.scale_log2), neg_m2 = make_float2(-m_run, -m_run);
        float2 part[2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int c = 0; c < kTile; c += 2) {
          const float2 a = __ffma2_rn(make_float2(s[c], s[c + 1]), scale2, neg_m2);
          const float2 e = ((c >> 1) & 3) == 3 ? rel_ex2_poly2(a) : make_float2(rel_ex2(a.x), rel_ex2(a.y));
          part[(c >> 1) & 1] = __fadd2_rn(part[(c >> 1) & 1], e);
        }
        l_run += (part[0].x + part[0].y) + (part[1].x + part[1].y);
      } else {
        const long long key = key0 + r;
        const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);
        float2 part[2] = {{0.f, 0.f}, {0.f, 0.f}};
        const float4* lse4 = reinterpret_cast<const float4*>(lse_s);
#pragma unroll
        for (int c4 = 0; c4 < kTile / 4; ++c4) {
          const float4 l4 = lse4[c4];                     // the same address for every lane: a broadcast
          const float2 a0 = __ffma2_rn(make_float2(s[4 * c4], s[4 * c4 + 1]), scale2, make_float2(l4.x, l4.y));
          const float2 a1 = __ffma2_rn(make_float2(s[4 * c4 + 2], s[4 * c4 + 3]), scale2, make_float2(l4.z, l4.w));
          part[0] = __fadd2_rn(part[0], make_float2(rel_ex2(a0.x), rel_ex2(a0.y)));
          part[1] = __fadd2_rn(part[1], (c4 & 1) ? rel_ex2_poly2(a1) : make_float2(rel_ex2(a1.x), rel_ex2(a1.y)));
        }
        float v = (part[0].x + part[0].y) + (part[1].x + part[1].y);
        int id = -1;
        if (key < p.pool_tokens) id = p.tok_shot[key]; else v = 0.f;
        // shots are runs of consecutive keys: segmented inclusive sum along the lanes, the last
        // lane of every run adds the run's mass to its shot
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float u = __shfl_up_sync(0xffffffffu, v, o);
          const int iu = __shfl_up_sync(0xffffffffu, id, o);
          if (lane >= o && iu == id) v += u;
        }
        const int idn = __shfl_down_sync(0xffffffffu, id, 1);
        if (id >= 0 && (lane == 31 || idn != id)) atomicAdd(p.mass + (long long)b * p.n_shots + id, (double)v);
      }
    }
    if (PASS == 1 && ok) {
      float* out = p.ml_part + (((long long)unit * p.splits + split) * kTile + r) * 2;
      out[0] = m_run;
      out[1] = l_run;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) ads_set_status(p.status, ADAPSHOT_ETIMEOUT);
}

// lse2[unit][row] = log2 sum_keys 2^(s c) from the per-range (max, sum) pairs; one thread per row.
__global__ void __launch_bounds__(128) rel_merge_kernel(const float* __restrict__ ml_part, int splits,
                                                        float* __restrict__ lse2) {
  const long long unit = blockIdx.x;
  const int r = threadIdx.x;
  float M = -1.0e30f;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, ml_part[((unit * splits + s) * kTile + r) * 2]);
  float l = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float* ml = ml_part + ((unit * splits + s) * kTile + r) * 2;
    l += ml[1] * exp2f(ml[0] - M);
  }
  lse2[unit * kTile + r] = l > 0.f ? M + log2f(l) : 0.f;
}

// score[b][i] = mass[b][i] / (T_q * Hq) (and / T_i with per_token); writes the sort keys and the ids.
__global__ void __launch_bounds__(256) rel_scores_kernel(const double* __restrict__ mass,
                                                         const long long* __restrict__ shot_off, int B, int n_shots,
                                                         double inv_rows, int per_token,
                                                         unsigned long long* __restrict__ keys, int* __restrict__ ids) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * n_shots) return;
  const int shot = (int)(i % n_shots);
  double s = mass[i] * inv_rows;
  if (per_token) s /= (double)(shot_off[shot + 1] - shot_off[shot]);
  keys[i] = ads_desc_key(s);
  ids[i] = shot;
}

struct RelPlan {
  int G, n_mt, rows, rows_pad, n_tiles, splits, tiles_per_split;
  size_t off_qpack, off_ml, off_lse, off_tokshot, off_mass, off_keys, off_ids, off_cand, total;
};

RelPlan rel_plan(const adapshot_model_t* model, const adapshot_pool_t* pool, int B, int Tq, int k) {
  RelPlan pl;
  const int D = model->head_dim, Hkv = model->n_kv_heads;
  pl.G = model->n_q_heads / Hkv;
  pl.rows = Tq * pl.G;
  pl.n_mt = (pl.rows + kTile - 1) / kTile;
  pl.rows_pad = pl.n_mt * kTile;
  pl.n_tiles = (int)((pool->pool_tokens + kTile - 1) / kTile);
  // Key ranges per unit: units * splits CTAs run in waves of 296 (two per SM on 148 SMs; a fixed
  // figure, so that the workspace size does not depend on the device), each CTA costs its tiles plus
  // about four tiles' time of start-up; the split with the cheapest waves * (tiles + 4) is taken,
  // every range at least eight key tiles.
  const long long units = (long long)B * pl.n_mt * Hkv;
  const int most = (pl.n_tiles + 7) / 8 < 256 ? (pl.n_tiles + 7) / 8 : 256;
  int best_s = 1;
  long long best_cost = 0;
  for (int sp = 1; sp <= most; ++sp) {
    const long long tiles = (pl.n_tiles + sp - 1) / sp;
    const long long waves = (units * sp + 295) / 296;
    const long long cost = waves * (tiles + 4);
    if (sp == 1 || cost < best_cost) {
      best_s = sp;
      best_cost = cost;
    }
  }
  pl.tiles_per_split = (pl.n_tiles + best_s - 1) / best_s;
  pl.splits = (pl.n_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
  size_t off = 0;
  pl.off_qpack = off;   off += ads_round_up((size_t)B * Hkv * pl.rows_pad * D * 2, 256);
  pl.off_ml = off;      off += ads_round_up((size_t)units * pl.splits * kTile * 2 * 4, 256);
  pl.off_lse = off;     off += ads_round_up((size_t)units * kTile * 4, 256);
  pl.off_tokshot = off; off += ads_round_up((size_t)pool->pool_tokens * 4, 256);
  pl.off_mass = off;    off += ads_round_up((size_t)B * pool->n_shots * 8, 256);
  pl.off_keys = off;    off += ads_round_up((size_t)B * pool->n_shots * 8, 256);
  pl.off_ids = off;     off += ads_round_up((size_t)B * pool->n_shots * 4, 256);
  pl.off_cand = off;    off += ads_topk_scratch_bytes(pool->n_shots, B, k);
  pl.total = off;
  return pl;
}

bool rel_shape_ok(const adapshot_model_t* m) {
  return (m->head_dim == 64 || m->head_dim == 128) && m->n_kv_heads > 0 && m->n_q_heads > 0 &&
         m->n_q_heads % m->n_kv_heads == 0;
}

template <int D>
int rel_launch(const adapshot_model_t* model, const adapshot_pool_t* pool, int layer, const void* q, int B, int Tq,
               int k, uint32_t flags, int32_t* sel_idx, float* sel_score, const RelPlan& pl, void* ws,
               int32_t* status, cudaStream_t st) {
  const int Hq = model->n_q_heads, Hkv = model->n_kv_heads;
  unsigned char* wsb = static_cast<unsigned char*>(ws);
  __nv_bfloat16* q_pack = reinterpret_cast<__nv_bfloat16*>(wsb + pl.off_qpack);
  float* ml_part = reinterpret_cast<float*>(wsb + pl.off_ml);
  float* lse2 = reinterpret_cast<float*>(wsb + pl.off_lse);
  int* tok_shot = reinterpret_cast<int*>(wsb + pl.off_tokshot);
  double* mass = reinterpret_cast<double*>(wsb + pl.off_mass);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(wsb + pl.off_keys);
  int* ids = reinterpret_cast<int*>(wsb + pl.off_ids);
  const long long units = (long long)B * pl.n_mt * Hkv;

  CUtensorMap tm_q, tm_k;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)pl.rows_pad, (uint64_t)B * Hkv};
    const uint64_t str[2] = {(uint64_t)D * 2, (uint64_t)pl.rows_pad * D * 2};
    const uint32_t box[3] = {64, (uint32_t)kTile, 1};
    if (!ads_make_bf16_map(&tm_q, q_pack, 3, dims, str, box)) return ADAPSHOT_ECUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)Hkv, (uint64_t)pool->pool_tokens, (uint64_t)model->n_layers};
    const uint64_t str[3] = {(uint64_t)D * 2, (uint64_t)Hkv * D * 2, (uint64_t)pool->pool_tokens * Hkv * D * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)kTile, 1};
    if (!ads_make_bf16_map(&tm_k, pool->k, 4, dims, str, box)) return ADAPSHOT_ECUDA;
  }

  const long long n_vec = (long long)B * Hkv * pl.rows_pad * (D / 8);
  rel_pack_q_kernel<D><<<(unsigned)((n_vec + 255) / 256), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(q), q_pack, B,
                                                                       Tq, Hq, Hkv, pl.rows_pad);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  rel_token_shot_kernel<<<(unsigned)((pool->pool_tokens + 255) / 256), 256, 0, st>>>(
      reinterpret_cast<const long long*>(pool->shot_off), pool->n_shots, pool->pool_tokens, tok_shot);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  ADS_CHECK_CUDA(cudaMemsetAsync(mass, 0, (size_t)B * pool->n_shots * 8, st));

  RelParams rp;
  rp.ml_part = ml_part; rp.lse2 = lse2; rp.mass = mass; rp.tok_shot = tok_shot; rp.status = status;
  rp.pool_tokens = pool->pool_tokens;
  rp.B = B; rp.Hkv = Hkv; rp.n_mt = pl.n_mt; rp.rows = pl.rows; rp.n_shots = pool->n_shots; rp.layer = layer;
  rp.n_tiles = pl.n_tiles; rp.splits = pl.splits; rp.tiles_per_split = pl.tiles_per_split;
  const float scale = model->softmax_scale > 0.f ? model->softmax_scale : 1.0f / sqrtf((float)D);
  rp.scale_log2 = scale * 1.4426950408889634f;

  const int smem = (int)RelSmem<D>::kTotal;
  static bool attr_done[2][kAdsMaxDevices] = {{false}, {false}};
  if (ads_set_max_smem(rel_pass_kernel<D, 1>, smem, attr_done[0]) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  if (ads_set_max_smem(rel_pass_kernel<D, 2>, smem, attr_done[1]) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  const dim3 grid((unsigned)(B * pl.n_mt), (unsigned)pl.splits, (unsigned)Hkv);
  rel_pass_kernel<D, 1><<<grid, kRelThreads, smem, st>>>(tm_q, tm_k, rp);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  rel_merge_kernel<<<(unsigned)units, 128, 0, st>>>(ml_part, pl.splits, lse2);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  rel_pass_kernel<D, 2><<<grid, kRelThreads, smem, st>>>(tm_q, tm_k, rp);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  const long long n_sc = (long long)B * pool->n_shots;
  rel_scores_kernel<<<(unsigned)((n_sc + 255) / 256), 256, 0, st>>>(
      mass, reinterpret_cast<const long long*>(pool->shot_off), B, pool->n_shots, 1.0 / ((double)Tq * Hq),
      (flags & ADAPSHOT_RELEVANCE_PER_TOKEN) ? 1 : 0, keys, ids);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  return ads_topk_from_keys(keys, ids, pool->n_shots, B, k, wsb + pl.off_cand, sel_idx, sel_score, st);
}

}  // namespace

extern "C" size_t adapshot_select_attn_workspace_bytes(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                                       int32_t B, int32_t Tq, int32_t k) {
  if (model == nullptr || pool == nullptr || !rel_shape_ok(model) || B <= 0 || Tq <= 0 || k <= 0 ||
      pool->n_shots <= 0 || pool->pool_tokens <= 0)
    return 0;
  return rel_plan(model, pool, B, Tq, k).total;
}

extern "C" int adapshot_select_attn(const adapshot_model_t* model, const adapshot_pool_t* pool, int32_t layer,
                                    const void* q, int32_t B, int32_t Tq, int32_t k, uint32_t flags,
                                    int32_t* sel_idx, float* sel_score, void* ws, size_t ws_bytes,
                                    int32_t* status, void* stream) {
  if (model == nullptr || pool == nullptr || q == nullptr || sel_idx == nullptr || ws == nullptr)
    return ADAPSHOT_EINVAL;
  if (pool->k == nullptr || pool->shot_off == nullptr || pool->n_shots <= 0 || pool->pool_tokens <= 0 || B <= 0 ||
      Tq <= 0 || (flags & ~ADAPSHOT_RELEVANCE_PER_TOKEN) != 0)
    return ADAPSHOT_EINVAL;
  if (model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (!rel_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (layer < 0 || layer >= model->n_layers) return ADAPSHOT_ESHAPE;
  if (k < 1 || k > pool->n_shots) return ADAPSHOT_ESHAPE;
  if (pool->n_shots > 8192 && k > 4096) return ADAPSHOT_EUNSUPPORTED;
  if (pool->pool_tokens > (1ll << 31) - 256) return ADAPSHOT_ESHAPE;
  if (!ads_aligned16(pool->k) || !ads_aligned16(q) || ((uintptr_t)ws & 255u) || ((uintptr_t)pool->shot_off & 7u))
    return ADAPSHOT_EALIGN;
  const RelPlan pl = rel_plan(model, pool, B, Tq, k);
  if ((long long)B * pl.n_mt > 0x7fffffffll || pl.splits > 65535 || model->n_kv_heads > 65535) return ADAPSHOT_ESHAPE;
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (model->head_dim == 128)
    return rel_launch<128>(model, pool, layer, q, B, Tq, k, flags, sel_idx, sel_score, pl, ws, status, st);
  return rel_launch<64>(model, pool, layer, q, B, Tq, k, flags, sel_idx, sel_score, pl, ws, status, st);
}
