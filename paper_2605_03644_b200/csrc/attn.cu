// Probe attention over the reused cache (paper Eq. 1 with the tree mask of Sec. 4.1:
// probe j sees the first n_j shots of the assembled context and, causally, its own
// tokens; scores scaled by 1/sqrt(d) as in Eq. 5; rotary positions of Eq. 6).
//
// Three kernels:
//   attn_prep     rotates Q and the probe's own K to their positions L_j + t and
//                 packs Q rows of one KV head (GQA) into an M-major tile layout;
//   attn_main     one CTA per (query, layer, probe, kv head, 128-row M tile, context
//                 chunk): TMA stages K/V tiles, tcgen05 UMMA computes S = Q K^T and
//                 O += P V with accumulators in TMEM, four warps run the online
//                 softmax (one thread per row); un-normalised partial results go to
//                 the workspace;
//   attn_combine  log-sum-exp merge of the chunk partials, normalise, store bf16.
#include <cuda.h>
#include <float.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kMaxProbes = 16;
constexpr int kTileM = 128;          // query rows per CTA (TMEM lanes)
constexpr int kTileN = 128;          // keys per tile
constexpr int kAttnThreads = 192;    // warp 0 TMA, warp 1 MMA, warps 2-5 softmax
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;   // log2 units: rescale O only when the max grows by 2^8
constexpr float kNegSentinel = -1.0e30f;

struct AttnParams {
  const long long* ctx_off;   // [B][k+1]
  float* o_part;              // [items][128][D] fp32, un-normalised
  float* ml_part;             // [items][128][2]  (running max in log2 units, row sum)
  int32_t* status;
  long long ctx_cap;
  int B, k, P, Tq, Hq, Hkv, G, nl;
  int n_mt, n_chunks, tiles_per_chunk;
  float scale_log2;           // softmax_scale * log2(e)
  int nshots[kMaxProbes];
};

struct PrepParams {
  const __nv_bfloat16* q;     // [B][nl][P][Tq][Hq][D]
  const __nv_bfloat16* kq;    // [B][nl][P][Tq][Hkv][D]
  __nv_bfloat16* q_rot;       // [B*nl*P*Hkv][Tq*G][D]
  __nv_bfloat16* kq_rot;      // layout of kq
  const long long* ctx_off;
  int B, k, P, Tq, Hq, Hkv, nl;
  double rope_base;
  int nshots[kMaxProbes];
};

__device__ __forceinline__ void bf16x8_unpack(const uint4& r, float* x) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    x[2 * j] = __uint_as_float(w[j] << 16);
    x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint4 bf16x8_pack(const float* x) {
  return make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]), pack_bf16x2(x[4], x[5]),
                    pack_bf16x2(x[6], x[7]));
}

// One warp per probe token (b, l, j, t): all Hq query heads and Hkv key heads of the
// token rotate by the same angles (L_j + t) * theta_i.
template <int D>
__global__ void __launch_bounds__(256) attn_prep_kernel(const PrepParams p) {
  constexpr int VPH = D / 8, HALF_V = VPH / 2;
  const int lane = threadIdx.x & 31;
  __shared__ double theta_sh[D / 2];   // theta_i once per CTA: fp64 pow is slow
  if (threadIdx.x < D / 2) theta_sh[threadIdx.x] = pow(p.rope_base, -2.0 * (double)threadIdx.x / (double)D);
  __syncthreads();
  const long long tok = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_tok = (long long)p.B * p.nl * p.P * p.Tq;
  if (tok >= n_tok) return;
  const int t = (int)(tok % p.Tq);
  const long long bpj = tok / p.Tq;                 // (b*nl + l)*P + j
  const int j = (int)(bpj % p.P);
  const int b = (int)(bpj / ((long long)p.P * p.nl));
  const long long Lj = p.ctx_off[(long long)b * (p.k + 1) + p.nshots[j]];
  const double pos = (double)(Lj + t);
  const int G = p.Hq / p.Hkv;

  const int jcol = lane % HALF_V;
  float sn[8], cs[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    rope_sincos(pos, theta_sh[jcol * 8 + e], &sn[e], &cs[e]);
  }
  const uint4* qsrc = reinterpret_cast<const uint4*>(p.q) + tok * p.Hq * VPH;
  const uint4* ksrc = reinterpret_cast<const uint4*>(p.kq) + tok * p.Hkv * VPH;
  uint4* kdst = reinterpret_cast<uint4*>(p.kq_rot) + tok * p.Hkv * VPH;
  uint4* qdst_base = reinterpret_cast<uint4*>(p.q_rot);
  const int units = (p.Hq + p.Hkv) * HALF_V;
  for (int u = lane; u < units; u += 32) {
    const int head = u / HALF_V;                    // column == jcol since 32 % HALF_V == 0
    const bool is_q = head < p.Hq;
    const uint4* src = is_q ? qsrc + head * VPH + jcol : ksrc + (head - p.Hq) * VPH + jcol;
    float x[8], y[8], xr[8], yr[8];
    bf16x8_unpack(src[0], x);
    bf16x8_unpack(src[HALF_V], y);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      xr[e] = x[e] * cs[e] - y[e] * sn[e];
      yr[e] = y[e] * cs[e] + x[e] * sn[e];
    }
    uint4* dst;
    if (is_q) {
      const int g = head / G, hh = head % G;
      const long long row = ((bpj * p.Hkv + g) * ((long long)p.Tq * G)) + (long long)t * G + hh;
      dst = qdst_base + row * VPH + jcol;
    } else {
      dst = kdst + (head - p.Hq) * VPH + jcol;
    }
    dst[0] = bf16x8_pack(xr);
    dst[HALF_V] = bf16x8_pack(yr);
  }
}

constexpr int kMaxPairs = 256;       // (probe, query) pairs one call may hold: B * P <= 256

// Shared-memory plan.  Every operand tile is made of [128 rows][128 bytes] sub-tiles
// written by TMA with the 128-byte swizzle; D = 128 needs two of them per tile.
template <int D>
struct AttnSmem {
  static constexpr int kKStages = D == 128 ? 2 : 3;
  static constexpr int kVStages = 3;
  static constexpr uint32_t kTileBytes = (D / 64) * 16384u;
  static constexpr uint32_t kOffQ = 0;                                    // 2 buffers
  static constexpr uint32_t kOffK = kOffQ + 2 * kTileBytes;
  static constexpr uint32_t kOffV = kOffK + kKStages * kTileBytes;
  static constexpr uint32_t kOffBar = kOffV + kVStages * kTileBytes;
  static constexpr uint32_t kOffPairs = kOffBar + 256;
  static constexpr uint32_t kTotal = kOffPairs + (kMaxPairs + 1) * 4 + 1024;   // + alignment slack
};

// mbarrier slots (8 bytes each)
enum Bar {
  kBarQFull = 0, kBarQEmpty = 2, kBarKFull = 4, kBarKEmpty = 7, kBarVFull = 10, kBarVEmpty = 13,
  kBarSFull = 16, kBarPFull = 18, kBarPVDone = 20, kBarOFull = 21, kBarOEmpty = 23, kBarDrain = 25,
  kNumBars = 26
};

struct WorkItem {
  int b, l, j, g, mt, c;
  long long Lj;
  int t_begin, n_ctx, n_own, n_tiles;
  int outer_ctx, outer_own, outer_q;
  long long item_out;
};

// idx-th non-empty piece of work.  prefix[pi] = first index of pair pi = jj * B + b,
// jj = P-1-j (longest probes first); inside a pair: chunk, layer, kv head, M tile
// (M tile fastest, so CTAs that share a K/V chunk run at the same time).
__device__ __forceinline__ void decode_item(const AttnParams& p, const int* prefix, int n_pairs, int idx,
                                            WorkItem& w) {
  int lo = 0, hi = n_pairs;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= idx) lo = mid; else hi = mid;
  }
  int local = idx - prefix[lo];
  w.j = p.P - 1 - lo / p.B;
  w.b = lo % p.B;
  w.mt = local % p.n_mt; local /= p.n_mt;
  w.g = local % p.Hkv; local /= p.Hkv;
  w.l = local % p.nl;
  w.c = local / p.nl;
  long long Lj = p.ctx_off[(long long)w.b * (p.k + 1) + p.nshots[w.j]];
  Lj = Lj > p.ctx_cap ? p.ctx_cap : (Lj < 0 ? 0 : Lj);
  w.Lj = Lj;
  const int n_tiles_ctx = (int)((Lj + kTileN - 1) / kTileN);
  const int c_last = n_tiles_ctx > 0 ? (n_tiles_ctx - 1) / p.tiles_per_chunk : 0;
  w.t_begin = w.c * p.tiles_per_chunk;
  w.n_ctx = max(0, min(n_tiles_ctx, w.t_begin + p.tiles_per_chunk) - w.t_begin);
  w.n_own = 0;
  if (w.c == c_last) {   // the last chunk also takes the probe's own tokens (causal part)
    const int row_hi = min(p.Tq * p.G - 1, w.mt * kTileM + kTileM - 1);
    w.n_own = (row_hi / p.G) / kTileN + 1;
  }
  w.n_tiles = w.n_ctx + w.n_own;
  w.outer_ctx = w.b * p.nl + w.l;
  w.outer_own = w.outer_ctx * p.P + w.j;
  w.outer_q = w.outer_own * p.Hkv + w.g;
  w.item_out = (((long long)w.outer_own * p.Hkv + w.g) * p.n_mt + w.mt) * p.n_chunks + w.c;
}

// Persistent kernel: one CTA per SM walks over the non-empty work items round-robin.
// TMEM: S/P buffers at columns 0 and 128 (P, as packed bf16, overwrites the S tile it
// was computed from), O accumulators at 256 and 384 (alternating per item so that the
// read-out of one item overlaps the MMAs of the next).
template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_main_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kctx,
                 const __grid_constant__ CUtensorMap tm_vctx, const __grid_constant__ CUtensorMap tm_kown,
                 const __grid_constant__ CUtensorMap tm_vown, const AttnParams p) {
  using SM = AttnSmem<D>;
  constexpr int SUB = D / 64;
  constexpr int KS = SM::kKStages, VS = SM::kVStages;
  constexpr uint32_t kTileBytes = SM::kTileBytes;
  constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kTileN, 0);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, 1);
  constexpr uint32_t kTmemS = 0, kTmemO = 256;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - raw_addr);
  const uint32_t bar0 = base + SM::kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + SM::kOffBar + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + SM::kOffBar + 8 * kNumBars + 8);
  int* prefix = reinterpret_cast<int*>(base_ptr + SM::kOffPairs);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pairs = p.P * p.B;

  // ---- how many non-empty items every (probe, query) pair has
  const int per_chunk = p.nl * p.Hkv * p.n_mt;
  for (int pi = threadIdx.x; pi < n_pairs; pi += kAttnThreads) {
    const int j = p.P - 1 - pi / p.B, b = pi % p.B;
    long long Lj = p.ctx_off[(long long)b * (p.k + 1) + p.nshots[j]];
    Lj = Lj > p.ctx_cap ? p.ctx_cap : (Lj < 0 ? 0 : Lj);
    const int n_tiles_ctx = (int)((Lj + kTileN - 1) / kTileN);
    const int n_valid = n_tiles_ctx > 0 ? (n_tiles_ctx - 1) / p.tiles_per_chunk + 1 : 1;
    prefix[pi + 1] = n_valid * per_chunk;
  }
  if (threadIdx.x == 32) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kBarQFull + i), 1);
      mbar_init(bar(kBarQEmpty + i), 1);
      mbar_init(bar(kBarSFull + i), 1);
      mbar_init(bar(kBarPFull + i), 128);
      mbar_init(bar(kBarOFull + i), 1);
      mbar_init(bar(kBarOEmpty + i), 128);
    }
    for (int i = 0; i < 3; ++i) {
      mbar_init(bar(kBarKFull + i), 1);
      mbar_init(bar(kBarKEmpty + i), 1);
      mbar_init(bar(kBarVFull + i), 1);
      mbar_init(bar(kBarVEmpty + i), 1);
    }
    mbar_init(bar(kBarPVDone), 1);
    mbar_init(bar(kBarDrain), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    prefix[0] = 0;
    for (int pi = 0; pi < n_pairs; ++pi) prefix[pi + 1] += prefix[pi];
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = prefix[n_pairs];

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kctx); tma_prefetch_desc(&tm_vctx);
      uint32_t tk = 0, tv = 0;
      int n = 0;
      bool ok = true;
      for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++n) {
        WorkItem w;
        decode_item(p, prefix, n_pairs, idx, w);
        const int qb = n & 1;
        ok = mbar_wait(bar(kBarQEmpty + qb), ((n >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar(kBarQFull + qb), kTileBytes);
#pragma unroll
        for (int s = 0; s < SUB; ++s)
          tma_load_3d(base + SM::kOffQ + qb * kTileBytes + s * 16384u, &tm_q, bar(kBarQFull + qb), s * 64,
                      w.mt * kTileM, w.outer_q);
        for (int i = 0; i < w.n_tiles; ++i) {
          const bool own = i >= w.n_ctx;
          const CUtensorMap* mk = own ? &tm_kown : &tm_kctx;
          const CUtensorMap* mv = own ? &tm_vown : &tm_vctx;
          const int row = own ? (i - w.n_ctx) * kTileN : (w.t_begin + i) * kTileN;
          const int outer = own ? w.outer_own : w.outer_ctx;
          const int sk = tk % KS;
          ok = mbar_wait(bar(kBarKEmpty + sk), ((tk / KS) & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(bar(kBarKFull + sk), kTileBytes);
#pragma unroll
          for (int s = 0; s < SUB; ++s)
            tma_load_4d(base + SM::kOffK + sk * kTileBytes + s * 16384u, mk, bar(kBarKFull + sk), s * 64, w.g, row,
                        outer);
          ++tk;
          const int sv = tv % VS;
          ok = mbar_wait(bar(kBarVEmpty + sv), ((tv / VS) & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(bar(kBarVFull + sv), kTileBytes);
#pragma unroll
          for (int s = 0; s < SUB; ++s)
            tma_load_4d(base + SM::kOffV + sv * kTileBytes + s * 16384u, mv, bar(kBarVFull + sv), s * 64, w.g, row,
                        outer);
          ++tv;
        }
      }
      if (!ok) {
        // gave up: let the copies already in flight land before the CTA retires
        for (uint32_t t = tk > (uint32_t)KS ? tk - KS : 0; t < tk; ++t)
          mbar_wait(bar(kBarKFull + t % KS), (t / KS) & 1, abort_flag + 1);
        for (uint32_t t = tv > (uint32_t)VS ? tv - VS : 0; t < tv; ++t)
          mbar_wait(bar(kBarVFull + t % VS), (t / VS) & 1, abort_flag + 1);
        for (int t = max(0, n - 1); t <= n; ++t)
          mbar_wait(bar(kBarQFull + (t & 1)), (t >> 1) & 1, abort_flag + 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      struct Pending { int sb, sv, vphase, pphase, ob, ophase, first, last; };
      Pending prev{};
      bool have_prev = false, ok = true;
      auto issue_pv = [&](const Pending& t) -> bool {
        if (t.first && !mbar_wait(bar(kBarOEmpty + t.ob), t.ophase ^ 1, abort_flag)) return false;
        if (!mbar_wait(bar(kBarPFull + t.sb), t.pphase, abort_flag)) return false;
        if (!mbar_wait(bar(kBarVFull + t.sv), t.vphase, abort_flag)) return false;
        tc_fence_after();
        const uint32_t v_base = base + SM::kOffV + t.sv * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kTileN / 16; ++ks) {
          // A = P from TMEM: 16 bf16 keys of one k-step occupy 8 packed columns
          umma_ts(tmem_base + kTmemO + t.ob * 128, tmem_base + kTmemS + t.sb * kTileN + ks * 8,
                  smem_desc_sw128(v_base + ks * 2048u, 16384, 1024), kIdescPV, (!t.first || ks > 0) ? 1u : 0u);
        }
        umma_commit(bar(kBarVEmpty + t.sv));
        umma_commit(bar(kBarPVDone));
        if (t.last) umma_commit(bar(kBarOFull + t.ob));
        return true;
      };
      uint32_t tk = 0, tv = 0, gt = 0;
      int n = 0;
      for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++n) {
        WorkItem w;
        decode_item(p, prefix, n_pairs, idx, w);
        const int qb = n & 1;
        ok = mbar_wait(bar(kBarQFull + qb), (n >> 1) & 1, abort_flag);
        const uint32_t q_base = base + SM::kOffQ + qb * kTileBytes;
        for (int i = 0; i < w.n_tiles && ok; ++i) {
          const int sk = tk % KS, sb = gt & 1;
          ok = mbar_wait(bar(kBarKFull + sk), (tk / KS) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k_base = base + SM::kOffK + sk * kTileBytes;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t o = (ks / 4) * 16384u + (ks % 4) * 32u;
            umma_ss(tmem_base + kTmemS + sb * kTileN, smem_desc_sw128(q_base + o, 16, 1024),
                    smem_desc_sw128(k_base + o, 16, 1024), kIdescQK, ks > 0 ? 1u : 0u);
          }
          umma_commit(bar(kBarSFull + sb));
          umma_commit(bar(kBarKEmpty + sk));
          if (i == w.n_tiles - 1) umma_commit(bar(kBarQEmpty + qb));
          ++tk;
          if (have_prev) ok = issue_pv(prev);
          prev.sb = sb; prev.sv = tv % VS; prev.vphase = (tv / VS) & 1; prev.pphase = (gt >> 1) & 1;
          prev.ob = n & 1; prev.ophase = (n >> 1) & 1; prev.first = i == 0; prev.last = i == w.n_tiles - 1;
          have_prev = true;
          ++tv; ++gt;
        }
      }
      if (ok && have_prev) ok = issue_pv(prev);
      if (!ok) {
        umma_commit(bar(kBarDrain));
        mbar_wait(bar(kBarDrain), 0, abort_flag + 1);
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------- softmax + correction
    const int quarter = warp & 3;                  // TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;             // row of the M tile
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    uint32_t gt = 0;
    int n = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++n) {
      WorkItem w;
      decode_item(p, prefix, n_pairs, idx, w);
      const int ob = n & 1;
      const int t_row = (w.mt * kTileM + r) / p.G;   // probe token of this row
      float m_used = kNegSentinel, l_sum = 0.f;
      for (int i = 0; i < w.n_tiles; ++i, ++gt) {
        const int sb = gt & 1;
        const uint32_t s_addr = tmem_base + lane_addr + kTmemS + sb * kTileN;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull + sb), (gt >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        float s[kTileN];
        tmem_ld128(s_addr, reinterpret_cast<uint32_t*>(s));

        // mask: context keys at or beyond L_j; own keys after the row's token (causal).
        // Only the last context tile and the own-token tiles can hide anything.
        int limit = kTileN;                          // columns < limit are visible
        if (i < w.n_ctx) {
          const long long first = (long long)(w.t_begin + i) * kTileN;
          if (first + kTileN > w.Lj) limit = (int)(w.Lj - first);
        } else {
          limit = min(t_row, p.Tq - 1) - (i - w.n_ctx) * kTileN + 1;   // <= 0: the whole tile is hidden
        }
        if (__any_sync(0xffffffffu, limit < kTileN)) {
#pragma unroll
          for (int cidx = 0; cidx < kTileN; ++cidx) s[cidx] = cidx < limit ? s[cidx] : -INFINITY;
        }
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int cidx = 0; cidx < kTileN; cidx += 8) {
#pragma unroll
          for (int u = 0; u < 4; ++u) mx[u] = fmax3(mx[u], s[cidx + 2 * u], s[cidx + 2 * u + 1]);
        }
        const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale_log2;
        float alpha = 1.f;
        const bool need = tile_max > m_used + kRescaleThreshold;
        if (need) {
          alpha = exp2f(m_used - tile_max);
          m_used = tile_max;
          l_sum *= alpha;
        }
        // P = 2^(s * scale - m) as packed bf16 back into the S columns (two keys per column);
        // scale-and-shift and the row sum run two columns per instruction (packed fp32)
        const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);
        const float2 neg_m2 = make_float2(-m_used, -m_used);
        float2 part[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
        uint32_t pk[kTileN / 2];
#pragma unroll
        for (int c2 = 0; c2 < kTileN / 2; ++c2) {
          const float2 x = __ffma2_rn(make_float2(s[2 * c2], s[2 * c2 + 1]), scale2, neg_m2);
          const float2 e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
          part[c2 & 3] = __fadd2_rn(part[c2 & 3], e);
          pk[c2] = pack_bf16x2(e.x, e.y);
        }
        const float2 tot = __fadd2_rn(__fadd2_rn(part[0], part[1]), __fadd2_rn(part[2], part[3]));
        l_sum += tot.x + tot.y;
        tmem_st64(s_addr, pk);
        if (i > 0 && __any_sync(0xffffffffu, need)) {
          // O may only be rescaled between PV(i-1) and PV(i).  PV(i) cannot start before this
          // thread has arrived on PFull below, so the barrier is never more than one phase ahead.
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarPVDone), (gt - 1) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int q4 = 0; q4 < D / 32; ++q4) {
            float o[32];
            const uint32_t addr = tmem_base + lane_addr + kTmemO + ob * 128 + q4 * 32;
            tmem_ld32(addr, reinterpret_cast<uint32_t*>(o));
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] *= alpha;
            tmem_st32(addr, reinterpret_cast<const uint32_t*>(o));
          }
        }
        tc_fence_before();
        mbar_arrive(bar(kBarPFull + sb));
      }
      if (!ok) break;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarOFull + ob), (n >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      float* orow = p.o_part + (w.item_out * kTileM + r) * D;
#pragma unroll
      for (int q4 = 0; q4 < D / 32; ++q4) {
        float o[32];
        tmem_ld32(tmem_base + lane_addr + kTmemO + ob * 128 + q4 * 32, reinterpret_cast<uint32_t*>(o));
#pragma unroll
        for (int e = 0; e < 32; e += 4)
          *reinterpret_cast<float4*>(orow + q4 * 32 + e) = make_float4(o[e], o[e + 1], o[e + 2], o[e + 3]);
      }
      tc_fence_before();
      mbar_arrive(bar(kBarOEmpty + ob));
      float* ml = p.ml_part + (w.item_out * kTileM + r) * 2;
      ml[0] = m_used;
      ml[1] = l_sum;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) ads_set_status(p.status, ADAPSHOT_ETIMEOUT);
}

struct CombineParams {
  const long long* ctx_off;
  const float* o_part;
  const float* ml_part;
  __nv_bfloat16* out;   // [B][nl][P][Tq][Hq][D]
  float* lse;           // [B][nl][P][Hq][Tq] or null
  long long ctx_cap;
  int B, k, P, Tq, Hq, Hkv, G, nl, n_mt, n_chunks, tiles_per_chunk;
  int nshots[kMaxProbes];
};

// One warp per output row (b, l, j, t, h): merge the chunk partials.
template <int D>
__global__ void __launch_bounds__(256) attn_combine_kernel(const CombineParams p) {
  const int lane = threadIdx.x & 31;
  const long long row_id = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_rows = (long long)p.B * p.nl * p.P * p.Tq * p.Hq;
  if (row_id >= n_rows) return;
  const int h = (int)(row_id % p.Hq);
  const int t = (int)((row_id / p.Hq) % p.Tq);
  const long long bpj = row_id / ((long long)p.Hq * p.Tq);
  const int j = (int)(bpj % p.P);
  const int b = (int)(bpj / ((long long)p.P * p.nl));
  const int g = h / p.G, hh = h % p.G;
  const int m = t * p.G + hh, mt = m / kTileM, r = m % kTileM;

  long long Lj = p.ctx_off[(long long)b * (p.k + 1) + p.nshots[j]];
  Lj = Lj > p.ctx_cap ? p.ctx_cap : (Lj < 0 ? 0 : Lj);
  const int n_tiles_ctx = (int)((Lj + kTileN - 1) / kTileN);
  const int c_last = n_tiles_ctx > 0 ? (n_tiles_ctx - 1) / p.tiles_per_chunk : 0;
  const long long item0 = ((bpj * p.Hkv + g) * p.n_mt + mt) * (long long)p.n_chunks;

  float M = kNegSentinel;
  for (int c = 0; c <= c_last; ++c) M = fmaxf(M, p.ml_part[((item0 + c) * kTileM + r) * 2]);
  constexpr int EPL = D / 32;                      // output elements per lane
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  float lsum = 0.f;
  for (int c = 0; c <= c_last; ++c) {
    const float* ml = p.ml_part + ((item0 + c) * kTileM + r) * 2;
    const float w = exp2f(ml[0] - M);
    lsum += ml[1] * w;
    const float* o = p.o_part + ((item0 + c) * kTileM + r) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += o[e] * w;
  }
  const float inv = 1.f / lsum;
  __nv_bfloat16* dst = p.out + row_id * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; e += 2)
    *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
  if (p.lse != nullptr && lane == 0)
    p.lse[(bpj * p.Hq + h) * p.Tq + t] = (M + log2f(lsum)) * 0.6931471805599453f;
}

// ----------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor, innermost dim contiguous, 128-byte swizzle, zero fill outside the bounds
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t gd[5], gs[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

struct AttnPlan {
  int n_mt, n_chunks, tiles_per_chunk;
  long long items;
  size_t off_qrot, off_kqrot, off_opart, off_ml, total;
};

AttnPlan make_plan(const adapshot_model_t* model, int B, int P, int Tq, int nl, long long ctx_cap,
                   uint32_t flags) {
  AttnPlan pl;
  const int G = model->n_q_heads / model->n_kv_heads;
  const int D = model->head_dim;
  pl.n_mt = (Tq * G + kTileM - 1) / kTileM;
  const long long tiles_cap = (ctx_cap + kTileN - 1) / kTileN;
  const long long base_items = (long long)B * nl * P * model->n_kv_heads * pl.n_mt;
  long long tpc = flags & 0xffffu;
  if (tpc == 0) {
    // about four waves of 148 CTAs when the context allows it, at least 8 tiles each
    long long want = (4 * 148 + base_items - 1) / base_items;
    tpc = (tiles_cap + want - 1) / want;
    if (tpc < 8) tpc = 8;
  }
  if (tpc > tiles_cap) tpc = tiles_cap > 0 ? tiles_cap : 1;
  pl.tiles_per_chunk = (int)tpc;
  pl.n_chunks = (int)((tiles_cap + tpc - 1) / tpc);
  if (pl.n_chunks < 1) pl.n_chunks = 1;
  pl.items = base_items * pl.n_chunks;
  size_t off = 0;
  pl.off_qrot = off;  off += ads_round_up((size_t)B * nl * P * Tq * model->n_q_heads * D * 2, 256);
  pl.off_kqrot = off; off += ads_round_up((size_t)B * nl * P * Tq * model->n_kv_heads * D * 2, 256);
  pl.off_opart = off; off += ads_round_up((size_t)pl.items * kTileM * D * 4, 256);
  pl.off_ml = off;    off += ads_round_up((size_t)pl.items * kTileM * 2 * 4, 256);
  pl.total = off;
  return pl;
}

bool attn_shape_ok(const adapshot_model_t* m) {
  return (m->head_dim == 64 || m->head_dim == 128) && m->n_kv_heads > 0 && m->n_q_heads > 0 &&
         m->n_q_heads % m->n_kv_heads == 0;
}

template <int D>
int launch_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx, int64_t ctx_cap,
                const int64_t* ctx_off, int B, int k, const int32_t* probe_nshots, int P, const void* q,
                const void* kq, const void* vq, int Tq, int nl, void* out, float* lse, const AttnPlan& pl,
                void* ws, int32_t* status, cudaStream_t st) {
  const int Hq = model->n_q_heads, Hkv = model->n_kv_heads, G = Hq / Hkv;
  unsigned char* wsb = static_cast<unsigned char*>(ws);
  __nv_bfloat16* q_rot = reinterpret_cast<__nv_bfloat16*>(wsb + pl.off_qrot);
  __nv_bfloat16* kq_rot = reinterpret_cast<__nv_bfloat16*>(wsb + pl.off_kqrot);
  float* o_part = reinterpret_cast<float*>(wsb + pl.off_opart);
  float* ml_part = reinterpret_cast<float*>(wsb + pl.off_ml);

  // ---- tensor maps
  CUtensorMap tm_q, tm_kctx, tm_vctx, tm_kown, tm_vown;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)Tq * G, (uint64_t)B * nl * P * Hkv};
    const uint64_t str[2] = {(uint64_t)D * 2, (uint64_t)Tq * G * D * 2};
    const uint32_t box[3] = {64, (uint32_t)kTileM, 1};
    if (!make_map(&tm_q, q_rot, 3, dims, str, box)) return ADAPSHOT_ECUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)Hkv, (uint64_t)ctx_cap, (uint64_t)B * nl};
    const uint64_t str[3] = {(uint64_t)D * 2, (uint64_t)Hkv * D * 2, (uint64_t)ctx_cap * Hkv * D * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)kTileN, 1};
    if (!make_map(&tm_kctx, k_ctx, 4, dims, str, box)) return ADAPSHOT_ECUDA;
    if (!make_map(&tm_vctx, v_ctx, 4, dims, str, box)) return ADAPSHOT_ECUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)Hkv, (uint64_t)Tq, (uint64_t)B * nl * P};
    const uint64_t str[3] = {(uint64_t)D * 2, (uint64_t)Hkv * D * 2, (uint64_t)Tq * Hkv * D * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)kTileN, 1};
    if (!make_map(&tm_kown, kq_rot, 4, dims, str, box)) return ADAPSHOT_ECUDA;
    if (!make_map(&tm_vown, vq, 4, dims, str, box)) return ADAPSHOT_ECUDA;
  }

  // ---- rotate Q and the probe's own K
  PrepParams pp;
  pp.q = static_cast<const __nv_bfloat16*>(q); pp.kq = static_cast<const __nv_bfloat16*>(kq);
  pp.q_rot = q_rot; pp.kq_rot = kq_rot; pp.ctx_off = reinterpret_cast<const long long*>(ctx_off);
  pp.B = B; pp.k = k; pp.P = P; pp.Tq = Tq; pp.Hq = Hq; pp.Hkv = Hkv; pp.nl = nl;
  pp.rope_base = model->rope_base;
  for (int i = 0; i < kMaxProbes; ++i) pp.nshots[i] = i < P ? probe_nshots[i] : 0;
  const long long n_tok = (long long)B * nl * P * Tq;
  attn_prep_kernel<D><<<(unsigned)((n_tok + 7) / 8), 256, 0, st>>>(pp);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  // ---- main kernel
  AttnParams ap;
  ap.ctx_off = reinterpret_cast<const long long*>(ctx_off);
  ap.o_part = o_part; ap.ml_part = ml_part; ap.status = status; ap.ctx_cap = ctx_cap;
  ap.B = B; ap.k = k; ap.P = P; ap.Tq = Tq; ap.Hq = Hq; ap.Hkv = Hkv; ap.G = G; ap.nl = nl;
  ap.n_mt = pl.n_mt; ap.n_chunks = pl.n_chunks; ap.tiles_per_chunk = pl.tiles_per_chunk;
  const float scale = model->softmax_scale > 0.f ? model->softmax_scale : 1.0f / sqrtf((float)D);
  ap.scale_log2 = scale * 1.4426950408889634f;
  for (int i = 0; i < kMaxProbes; ++i) ap.nshots[i] = pp.nshots[i];
  const int smem = (int)AttnSmem<128>::kTotal;     // same request for D = 64: one CTA per SM
  static bool attr_done[2] = {false, false};
  if (!attr_done[D == 128]) {
    ADS_CHECK_CUDA(cudaFuncSetAttribute(attn_main_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_done[D == 128] = true;
  }
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    ADS_CHECK_CUDA(cudaGetDevice(&dev));
    ADS_CHECK_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  }
  const unsigned grid = (unsigned)(pl.items < n_sm ? pl.items : n_sm);   // persistent: one CTA per SM
  attn_main_kernel<D><<<grid, kAttnThreads, smem, st>>>(tm_q, tm_kctx, tm_vctx, tm_kown, tm_vown, ap);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  // ---- merge
  CombineParams cp;
  cp.ctx_off = ap.ctx_off; cp.o_part = o_part; cp.ml_part = ml_part;
  cp.out = static_cast<__nv_bfloat16*>(out); cp.lse = lse; cp.ctx_cap = ctx_cap;
  cp.B = B; cp.k = k; cp.P = P; cp.Tq = Tq; cp.Hq = Hq; cp.Hkv = Hkv; cp.G = G; cp.nl = nl;
  cp.n_mt = pl.n_mt; cp.n_chunks = pl.n_chunks; cp.tiles_per_chunk = pl.tiles_per_chunk;
  for (int i = 0; i < kMaxProbes; ++i) cp.nshots[i] = pp.nshots[i];
  const long long n_rows = n_tok * Hq;
  attn_combine_kernel<D><<<(unsigned)((n_rows + 7) / 8), 256, 0, st>>>(cp);
  return ads_launch_status();
}

}  // namespace

extern "C" size_t adapshot_attn_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                                int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap) {
  if (model == nullptr || !attn_shape_ok(model) || B <= 0 || P <= 0 || Tq <= 0 || n_layers_in_call <= 0 ||
      ctx_cap <= 0)
    return 0;
  // sized for the finest split a caller may request through `flags`
  AttnPlan a = make_plan(model, B, P, Tq, n_layers_in_call, ctx_cap, 0);
  AttnPlan f = make_plan(model, B, P, Tq, n_layers_in_call, ctx_cap, 8);
  return a.total > f.total ? a.total : f.total;
}

extern "C" int adapshot_query_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx,
                                   int64_t ctx_cap, const int64_t* ctx_off, int32_t B, int32_t k,
                                   const int32_t* probe_nshots, int32_t P, const void* q, const void* kq,
                                   const void* vq, int32_t Tq, int32_t layer_begin, int32_t layer_end,
                                   void* out, float* lse, uint32_t flags, void* ws, size_t ws_bytes,
                                   int32_t* status, void* stream) {
  if (model == nullptr || k_ctx == nullptr || v_ctx == nullptr || ctx_off == nullptr || probe_nshots == nullptr ||
      q == nullptr || kq == nullptr || vq == nullptr || out == nullptr || ws == nullptr)
    return ADAPSHOT_EINVAL;
  if (B <= 0 || k <= 0 || Tq <= 0 || ctx_cap <= 0 || (flags & ~0xffffu) != 0) return ADAPSHOT_EINVAL;
  if (model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (!attn_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
  if (P < 1 || P > kMaxProbes || (long long)P * B > kMaxPairs) return ADAPSHOT_ESHAPE;
  for (int i = 0; i < P; ++i) {
    if (probe_nshots[i] < 1 || probe_nshots[i] > k) return ADAPSHOT_ESHAPE;
    if (i > 0 && probe_nshots[i] <= probe_nshots[i - 1]) return ADAPSHOT_ESHAPE;
  }
  if ((flags & 0xffffu) != 0 && (flags & 0xffffu) < 8) return ADAPSHOT_EINVAL;
  if (!ads_aligned16(k_ctx) || !ads_aligned16(v_ctx) || !ads_aligned16(q) || !ads_aligned16(kq) ||
      !ads_aligned16(vq) || !ads_aligned16(out) || ((uintptr_t)ws & 255u))
    return ADAPSHOT_EALIGN;
  if (ctx_cap > (1ll << 31) - 256) return ADAPSHOT_ESHAPE;
  const int nl = layer_end - layer_begin;
  const AttnPlan pl = make_plan(model, B, P, Tq, nl, ctx_cap, flags);
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  if (pl.items > 0x7fffffffll) return ADAPSHOT_ESHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (model->head_dim == 128)
    return launch_attn<128>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                            lse, pl, ws, status, st);
  return launch_attn<64>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                         lse, pl, ws, status, st);
}
