// Probe attention over the reused cache (paper Eq. 1 with the tree mask of Sec. 4.1:
// probe j sees the first n_j shots of the assembled context and, causally, its own
// tokens; scores scaled by 1/sqrt(d) as in Eq. 5; rotary positions of Eq. 6).
//
// Three kernels:
//   attn_prep     rotates Q and the probe's own K to their positions L_j + t, packs the
//                 Q rows of one KV head (GQA) into an M-major tile layout, and writes
//                 the schedule (how many 128-key tiles every (probe, query) pair has
//                 and where the tile sequence is cut into ranges of equal cost);
//   attn_main     persistent CTAs.  A CTA works on two 128-row M tiles of one KV head
//                 at a time ("M pair"): TMA stages each K/V tile once for both, one
//                 thread issues tcgen05 UMMAs (S = Q K^T, O += P V, accumulators in
//                 TMEM, P kept in TMEM), two groups of four warps run the online
//                 softmax of the two M tiles (one thread per row) and alternate on the
//                 tensor pipe.  The global tile sequence is cut into ranges of equal
//                 cost, one per gang of CTAs (the CTAs of a gang take the M pairs of the
//                 same K/V tiles, so the tiles are shared through L2).  A range that
//                 covers a whole unit stores the final bf16 rows (staged through shared
//                 memory into whole row segments); a range that cuts a unit stores
//                 un-normalised partials;
//   attn_combine  log-sum-exp merge of the partials of the cut units.
// The fused variant (adapshot_query_attn_fused) adds attn_fused_plan (row map and rotary
// table, once per call) and runs attn_main with two loader warps that copy the context
// K/V tiles from the pool and re-encode K (Eq. 7) in shared memory, instead of TMA loads
// from an assembled cache.  The V-from-pool variant (adapshot_query_attn_vpool) sits between
// the two: K tiles come by TMA from a cache that holds the re-encoded K only, V tiles (which
// Eq. 7 leaves as they are) are copied from the pool through the row map, so that the gather
// moves half the bytes.
#include <cuda.h>
#include <float.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace {

using namespace sm100;

constexpr int kMaxProbes = 16;
constexpr int kMaxPairs = 256;       // (probe, query) pairs one call may hold: B * P <= 256
constexpr int kMaxCtas = 160;        // persistent grid: one CTA per SM, at most this many
constexpr int kMaxGang = 8;          // CTAs that share one range of K/V tiles
constexpr int kUnitCost = 4;          // fixed cost of starting a unit, in tiles (measured: about 10 k clocks)
constexpr int kTileM = 128;          // query rows per M tile (TMEM lanes)
constexpr int kTileN = 128;          // keys per tile
constexpr int kAttnThreads = 320;    // warp 0 TMA, warp 1 MMA, warps 2-5 softmax A, warps 6-9 softmax B
constexpr int kFusedThreads = 384;   // fused variant: warps 2-3 load and rotate K/V, softmax on warps 4-11
constexpr int kVPoolThreads = 352;   // V-from-pool variant: the cache variant's warps plus warp 10, which gathers V
constexpr int kModeCache = 0;        // K and V tiles by TMA from the assembled cache
constexpr int kModeFused = 1;        // K and V tiles from the pool, K re-encoded in shared memory
constexpr int kModeVPool = 2;        // K tiles by TMA from a K-only cache, V tiles from the pool
constexpr int kLoaders = 64;         // threads of the two loader warps
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;   // log2 units: rescale O only when the max grows by 2^8
constexpr float kNegSentinel = -1.0e30f;
constexpr float kLn2 = 0.6931471805599453f;

// Schedule shared by the main and the combine kernel (lives in the workspace).
// Pairs are ordered longest probe first: pair = (P-1-j) * B + b.  Every pair owns
// nl * Hkv units (layer, kv head) of n_su tiles each: n_ctx context tiles followed by
// n_own tiles of the probe's own tokens.  The ranges are equal in cost, not in tiles: every
// unit that starts in a range adds kUnitCost tiles' worth of time to it (Q load and pipeline
// fill, read-out of O), which matters when the units are as short as a range.
struct Sched {
  long long total;                   // tiles of all units
  long long start[kMaxCtas + 1];     // first tile of every gang's range; start[n_gangs] = total
  int first_pair[kMaxCtas + 1];      // pair that holds start[q]
  long long prefix[kMaxPairs + 1];   // first tile of every pair in the global sequence
  long long Lj[kMaxPairs];           // context length of the pair's probe (clamped to ctx_cap)
  int n_ctx[kMaxPairs];
  int n_su[kMaxPairs];
};

struct AttnParams {
  const Sched* sched;
  float* o_part;              // [slots][2][D/4][128][4] fp32, un-normalised (rows contiguous per 4 columns)
  float* ml_part;             // [slots][2][128][2]  (running max in log2 units, row sum)
  __nv_bfloat16* out;         // [B][nl][P][Tq][Hq][D]
  float* lse;                 // [B][nl][P][Hq][Tq] or null
  int32_t* status;
  int B, P, Tq, Hq, Hkv, G, nl;
  int To;                     // own tokens per probe (>= Tq): the Tq rows are the last Tq of them
  int n_mt, n_mp, gang, n_gangs;
  float scale_log2;           // softmax_scale * log2(e)
  // fused variant only: K/V tiles come from the pool (and from the probe's own rotated keys)
  const __nv_bfloat16* k_pool;   // [n_layers][pool_tokens][Hkv][D]
  const __nv_bfloat16* v_pool;
  const __nv_bfloat16* kq_rot;   // [B*nl*P][To][Hkv][D], rotated by the prep kernel
  const __nv_bfloat16* vq;
  const int* row_map;            // [B][ctx_cap]: pool token of every context position, -1 beyond L
  const int* off_map;            // [B][ctx_cap]: first position of the shot a position lies in (k_pos_mode 1)
  int k_pos_mode;                // 0: angle = position; 1: angle = the shot's first position (Eq. 7 as printed)
  const float2* rope_tab;        // [ctx_cap rounded up to 128][D/2]: (cos, sin) of position * theta_i
  long long pool_tokens, ctx_cap;
  int layer_begin;
  double rope_base_f;
};

struct PrepParams {
  const __nv_bfloat16* q;     // [B][nl][P][Tq][Hq][D]
  const __nv_bfloat16* kq;    // [B][nl][P][To][Hkv][D]
  __nv_bfloat16* q_rot;       // [B*nl*P*Hkv][Tq*G][D]
  __nv_bfloat16* kq_rot;      // layout of kq
  const long long* ctx_off;
  Sched* sched;
  long long ctx_cap;
  int B, k, P, Tq, Hq, Hkv, nl, n_gangs;
  int To;                     // own tokens per probe: the Tq query rows are the last Tq of them
  const int* nshots_dev;      // per-query shot count of the (single) probe, device memory, or null
  int32_t* status;
  double rope_base;
  double theta[64];           // theta_i = rope_base^(-2i/D), formed on the host
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

constexpr int kPrepParts = 4;

// Shots of probe j of query b: from the host list, or (decode over the prefix each query chose)
// from a per-query device array; a count outside 1..k is reported and clamped.
__device__ __forceinline__ int probe_shots(const PrepParams& p, int b, int j) {
  if (p.nshots_dev == nullptr) return p.nshots[j];
  int n = p.nshots_dev[b];
  if (n < 1 || n > p.k) {
    ads_set_status(p.status, ADAPSHOT_EINDEX);
    n = n < 1 ? 1 : p.k;
  }
  return n;
}

// kPrepParts warps per probe token (b, l, j, t): all Hq query heads and Hkv key heads of the
// token rotate by the same angles (L_j + t) * theta_i.  The last block writes the schedule instead.
template <int D>
__global__ void __launch_bounds__(256) attn_prep_kernel(const PrepParams p) {
  constexpr int VPH = D / 8, HALF_V = VPH / 2;
  const int lane = threadIdx.x & 31;

  if (blockIdx.x == gridDim.x - 1) {
    // the schedule, by a block of its own (beside the rotation, not in front of a share of it);
    // intermediate values stay in shared memory
    __shared__ long long s_pre[kMaxPairs + 1], s_vpre[kMaxPairs + 1];
    __shared__ int s_nsu[kMaxPairs];
    Sched* sc = p.sched;
    const int n_pairs = p.P * p.B;
    const int n_own = (p.To + kTileN - 1) / kTileN;
    const long long units_per_pair = (long long)p.nl * p.Hkv;
    for (int pi = threadIdx.x; pi < n_pairs; pi += blockDim.x) {
      const int j = p.P - 1 - pi / p.B, b = pi % p.B;
      long long Lj = p.ctx_off[(long long)b * (p.k + 1) + probe_shots(p, b, j)];
      Lj = Lj > p.ctx_cap ? p.ctx_cap : (Lj < 0 ? 0 : Lj);
      const int n_ctx = (int)((Lj + kTileN - 1) / kTileN);
      sc->Lj[pi] = Lj;
      sc->n_ctx[pi] = n_ctx;
      sc->n_su[pi] = n_ctx + n_own;
      s_nsu[pi] = n_ctx + n_own;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      long long acc = 0, vacc = 0;
      for (int pi = 0; pi < n_pairs; ++pi) {
        s_pre[pi] = acc;
        s_vpre[pi] = vacc;
        sc->prefix[pi] = acc;
        acc += (long long)s_nsu[pi] * units_per_pair;
        vacc += (long long)(s_nsu[pi] + kUnitCost) * units_per_pair;
      }
      s_pre[n_pairs] = acc;
      s_vpre[n_pairs] = vacc;
      sc->prefix[n_pairs] = acc;
      sc->total = acc;
    }
    __syncthreads();
    // Range q starts where the cost sequence (every unit preceded by kUnitCost virtual tiles)
    // reaches q / n_gangs of its length: threads q = 0 .. n_gangs, independently.
    const long long vtotal = s_vpre[n_pairs];
    for (int q = threadIdx.x; q <= p.n_gangs; q += blockDim.x) {
      const long long v = (long long)q * vtotal / p.n_gangs;
      long long real = s_pre[n_pairs];
      int fp = n_pairs - 1;
      if (v < vtotal) {
        int lo = 0, hi = n_pairs;                   // pair with s_vpre[lo] <= v < s_vpre[lo + 1]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (s_vpre[mid] <= v) lo = mid; else hi = mid;
        }
        const long long lv = s_nsu[lo] + kUnitCost;
        const long long rel = v - s_vpre[lo];
        const long long su = rel / lv, off = rel % lv;
        real = s_pre[lo] + su * s_nsu[lo] + (off > kUnitCost ? off - kUnitCost : 0);
        fp = lo;
      }
      sc->start[q] = real;
      sc->first_pair[q] = fp;
    }
    return;
  }
  const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long tok = gw / kPrepParts;            // kPrepParts warps share the heads of one own token
  const int part = (int)(gw % kPrepParts);
  const long long n_tok = (long long)p.B * p.nl * p.P * p.To;
  if (tok >= n_tok) return;
  const int u_own = (int)(tok % p.To);              // own token u sits at position L_j + u
  const long long bpj = tok / p.To;                 // (b*nl + l)*P + j
  const int j = (int)(bpj % p.P);
  const int b = (int)(bpj / ((long long)p.P * p.nl));
  const long long Lj = p.ctx_off[(long long)b * (p.k + 1) + probe_shots(p, b, j)];
  const double pos = (double)(Lj + u_own);
  const int G = p.Hq / p.Hkv;
  const int t = u_own - (p.To - p.Tq);              // query row of this token (the last Tq own tokens have one)
  const bool has_q = t >= 0;

  const int jcol = lane % HALF_V;
  float sn[8], cs[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    rope_sincos(pos, p.theta[jcol * 8 + e], &sn[e], &cs[e]);
  }
  const uint4* qsrc = reinterpret_cast<const uint4*>(p.q) + (bpj * p.Tq + (has_q ? t : 0)) * p.Hq * VPH;
  const uint4* ksrc = reinterpret_cast<const uint4*>(p.kq) + tok * p.Hkv * VPH;
  uint4* kdst = reinterpret_cast<uint4*>(p.kq_rot) + tok * p.Hkv * VPH;
  uint4* qdst_base = reinterpret_cast<uint4*>(p.q_rot);
  const int units = (p.Hq + p.Hkv) * HALF_V;
  for (int u = part * 32 + lane; u < units; u += 32 * kPrepParts) {
    const int head = u / HALF_V;                    // column == jcol since 32 % HALF_V == 0
    const bool is_q = head < p.Hq;
    if (is_q && !has_q) continue;
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

// Fused variant, once per call: the pool token behind every context position of every query
// (the gather's plan lookup, stored instead of applied) and the rotary table of the context
// positions, (cos, sin)(p * theta_i) from fp64 angles.
struct FusedPlanParams {
  const long long* ctx_off;   // [B][k+1]
  const int32_t* sel_idx;     // [B][k]
  const long long* shot_off;  // [n_shots+1]
  int* row_map;               // [B][ctx_cap]
  int* off_map;               // [B][ctx_cap]: first position of the position's shot
  float2* rope_tab;           // [tab_rows][D/2]
  long long ctx_cap, tab_rows;
  int B, k, n_shots, half_d;
  double rope_base;
};

__global__ void __launch_bounds__(256) attn_fused_plan_kernel(const FusedPlanParams p) {
  const long long n_map = (long long)p.B * p.ctx_cap;
  const long long n_tab = p.tab_rows * p.half_d;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < n_map + n_tab; u += stride) {
    if (u < n_map) {
      const int b = (int)(u / p.ctx_cap);
      const long long pos = u % p.ctx_cap;
      const long long* off = p.ctx_off + (long long)b * (p.k + 1);
      int row = -1, first = 0;
      if (pos < off[p.k]) {
        int lo = 0, hi = p.k;          // shot slot with off[lo] <= pos < off[lo+1]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (off[mid] <= pos) lo = mid; else hi = mid;
        }
        const int s = p.sel_idx[(long long)b * p.k + lo];
        if (s >= 0 && s < p.n_shots) row = (int)(p.shot_off[s] + (pos - off[lo]));
        first = (int)off[lo];
      }
      p.row_map[u] = row;
      p.off_map[u] = first;
    } else {
      const long long v = u - n_map;
      const long long pos = v / p.half_d;
      const int i = (int)(v % p.half_d);
      const double theta = pow(p.rope_base, -(double)i / (double)p.half_d);
      float sn, cs;
      rope_sincos((double)pos, theta, &sn, &cs);
      p.rope_tab[v] = make_float2(cs, sn);
    }
  }
}

// Shared-memory plan.  Every operand tile is made of [128 rows][128 bytes] sub-tiles
// written by TMA with the 128-byte swizzle; D = 128 needs two of them per tile.
// The fused variant's loader warps take the stages of tile i+1 before they hand over tile i,
// which needs a third V stage; the room goes at the expense of the read-out staging.
template <int D, int MODE>
struct AttnSmem {
  static constexpr int kKStages = 2;
  static constexpr int kVStages = MODE == kModeFused ? 3 : 2;
  static constexpr uint32_t kStageBytes = MODE == kModeFused ? 0 : 4096;  // per softmax warp: 32 rows x 128 bytes
  static constexpr uint32_t kTileBytes = (D / 64) * 16384u;
  static constexpr uint32_t kOffQ = 0;                                    // Q of M tile A, then of M tile B
  static constexpr uint32_t kOffK = kOffQ + 2 * kTileBytes;
  static constexpr uint32_t kOffV = kOffK + kKStages * kTileBytes;
  static constexpr uint32_t kOffStage = kOffV + kVStages * kTileBytes;    // read-out staging of the 8 softmax warps
  static constexpr uint32_t kOffBar = kOffStage + 8 * kStageBytes;
  static constexpr uint32_t kOffRows = kOffBar + 256 + 1024;              // V-from-pool variant: pool rows of a tile
  static constexpr uint32_t kTotal = kOffRows + (MODE == kModeVPool ? 512 : 0) + 1024;   // + alignment slack
};

// mbarrier slots (8 bytes each)
enum Bar {
  kBarQFull = 0, kBarQEmpty = 2, kBarKFull = 4, kBarKEmpty = 7, kBarVFull = 10, kBarVEmpty = 13,
  kBarSFull = 16, kBarPFull = 18, kBarOFull = 20, kBarOEmpty = 22, kBarDrain = 24,
  kNumBars = 25
};

// A piece = the part of one unit (pair, layer, kv head) that falls into a gang's range.
struct Piece {
  int pair, su, t0, t1, n_su, n_ctx;
  long long Lj;
  bool first_of_gang;
};

struct Walker {
  long long x, begin, end;
  int pair;                      // pair that holds x (pieces only move forward)
};

// The part of the schedule a CTA walks, copied to shared memory once: the pairs from the
// one its range starts in.  Pairs beyond the copy (a range that spans more than
// kCachePairs pairs) are read from the workspace.
constexpr int kCachePairs = 40;
struct SchedCache {
  long long prefix[kCachePairs + 1];
  long long Lj[kCachePairs];
  int n_ctx[kCachePairs];
  int n_su[kCachePairs];
  long long begin, end;
  int p0, n;
};
static_assert(sizeof(SchedCache) <= 1024, "the schedule cache has 1 KiB of shared memory");
struct PairInfo {
  long long prefix, next_prefix, Lj;
  int n_ctx, n_su;
};
__device__ __forceinline__ PairInfo pair_info(const Sched* sc, const SchedCache* c, int pair) {
  PairInfo pi;
  const int k = pair - c->p0;
  if (k >= 0 && k < c->n) {
    pi.prefix = c->prefix[k]; pi.next_prefix = c->prefix[k + 1]; pi.Lj = c->Lj[k];
    pi.n_ctx = c->n_ctx[k]; pi.n_su = c->n_su[k];
  } else {
    pi.prefix = sc->prefix[pair]; pi.next_prefix = sc->prefix[pair + 1]; pi.Lj = sc->Lj[pair];
    pi.n_ctx = sc->n_ctx[pair]; pi.n_su = sc->n_su[pair];
  }
  return pi;
}

__device__ __forceinline__ int find_pair(const Sched* sc, int n_pairs, long long x) {
  int lo = 0, hi = n_pairs;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (sc->prefix[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ bool next_piece(const Sched* sc, const SchedCache* cache, int n_pairs, Walker& wk,
                                           Piece& pc) {
  if (wk.x >= wk.end) return false;
  PairInfo pi = pair_info(sc, cache, wk.pair);
  while (wk.pair + 1 < n_pairs && pi.next_prefix <= wk.x) pi = pair_info(sc, cache, ++wk.pair);
  const int lo = wk.pair;
  const int nsu = pi.n_su;
  const long long rel = wk.x - pi.prefix;
  pc.pair = lo;
  pc.su = (int)(rel / nsu);
  pc.t0 = (int)(rel % nsu);
  const long long room = wk.end - wk.x;
  pc.t1 = (int)(room < (long long)(nsu - pc.t0) ? pc.t0 + room : nsu);
  pc.n_su = nsu;
  pc.n_ctx = pi.n_ctx;
  pc.Lj = pi.Lj;
  pc.first_of_gang = wk.x == wk.begin;
  wk.x += pc.t1 - pc.t0;
  return true;
}

// One M pair of one piece: what a CTA works on between two read-outs of O.
struct Item {
  int b, l, j, g, mp;
  bool has_b, whole;
  int ctx_begin, n_ctx, own_begin, n_own, n_tiles;
  long long Lj;
  int outer_ctx, outer_own, outer_q;
  long long slot;
};

__device__ __forceinline__ void make_item(const AttnParams& p, const Piece& pc, int gang_id, int mp, Item& w) {
  w.j = p.P - 1 - pc.pair / p.B;
  w.b = pc.pair % p.B;
  w.l = pc.su / p.Hkv;
  w.g = pc.su % p.Hkv;
  w.mp = mp;
  w.has_b = 2 * mp + 1 < p.n_mt;
  w.whole = pc.t0 == 0 && pc.t1 == pc.n_su;
  w.Lj = pc.Lj;
  const int ctx_end = min(pc.t1, pc.n_ctx);
  w.ctx_begin = pc.t0;
  w.n_ctx = max(0, ctx_end - pc.t0);
  // own-token tiles this M pair can see (causal): tokens up to the pair's last row
  const int row_hi = min(p.Tq * p.G - 1, mp * 2 * kTileM + 2 * kTileM - 1);
  const int own_need = (p.To - p.Tq + row_hi / p.G) / kTileN + 1;
  w.own_begin = max(pc.t0, pc.n_ctx) - pc.n_ctx;
  const int own_end = min(pc.t1 - pc.n_ctx, own_need);
  w.n_own = max(0, own_end - w.own_begin);
  w.n_tiles = w.n_ctx + w.n_own;
  w.outer_ctx = w.b * p.nl + w.l;
  w.outer_own = w.outer_ctx * p.P + w.j;
  w.outer_q = w.outer_own * p.Hkv + w.g;
  w.slot = ((long long)(2 * gang_id + (pc.first_of_gang ? 0 : 1)) * p.n_mp + mp);
}

// V-from-pool variant: maps over the pool's V with boxes of 1, 2, 4, ..., 128 rows, from which a
// tile is stitched run by run (a run = consecutive context positions that are consecutive pool rows).
struct VPoolMaps {
  CUtensorMap m[8];
};

// TMEM: S/P of M tile A at columns 0..127, of M tile B at 128..255 (P, as packed bf16,
// overwrites the S tile it was computed from); O accumulators at 256 and 384.
// FUSED: the context K/V tiles are read from the pool through the row map (per-thread async
// copies into the swizzled tile layout) and K is rotated in shared memory by two loader warps,
// so that no re-encoded cache is ever written to HBM; TMA then only brings Q.
template <int D, int MODE>
__global__ void __launch_bounds__(MODE == kModeFused ? kFusedThreads : (MODE == kModeVPool ? kVPoolThreads : kAttnThreads), 1)
attn_main_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kctx,
                 const __grid_constant__ CUtensorMap tm_vctx, const __grid_constant__ CUtensorMap tm_kown,
                 const __grid_constant__ CUtensorMap tm_vown, const __grid_constant__ VPoolMaps vmaps,
                 const AttnParams p) {
  constexpr bool FUSED = MODE == kModeFused;
  constexpr bool VPOOL = MODE == kModeVPool;
  using SM = AttnSmem<D, MODE>;
  constexpr int SUB = D / 64;
  constexpr int KS = SM::kKStages, VS = SM::kVStages;
  constexpr uint32_t kTileBytes = SM::kTileBytes;
  constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kTileN, 0);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, 1);
  constexpr uint32_t kTmemS = 0, kTmemO = 256;
  constexpr int kSoftmaxWarp0 = FUSED ? 4 : 2;          // first of the eight softmax warps
  constexpr int kGatherWarp = kSoftmaxWarp0 + 8;        // V-from-pool variant: the warp that gathers the V tiles

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - raw_addr);
  const uint32_t bar0 = base + SM::kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + SM::kOffBar + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + SM::kOffBar + 8 * kNumBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pairs = p.P * p.B;
  const int gang_id = blockIdx.x / p.gang, rank = blockIdx.x % p.gang;
  const Sched* sc = p.sched;

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
      mbar_init(bar(kBarKFull + i), FUSED ? kLoaders : 1);
      mbar_init(bar(kBarKEmpty + i), 1);
      mbar_init(bar(kBarVFull + i), FUSED ? kLoaders : 1);
      mbar_init(bar(kBarVEmpty + i), 1);
    }
    mbar_init(bar(kBarDrain), 1);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    mbar_fence_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  // the CTA's part of the schedule, fetched by two otherwise idle warps while the rest is set up
  SchedCache* cache = reinterpret_cast<SchedCache*>(base_ptr + SM::kOffBar + 256);
  if (warp >= 2 && warp < 4) {
    const int p0 = sc->first_pair[gang_id];
    const int n = min(kCachePairs, n_pairs - p0);
    for (int k = threadIdx.x - 64; k <= n; k += 64) {
      cache->prefix[k] = sc->prefix[p0 + k];
      if (k < n) {
        cache->Lj[k] = sc->Lj[p0 + k];
        cache->n_ctx[k] = sc->n_ctx[p0 + k];
        cache->n_su[k] = sc->n_su[p0 + k];
      }
    }
    if (threadIdx.x == 64) {
      cache->begin = sc->start[gang_id];
      cache->end = sc->start[gang_id + 1];
      cache->p0 = p0;
      cache->n = n;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  Walker wk0;
  wk0.begin = cache->begin;
  wk0.end = cache->end;
  wk0.x = wk0.begin;
  wk0.pair = cache->p0;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kctx); tma_prefetch_desc(&tm_vctx);
      uint32_t tk = 0, tv = 0, nq[2] = {0, 0};
      bool ok = true;
      Walker wk = wk0;
      Piece pc;
      while (ok && next_piece(sc, cache, n_pairs, wk, pc)) {
        for (int mp = rank; mp < p.n_mp && ok; mp += p.gang) {
          Item w;
          make_item(p, pc, gang_id, mp, w);
          if (w.n_tiles == 0) continue;
          for (int x = 0; x < (w.has_b ? 2 : 1) && ok; ++x) {
            ok = mbar_wait(bar(kBarQEmpty + x), (nq[x] & 1) ^ 1, abort_flag);
            if (!ok) break;
            mbar_arrive_expect_tx(bar(kBarQFull + x), kTileBytes);
#pragma unroll
            for (int s = 0; s < SUB; ++s)
              tma_load_3d(base + SM::kOffQ + x * kTileBytes + s * 16384u, &tm_q, bar(kBarQFull + x), s * 64,
                          (2 * mp + x) * kTileM, w.outer_q);
            ++nq[x];
          }
          for (int i = 0; i < (FUSED ? 0 : w.n_tiles) && ok; ++i) {
            const bool own = i >= w.n_ctx;
            const CUtensorMap* mk = own ? &tm_kown : &tm_kctx;
            const CUtensorMap* mv = own ? &tm_vown : &tm_vctx;
            const int row = own ? (w.own_begin + i - w.n_ctx) * kTileN : (w.ctx_begin + i) * kTileN;
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
            if constexpr (!VPOOL) {
              const int sv = tv % VS;
              ok = mbar_wait(bar(kBarVEmpty + sv), ((tv / VS) & 1) ^ 1, abort_flag);
              if (!ok) break;
              mbar_arrive_expect_tx(bar(kBarVFull + sv), kTileBytes);
#pragma unroll
              for (int s = 0; s < SUB; ++s)
                tma_load_4d(base + SM::kOffV + sv * kTileBytes + s * 16384u, mv, bar(kBarVFull + sv), s * 64, w.g,
                            row, outer);
              ++tv;
            }
          }
        }
      }
      if (!ok && !FUSED) {
        // gave up: let the copies already in flight land before the CTA retires
        for (uint32_t t = tk > (uint32_t)KS ? tk - KS : 0; t < tk; ++t)
          mbar_wait(bar(kBarKFull + t % KS), (t / KS) & 1, abort_flag + 1);
        if constexpr (!VPOOL)
          for (uint32_t t = tv > (uint32_t)VS ? tv - VS : 0; t < tv; ++t)
            mbar_wait(bar(kBarVFull + t % VS), (t / VS) & 1, abort_flag + 1);
      }
      if (!ok) {
        for (int x = 0; x < 2; ++x)
          if (nq[x] > 0) mbar_wait(bar(kBarQFull + x), (nq[x] - 1) & 1, abort_flag + 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // The tensor pipe takes only a few UMMAs ahead of the one it runs: whatever this thread
      // does between two issues is time the pipe may idle, so the per-tile path is kept short
      // (scalar counters, no indexed arrays, descriptors as a constant high half plus a low
      // half = (address >> 4) with an immediate per k-step).
      uint32_t tk = 0, tv = 0, np0 = 0, np1 = 0, ni0 = 0, ni1 = 0;
      bool ok = true;
      Walker wk = wk0;
      Piece pc;
      constexpr uint32_t kHi = smem_desc_hi_sw128(1024);
      const uint32_t q_lo0 = smem_desc_lo(base + SM::kOffQ, 16);
      const uint32_t k_lo0 = smem_desc_lo(base + SM::kOffK, 16);
      const uint32_t v_lo0 = smem_desc_lo(base + SM::kOffV, 16384);
      auto issue_qk = [&](const int x, uint32_t k_stage) {
        const uint32_t q_lo = q_lo0 + x * (kTileBytes >> 4);
        const uint32_t k_lo = k_lo0 + k_stage * (kTileBytes >> 4);
        const uint32_t d = tmem_base + kTmemS + x * kTileN;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t o = ((ks / 4) * 16384u + (ks % 4) * 32u) >> 4;
          umma_ss_lohi(d, q_lo + o, kHi, k_lo + o, kHi, kIdescQK, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar(kBarSFull + x));
      };
      auto issue_pv = [&](const int x, uint32_t v_stage, bool first) {
        const uint32_t v_lo = v_lo0 + v_stage * (kTileBytes >> 4);
        const uint32_t d = tmem_base + kTmemO + x * 128;
        const uint32_t a = tmem_base + kTmemS + x * kTileN;
        // A = P from TMEM: 16 bf16 keys of one k-step occupy 8 packed columns
        umma_ts_lohi(d, a, v_lo, kHi, kIdescPV, first ? 0u : 1u);
#pragma unroll
        for (int ks = 1; ks < kTileN / 16; ++ks)
          umma_ts_lohi(d, a + ks * 8, v_lo + ((ks * 2048u) >> 4), kHi, kIdescPV, 1u);
      };
      // one M tile's share of tile i: O += P V, then S of the next tile (in place of P: the
      // tensor pipe runs its operations in order)
      auto chain = [&](const int x, uint32_t& np_x, const uint32_t ni_x, int i, int n_tiles, uint32_t k_stage,
                       uint32_t v_stage) -> bool {
        // O of the previous item must have been read out before the first PV overwrites it
        if (i == 0 && !mbar_wait(bar(kBarOEmpty + x), (ni_x & 1) ^ 1, abort_flag)) return false;
        if (!mbar_wait(bar(kBarPFull + x), np_x & 1, abort_flag)) return false;
        ++np_x;
        tc_fence_after();
        issue_pv(x, v_stage, i == 0);
        if (i + 1 < n_tiles) {
          issue_qk(x, k_stage);
          if (i + 2 == n_tiles) umma_commit(bar(kBarQEmpty + x));
        } else {
          umma_commit(bar(kBarOFull + x));
        }
        return true;
      };
      while (ok && next_piece(sc, cache, n_pairs, wk, pc)) {
        for (int mp = rank; mp < p.n_mp && ok; mp += p.gang) {
          Item w;
          make_item(p, pc, gang_id, mp, w);
          if (w.n_tiles == 0) continue;
          // S of the first tile for both M tiles
          ok = mbar_wait(bar(kBarQFull + 0), ni0 & 1, abort_flag);
          if (ok && w.has_b) ok = mbar_wait(bar(kBarQFull + 1), ni1 & 1, abort_flag);
          if (ok) ok = mbar_wait(bar(kBarKFull + tk % KS), (tk / KS) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_qk(0, tk % KS);
          if (w.n_tiles == 1) umma_commit(bar(kBarQEmpty + 0));
          if (w.has_b) {
            issue_qk(1, tk % KS);
            if (w.n_tiles == 1) umma_commit(bar(kBarQEmpty + 1));
          }
          umma_commit(bar(kBarKEmpty + tk % KS));
          ++tk;
          for (int i = 0; i < w.n_tiles && ok; ++i) {
            const bool next = i + 1 < w.n_tiles;
            const uint32_t k_stage = tk % KS, v_stage = tv % VS;
            if (next) ok = mbar_wait(bar(kBarKFull + k_stage), (tk / KS) & 1, abort_flag);
            if (ok) ok = mbar_wait(bar(kBarVFull + v_stage), (tv / VS) & 1, abort_flag);
            if (ok) ok = chain(0, np0, ni0, i, w.n_tiles, k_stage, v_stage);
            if (ok && w.has_b) ok = chain(1, np1, ni1, i, w.n_tiles, k_stage, v_stage);
            if (!ok) break;
            umma_commit(bar(kBarVEmpty + v_stage));
            ++tv;
            if (next) {
              umma_commit(bar(kBarKEmpty + k_stage));
              ++tk;
            }
          }
          ++ni0;
          if (w.has_b) ++ni1;
        }
      }
      if (!ok) {
        umma_commit(bar(kBarDrain));
        mbar_wait(bar(kBarDrain), 0, abort_flag + 1);
      }
    }
    __syncwarp();
  } else if (FUSED && warp < 4) {
    // ------------------------------------------- loader: K/V tiles straight from the pool
    // A thread owns the same rotary pairs of every tile: pair c = lt + 64 u is row c / PPR,
    // 16-byte chunk jj = c % PPR of the low half and chunk jj + PPR of the high half, so its
    // eight frequencies never change and consecutive pairs are kRowStep positions apart: the
    // (cos, sin) of the first row come from the table, the others by one complex
    // multiplication with (cos, sin)(kRowStep * theta).  Copies are per-thread async copies
    // (no registers, zero fill for rows beyond the context), written in the 128-byte swizzle
    // the UMMA descriptors expect; K is rotated in place by the thread that copied it.
    constexpr int PPR = D / 16;
    constexpr int kRowStep = kLoaders / PPR;
    constexpr int PAIRS = kTileN / kRowStep;
    const int lt = threadIdx.x - 64;
    const int jj = lt % PPR, row0 = lt / PPR;
    uint32_t dst_off[2];                              // tile offsets of row 0's two chunks, before the row term
#pragma unroll
    for (int h = 0; h < 2; ++h) dst_off[h] = ((jj + h * PPR) / 8) * 16384u;
    float2 step[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const double theta = pow((double)p.rope_base_f, -(double)(jj * 8 + e) / (double)(D / 2));
      float sn, cs;
      rope_sincos((double)kRowStep, theta, &sn, &cs);
      step[e] = make_float2(cs, sn);
    }
    uint32_t tk = 0, tv = 0;
    bool ok = true;
    Walker wk = wk0;
    Piece pc;
    auto chunk_addr = [&](int row, int h) -> uint32_t {
      const int j = (jj + h * PPR) & 7;
      return dst_off[h] + row * 128u + ((j ^ (row & 7)) << 4);
    };
    auto issue = [&](const Item& w, int i, uint32_t sk, uint32_t sv) {
      const bool own = i >= w.n_ctx;
      const uint32_t k_base = base + SM::kOffK + sk * kTileBytes, v_base = base + SM::kOffV + sv * kTileBytes;
      long long src[PAIRS];                            // element offset of the row's head, -1: zero fill
#pragma unroll
      for (int u = 0; u < PAIRS; ++u) {
        const int row = row0 + u * kRowStep;
        if (!own) {
          const long long pos = (long long)(w.ctx_begin + i) * kTileN + row;
          const int r = pos < p.ctx_cap ? p.row_map[(long long)w.b * p.ctx_cap + pos] : -1;
          src[u] = r < 0 ? -1 : (((long long)(p.layer_begin + w.l) * p.pool_tokens + r) * p.Hkv + w.g) * D;
        } else {
          const int t = (w.own_begin + i - w.n_ctx) * kTileN + row;
          src[u] = t >= p.To ? -1 : (((long long)w.outer_own * p.To + t) * p.Hkv + w.g) * D;
        }
      }
      const __nv_bfloat16* kb = own ? p.kq_rot : p.k_pool;
      const __nv_bfloat16* vb = own ? p.vq : p.v_pool;
#pragma unroll
      for (int u = 0; u < PAIRS; ++u) {
        const int row = row0 + u * kRowStep;
        const uint32_t n = src[u] < 0 ? 0u : 16u;
        const __nv_bfloat16* g = kb + (src[u] < 0 ? 0 : src[u]) + jj * 8;
        cp_async16(k_base + chunk_addr(row, 0), g, n);
        cp_async16(k_base + chunk_addr(row, 1), g + D / 2, n);
      }
      cp_async_commit();
#pragma unroll
      for (int u = 0; u < PAIRS; ++u) {
        const int row = row0 + u * kRowStep;
        const uint32_t n = src[u] < 0 ? 0u : 16u;
        const __nv_bfloat16* g = vb + (src[u] < 0 ? 0 : src[u]) + jj * 8;
        cp_async16(v_base + chunk_addr(row, 0), g, n);
        cp_async16(v_base + chunk_addr(row, 1), g + D / 2, n);
      }
      cp_async_commit();
    };
    auto rotate = [&](const Item& w, int i, uint32_t sk) {
      unsigned char* kt = base_ptr + SM::kOffK + sk * kTileBytes;
      const long long pos0 = (long long)(w.ctx_begin + i) * kTileN + row0;
      float2 cur[8];
      auto load_angles = [&](long long table_row) {
        const float4* tab = reinterpret_cast<const float4*>(p.rope_tab + table_row * (D / 2) + jj * 8);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float4 t4 = tab[e];
          cur[2 * e] = make_float2(t4.x, t4.y);
          cur[2 * e + 1] = make_float2(t4.z, t4.w);
        }
      };
      const bool per_shot = p.k_pos_mode == 1;     // the angle is that of the shot's first position
      if (!per_shot) load_angles(pos0);
#pragma unroll
      for (int u = 0; u < PAIRS; ++u) {
        const int row = row0 + u * kRowStep;
        uint4* lo = reinterpret_cast<uint4*>(kt + chunk_addr(row, 0));
        uint4* hi = reinterpret_cast<uint4*>(kt + chunk_addr(row, 1));
        if (per_shot) {
          const long long pos = pos0 + u * kRowStep;
          load_angles(pos < p.ctx_cap ? p.off_map[(long long)w.b * p.ctx_cap + pos] : 0);
        }
        float x[8], y[8], xr[8], yr[8];
        bf16x8_unpack(*lo, x);
        bf16x8_unpack(*hi, y);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          xr[e] = x[e] * cur[e].x - y[e] * cur[e].y;
          yr[e] = y[e] * cur[e].x + x[e] * cur[e].y;
        }
        *lo = bf16x8_pack(xr);
        *hi = bf16x8_pack(yr);
        if (!per_shot && u + 1 < PAIRS) {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float c = cur[e].x * step[e].x - cur[e].y * step[e].y;
            const float sn = cur[e].y * step[e].x + cur[e].x * step[e].y;
            cur[e] = make_float2(c, sn);
          }
        }
      }
    };
    while (ok && next_piece(sc, cache, n_pairs, wk, pc)) {
      for (int mp = rank; mp < p.n_mp && ok; mp += p.gang) {
        Item w;
        make_item(p, pc, gang_id, mp, w);
        if (w.n_tiles == 0) continue;
        ok = mbar_wait(bar(kBarKEmpty + tk % KS), ((tk / KS) & 1) ^ 1, abort_flag) &&
             mbar_wait(bar(kBarVEmpty + tv % VS), ((tv / VS) & 1) ^ 1, abort_flag);
        if (!ok) break;
        issue(w, 0, tk % KS, tv % VS);
        for (int i = 0; i < w.n_tiles; ++i) {
          const uint32_t sk = tk % KS, sv = tv % VS;
          const bool next = i + 1 < w.n_tiles;
          if (next) {
            ok = mbar_wait(bar(kBarKEmpty + (tk + 1) % KS), (((tk + 1) / KS) & 1) ^ 1, abort_flag) &&
                 mbar_wait(bar(kBarVEmpty + (tv + 1) % VS), (((tv + 1) / VS) & 1) ^ 1, abort_flag);
            if (!ok) break;
            issue(w, i + 1, (tk + 1) % KS, (tv + 1) % VS);
            cp_async_wait<3>();                         // K of tile i has landed
          } else {
            cp_async_wait<1>();
          }
          if (i < w.n_ctx) rotate(w, i, sk);
          fence_proxy_async_smem();
          mbar_arrive(bar(kBarKFull + sk));
          if (next) cp_async_wait<2>(); else cp_async_wait<0>();   // V of tile i
          fence_proxy_async_smem();
          mbar_arrive(bar(kBarVFull + sv));
          ++tk;
          ++tv;
        }
      }
    }
    cp_async_wait<0>();
  } else if (VPOOL && warp == kGatherWarp) {
    // ----------------------------------------------- V tiles straight from the pool, stitched by TMA
    // Eq. 7 corrects K only, so V needs no assembled copy.  The 128 context positions of a tile map
    // to a few runs of consecutive pool rows (one per selected shot the tile touches): the lanes look
    // the positions up and mark where a run ends; every run is brought as one or two power-of-two boxes
    // (maps with 128, 64, ..., 1-row boxes over the pool; a box may start at any row, its shared-memory
    // address only has to be 128-byte aligned), one box per lane, all found before the stage is waited
    // for.  Positions beyond the context continue the last run (their P is exactly zero; rows outside
    // the pool arrive as zeros).  The probe's own tokens are one run of the own-token tensor.
    int* rows_s = reinterpret_cast<int*>(base_ptr + SM::kOffRows);
    uint32_t tv = 0;
    bool ok = true;
    Walker wk = wk0;
    Piece pc;
    if (lane == 0) {
      tma_prefetch_desc(&tm_vown);
#pragma unroll
      for (int e = 0; e < 8; ++e) tma_prefetch_desc(&vmaps.m[e]);
    }
    while (ok && next_piece(sc, cache, n_pairs, wk, pc)) {
      for (int mp = rank; mp < p.n_mp && ok; mp += p.gang) {
        Item w;
        make_item(p, pc, gang_id, mp, w);
        for (int i = 0; i < w.n_tiles; ++i, ++tv) {
          const uint32_t sv = tv % VS;
          const uint32_t v_dst = base + SM::kOffV + sv * kTileBytes;
          if (i >= w.n_ctx) {
            // own tokens: one tiled box (rows beyond the last own token arrive as zeros)
            if (lane == 0) {
              ok = mbar_wait(bar(kBarVEmpty + sv), ((tv / VS) & 1) ^ 1, abort_flag);
              if (ok) {
                mbar_arrive_expect_tx(bar(kBarVFull + sv), kTileBytes);
#pragma unroll
                for (int s2 = 0; s2 < SUB; ++s2)
                  tma_load_4d(v_dst + s2 * 16384u, &tm_vown, bar(kBarVFull + sv), s2 * 64, w.g,
                              (w.own_begin + i - w.n_ctx) * kTileN, w.outer_own);
              }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            continue;
          }
          // pool row of positions lane, lane + 32, lane + 64, lane + 96 of the tile (looked up while the
          // stage may still be in use); beyond the context the last run is continued
          const long long pos0 = (long long)(w.ctx_begin + i) * kTileN;
          const long long L_all = p.ctx_cap;            // (row map entries beyond a query's context are -1)
          int r[4];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const long long pos = pos0 + lane + 32 * q4;
            r[q4] = pos < L_all ? p.row_map[(long long)w.b * p.ctx_cap + pos] : -1;
          }
          // the number of valid positions of the tile: they form a prefix (valid positions are 0 .. L-1)
          unsigned valid_mask[4];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) valid_mask[q4] = __ballot_sync(0xffffffffu, r[q4] >= 0);
          const int n_valid = __popc(valid_mask[0]) + __popc(valid_mask[1]) + __popc(valid_mask[2]) + __popc(valid_mask[3]);
          __syncwarp();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) rows_s[lane + 32 * q4] = r[q4];
          __syncwarp();
          const int last_row = n_valid > 0 ? rows_s[n_valid - 1] : 0;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int pidx = lane + 32 * q4;
            if (pidx >= n_valid) r[q4] = last_row + (pidx - n_valid + 1);
          }
          __syncwarp();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) rows_s[lane + 32 * q4] = r[q4];
          // a run ends after position pidx when the next position is not the next pool row
          unsigned brk[4];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            int nxt = __shfl_down_sync(0xffffffffu, r[q4], 1);
            const int wrap = __shfl_sync(0xffffffffu, q4 < 3 ? r[q4 + 1 < 4 ? q4 + 1 : 3] : 0, 0);
            if (lane == 31) nxt = wrap;
            const bool last = lane == 31 && q4 == 3;
            brk[q4] = __ballot_sync(0xffffffffu, last || nxt != r[q4] + 1);
          }
          // the run ends as one 128-bit mask in every lane; lane j then finds the j-th box on its own.
          // A run of n rows takes the largest power-of-two box that fits, once from its first row and,
          // unless n is that power of two, once more ending at its last row: the two overlap, both write
          // the same values there, and no run needs more than two copy instructions (the copy engine's
          // time goes with the number of instructions, not with the bytes)
          __syncwarp();
          int my_pidx = -1, my_row = 0, my_lg = 0, n_boxes = 0;
          uint32_t tile_bytes = 0;                 // what the boxes deliver in all (overlaps are copied twice)
          {
            int pidx = 0;
            while (pidx < kTileN) {
              int e = pidx;                       // end of the run that starts at pidx: first set bit at or after it
              for (;;) {
                const unsigned word = (e < 32 ? brk[0] : e < 64 ? brk[1] : e < 96 ? brk[2] : brk[3]) >> (e & 31);
                if (word != 0) { e += __ffs(word) - 1; break; }
                e = (e | 31) + 1;
              }
              const int n = e - pidx + 1;
              const int lg = 31 - __clz(n);        // the largest power-of-two box that fits
              if (n_boxes == lane) { my_pidx = pidx; my_lg = lg; }
              ++n_boxes;
              if (n > (1 << lg)) {                 // the rest of the run: the same box once more, ending at the run's end
                if (n_boxes == lane) { my_pidx = e + 1 - (1 << lg); my_lg = lg; }
                ++n_boxes;
              }
              tile_bytes += (n > (1 << lg) ? 2u : 1u) * ((uint32_t)SUB << (lg + 7));
              pidx = e + 1;
            }
          }
          if (my_pidx >= 0) my_row = rows_s[my_pidx];
          // (tiles of more than 32 boxes - many one-token shots - take further rounds of the same walk)
          if (lane == 0) {
            ok = mbar_wait(bar(kBarVEmpty + sv), ((tv / VS) & 1) ^ 1, abort_flag);
            if (ok) mbar_arrive_expect_tx(bar(kBarVFull + sv), tile_bytes);
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
          const int layer = p.layer_begin + w.l;
          if (my_pidx >= 0) {
#pragma unroll
            for (int s2 = 0; s2 < SUB; ++s2)
              tma_load_4d(v_dst + s2 * 16384u + (uint32_t)my_pidx * 128u, &vmaps.m[my_lg], bar(kBarVFull + sv), s2 * 64,
                          w.g, my_row, layer);
          }
          for (int round = 1; round * 32 < n_boxes; ++round) {      // rare: more than 32 boxes in the tile
            int pidx = 0, idx = 0, bp = -1, bl = 0;
            while (pidx < kTileN) {
              int e = pidx;
              for (;;) {
                const unsigned word = (e < 32 ? brk[0] : e < 64 ? brk[1] : e < 96 ? brk[2] : brk[3]) >> (e & 31);
                if (word != 0) { e += __ffs(word) - 1; break; }
                e = (e | 31) + 1;
              }
              const int n = e - pidx + 1;
              const int lg = 31 - __clz(n);
              if (idx == round * 32 + lane) { bp = pidx; bl = lg; }
              ++idx;
              if (n > (1 << lg)) {
                if (idx == round * 32 + lane) { bp = e + 1 - (1 << lg); bl = lg; }
                ++idx;
              }
              pidx = e + 1;
            }
            if (bp >= 0) {
              const int brow = rows_s[bp];
#pragma unroll
              for (int s2 = 0; s2 < SUB; ++s2)
                tma_load_4d(v_dst + s2 * 16384u + (uint32_t)bp * 128u, &vmaps.m[bl], bar(kBarVFull + sv), s2 * 64, w.g,
                            brow, layer);
            }
          }
          __syncwarp();
        }
      }
    }
    if (!ok && lane == 0) {
      // gave up: let the copies already in flight land before the CTA retires
      for (uint32_t t = tv > (uint32_t)VS ? tv - VS : 0; t < tv; ++t)
        mbar_wait(bar(kBarVFull + t % VS), (t / VS) & 1, abort_flag + 1);
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------- softmax + read-out of O
    const int x = (warp - kSoftmaxWarp0) >> 2;     // 0: M tile A, 1: M tile B
    const int quarter = warp & 3;                  // TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;             // row of the M tile
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_addr + kTmemS + x * kTileN;
    const uint32_t o_addr = tmem_base + lane_addr + kTmemO + x * 128;
    uint32_t ns = 0, ni = 0;
    bool ok = true;
    Walker wk = wk0;
    Piece pc;
    while (ok && next_piece(sc, cache, n_pairs, wk, pc)) {
      for (int mp = rank; mp < p.n_mp && ok; mp += p.gang) {
        Item w;
        make_item(p, pc, gang_id, mp, w);
        if (x == 1 && !w.has_b) continue;
        const int mt = 2 * mp + x;
        const int m = mt * kTileM + r;               // row of the unit: token m / G, head m % G
        const int t_row = m / p.G;
        float m_used = kNegSentinel, l_sum = 0.f;
        for (int i = 0; i < w.n_tiles; ++i, ++ns) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull + x), ns & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          float s[kTileN];
          tmem_ld128(s_addr, reinterpret_cast<uint32_t*>(s));

          // mask: context keys at or beyond L_j; own keys after the row's token (causal).
          // Only the last context tile and the own-token tiles can hide anything.
          int limit = kTileN;                          // columns < limit are visible
          if (i < w.n_ctx) {
            const long long first = (long long)(w.ctx_begin + i) * kTileN;
            if (first + kTileN > w.Lj) limit = (int)(w.Lj - first);
          } else {
            limit = p.To - p.Tq + min(t_row, p.Tq - 1) - (w.own_begin + i - w.n_ctx) * kTileN + 1;   // <= 0: all hidden
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
          // the packed pair c2 goes into the register that held score c2 (already consumed:
          // c2 <= 2 c2), so the row never needs more than its 128 registers
          uint32_t* pk = reinterpret_cast<uint32_t*>(s);
#pragma unroll
          for (int c2 = 0; c2 < kTileN / 2; ++c2) {
            const float2 xs = __ffma2_rn(make_float2(s[2 * c2], s[2 * c2 + 1]), scale2, neg_m2);
            const float2 e = make_float2(ex2_approx(xs.x), ex2_approx(xs.y));
            part[c2 & 3] = __fadd2_rn(part[c2 & 3], e);
            pk[c2] = pack_bf16x2(e.x, e.y);
          }
          const float2 tot = __fadd2_rn(__fadd2_rn(part[0], part[1]), __fadd2_rn(part[2], part[3]));
          l_sum += tot.x + tot.y;
          tmem_st64(s_addr, pk);
          if (i > 0 && __any_sync(0xffffffffu, need)) {
            // S(i) is complete, so PV(i-1), issued before it, is complete too; PV(i) waits for
            // the arrival below: O is quiescent here.
#pragma unroll
            for (int q4 = 0; q4 < D / 32; ++q4) {
              float o[32];
              tmem_ld32(o_addr + q4 * 32, reinterpret_cast<uint32_t*>(o));
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] *= alpha;
              tmem_st32(o_addr + q4 * 32, reinterpret_cast<const uint32_t*>(o));
            }
          }
          tc_fence_before();
          mbar_arrive(bar(kBarPFull + x));
        }
        if (!ok) break;
        const bool row_ok = m < p.Tq * p.G;
        if (w.n_tiles == 0) {
          // nothing of this M pair falls into the piece: a neutral partial (a whole unit is never empty)
          float4* otile = reinterpret_cast<float4*>(p.o_part) + (w.slot * 2 + x) * (long long)(D / 4) * kTileM + r;
#pragma unroll
          for (int c4 = 0; c4 < D / 4; ++c4) otile[c4 * kTileM] = make_float4(0.f, 0.f, 0.f, 0.f);
          float* ml = p.ml_part + ((w.slot * 2 + x) * kTileM + r) * 2;
          ml[0] = kNegSentinel;
          ml[1] = 0.f;
          continue;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarOFull + x), ni & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (w.whole) {
          // The piece covers the unit: normalise and store the final rows.  A thread owns a
          // row, and rows are far apart in the output, so a direct store would touch 32 lines
          // per instruction; instead the warp passes 64 columns at a time through its staging
          // area (16-byte chunks swizzled by the row) and writes four rows' 128-byte segments
          // per instruction.
          const float inv = 1.f / l_sum;
          const long long bpj = w.outer_own;
          unsigned char* stg = base_ptr + SM::kOffStage + (warp - kSoftmaxWarp0) * SM::kStageBytes;
          const int sub = lane >> 3, ch = lane & 7;            // read-back: row 4 j + sub, chunk ch
          const int m0 = mt * kTileM + quarter * 32;
          if constexpr (FUSED) {
            // (no staging area in the fused variant's shared-memory plan: one row per thread)
            const int hq = w.g * p.G + m % p.G;
            __nv_bfloat16* dst = p.out + (((bpj * p.Tq + t_row) * p.Hq) + hq) * (long long)D;
#pragma unroll
            for (int q4 = 0; q4 < D / 32; ++q4) {
              float o[32];
              tmem_ld32(o_addr + q4 * 32, reinterpret_cast<uint32_t*>(o));
              if (q4 == D / 32 - 1) {
                tc_fence_before();
                mbar_arrive(bar(kBarOEmpty + x));
              }
              if (row_ok) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                  float v8[8];
#pragma unroll
                  for (int u = 0; u < 8; ++u) v8[u] = o[e + u] * inv;
                  *reinterpret_cast<uint4*>(dst + q4 * 32 + e) = bf16x8_pack(v8);
                }
              }
            }
          } else {
#pragma unroll
          for (int h = 0; h < D / 64; ++h) {
            float o[64];
            tmem_ld32(o_addr + h * 64, reinterpret_cast<uint32_t*>(o));
            tmem_ld32(o_addr + h * 64 + 32, reinterpret_cast<uint32_t*>(o + 32));
            if (h == D / 64 - 1) {             // O is in registers: the next item may overwrite it
              tc_fence_before();
              mbar_arrive(bar(kBarOEmpty + x));
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              float v8[8];
#pragma unroll
              for (int u = 0; u < 8; ++u) v8[u] = o[c * 8 + u] * inv;
              *reinterpret_cast<uint4*>(stg + lane * 128 + ((c ^ (lane & 7)) << 4)) = bf16x8_pack(v8);
            }
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int row = 4 * j + sub;
              const int mm = m0 + row;
              const uint4 v = *reinterpret_cast<const uint4*>(stg + row * 128 + ((ch ^ (row & 7)) << 4));
              if (mm < p.Tq * p.G) {
                const int tt = mm / p.G, hq = w.g * p.G + mm % p.G;
                __nv_bfloat16* dst = p.out + (((bpj * p.Tq + tt) * p.Hq) + hq) * (long long)D;
                *reinterpret_cast<uint4*>(dst + h * 64 + ch * 8) = v;
              }
            }
            __syncwarp();
          }
          }
          if (row_ok && p.lse != nullptr) {
            const int hh = m % p.G, hq = w.g * p.G + hh;
            p.lse[(bpj * p.Hq + hq) * p.Tq + t_row] = (m_used + log2f(l_sum)) * kLn2;
          }
        } else {
          // un-normalised partial, four columns of 128 rows at a time ([D/4][128][4] per M tile):
          // a warp's 32 rows are 512 contiguous bytes per store
          float4* otile = reinterpret_cast<float4*>(p.o_part) + (w.slot * 2 + x) * (long long)(D / 4) * kTileM + r;
#pragma unroll
          for (int q4 = 0; q4 < D / 32; ++q4) {
            float o[32];
            tmem_ld32(o_addr + q4 * 32, reinterpret_cast<uint32_t*>(o));
            if (q4 == D / 32 - 1) {
              tc_fence_before();
              mbar_arrive(bar(kBarOEmpty + x));
            }
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              otile[(q4 * 8 + e / 4) * kTileM] = make_float4(o[e], o[e + 1], o[e + 2], o[e + 3]);
          }
          float* ml = p.ml_part + ((w.slot * 2 + x) * kTileM + r) * 2;
          ml[0] = m_used;
          ml[1] = l_sum;
        }
        ++ni;
      }
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
  const Sched* sched;
  const float* o_part;
  const float* ml_part;
  __nv_bfloat16* out;   // [B][nl][P][Tq][Hq][D]
  float* lse;           // [B][nl][P][Hq][Tq] or null
  int B, P, Tq, Hq, Hkv, G, nl, n_mp, n_gangs;
};

constexpr int kCombineRows = 8;      // rows per warp

// Block (q, y): if the range of gang q ends inside a unit that starts in that range, the
// unit was cut; its pieces sit with gangs q .. q_last.  One warp merges eight rows.
template <int D>
__global__ void __launch_bounds__(256) attn_combine_kernel(const CombineParams p) {
  const Sched* sc = p.sched;
  const int q = blockIdx.x;
  const long long total = sc->total;
  const long long cut = sc->start[q + 1];
  if (cut >= total) return;
  const int n_pairs = p.P * p.B;
  const int pair = find_pair(sc, n_pairs, cut);
  const int nsu = sc->n_su[pair];
  const long long rel = cut - sc->prefix[pair];
  if (rel % nsu == 0) return;                       // the cut falls between two units
  const int su = (int)(rel / nsu);
  const long long s_u = sc->prefix[pair] + (long long)su * nsu, e_u = s_u + nsu;
  if (s_u < sc->start[q]) return;                   // an earlier gang holds the unit's first piece
  int q_last = q + 1;                               // last gang whose range begins inside the unit
  while (q_last + 1 < p.n_gangs && sc->start[q_last + 1] < e_u) ++q_last;

  const int lane = threadIdx.x & 31;
  const int j = p.P - 1 - pair / p.B, b = pair % p.B;
  const int l = su / p.Hkv, g = su % p.Hkv;
  const long long bpj = ((long long)b * p.nl + l) * p.P + j;
  // A warp merges 8 rows: lane = (row r_sub, 4-column chunk c_sub of the 16 columns of one
  // step), so that a load is 8 rows x 16 bytes contiguous per chunk in the partial layout
  // ([D/4][128 rows][4] per M tile) and a store fills one 32-byte sector per row.
  const int r_sub = lane & 7, c_sub = lane >> 3;
  const int m = (blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5)) * kCombineRows + r_sub;
  if (m >= p.Tq * p.G) return;
  const int mt = m / kTileM, r = m % kTileM, mp = mt >> 1, x = mt & 1;
  const int t = m / p.G, hh = m % p.G, h = g * p.G + hh;
  auto slot_tile = [&](int qq) -> long long {
    const int which = sc->start[qq] >= s_u ? 0 : 1;           // the gang's first piece, or its last
    return ((long long)(2 * qq + which) * p.n_mp + mp) * 2 + x;
  };
  // (when there are fewer tiles than gangs, empty ranges lie between the pieces)
  auto has_piece = [&](int qq) -> bool { return sc->start[qq] < sc->start[qq + 1]; };
  float M = kNegSentinel;
  for (int qq = q; qq <= q_last; ++qq)
    if (has_piece(qq)) M = fmaxf(M, p.ml_part[(slot_tile(qq) * kTileM + r) * 2]);
  const float4* o4 = reinterpret_cast<const float4*>(p.o_part);
  float4 acc[D / 16];
#pragma unroll
  for (int it = 0; it < D / 16; ++it) acc[it] = make_float4(0.f, 0.f, 0.f, 0.f);
  float lsum = 0.f;
  for (int qq = q; qq <= q_last; ++qq) {
    if (!has_piece(qq)) continue;
    const long long tile = slot_tile(qq);
    const float* ml = p.ml_part + (tile * kTileM + r) * 2;
    const float wgt = exp2f(ml[0] - M);
    lsum += ml[1] * wgt;
    float4 v[D / 16];
#pragma unroll
    for (int it = 0; it < D / 16; ++it) v[it] = o4[(tile * (D / 4) + it * 4 + c_sub) * kTileM + r];
#pragma unroll
    for (int it = 0; it < D / 16; ++it) {
      acc[it].x += v[it].x * wgt; acc[it].y += v[it].y * wgt;
      acc[it].z += v[it].z * wgt; acc[it].w += v[it].w * wgt;
    }
  }
  const float inv = 1.f / lsum;
  __nv_bfloat16* dst = p.out + (((bpj * p.Tq + t) * p.Hq) + h) * (long long)D;
#pragma unroll
  for (int it = 0; it < D / 16; ++it) {
    uint2 packed;
    packed.x = pack_bf16x2(acc[it].x * inv, acc[it].y * inv);
    packed.y = pack_bf16x2(acc[it].z * inv, acc[it].w * inv);
    *reinterpret_cast<uint2*>(dst + (it * 4 + c_sub) * 4) = packed;
  }
  if (p.lse != nullptr && c_sub == 0)
    p.lse[(bpj * p.Hq + h) * p.Tq + t] = (M + log2f(lsum)) * kLn2;
}

// Self-test of the bounded wait every pipeline barrier uses: warp 0 waits (with a limit of about a
// millisecond) on a barrier that nothing will ever complete, gives up, raises the CTA's abort flag
// and reports ADAPSHOT_ETIMEOUT; warp 1 waits on the same barrier with the long limit and must
// return as soon as it sees the flag.  The kernel ends normally: the context stays usable.
__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(int32_t* status, long long* cycles) {
  __shared__ __align__(8) unsigned long long barmem;
  __shared__ int abort_flag[2];
  const uint32_t b = smem_u32(&barmem);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    abort_flag[0] = abort_flag[1] = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait_limit(b, 0, abort_flag, 2000000ll);
  if (threadIdx.x == 32) ok = mbar_wait(b, 0, abort_flag);
  if ((threadIdx.x & 31) == 0) cycles[threadIdx.x >> 5] = ok ? -1 : clock64() - t0;
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag[0] != 0) ads_set_status(status, ADAPSHOT_ETIMEOUT);
}

// ----------------------------------------------------------------- host side
// bf16 tensor, innermost dim contiguous, 128-byte swizzle, zero fill outside the bounds
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box) {
  return ads_make_bf16_map(m, base, rank, dims, strides_bytes, box);
}

// Optional timing of the main kernel alone (adapshot_profile): two events around its launch.
bool g_profile = false;
bool g_profile_valid = false;
cudaEvent_t g_profile_ev[2] = {nullptr, nullptr};

struct AttnPlan {
  int n_mt, n_mp, gang;
  size_t off_qrot, off_kqrot, off_sched, off_opart, off_ml, off_rowmap, off_offmap, off_tab, total;
  long long tab_rows;
};

// Own tokens beyond the query rows, and a per-query shot count on the device (decode calls).
struct AttnExtra {
  int To = 0;                        // 0: as many own tokens as query rows
  const int32_t* nshots_dev = nullptr;
};

// What the fused variant reads instead of an assembled cache.
struct FusedSrc {
  const adapshot_pool_t* pool;
  const int32_t* sel_idx;
  int layer_begin;
};

// The gang (CTAs that walk the same K/V tiles, one M pair each per round) is the number of
// M pairs when that is at most kMaxGang, else the M pairs are dealt out in rounds.
AttnPlan make_plan(const adapshot_model_t* model, int B, int P, int Tq, int nl, long long fused_ctx_cap = 0,
                   bool with_table = true, int To = 0) {
  if (To < Tq) To = Tq;
  AttnPlan pl;
  const int G = model->n_q_heads / model->n_kv_heads;
  const int D = model->head_dim;
  pl.n_mt = (Tq * G + kTileM - 1) / kTileM;
  pl.n_mp = (pl.n_mt + 1) / 2;
  const int rounds = (pl.n_mp + kMaxGang - 1) / kMaxGang;
  pl.gang = (pl.n_mp + rounds - 1) / rounds;
  const size_t slots = (size_t)2 * kMaxCtas * pl.n_mp;     // two cut pieces per gang at most
  size_t off = 0;
  pl.off_qrot = off;  off += ads_round_up((size_t)B * nl * P * Tq * model->n_q_heads * D * 2, 256);
  pl.off_kqrot = off; off += ads_round_up((size_t)B * nl * P * To * model->n_kv_heads * D * 2, 256);
  pl.off_sched = off; off += ads_round_up(sizeof(Sched), 256);
  pl.off_opart = off; off += ads_round_up(slots * 2 * kTileM * D * 4, 256);
  pl.off_ml = off;    off += ads_round_up(slots * 2 * kTileM * 2 * 4, 256);
  pl.off_rowmap = pl.off_offmap = pl.off_tab = off;
  pl.tab_rows = 0;
  if (fused_ctx_cap > 0) {
    pl.tab_rows = with_table ? (fused_ctx_cap + kTileN - 1) / kTileN * kTileN : 0;
    pl.off_rowmap = off; off += ads_round_up((size_t)B * fused_ctx_cap * 4, 256);
    pl.off_offmap = off; off += ads_round_up((size_t)B * fused_ctx_cap * 4, 256);
    pl.off_tab = off;    off += ads_round_up((size_t)pl.tab_rows * (D / 2) * 8, 256);
  }
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
                void* ws, int32_t* status, cudaStream_t st, const FusedSrc* fused = nullptr,
                int mode = kModeCache, AttnExtra extra = AttnExtra()) {
  const int To = extra.To > Tq ? extra.To : Tq;
  const int Hq = model->n_q_heads, Hkv = model->n_kv_heads, G = Hq / Hkv;
  unsigned char* wsb = static_cast<unsigned char*>(ws);
  __nv_bfloat16* q_rot = reinterpret_cast<__nv_bfloat16*>(wsb + pl.off_qrot);
  __nv_bfloat16* kq_rot = reinterpret_cast<__nv_bfloat16*>(wsb + pl.off_kqrot);
  Sched* sched = reinterpret_cast<Sched*>(wsb + pl.off_sched);
  float* o_part = reinterpret_cast<float*>(wsb + pl.off_opart);
  float* ml_part = reinterpret_cast<float*>(wsb + pl.off_ml);

  const int n_sm = ads_sm_count();
  if (n_sm <= 0) return ADAPSHOT_ECUDA;
  const int n_cta = n_sm < kMaxCtas ? n_sm : kMaxCtas;
  const int n_gangs = n_cta / pl.gang > 0 ? n_cta / pl.gang : 1;

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
    tm_kctx = tm_q;                    // (a map the mode never uses: its loader warps read the pool)
    tm_vctx = tm_q;
    if (mode != kModeFused && !make_map(&tm_kctx, k_ctx, 4, dims, str, box)) return ADAPSHOT_ECUDA;
    if (mode == kModeCache && !make_map(&tm_vctx, v_ctx, 4, dims, str, box)) return ADAPSHOT_ECUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)Hkv, (uint64_t)To, (uint64_t)B * nl * P};
    const uint64_t str[3] = {(uint64_t)D * 2, (uint64_t)Hkv * D * 2, (uint64_t)To * Hkv * D * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)kTileN, 1};
    if (!make_map(&tm_kown, kq_rot, 4, dims, str, box)) return ADAPSHOT_ECUDA;
    if (!make_map(&tm_vown, vq, 4, dims, str, box)) return ADAPSHOT_ECUDA;
  }
  VPoolMaps vmaps;
  for (int e = 0; e < 8; ++e) vmaps.m[e] = tm_q;       // (unused outside the V-from-pool variant)
  if (mode == kModeVPool) {
    // the pool's V with boxes of 1, 2, ..., 128 rows (the layout of the cache maps, over the pool)
    const uint64_t pt = (uint64_t)fused->pool->pool_tokens;
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)Hkv, pt, (uint64_t)model->n_layers};
    const uint64_t str[3] = {(uint64_t)D * 2, (uint64_t)Hkv * D * 2, pt * Hkv * D * 2};
    for (int e = 0; e < 8; ++e) {
      const uint32_t box[4] = {64, 1, 1u << e, 1};
      if (!make_map(&vmaps.m[e], fused->pool->v, 4, dims, str, box)) return ADAPSHOT_ECUDA;
    }
  }

  // ---- fused variant: row map and rotary table
  int* row_map = reinterpret_cast<int*>(wsb + pl.off_rowmap);
  int* off_map = reinterpret_cast<int*>(wsb + pl.off_offmap);
  float2* rope_tab = reinterpret_cast<float2*>(wsb + pl.off_tab);
  if (fused != nullptr) {
    FusedPlanParams fp;
    fp.ctx_off = reinterpret_cast<const long long*>(ctx_off);
    fp.sel_idx = fused->sel_idx;
    fp.shot_off = reinterpret_cast<const long long*>(fused->pool->shot_off);
    fp.row_map = row_map; fp.off_map = off_map; fp.rope_tab = rope_tab;
    fp.ctx_cap = ctx_cap; fp.tab_rows = pl.tab_rows;
    fp.B = B; fp.k = k; fp.n_shots = fused->pool->n_shots; fp.half_d = D / 2;
    fp.rope_base = model->rope_base;
    const long long work = (long long)B * ctx_cap + pl.tab_rows * (D / 2);
    long long blocks = (work + 255) / 256;
    if (blocks > n_sm * 16) blocks = n_sm * 16;
    attn_fused_plan_kernel<<<(unsigned)blocks, 256, 0, st>>>(fp);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  }

  // ---- rotate Q and the probe's own K, write the schedule
  PrepParams pp;
  pp.q = static_cast<const __nv_bfloat16*>(q); pp.kq = static_cast<const __nv_bfloat16*>(kq);
  pp.q_rot = q_rot; pp.kq_rot = kq_rot; pp.ctx_off = reinterpret_cast<const long long*>(ctx_off);
  pp.sched = sched; pp.ctx_cap = ctx_cap;
  pp.B = B; pp.k = k; pp.P = P; pp.Tq = Tq; pp.Hq = Hq; pp.Hkv = Hkv; pp.nl = nl; pp.n_gangs = n_gangs;
  pp.To = To; pp.nshots_dev = extra.nshots_dev; pp.status = status;
  pp.rope_base = model->rope_base;
  for (int i = 0; i < D / 2; ++i) pp.theta[i] = pow(model->rope_base, -2.0 * (double)i / (double)D);
  for (int i = 0; i < kMaxProbes; ++i) pp.nshots[i] = i < P ? probe_nshots[i] : 0;
  const long long n_tok = (long long)B * nl * P * To;
  attn_prep_kernel<D><<<(unsigned)((n_tok * kPrepParts + 7) / 8) + 1, 256, 0, st>>>(pp);   // + the schedule block
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  // ---- main kernel
  AttnParams ap = {};
  ap.sched = sched; ap.o_part = o_part; ap.ml_part = ml_part;
  ap.out = static_cast<__nv_bfloat16*>(out); ap.lse = lse; ap.status = status;
  ap.B = B; ap.P = P; ap.Tq = Tq; ap.Hq = Hq; ap.Hkv = Hkv; ap.G = G; ap.nl = nl; ap.To = To;
  ap.n_mt = pl.n_mt; ap.n_mp = pl.n_mp; ap.gang = pl.gang; ap.n_gangs = n_gangs;
  const float scale = model->softmax_scale > 0.f ? model->softmax_scale : 1.0f / sqrtf((float)D);
  ap.scale_log2 = scale * 1.4426950408889634f;
  // the same request for D = 64 as for D = 128: one CTA per SM in every variant
  const int smem = mode == kModeVPool ? (int)AttnSmem<128, kModeVPool>::kTotal : (int)AttnSmem<128, kModeCache>::kTotal;
  static bool attr_done[3][kAdsMaxDevices] = {{false}, {false}, {false}};   // per template instance (D, mode) and device
  if (g_profile) ADS_CHECK_CUDA(cudaEventRecord(g_profile_ev[0], st));
  if (mode == kModeCache) {
    if (ads_set_max_smem(attn_main_kernel<D, kModeCache>, smem, attr_done[0]) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
    attn_main_kernel<D, kModeCache><<<(unsigned)(n_gangs * pl.gang), kAttnThreads, smem, st>>>(
        tm_q, tm_kctx, tm_vctx, tm_kown, tm_vown, vmaps, ap);
  } else {
    ap.k_pool = static_cast<const __nv_bfloat16*>(fused->pool->k);
    ap.v_pool = static_cast<const __nv_bfloat16*>(fused->pool->v);
    ap.kq_rot = kq_rot;
    ap.vq = static_cast<const __nv_bfloat16*>(vq);
    ap.row_map = row_map; ap.off_map = off_map; ap.k_pos_mode = model->k_pos_mode; ap.rope_tab = rope_tab;
    ap.pool_tokens = fused->pool->pool_tokens; ap.ctx_cap = ctx_cap;
    ap.layer_begin = fused->layer_begin; ap.rope_base_f = model->rope_base;
    if (mode == kModeFused) {
      if (ads_set_max_smem(attn_main_kernel<D, kModeFused>, smem, attr_done[1]) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
      attn_main_kernel<D, kModeFused><<<(unsigned)(n_gangs * pl.gang), kFusedThreads, smem, st>>>(
          tm_q, tm_kctx, tm_vctx, tm_kown, tm_vown, vmaps, ap);
    } else {
      if (ads_set_max_smem(attn_main_kernel<D, kModeVPool>, smem, attr_done[2]) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
      attn_main_kernel<D, kModeVPool><<<(unsigned)(n_gangs * pl.gang), kVPoolThreads, smem, st>>>(
          tm_q, tm_kctx, tm_vctx, tm_kown, tm_vown, vmaps, ap);
    }
  }
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  if (g_profile) {
    ADS_CHECK_CUDA(cudaEventRecord(g_profile_ev[1], st));
    g_profile_valid = true;
  }

  // ---- merge the units that a range boundary cut
  CombineParams cp;
  cp.sched = sched; cp.o_part = o_part; cp.ml_part = ml_part;
  cp.out = ap.out; cp.lse = lse;
  cp.B = B; cp.P = P; cp.Tq = Tq; cp.Hq = Hq; cp.Hkv = Hkv; cp.G = G; cp.nl = nl;
  cp.n_mp = pl.n_mp; cp.n_gangs = n_gangs;
  const dim3 grid((unsigned)n_gangs, (unsigned)((Tq * G + 8 * kCombineRows - 1) / (8 * kCombineRows)));
  attn_combine_kernel<D><<<grid, 256, 0, st>>>(cp);
  return ads_launch_status();
}

}  // namespace

extern "C" size_t adapshot_attn_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                                int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap) {
  if (model == nullptr || !attn_shape_ok(model) || B <= 0 || P <= 0 || Tq <= 0 || n_layers_in_call <= 0 ||
      ctx_cap <= 0)
    return 0;
  return make_plan(model, B, P, Tq, n_layers_in_call).total;
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
  if (B <= 0 || k <= 0 || Tq <= 0 || ctx_cap <= 0 || flags != 0) return ADAPSHOT_EINVAL;
  if (model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (!attn_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
  if (P < 1 || P > kMaxProbes || (long long)P * B > kMaxPairs) return ADAPSHOT_ESHAPE;
  for (int i = 0; i < P; ++i) {
    if (probe_nshots[i] < 1 || probe_nshots[i] > k) return ADAPSHOT_ESHAPE;
    if (i > 0 && probe_nshots[i] <= probe_nshots[i - 1]) return ADAPSHOT_ESHAPE;
  }
  if (!ads_aligned16(k_ctx) || !ads_aligned16(v_ctx) || !ads_aligned16(q) || !ads_aligned16(kq) ||
      !ads_aligned16(vq) || !ads_aligned16(out) || ((uintptr_t)ws & 255u))
    return ADAPSHOT_EALIGN;
  if (ctx_cap > (1ll << 31) - 256) return ADAPSHOT_ESHAPE;
  const int nl = layer_end - layer_begin;
  const AttnPlan pl = make_plan(model, B, P, Tq, nl);
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (model->head_dim == 128)
    return launch_attn<128>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                            lse, pl, ws, status, st);
  return launch_attn<64>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                         lse, pl, ws, status, st);
}

extern "C" size_t adapshot_attn_fused_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                                      int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap) {
  if (model == nullptr || !attn_shape_ok(model) || B <= 0 || P <= 0 || Tq <= 0 || n_layers_in_call <= 0 ||
      ctx_cap <= 0)
    return 0;
  return make_plan(model, B, P, Tq, n_layers_in_call, ctx_cap).total;
}

extern "C" int adapshot_query_attn_fused(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                         const int32_t* sel_idx, const int64_t* ctx_off, int64_t ctx_cap,
                                         int32_t B, int32_t k, const int32_t* probe_nshots, int32_t P,
                                         const void* q, const void* kq, const void* vq, int32_t Tq,
                                         int32_t layer_begin, int32_t layer_end, void* out, float* lse,
                                         uint32_t flags, void* ws, size_t ws_bytes, int32_t* status,
                                         void* stream) {
  if (model == nullptr || pool == nullptr || sel_idx == nullptr || ctx_off == nullptr || probe_nshots == nullptr ||
      q == nullptr || kq == nullptr || vq == nullptr || out == nullptr || ws == nullptr)
    return ADAPSHOT_EINVAL;
  if (pool->k == nullptr || pool->v == nullptr || pool->shot_off == nullptr || pool->n_shots <= 0 ||
      pool->pool_tokens <= 0)
    return ADAPSHOT_EINVAL;
  if (B <= 0 || k <= 0 || Tq <= 0 || ctx_cap <= 0 || flags != 0) return ADAPSHOT_EINVAL;
  if (model->dtype != ADAPSHOT_BF16 || (model->k_pos_mode != 0 && model->k_pos_mode != 1)) return ADAPSHOT_EUNSUPPORTED;
  if (!attn_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (!(model->rope_base > 1.0)) return ADAPSHOT_EINVAL;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
  if (P < 1 || P > kMaxProbes || (long long)P * B > kMaxPairs || k > pool->n_shots) return ADAPSHOT_ESHAPE;
  for (int i = 0; i < P; ++i) {
    if (probe_nshots[i] < 1 || probe_nshots[i] > k) return ADAPSHOT_ESHAPE;
    if (i > 0 && probe_nshots[i] <= probe_nshots[i - 1]) return ADAPSHOT_ESHAPE;
  }
  if (!ads_aligned16(pool->k) || !ads_aligned16(pool->v) || !ads_aligned16(q) || !ads_aligned16(kq) ||
      !ads_aligned16(vq) || !ads_aligned16(out) || ((uintptr_t)ws & 255u) || ((uintptr_t)sel_idx & 3u))
    return ADAPSHOT_EALIGN;
  if (ctx_cap > (1ll << 31) - 256 || pool->pool_tokens > (1ll << 31) - 1) return ADAPSHOT_ESHAPE;
  const int nl = layer_end - layer_begin;
  const AttnPlan pl = make_plan(model, B, P, Tq, nl, ctx_cap);
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FusedSrc src;
  src.pool = pool; src.sel_idx = sel_idx; src.layer_begin = layer_begin;
  if (model->head_dim == 128)
    return launch_attn<128>(model, nullptr, nullptr, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl,
                            out, lse, pl, ws, status, st, &src, kModeFused);
  return launch_attn<64>(model, nullptr, nullptr, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                         lse, pl, ws, status, st, &src, kModeFused);
}

extern "C" size_t adapshot_attn_vpool_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t P,
                                                      int32_t Tq, int32_t n_layers_in_call, int64_t ctx_cap) {
  if (model == nullptr || !attn_shape_ok(model) || B <= 0 || P <= 0 || Tq <= 0 || n_layers_in_call <= 0 ||
      ctx_cap <= 0)
    return 0;
  return make_plan(model, B, P, Tq, n_layers_in_call, ctx_cap, false).total;
}

extern "C" int adapshot_query_attn_vpool(const adapshot_model_t* model, const adapshot_pool_t* pool,
                                         const int32_t* sel_idx, const void* k_ctx, int64_t ctx_cap,
                                         const int64_t* ctx_off, int32_t B, int32_t k,
                                         const int32_t* probe_nshots, int32_t P, const void* q, const void* kq,
                                         const void* vq, int32_t Tq, int32_t layer_begin, int32_t layer_end,
                                         void* out, float* lse, uint32_t flags, void* ws, size_t ws_bytes,
                                         int32_t* status, void* stream) {
  if (model == nullptr || pool == nullptr || sel_idx == nullptr || k_ctx == nullptr || ctx_off == nullptr ||
      probe_nshots == nullptr || q == nullptr || kq == nullptr || vq == nullptr || out == nullptr || ws == nullptr)
    return ADAPSHOT_EINVAL;
  if (pool->v == nullptr || pool->shot_off == nullptr || pool->n_shots <= 0 || pool->pool_tokens <= 0)
    return ADAPSHOT_EINVAL;
  if (B <= 0 || k <= 0 || Tq <= 0 || ctx_cap <= 0 || flags != 0) return ADAPSHOT_EINVAL;
  if (model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (!attn_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
  if (P < 1 || P > kMaxProbes || (long long)P * B > kMaxPairs || k > pool->n_shots) return ADAPSHOT_ESHAPE;
  for (int i = 0; i < P; ++i) {
    if (probe_nshots[i] < 1 || probe_nshots[i] > k) return ADAPSHOT_ESHAPE;
    if (i > 0 && probe_nshots[i] <= probe_nshots[i - 1]) return ADAPSHOT_ESHAPE;
  }
  if (!ads_aligned16(pool->v) || !ads_aligned16(k_ctx) || !ads_aligned16(q) || !ads_aligned16(kq) ||
      !ads_aligned16(vq) || !ads_aligned16(out) || ((uintptr_t)ws & 255u) || ((uintptr_t)sel_idx & 3u))
    return ADAPSHOT_EALIGN;
  if (ctx_cap > (1ll << 31) - 256 || pool->pool_tokens > (1ll << 31) - 1) return ADAPSHOT_ESHAPE;
  const int nl = layer_end - layer_begin;
  const AttnPlan pl = make_plan(model, B, P, Tq, nl, ctx_cap, false);
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FusedSrc src;
  src.pool = pool; src.sel_idx = sel_idx; src.layer_begin = layer_begin;
  if (model->head_dim == 128)
    return launch_attn<128>(model, k_ctx, nullptr, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out,
                            lse, pl, ws, status, st, &src, kModeVPool);
  return launch_attn<64>(model, k_ctx, nullptr, ctx_cap, ctx_off, B, k, probe_nshots, P, q, kq, vq, Tq, nl, out, lse,
                         pl, ws, status, st, &src, kModeVPool);
}

// ---------------------------------------------------------------- literal tree layout
namespace {
// Position ids of the probe tokens of the interleaved sequence: token t of probe j of query b sits
// at L_j + t (the shots keep the positions 0 .. L-1 of their plain concatenation).
struct TreePosArgs { int n[kMaxProbes]; };
__global__ void tree_positions_kernel(const long long* __restrict__ ctx_off, int B, int k, int P, int Tq,
                                           const TreePosArgs a, long long* __restrict__ pos) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * P * Tq) return;
  const int t = (int)(i % Tq), j = (int)((i / Tq) % P), b = (int)(i / ((long long)Tq * P));
  pos[i] = ctx_off[(long long)b * (k + 1) + a.n[j]] + t;
}
}  // namespace

extern "C" int adapshot_tree_layout(const int32_t* seg_kind, const int32_t* seg_len, int32_t n_seg, int32_t k,
                                    int32_t* probe_nshots, int32_t* P_out, int32_t* Tq_out) {
  if (seg_kind == nullptr || seg_len == nullptr || probe_nshots == nullptr || P_out == nullptr || Tq_out == nullptr ||
      n_seg <= 0)
    return ADAPSHOT_EINVAL;
  int shots = 0, P = 0, Tq = 0;
  bool shots_since_probe = false;
  for (int i = 0; i < n_seg; ++i) {
    if (seg_len[i] <= 0) return ADAPSHOT_ESHAPE;
    if (seg_kind[i] == ADAPSHOT_SEG_SHOTS) {
      shots += seg_len[i];
      if (shots > k) return ADAPSHOT_ESHAPE;
      shots_since_probe = true;
    } else if (seg_kind[i] == ADAPSHOT_SEG_PROBE) {
      // every probe follows at least one new shot (nested counts are strictly ascending) and all
      // probes have the same number of tokens
      if (!shots_since_probe || P >= kMaxProbes) return ADAPSHOT_ESHAPE;
      if (P == 0) Tq = seg_len[i];
      else if (seg_len[i] != Tq) return ADAPSHOT_ESHAPE;
      probe_nshots[P++] = shots;
      shots_since_probe = false;
    } else {
      return ADAPSHOT_EINVAL;
    }
  }
  if (P == 0 || shots_since_probe) return ADAPSHOT_ESHAPE;      // the sequence ends with a probe
  *P_out = P;
  *Tq_out = Tq;
  return ADAPSHOT_OK;
}

extern "C" int adapshot_tree_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx,
                                  int64_t ctx_cap, const int64_t* ctx_off, int32_t B, int32_t k,
                                  const int32_t* seg_kind, const int32_t* seg_len, int32_t n_seg,
                                  const void* q_seq, const void* kq_seq, const void* vq_seq,
                                  int32_t layer_begin, int32_t layer_end, void* out_seq, float* lse,
                                  int64_t* pos_seq, uint32_t flags, void* ws, size_t ws_bytes, int32_t* status,
                                  void* stream) {
  int32_t nshots[kMaxProbes], P = 0, Tq = 0;
  if (model == nullptr || ctx_off == nullptr) return ADAPSHOT_EINVAL;
  const int rc = adapshot_tree_layout(seg_kind, seg_len, n_seg, k, nshots, &P, &Tq);
  if (rc != ADAPSHOT_OK) return rc;
  // the probe tokens of the sequence, in sequence order, are [P][T_q]: the per-probe call's layout
  const int rc2 = adapshot_query_attn(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, nshots, P, q_seq, kq_seq, vq_seq,
                                      Tq, layer_begin, layer_end, out_seq, lse, flags, ws, ws_bytes, status, stream);
  if (rc2 != ADAPSHOT_OK || pos_seq == nullptr) return rc2;
  if ((uintptr_t)pos_seq & 7u) return ADAPSHOT_EALIGN;
  TreePosArgs a;
  for (int i = 0; i < kMaxProbes; ++i) a.n[i] = i < P ? nshots[i] : 0;
  const long long n = (long long)B * P * Tq;
  tree_positions_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const long long*>(ctx_off), B, k, P, Tq, a, reinterpret_cast<long long*>(pos_seq));
  return ads_launch_status();
}

// ------------------------------------------------------------------------ decode step
extern "C" size_t adapshot_decode_workspace_bytes(const adapshot_model_t* model, int32_t B, int32_t T_new,
                                                  int32_t T_own, int32_t n_layers_in_call) {
  if (model == nullptr || !attn_shape_ok(model) || B <= 0 || T_new <= 0 || T_own < T_new || n_layers_in_call <= 0)
    return 0;
  return make_plan(model, B, 1, T_new, n_layers_in_call, 0, true, T_own).total;
}

extern "C" int adapshot_decode_attn(const adapshot_model_t* model, const void* k_ctx, const void* v_ctx,
                                    int64_t ctx_cap, const int64_t* ctx_off, int32_t B, int32_t k,
                                    const int32_t* n_shots, const void* q_new, const void* k_own,
                                    const void* v_own, int32_t T_new, int32_t T_own, int32_t layer_begin,
                                    int32_t layer_end, void* out, float* lse, uint32_t flags, void* ws,
                                    size_t ws_bytes, int32_t* status, void* stream) {
  if (model == nullptr || k_ctx == nullptr || v_ctx == nullptr || ctx_off == nullptr || n_shots == nullptr ||
      q_new == nullptr || k_own == nullptr || v_own == nullptr || out == nullptr || ws == nullptr)
    return ADAPSHOT_EINVAL;
  if (B <= 0 || k <= 0 || T_new <= 0 || ctx_cap <= 0 || flags != 0) return ADAPSHOT_EINVAL;
  if (T_own < T_new) return ADAPSHOT_ESHAPE;
  if (model->dtype != ADAPSHOT_BF16) return ADAPSHOT_EUNSUPPORTED;
  if (!attn_shape_ok(model)) return ADAPSHOT_ESHAPE;
  if (layer_begin < 0 || layer_end <= layer_begin || layer_end > model->n_layers) return ADAPSHOT_ESHAPE;
  if (B > kMaxPairs) return ADAPSHOT_ESHAPE;
  if (!ads_aligned16(k_ctx) || !ads_aligned16(v_ctx) || !ads_aligned16(q_new) || !ads_aligned16(k_own) ||
      !ads_aligned16(v_own) || !ads_aligned16(out) || ((uintptr_t)ws & 255u) || ((uintptr_t)n_shots & 3u))
    return ADAPSHOT_EALIGN;
  if (ctx_cap > (1ll << 31) - 256) return ADAPSHOT_ESHAPE;
  const int nl = layer_end - layer_begin;
  const AttnPlan pl = make_plan(model, B, 1, T_new, nl, 0, true, T_own);
  if (ws_bytes < pl.total) return ADAPSHOT_ECAPACITY;
  AttnExtra extra;
  extra.To = T_own;
  extra.nshots_dev = n_shots;
  const int32_t one = 1;      // (placeholder for the host list: the per-query device counts are used)
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (model->head_dim == 128)
    return launch_attn<128>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, &one, 1, q_new, k_own, v_own, T_new, nl, out,
                            lse, pl, ws, status, st, nullptr, kModeCache, extra);
  return launch_attn<64>(model, k_ctx, v_ctx, ctx_cap, ctx_off, B, k, &one, 1, q_new, k_own, v_own, T_new, nl, out,
                         lse, pl, ws, status, st, nullptr, kModeCache, extra);
}

extern "C" int adapshot_profile(int enable) {
  if (enable && g_profile_ev[0] == nullptr) {
    ADS_CHECK_CUDA(cudaEventCreate(&g_profile_ev[0]));
    ADS_CHECK_CUDA(cudaEventCreate(&g_profile_ev[1]));
  }
  g_profile = enable != 0;
  g_profile_valid = false;
  return ADAPSHOT_OK;
}

extern "C" float adapshot_profile_attn_main_ms(void) {
  if (!g_profile_valid) return -1.f;
  float ms = -1.f;
  if (cudaEventSynchronize(g_profile_ev[1]) != cudaSuccess) return -1.f;
  if (cudaEventElapsedTime(&ms, g_profile_ev[0], g_profile_ev[1]) != cudaSuccess) return -1.f;
  return ms;
}

extern "C" int adapshot_selftest_wait_timeout(int32_t* status, long long* cycles, void* stream) {
  if (status == nullptr || cycles == nullptr) return ADAPSHOT_EINVAL;
  wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, cycles);
  return ads_launch_status();
}
