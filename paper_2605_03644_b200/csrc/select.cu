// Semantic shot selection (paper Sec. 4.1 ranking, Sec. 4.2 "rank in descending
// order and select the top k"): cosine of the query embedding against every cached
// shot embedding, then the top k with ties broken by the lower shot id (by rank counting
// for pools of up to 4096 shots, by chunked block-wide sorts beyond).
//
// The ranking must equal that of an fp64 evaluation of the same formula, so the
// fp32 products (exact in fp64) are accumulated in fp64 and scores are compared in
// fp64; the table is read once and the kernel stays bandwidth-bound.
#include "common.cuh"

namespace {

constexpr int kSortCap = 8192;      // candidates one CTA sorts in shared memory
constexpr int kSortThreads = 1024;

__device__ __forceinline__ unsigned long long desc_key(double s) { return ads_desc_key(s); }
__device__ __forceinline__ double key_score(unsigned long long k) { return ads_key_score(k); }

// One warp per pool row i: dots[b][i] = <q_b, e_i> for all b, enorm[i] = |e_i|.  With
// keys_out set (pools that the rank kernel handles) the warp also forms |q_b| from the values
// it loads anyway and writes the sort key of cos(q_b, e_i) in place of the dot product, so
// that the ranking kernel's CTAs do not each redo N fp64 divisions.
// NV > 0: E = 128 NV, the row is widened to fp64 once and kept in registers for all B queries
// (the fp32 -> fp64 conversions, not the fp64 FMAs, are what a row-times-many-queries pass pays for);
// NV = 0: any E.
template <int NV>
__global__ void __launch_bounds__(256)
cosine_dots_kernel(const float* __restrict__ emb, const float* __restrict__ q_emb, int N, int E,
                   int B, double* __restrict__ dots, double* __restrict__ enorm, int keys_out) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= N) return;
  const float* e = emb + (long long)row * E;
  double nn = 0.0;
  if constexpr (NV > 0) {
    double ev[4 * NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const float4 v = *reinterpret_cast<const float4*>(e + lane * 4 + 128 * i);
      ev[4 * i] = v.x; ev[4 * i + 1] = v.y; ev[4 * i + 2] = v.z; ev[4 * i + 3] = v.w;
    }
#pragma unroll
    for (int j = 0; j < 4 * NV; ++j) nn += ev[j] * ev[j];
    nn = warp_sum(nn);
    if (lane == 0) enorm[row] = sqrt(nn);
    for (int b = 0; b < B; ++b) {
      const float* q = q_emb + (long long)b * E;
      double acc = 0.0, qq = 0.0;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float4 w = __ldg(reinterpret_cast<const float4*>(q + lane * 4 + 128 * i));
        const double w0 = w.x, w1 = w.y, w2 = w.z, w3 = w.w;
        acc += ev[4 * i] * w0 + ev[4 * i + 1] * w1 + ev[4 * i + 2] * w2 + ev[4 * i + 3] * w3;
        if (keys_out) qq += w0 * w0 + w1 * w1 + w2 * w2 + w3 * w3;
      }
      acc = warp_sum(acc);
      if (keys_out) {
        qq = warp_sum(qq);
        if (lane == 0) {
          const double den = sqrt(qq) * sqrt(nn);
          reinterpret_cast<unsigned long long*>(dots)[(long long)b * N + row] = desc_key(den > 0.0 ? acc / den : 0.0);
        }
      } else if (lane == 0) {
        dots[(long long)b * N + row] = acc;
      }
    }
    return;
  }
  const bool vec_ok = (E & 3) == 0;
  if (vec_ok) {
    for (int i = lane * 4; i < E; i += 128) {
      float4 v = *reinterpret_cast<const float4*>(e + i);
      nn += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
    }
  } else {
    for (int i = lane; i < E; i += 32) nn += (double)e[i] * e[i];
  }
  nn = warp_sum(nn);
  if (lane == 0) enorm[row] = sqrt(nn);
  for (int b = 0; b < B; ++b) {
    const float* q = q_emb + (long long)b * E;
    double acc = 0.0, qq = 0.0;
    if (vec_ok) {
      for (int i = lane * 4; i < E; i += 128) {
        float4 v = *reinterpret_cast<const float4*>(e + i);   // L1-resident after the first pass
        float4 w = __ldg(reinterpret_cast<const float4*>(q + i));
        acc += (double)v.x * w.x + (double)v.y * w.y + (double)v.z * w.z + (double)v.w * w.w;
        qq += (double)w.x * w.x + (double)w.y * w.y + (double)w.z * w.z + (double)w.w * w.w;
      }
    } else {
      for (int i = lane; i < E; i += 32) {
        acc += (double)e[i] * q[i];
        qq += (double)q[i] * q[i];
      }
    }
    acc = warp_sum(acc);
    if (keys_out) {
      qq = warp_sum(qq);
      if (lane == 0) {
        const double den = sqrt(qq) * sqrt(nn);
        reinterpret_cast<unsigned long long*>(dots)[(long long)b * N + row] = desc_key(den > 0.0 ? acc / den : 0.0);
      }
    } else if (lane == 0) {
      dots[(long long)b * N + row] = acc;
    }
  }
}

__device__ __forceinline__ bool pair_less(unsigned long long ka, int ia, unsigned long long kb, int ib) {
  return ka < kb || (ka == kb && ia < ib);
}

// grid (n_chunks, B).  Sorts candidates [chunk*kSortCap, ...) of query b and writes
// the first min(k, n_in_chunk) of them to out_key/out_id at [b][chunk*k + r].
// Round 0 builds the candidates from dots / norms (in_key == nullptr).
__global__ void __launch_bounds__(kSortThreads)
topk_sort_kernel(const double* __restrict__ dots, const double* __restrict__ enorm,
                 const float* __restrict__ q_emb, int E,
                 const unsigned long long* __restrict__ in_key, const int* __restrict__ in_id,
                 int n_in, int in_stride, int k, unsigned long long* __restrict__ out_key,
                 int* __restrict__ out_id,
                 int out_stride, int32_t* __restrict__ final_idx, float* __restrict__ final_score) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  int* ids = reinterpret_cast<int*>(keys + kSortCap);
  __shared__ double red[kSortThreads / 32];
  __shared__ double qnorm_sh;

  const int b = blockIdx.y, chunk = blockIdx.x;
  const int begin = chunk * kSortCap;
  const int n = min(kSortCap, n_in - begin);
  int n_pow2 = 1;
  while (n_pow2 < n) n_pow2 <<= 1;

  if (in_key == nullptr) {
    // |q_b| in fp64, once per CTA
    const float* q = q_emb + (long long)b * E;
    double acc = 0.0;
    for (int i = threadIdx.x; i < E; i += kSortThreads) acc += (double)q[i] * q[i];
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {
      double v = red[threadIdx.x];
      v = warp_sum(v);
      if (threadIdx.x == 0) qnorm_sh = sqrt(v);
    }
    __syncthreads();
    const double qn = qnorm_sh;
    for (int i = threadIdx.x; i < n_pow2; i += kSortThreads) {
      if (i < n) {
        double den = qn * enorm[begin + i];
        double s = den > 0.0 ? dots[(long long)b * in_stride + begin + i] / den : 0.0;
        keys[i] = desc_key(s);
        ids[i] = begin + i;
      } else {
        keys[i] = ~0ull;             // padding sorts last
        ids[i] = 0x7fffffff;
      }
    }
  } else {
    for (int i = threadIdx.x; i < n_pow2; i += kSortThreads) {
      if (i < n) {
        keys[i] = in_key[(long long)b * in_stride + begin + i];
        ids[i] = in_id[(long long)b * in_stride + begin + i];
      } else {
        keys[i] = ~0ull;
        ids[i] = 0x7fffffff;
      }
    }
  }
  __syncthreads();

  // bitonic sort, ascending on (key, id); ids are unique so the order is total
  for (int size = 2; size <= n_pow2; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < (n_pow2 >> 1); t += kSortThreads) {
        int lo = 2 * t - (t & (stride - 1));
        int hi = lo + stride;
        bool up = (lo & size) == 0;
        unsigned long long ka = keys[lo], kb = keys[hi];
        int ia = ids[lo], ib = ids[hi];
        bool swap = up ? pair_less(kb, ib, ka, ia) : pair_less(ka, ia, kb, ib);
        if (swap) {
          keys[lo] = kb; keys[hi] = ka;
          ids[lo] = ib; ids[hi] = ia;
        }
      }
      __syncthreads();
    }
  }

  const int n_out = min(k, n);
  if (final_idx != nullptr) {
    for (int r = threadIdx.x; r < n_out; r += kSortThreads) {
      final_idx[(long long)b * k + r] = ids[r];
      if (final_score != nullptr) final_score[(long long)b * k + r] = (float)key_score(keys[r]);
    }
  } else {
    for (int r = threadIdx.x; r < n_out; r += kSortThreads) {
      out_key[(long long)b * out_stride + chunk * k + r] = keys[r];
      out_id[(long long)b * out_stride + chunk * k + r] = ids[r];
    }
  }
}

// Top-k by counting, for pools of up to kRankMaxN shots: the rank of shot i in the order
// (score descending, id ascending) is the number of shots that precede it; every shot with
// rank < k writes its id to position rank.  No sort and no serial phases: grid (N / 16, B),
// 16 candidates per CTA, the comparison range split over sixteen groups of 16 threads.
// "key_j precedes key_i" = key_j < key_i, or equal keys and j < i, = key_j < key_i + (j < i).
constexpr int kRankMaxN = 4096;
constexpr int kRankThreads = 256, kRankCand = 16, kRankTile = 2048;

__global__ void __launch_bounds__(kRankThreads)
rank_topk_kernel(const unsigned long long* __restrict__ all_keys, int N, int k,
                 int32_t* __restrict__ final_idx, float* __restrict__ final_score) {
  __shared__ unsigned long long keys[kRankTile];
  __shared__ int part_cnt[kRankThreads];
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  const unsigned long long* gkeys = all_keys + (long long)b * N;
  auto key_of = [&](int j) -> unsigned long long { return gkeys[j]; };
  const int i = blockIdx.x * kRankCand + (tid & (kRankCand - 1));
  const int part = tid / kRankCand;                       // which quarter of every tile this thread scans
  const unsigned long long ki = i < N ? key_of(i) : ~0ull;
  const unsigned long long ki_le = ki == ~0ull ? ki : ki + 1;   // threshold for j < i (equal keys precede)
  int cnt = 0;
  for (int tile0 = 0; tile0 < N; tile0 += kRankTile) {
    const int n_t = min(kRankTile, N - tile0);
    for (int t = tid; t < n_t; t += kRankThreads) keys[t] = key_of(tile0 + t);
    __syncthreads();
    const int per = kRankTile / (kRankThreads / kRankCand);
    const int j0 = part * per, j1 = min(n_t, j0 + per);
    const int split = max(j0, min(j1, i - tile0));        // [j0, split): j < i;  [split, j1): j >= i
    for (int j = j0; j < split; ++j) cnt += keys[j] < ki_le ? 1 : 0;
    for (int j = split; j < j1; ++j) cnt += keys[j] < ki ? 1 : 0;
    __syncthreads();
  }
  part_cnt[tid] = cnt;
  __syncthreads();
  if (part == 0 && i < N) {
    int rank = 0;
#pragma unroll
    for (int q4 = 0; q4 < kRankThreads / kRankCand; ++q4) rank += part_cnt[q4 * kRankCand + tid];
    if (rank < k) {
      final_idx[(long long)b * k + rank] = i;
      if (final_score != nullptr) final_score[(long long)b * k + rank] = (float)key_score(ki);
    }
  }
}

size_t sel_cand_entries(int n_shots, int k) {
  if (n_shots <= kSortCap) return 0;
  size_t chunks = ((size_t)n_shots + kSortCap - 1) / kSortCap;
  return chunks * (size_t)k;
}

}  // namespace

size_t ads_topk_scratch_bytes(int N, int B, int k) {
  const size_t cand = sel_cand_entries(N, k);
  return 2 * (ads_round_up((size_t)B * cand * 8, 256) + ads_round_up((size_t)B * cand * 4, 256));
}

int ads_topk_from_keys(const unsigned long long* keys, const int* ids, int N, int B, int k, void* cand_ws,
                       int32_t* sel_idx, float* sel_score, cudaStream_t st) {
  if (N > kSortCap && k > kSortCap / 2) return ADAPSHOT_EUNSUPPORTED;
  if (N <= kRankMaxN) {
    dim3 grid((N + kRankCand - 1) / kRankCand, B);
    rank_topk_kernel<<<grid, kRankThreads, 0, st>>>(keys, N, k, sel_idx, sel_score);
    return ads_launch_status();
  }
  const size_t smem = (size_t)kSortCap * (8 + 4);
  static bool attr_set[kAdsMaxDevices] = {false};
  if (ads_set_max_smem(topk_sort_kernel, (int)smem, attr_set) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
  const size_t cand = sel_cand_entries(N, k);
  unsigned char* p = static_cast<unsigned char*>(cand_ws);
  unsigned long long* ckey[2];
  int* cid[2];
  for (int i = 0; i < 2; ++i) {
    ckey[i] = reinterpret_cast<unsigned long long*>(p);
    p += ads_round_up((size_t)B * cand * 8, 256);
    cid[i] = reinterpret_cast<int*>(p);
    p += ads_round_up((size_t)B * cand * 4, 256);
  }
  int n_in = N, in_stride = N, round = 0;
  const unsigned long long* in_key = keys;
  const int* in_id = ids;
  while (true) {
    const int chunks = (n_in + kSortCap - 1) / kSortCap;
    const bool last = chunks == 1;
    dim3 grid(chunks, B);
    const int out_stride = chunks * k;
    topk_sort_kernel<<<grid, kSortThreads, smem, st>>>(
        nullptr, nullptr, nullptr, 0, in_key, in_id, n_in, in_stride, k, ckey[round & 1], cid[round & 1], out_stride,
        last ? sel_idx : nullptr, last ? sel_score : nullptr);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
    if (last) break;
    in_key = ckey[round & 1];
    in_id = cid[round & 1];
    const int last_n = n_in - (chunks - 1) * kSortCap;
    n_in = (chunks - 1) * k + (last_n < k ? last_n : k);
    in_stride = out_stride;
    ++round;
  }
  return ADAPSHOT_OK;
}

extern "C" size_t adapshot_select_workspace_bytes(int32_t n_shots, int32_t B, int32_t k) {
  if (n_shots <= 0 || B <= 0 || k <= 0) return 0;
  size_t bytes = ads_round_up((size_t)B * n_shots * sizeof(double), 256);   // dots
  bytes += ads_round_up((size_t)n_shots * sizeof(double), 256);             // |e_i|
  size_t cand = sel_cand_entries(n_shots, k);
  // two ping-pong candidate lists of (key, id)
  bytes += 2 * (ads_round_up((size_t)B * cand * 8, 256) + ads_round_up((size_t)B * cand * 4, 256));
  return bytes;
}

extern "C" int adapshot_select(const adapshot_pool_t* pool, const float* q_emb, int32_t B, int32_t k,
                               int32_t* sel_idx, float* sel_score, void* ws, size_t ws_bytes,
                               int32_t* status, void* stream) {
  (void)status;
  if (pool == nullptr || q_emb == nullptr || sel_idx == nullptr || ws == nullptr) return ADAPSHOT_EINVAL;
  if (pool->emb == nullptr || pool->n_shots <= 0 || pool->emb_dim <= 0 || B <= 0) return ADAPSHOT_EINVAL;
  const int N = pool->n_shots, E = pool->emb_dim;
  if (k < 1 || k > N) return ADAPSHOT_ESHAPE;
  if (N > kSortCap && k > kSortCap / 2) return ADAPSHOT_EUNSUPPORTED;
  if (!ads_aligned16(pool->emb) || !ads_aligned16(q_emb) || !ads_aligned16(ws)) return ADAPSHOT_EALIGN;
  if (ws_bytes < adapshot_select_workspace_bytes(N, B, k)) return ADAPSHOT_ECAPACITY;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* p = static_cast<unsigned char*>(ws);
  double* dots = reinterpret_cast<double*>(p);
  p += ads_round_up((size_t)B * N * sizeof(double), 256);
  double* enorm = reinterpret_cast<double*>(p);
  p += ads_round_up((size_t)N * sizeof(double), 256);
  const size_t cand = sel_cand_entries(N, k);
  unsigned long long* ckey[2];
  int* cid[2];
  for (int i = 0; i < 2; ++i) {
    ckey[i] = reinterpret_cast<unsigned long long*>(p);
    p += ads_round_up((size_t)B * cand * 8, 256);
    cid[i] = reinterpret_cast<int*>(p);
    p += ads_round_up((size_t)B * cand * 4, 256);
  }

  const int warps_per_block = 8;
  const unsigned cgrid = (unsigned)((N + warps_per_block - 1) / warps_per_block);
  const int keys_out = N <= kRankMaxN ? 1 : 0;
  if (E == 1024)
    cosine_dots_kernel<8><<<cgrid, warps_per_block * 32, 0, st>>>(pool->emb, q_emb, N, E, B, dots, enorm, keys_out);
  else if (E == 128)
    cosine_dots_kernel<1><<<cgrid, warps_per_block * 32, 0, st>>>(pool->emb, q_emb, N, E, B, dots, enorm, keys_out);
  else
    cosine_dots_kernel<0><<<cgrid, warps_per_block * 32, 0, st>>>(pool->emb, q_emb, N, E, B, dots, enorm, keys_out);
  if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  if (N <= kRankMaxN) {
    dim3 grid((N + kRankCand - 1) / kRankCand, B);
    rank_topk_kernel<<<grid, kRankThreads, 0, st>>>(reinterpret_cast<const unsigned long long*>(dots), N, k, sel_idx,
                                                    sel_score);
    return ads_launch_status();
  }

  const size_t smem = (size_t)kSortCap * (8 + 4);
  static bool attr_set[kAdsMaxDevices] = {false};
  if (ads_set_max_smem(topk_sort_kernel, (int)smem, attr_set) != ADAPSHOT_OK) return ADAPSHOT_ECUDA;

  int n_in = N, in_stride = N;
  int round = 0;
  const unsigned long long* in_key = nullptr;
  const int* in_id = nullptr;
  while (true) {
    const int chunks = (n_in + kSortCap - 1) / kSortCap;
    const bool last = chunks == 1;
    dim3 grid(chunks, B);
    const int out_stride = chunks * k;
    topk_sort_kernel<<<grid, kSortThreads, smem, st>>>(
        dots, enorm, q_emb, E, in_key, in_id, n_in, in_stride, k, ckey[round & 1], cid[round & 1], out_stride,
        last ? sel_idx : nullptr, last ? sel_score : nullptr);
    if (ads_launch_status() != ADAPSHOT_OK) return ADAPSHOT_ECUDA;
    if (last) break;
    in_key = ckey[round & 1];
    in_id = cid[round & 1];
    // every chunk but possibly the last holds >= k candidates (k <= kSortCap / 2)
    const int last_n = n_in - (chunks - 1) * kSortCap;
    n_in = (chunks - 1) * k + (last_n < k ? last_n : k);
    in_stride = out_stride;
    ++round;
  }
  return ADAPSHOT_OK;
}
