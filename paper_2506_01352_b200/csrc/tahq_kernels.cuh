// Kernels of the TAH-Quant boundary codec (sm_100a).  See tahq_device.cuh for the work decomposition.
//
//   encode:  stats_kernel        Eq. 1-2   tile -> entropy score                 (skipped for integer budgets)
//            hist_kernel         Sec. 3.2  per-group histogram of binned scores
//            gather_kernel       Sec. 3.2  threshold bin + candidates of that bin
//            resolve_kernel      Sec. 3.2  exact k_hi-th largest (score, index) key per group
//            bitmap_kernel       Sec. 3.2  1-bit map + hi-tile counts per 128 tiles
//            scan_kernel         Sec. 3.4  exclusive prefix of those counts (payload offsets)
//            quant_pack_kernel   Eq. 3-4, Sec. 3.3-3.4  pivot test, swap + Hadamard, quantise, pack
//   decode:  count_kernel + scan_kernel    bit map -> payload offsets, header check
//            decode_kernel       Sec. 3.3, Alg. 1 l.5  unpack, z + q*s, inverse transform, store
#pragma once

#include "tahq_device.cuh"

namespace tahq {

struct Args {
  const uint8_t *in;        // encode: tensor; decode: unused
  uint8_t *packed;          // packed buffer (decode reads it)
  uint8_t *out;             // decode: tensor
  uint64_t n_tiles, tiles_per_group, k_hi, n_groups;
  uint32_t lo, mixed;       // low width; 1 when two widths are in use
  uint64_t off_bitmap, off_sz, off_pivot, off_payload, payload_bytes, total_bytes;
  float tau, eps_l1, eps_log, eps_ratio;
  float *scores;            // [n_tiles]
  uint32_t *hist;           // [n_groups][kBins]
  uint32_t *ncand;          // [n_groups]
  uint2 *binsel;            // [n_groups] {threshold bin, rank inside the bin (1-based)}
  unsigned long long *theta;// [n_groups] key of the k_hi-th ranked tile
  unsigned long long *cand; // [n_groups][cand_cap]
  uint32_t cand_cap, cpg;   // candidate capacity per group; CTAs per group of hist/gather
  uint32_t direct;          // small groups: resolve_kernel ranks all scores of the group itself
  uint32_t *cnt128;         // [ceil(n_tiles/128)+2] hi tiles per 128 tiles, then their exclusive prefix
  uint32_t *status;         // device status word
  uint32_t header[32];      // the 128-byte header of the packed buffer
};

// ------------------------------------------------------------------------------------------
// Persistent multi-stage cp.async loop over the chunks of a CTA
// ------------------------------------------------------------------------------------------
template <class C, int NST, class Body>
__device__ __forceinline__ void chunk_pipeline(const uint8_t *in, uint64_t n_tiles, uint8_t *stages, Body &&body) {
  const uint64_t n_chunks = (n_tiles + C::TPC - 1) / C::TPC;
  uint64_t c_issue = blockIdx.x;
#pragma unroll
  for (int s = 0; s < NST - 1; ++s) {
    if (c_issue < n_chunks) issue_chunk<C>(in, n_tiles, c_issue, stages + (size_t)s * C::STAGE_BYTES);
    cp_async_commit();
    c_issue += gridDim.x;
  }
  int stage = 0;
  for (uint64_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
    cp_async_wait<NST - 2>();
    __syncthreads();   // chunk c has landed; everyone is done with the stage consumed last time
    {
      const int s2 = (stage + NST - 1) % NST;
      if (c_issue < n_chunks) issue_chunk<C>(in, n_tiles, c_issue, stages + (size_t)s2 * C::STAGE_BYTES);
      cp_async_commit();
      c_issue += gridDim.x;
    }
    body(c, stages + (size_t)stage * C::STAGE_BYTES);
    stage = (stage + 1) % NST;
  }
  cp_async_wait<0>();
}

// ------------------------------------------------------------------------------------------
// Eq. 1-2: entropy score per tile
// ------------------------------------------------------------------------------------------
template <class C, int NST>
__global__ void __launch_bounds__(kThreads) stats_kernel(const Args a) {
  extern __shared__ __align__(128) uint8_t smem[];
  chunk_pipeline<C, NST>(a.in, a.n_tiles, smem, [&](uint64_t c, const uint8_t *stage) {
    const float s = tile_score<C>(stage, a.eps_l1, a.eps_log);
    const uint64_t tile = c * C::TPC + threadIdx.x / C::LPT;
    if (tile < a.n_tiles && (C::LPT == 1 || !(threadIdx.x & 1))) a.scores[tile] = s;
  });
}

// ------------------------------------------------------------------------------------------
// Sec. 3.2: exact top-k_hi per ranking group
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void group_slice(const Args &a, uint64_t &g, uint64_t &lo, uint64_t &hi) {
  g = blockIdx.x / a.cpg;
  const uint64_t j = blockIdx.x % a.cpg;
  const uint64_t slice = (a.tiles_per_group + a.cpg - 1) / a.cpg;
  lo = j * slice;
  hi = lo + slice < a.tiles_per_group ? lo + slice : a.tiles_per_group;
  if (lo > hi) lo = hi;
}

__global__ void __launch_bounds__(kThreads) hist_kernel(const Args a) {
  __shared__ uint32_t h[kBins];
  for (int b = threadIdx.x; b < kBins; b += kThreads) h[b] = 0;
  __syncthreads();
  uint64_t g, lo, hi;
  group_slice(a, g, lo, hi);
  const float *sc = a.scores + g * a.tiles_per_group;
  for (uint64_t i = lo + threadIdx.x; i < hi; i += kThreads) atomicAdd(&h[score_bin(sc[i])], 1u);
  __syncthreads();
  uint32_t *gh = a.hist + g * kBins;
  for (int b = threadIdx.x; b < kBins; b += kThreads)
    if (h[b]) atomicAdd(&gh[b], h[b]);
}

__global__ void __launch_bounds__(kThreads) gather_kernel(const Args a) {
  __shared__ uint32_t h[kBins];
  __shared__ uint32_t part[kThreads];
  __shared__ uint32_t sel[2];
  uint64_t g, lo, hi;
  group_slice(a, g, lo, hi);
  const uint32_t *gh = a.hist + g * kBins;
  for (int b = threadIdx.x; b < kBins; b += kThreads) h[b] = gh[b];
  __syncthreads();
  constexpr int BPT = kBins / kThreads;   // bins per thread
  uint32_t mine = 0;
#pragma unroll
  for (int j = 0; j < BPT; ++j) mine += h[threadIdx.x * BPT + j];
  part[threadIdx.x] = mine;
  __syncthreads();
  uint32_t above = 0;   // tiles in bins above this thread's range
  for (int j = threadIdx.x + 1; j < kThreads; ++j) above += part[j];
  const uint32_t k = (uint32_t)a.k_hi;
  if (above < k && above + mine >= k) {   // the k-th ranked tile lies in one of this thread's bins
    for (int j = BPT - 1; j >= 0; --j) {
      const uint32_t n = h[threadIdx.x * BPT + j];
      if (above + n >= k) { sel[0] = threadIdx.x * BPT + j; sel[1] = k - above; break; }
      above += n;
    }
  }
  __syncthreads();
  const uint32_t B = sel[0];
  if (blockIdx.x % a.cpg == 0 && threadIdx.x == 0) a.binsel[g] = make_uint2(B, sel[1]);
  const float *sc = a.scores + g * a.tiles_per_group;
  for (uint64_t i = lo + threadIdx.x; i < hi; i += kThreads) {
    const float s = sc[i];
    if (score_bin(s) == B) {
      const uint32_t slot = atomicAdd(&a.ncand[g], 1u);
      if (slot < a.cand_cap) a.cand[g * a.cand_cap + slot] = rank_key(s, (uint32_t)i);
    }
  }
}

constexpr int kResolveThreads = 1024;

// r-th largest 64-bit key among the candidates of the threshold bin: radix select, 8 bits a pass.
__global__ void __launch_bounds__(kResolveThreads) resolve_kernel(const Args a) {
  __shared__ uint32_t h[256];
  __shared__ uint32_t pick[2];
  const uint64_t g = blockIdx.x;
  const uint32_t B = a.direct ? 0u : a.binsel[g].x;
  uint32_t r = a.direct ? (uint32_t)a.k_hi : a.binsel[g].y;
  const uint32_t n = a.direct ? 0u : a.hist[g * kBins + B];
  const bool listed = !a.direct && n <= a.cand_cap;   // otherwise take the candidates from the scores
  const unsigned long long *cand = a.cand + g * a.cand_cap;
  const float *sc = a.scores + g * a.tiles_per_group;
  const uint64_t count = listed ? n : a.tiles_per_group;
  unsigned long long prefix = 0, mask = 0;
  for (int shift = 56; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) h[threadIdx.x] = 0;
    __syncthreads();
    for (uint64_t i = threadIdx.x; i < count; i += kResolveThreads) {
      unsigned long long key;
      bool ok;
      if (listed) { key = cand[i]; ok = true; }
      else { const float s = sc[i]; ok = a.direct || score_bin(s) == B; key = rank_key(s, (uint32_t)i); }
      if (ok && (key & mask) == prefix) atomicAdd(&h[(unsigned)(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane L owns digits 255-8L .. 248-8L (descending); find where the running count reaches r
      const int top = 255 - 8 * (int)threadIdx.x;
      uint32_t mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += h[top - j];
      uint32_t incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o *= 2) {
        const uint32_t v = __shfl_up_sync(kFull, incl, o);
        if ((int)threadIdx.x >= o) incl += v;
      }
      uint32_t above = incl - mine;
      if (above < r && incl >= r) {
        for (int j = 0; j < 8; ++j) {
          const uint32_t c = h[top - j];
          if (above + c >= r) { pick[0] = (uint32_t)(top - j); pick[1] = r - above; break; }
          above += c;
        }
      }
    }
    __syncthreads();
    prefix |= (unsigned long long)pick[0] << shift;
    mask |= 0xffull << shift;
    r = pick[1];
    __syncthreads();
  }
  if (threadIdx.x == 0) a.theta[g] = prefix;
}

// Bit map (tile t -> bit t&31 of word t>>5) and the number of hi tiles in every 128 tiles.
__global__ void __launch_bounds__(kThreads) bitmap_kernel(const Args a) {
  __shared__ uint32_t wc[kThreads / 32];
  const uint64_t t = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  bool hi = false;
  if (t < a.n_tiles) {
    const uint64_t g = t / a.tiles_per_group;
    const uint32_t i = (uint32_t)(t - g * a.tiles_per_group);
    hi = rank_key(a.scores[t], i) >= a.theta[g];
  }
  const uint32_t word = __ballot_sync(kFull, hi);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    reinterpret_cast<uint32_t *>(a.packed + a.off_bitmap)[t >> 5] = word;
    wc[warp] = __popc(word);
  }
  __syncthreads();
  if (threadIdx.x < 2)
    a.cnt128[(uint64_t)blockIdx.x * 2 + threadIdx.x] =
        wc[4 * threadIdx.x] + wc[4 * threadIdx.x + 1] + wc[4 * threadIdx.x + 2] + wc[4 * threadIdx.x + 3];
}

// Single-CTA exclusive scan of cnt128[0..n) in place.  expect_total != ~0: flag a mismatch.
constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads) scan_kernel(uint32_t *v, uint64_t n, unsigned long long expect_total,
                                                            uint32_t *status) {
  __shared__ uint32_t wsum[32];
  const uint64_t per = (n + kScanThreads - 1) / kScanThreads;
  const uint64_t lo = per * threadIdx.x;
  const uint64_t hi = lo + per < n ? lo + per : n;
  uint32_t mine = 0;
  for (uint64_t i = lo; i < hi; ++i) mine += v[i];
  uint32_t incl = mine;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o *= 2) {
    const uint32_t u = __shfl_up_sync(kFull, incl, o);
    if (lane >= o) incl += u;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = wsum[lane];
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o *= 2) {
      const uint32_t u = __shfl_up_sync(kFull, wi, o);
      if (lane >= o) wi += u;
    }
    wsum[lane] = wi - w;
    if (lane == 31 && expect_total != ~0ull && (unsigned long long)wi != expect_total)
      atomicOr(status, 2u /* TAHQ_DEV_BAD_BITMAP */);
  }
  __syncthreads();
  uint32_t run = wsum[warp] + incl - mine;
  for (uint64_t i = lo; i < hi; ++i) {
    const uint32_t c = v[i];
    v[i] = run;
    run += c;
  }
}

// ------------------------------------------------------------------------------------------
// Widths and offsets of the tiles of one chunk, from the chunk's words of the bit map
// ------------------------------------------------------------------------------------------
template <class C>
struct ChunkPlan {
  uint32_t is_hi;       // this thread's tile uses the higher width
  uint32_t row_off;     // byte offset of this thread's codes inside the chunk's payload
  uint32_t bytes;       // payload bytes of the chunk
  uint64_t goff;        // byte offset of the chunk's payload inside the payload section
};

template <class C>
__device__ __forceinline__ ChunkPlan<C> plan_chunk(const Args &a, uint64_t c) {
  constexpr int NW = C::TPC / 32;
  const uint64_t tile0 = c * C::TPC;
  const int r = threadIdx.x / C::LPT, half = threadIdx.x % C::LPT;
  const int myw = r >> 5, mybit = r & 31;
  uint32_t hi_before = 0, total_hi = 0, myword = 0;
  if (a.mixed) {
    const uint32_t *bm = reinterpret_cast<const uint32_t *>(a.packed + a.off_bitmap) + tile0 / 32;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const uint64_t first = tile0 + 32ull * w;
      uint32_t word = 0;
      if (first < a.n_tiles) {
        const uint64_t left = a.n_tiles - first;
        word = __ldg(bm + w) & (left >= 32 ? 0xffffffffu : ((1u << (uint32_t)left) - 1u));
      }
      const uint32_t pc = __popc(word);
      total_hi += pc;
      hi_before += (w < myw) ? pc : 0u;
      myword = (w == myw) ? word : myword;
    }
  }
  hi_before += __popc(myword & ((1u << mybit) - 1u));
  ChunkPlan<C> p;
  p.is_hi = (myword >> mybit) & 1u;
  const uint32_t b = a.lo + p.is_hi;
  p.row_off = (C::G / 8) * (a.lo * r + hi_before) + half * (C::EPT / 8) * b;
  const uint64_t left = a.n_tiles - tile0;
  const uint32_t nvalid = left < (uint64_t)C::TPC ? (uint32_t)left : (uint32_t)C::TPC;
  p.bytes = (C::G / 8) * (a.lo * nvalid + total_hi);
  const uint64_t P = a.mixed ? (uint64_t)__ldg(a.cnt128 + tile0 / 128) : 0ull;
  p.goff = (uint64_t)(C::G / 8) * ((uint64_t)a.lo * tile0 + P);
  return p;
}

// ------------------------------------------------------------------------------------------
// Eq. 3-4 + Sec. 3.3-3.4: pivot test, swap + Hadamard, min-max quantisation, packing
// ------------------------------------------------------------------------------------------
template <class C, int W>
__device__ __forceinline__ void pack_store(const uint32_t (&code)[C::EPT], uint32_t *dst) {
  uint32_t w[C::EPT * W / 32];
  pack_words<W, C::EPT>(code, w);
#pragma unroll
  for (int j = 0; j < C::EPT * W / 32; ++j) dst[j] = w[j];
}

template <class C, int NST>
__global__ void __launch_bounds__(kThreads) quant_pack_kernel(const Args a) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint32_t *out = reinterpret_cast<uint32_t *>(smem + (size_t)NST * C::STAGE_BYTES);
  uint32_t *sz32 = reinterpret_cast<uint32_t *>(a.packed + a.off_sz);
  uint8_t *pivot = a.packed + a.off_pivot;

  if (blockIdx.x == 0) {   // header and the zero padding behind every section
    if (threadIdx.x < 32) reinterpret_cast<uint32_t *>(a.packed)[threadIdx.x] = a.header[threadIdx.x];
    const uint64_t pad[4][2] = {{a.off_bitmap + (a.n_tiles + 7) / 8, a.off_sz},
                                {a.off_sz + 4 * a.n_tiles, a.off_pivot},
                                {a.off_pivot + a.n_tiles, a.off_payload},
                                {a.off_payload + a.payload_bytes, a.total_bytes}};
    for (int s = 0; s < 4; ++s)
      for (uint64_t o = pad[s][0] + threadIdx.x; o < pad[s][1]; o += kThreads) a.packed[o] = 0;
  }

  chunk_pipeline<C, NST>(a.in, a.n_tiles, smem, [&](uint64_t c, const uint8_t *stage) {
    const uint64_t tile0 = c * C::TPC;
    const int half = threadIdx.x % C::LPT;
    const uint64_t tile = tile0 + threadIdx.x / C::LPT;
    const bool valid = tile < a.n_tiles;
    const ChunkPlan<C> plan = plan_chunk<C>(a, c);
    if (!a.mixed && threadIdx.x < C::TPC / 32)   // integer budget: the bit map is all zero
      reinterpret_cast<uint32_t *>(a.packed + a.off_bitmap)[tile0 / 32 + threadIdx.x] = 0;

    float x[C::EPT];
#pragma unroll
    for (int o = 0; o < C::NOCT; ++o) {
      float v[8];
      load_oct<C>(stage, o, v);
#pragma unroll
      for (int k = 0; k < 8; ++k) x[8 * o + k] = v[k];
    }

    // Eq. 3: largest magnitude (first index), largest among the others
    float a1 = fabsf(x[0]), a2 = 0.0f;
    int d = 0;
#pragma unroll
    for (int k = 1; k < C::EPT; ++k) {
      const float m = fabsf(x[k]);
      const bool gt = m > a1;
      a2 = gt ? a1 : fmaxf(a2, m);
      d = gt ? k : d;
      a1 = gt ? m : a1;
    }
    if constexpr (C::LPT == 2) {
      const float o1 = __shfl_xor_sync(kFull, a1, 1), o2 = __shfl_xor_sync(kFull, a2, 1);
      const int od = __shfl_xor_sync(kFull, d, 1);
      const float l1 = half ? o1 : a1, l2 = half ? o2 : a2, u1 = half ? a1 : o1, u2 = half ? a2 : o2;
      const int ld = half ? od : d, ud = half ? d : od;
      const bool lw = l1 >= u1;   // the lower half holds the lower indices: it wins ties
      a1 = lw ? l1 : u1;
      a2 = lw ? fmaxf(l2, u1) : fmaxf(u2, l1);
      d = lw ? ld : C::EPT + ud;
    }
    const float t1 = a2 + a.eps_ratio;
    const float t2 = a.tau * t1;
    const bool flag = a1 > t2;

    // Eq. 4: pivot swap + Hadamard on flagged tiles
    const unsigned fm = __ballot_sync(kFull, flag);
    if (flag) {
      if constexpr (C::LPT == 1) {
        const float xd = load_elem<C>(stage, d), x0 = x[0];
#pragma unroll
        for (int k = 1; k < C::EPT; ++k) x[k] = (k == d) ? x0 : x[k];
        x[0] = xd;
        butterfly<C::EPT>(x);
      } else {
        const int lane = threadIdx.x & 31, owner = d / C::EPT, dl = d % C::EPT;
        const float x0 = __shfl_sync(fm, x[0], lane & ~1);
        const float xd = __shfl_sync(fm, load_elem<C>(stage, dl), (lane & ~1) + owner);
        if (half == owner) {
#pragma unroll
          for (int k = 0; k < C::EPT; ++k) x[k] = (k == dl) ? x0 : x[k];
        }
        if (half == 0) x[0] = xd;
        butterfly<C::EPT>(x);
#pragma unroll
        for (int k = 0; k < C::EPT; ++k) {
          const float p = __shfl_xor_sync(fm, x[k], 1);
          x[k] = half ? (p - x[k]) : (x[k] + p);
        }
      }
      constexpr float cG = (C::G == 32) ? 0.17677669529663687f : (C::G == 64) ? 0.125f : 0.08838834764831845f;
#pragma unroll
      for (int k = 0; k < C::EPT; ++k) x[k] = x[k] * cG;
    }

    // Sec. 3.3: min-max range -> binary16 zero-point and scale
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int k = 1; k < C::EPT; ++k) { mn = fminf(mn, x[k]); mx = fmaxf(mx, x[k]); }
    if constexpr (C::LPT == 2) {
      mn = fminf(mn, __shfl_xor_sync(kFull, mn, 1));
      mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
    }
    const uint32_t b = a.lo + plan.is_hi;
    const float qmax = (float)((1u << b) - 1u);
    mn = mn + 0.0f;
    mn = fminf(fmaxf(mn, -65504.0f), 65504.0f);
    const __half zh = __float2half_rn(mn);
    const float z = __half2float(zh);
    float s = __fdiv_rn(mx - z, qmax);
    s = (s > 0.0f) ? s : 0.0f;
    s = fminf(s, 65504.0f);
    const __half sh = __float2half_rn(s);
    const float sf = __half2float(sh);
    const float inv_s = sf > 0.0f ? __fdiv_rn(1.0f, sf) : 0.0f;

    // q = rint(clamp((v - z) * inv_s, 0, qmax)); adding 1.5*2^23 rounds to nearest-even
    uint32_t code[C::EPT];
#pragma unroll
    for (int k = 0; k < C::EPT; ++k) {
      float y = (x[k] - z) * inv_s;
      y = fminf(fmaxf(y, 0.0f), qmax);
      code[k] = __float_as_uint(y + 12582912.0f) & 0x1ffu;
    }

    if (valid) {
      if (half == 0) {
        sz32[tile] = (uint32_t)__half_as_ushort(sh) | ((uint32_t)__half_as_ushort(zh) << 16);
        pivot[tile] = flag ? (uint8_t)(0x80 | d) : (uint8_t)0;
      }
      uint32_t *dst = out + plan.row_off / 4;
      switch (b) {
        case 2: pack_store<C, 2>(code, dst); break;
        case 3: pack_store<C, 3>(code, dst); break;
        case 4: pack_store<C, 4>(code, dst); break;
        case 5: pack_store<C, 5>(code, dst); break;
        case 6: pack_store<C, 6>(code, dst); break;
        case 7: pack_store<C, 7>(code, dst); break;
        default: pack_store<C, 8>(code, dst); break;
      }
    }
    __syncthreads();
    uint32_t *gdst = reinterpret_cast<uint32_t *>(a.packed + a.off_payload + plan.goff);
    for (uint32_t i = threadIdx.x; i < plan.bytes / 4; i += kThreads) gdst[i] = out[i];
  });
}

// ------------------------------------------------------------------------------------------
// Decode
// ------------------------------------------------------------------------------------------

// hi tiles per 128 tiles, straight from the received bit map; CTA 0 also checks the header.
__global__ void __launch_bounds__(kThreads) count_kernel(const Args a) {
  const uint64_t n128 = (a.n_tiles + 127) / 128;
  const uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  if (blockIdx.x == 0 && threadIdx.x < 32) {
    const uint32_t got = reinterpret_cast<const uint32_t *>(a.packed)[threadIdx.x];
    // seed / rounding / constants are part of the header, so a buffer from another configuration is refused
    if (got != a.header[threadIdx.x]) atomicOr(a.status, 1u /* TAHQ_DEV_BAD_HEADER */);
  }
  if (i >= n128) return;
  uint32_t n = 0;
  if (a.mixed) {
    const uint32_t *bm = reinterpret_cast<const uint32_t *>(a.packed + a.off_bitmap) + i * 4;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const uint64_t first = i * 128 + 32ull * w;
      if (first < a.n_tiles) {
        const uint64_t left = a.n_tiles - first;
        n += __popc(bm[w] & (left >= 32 ? 0xffffffffu : ((1u << (uint32_t)left) - 1u)));
      }
    }
  }
  a.cnt128[i] = n;
}

template <class C, int W>
__device__ __forceinline__ void load_unpack(const uint32_t *src, uint32_t (&code)[C::EPT]) {
  uint32_t w[C::EPT * W / 32];
#pragma unroll
  for (int j = 0; j < C::EPT * W / 32; ++j) w[j] = __ldg(src + j);
  unpack_words<W, C::EPT>(w, code);
}

template <class C>
__global__ void __launch_bounds__(kThreads) decode_kernel(const Args a) {
  extern __shared__ __align__(128) uint8_t smem[];   // one swizzled output stage
  if (*reinterpret_cast<volatile uint32_t *>(a.status) != 0) return;   // refused buffer: leave the output alone
  const uint32_t *sz32 = reinterpret_cast<const uint32_t *>(a.packed + a.off_sz);
  const uint8_t *pivot = a.packed + a.off_pivot;
  const uint64_t n_chunks = (a.n_tiles + C::TPC - 1) / C::TPC;
  for (uint64_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
    const uint64_t tile0 = c * C::TPC;
    const int half = threadIdx.x % C::LPT;
    const uint64_t tile = tile0 + threadIdx.x / C::LPT;
    const bool valid = tile < a.n_tiles;
    const ChunkPlan<C> plan = plan_chunk<C>(a, c);
    const uint32_t b = a.lo + plan.is_hi;

    float x[C::EPT];
    uint32_t pv = 0;
    if (valid) {
      const uint32_t szw = __ldg(sz32 + tile);
      const float s = __half2float(__ushort_as_half((unsigned short)(szw & 0xffffu)));
      const float z = __half2float(__ushort_as_half((unsigned short)(szw >> 16)));
      pv = __ldg(pivot + tile);
      const uint32_t *src = reinterpret_cast<const uint32_t *>(a.packed + a.off_payload + plan.goff + plan.row_off);
      uint32_t code[C::EPT];
      switch (b) {
        case 2: load_unpack<C, 2>(src, code); break;
        case 3: load_unpack<C, 3>(src, code); break;
        case 4: load_unpack<C, 4>(src, code); break;
        case 5: load_unpack<C, 5>(src, code); break;
        case 6: load_unpack<C, 6>(src, code); break;
        case 7: load_unpack<C, 7>(src, code); break;
        default: load_unpack<C, 8>(src, code); break;
      }
#pragma unroll
      for (int k = 0; k < C::EPT; ++k) x[k] = __fmaf_rn((float)code[k], s, z);
    } else {
#pragma unroll
      for (int k = 0; k < C::EPT; ++k) x[k] = 0.0f;
    }

    const bool flag = (pv & 0x80u) != 0;
    const unsigned fm = __ballot_sync(kFull, flag);
    if (flag) {
      const int d = pv & 0x7f;
      butterfly<C::EPT>(x);
      if constexpr (C::LPT == 2) {
#pragma unroll
        for (int k = 0; k < C::EPT; ++k) {
          const float p = __shfl_xor_sync(fm, x[k], 1);
          x[k] = half ? (p - x[k]) : (x[k] + p);
        }
      }
      constexpr float cG = (C::G == 32) ? 0.17677669529663687f : (C::G == 64) ? 0.125f : 0.08838834764831845f;
#pragma unroll
      for (int k = 0; k < C::EPT; ++k) x[k] = x[k] * cG;
      // un-swap coordinates 0 and d
      if constexpr (C::LPT == 1) {
        float xd = x[0];
#pragma unroll
        for (int k = 1; k < C::EPT; ++k) xd = (k == d) ? x[k] : xd;
        const float x0 = x[0];
#pragma unroll
        for (int k = 1; k < C::EPT; ++k) x[k] = (k == d) ? x0 : x[k];
        x[0] = xd;
      } else {
        const int lane = threadIdx.x & 31, owner = d / C::EPT, dl = d % C::EPT;
        float mine = x[0];
#pragma unroll
        for (int k = 1; k < C::EPT; ++k) mine = (k == dl) ? x[k] : mine;
        const float x0 = __shfl_sync(fm, x[0], lane & ~1);
        const float xd = __shfl_sync(fm, mine, (lane & ~1) + owner);
        if (half == owner) {
#pragma unroll
          for (int k = 0; k < C::EPT; ++k) x[k] = (k == dl) ? x0 : x[k];
        }
        if (half == 0) x[0] = xd;
      }
    }

    // stage the row (swizzled), then write the chunk out with coalesced 16-byte stores
    const int row = threadIdx.x;
    if constexpr (C::BF16) {
#pragma unroll
      for (int q = 0; q < C::CPR; ++q) {
        uint4 w;
        uint32_t u[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(x[8 * q + 2 * j], x[8 * q + 2 * j + 1]);
          u[j] = *reinterpret_cast<const uint32_t *>(&h2);
        }
        w.x = u[0]; w.y = u[1]; w.z = u[2]; w.w = u[3];
        *reinterpret_cast<uint4 *>(smem + (size_t)phys_chunk<C>(row, q) * 16) = w;
      }
    } else {
#pragma unroll
      for (int q = 0; q < C::CPR; ++q)
        *reinterpret_cast<float4 *>(smem + (size_t)phys_chunk<C>(row, q) * 16) =
            make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]);
    }
    __syncthreads();
    const uint64_t left = a.n_tiles - tile0;
    const uint32_t valid_bytes = (uint32_t)(left < (uint64_t)C::TPC ? left : (uint64_t)C::TPC) * C::G * C::ESZ;
    uint8_t *gout = a.out + tile0 * (uint64_t)(C::G * C::ESZ);
#pragma unroll
    for (int i = 0; i < C::CPR; ++i) {
      const int ci = i * kThreads + (int)threadIdx.x;
      if ((uint32_t)ci * 16u < valid_bytes)
        *reinterpret_cast<uint4 *>(gout + (size_t)ci * 16) =
            *reinterpret_cast<const uint4 *>(smem + (size_t)(ci ^ swz<C>(ci / C::CPR)) * 16);
    }
    __syncthreads();
  }
}

}  // namespace tahq
