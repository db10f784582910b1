// Warp-streaming encode kernel of the TAH-Quant boundary codec (sm_100a), for tiles owned by one lane
// (G = 32, 64).
//
// Every warp is an independent worker: it streams units of 32 consecutive tiles (one bit-map word)
// through a private cp.async ring in shared memory, one lane per tile, and never meets a CTA-wide
// barrier after the prologue.  Two things make that possible.
//   * Sec. 3.2 / 3.4: the widths are known before the kernel starts (scores and thresholds are in
//     memory), so the prologue turns the CTA's slice of scores into bit-map words, their running
//     population count, and (one look-back over the CTAs) the byte offset of every tile.
//   * Eq. 3-4: tiles that pass the pivot test cost about three times as much as the others.  A lane
//     handles an unflagged tile on the spot; tiles that may be flagged are only noted in a queue of
//     tile indices private to the warp.  When 32 are queued, their rows are fetched again (from L2,
//     where they were a moment ago) into a 32-row stage of the warp, and one iteration later the whole
//     warp runs the flagged path on them, one lane per row.  All warps therefore do the same amount
//     of work and no lane idles through the long path.
#pragma once

#include "tahq_kernels.cuh"

namespace tahq {

constexpr int kWarps = kThreads / 32;
constexpr int kSegWords = 1024;   // bit-map words (units) a CTA keeps in shared memory at a time

template <class C>
struct StreamCfg {
  static_assert(C::LPT == 1, "one lane per tile");
  static constexpr int UNIT_BYTES = 32 * C::ROWB;   // 32 rows
  static constexpr int WORDS = C::ROWB / 4;         // 32-bit words of one row
  static constexpr int smem_bytes(int nst) { return kWarps * (nst + 1) * UNIT_BYTES; }
};

// cp.async of unit u (tiles 32u .. 32u+31) into a warp-private slot, rows swizzled as everywhere
template <class C>
__device__ __forceinline__ void warp_issue_unit(const uint8_t *in, uint64_t n_tiles, uint64_t u, uint8_t *slot,
                                                int lane) {
  const uint64_t tile0 = u * 32;
  const uint8_t *src = in + tile0 * (uint64_t)C::ROWB + (size_t)lane * 16;
  if (tile0 + 32 <= n_tiles) {
#pragma unroll
    for (int i = 0; i < C::CPR; ++i) {
      const int piece = i * 32 + lane;
      cp_async16(slot + (size_t)phys_chunk<C>(piece / C::CPR, piece % C::CPR) * 16, src + (size_t)i * 512, 16);
    }
  } else {
    const uint32_t valid_bytes = tile0 < n_tiles ? (uint32_t)(n_tiles - tile0) * C::ROWB : 0u;
#pragma unroll
    for (int i = 0; i < C::CPR; ++i) {
      const int piece = i * 32 + lane;
      const bool ok = (uint32_t)piece * 16u < valid_bytes;
      cp_async16(slot + (size_t)phys_chunk<C>(piece / C::CPR, piece % C::CPR) * 16, ok ? src + (size_t)i * 512 : in,
                 ok ? 16 : 0);
    }
  }
}

// a row: shared memory <-> registers (raw words)
template <class C>
__device__ __forceinline__ void row_load_words(const uint8_t *stage, int row, uint32_t (&w)[C::ROWB / 4]) {
#pragma unroll
  for (int q = 0; q < C::CPR; ++q) {
    const uint4 v = *reinterpret_cast<const uint4 *>(stage + (size_t)phys_chunk<C>(row, q) * 16);
    w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
  }
}
template <class C>
__device__ __forceinline__ void row_store_words(uint8_t *stage, int row, const uint32_t (&w)[C::ROWB / 4]) {
#pragma unroll
  for (int q = 0; q < C::CPR; ++q)
    *reinterpret_cast<uint4 *>(stage + (size_t)phys_chunk<C>(row, q) * 16) =
        make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
}

// smallest and largest element of a row held as raw words
template <class C>
__device__ __forceinline__ void words_minmax(const uint32_t (&w)[C::ROWB / 4], float &mn, float &mx) {
  constexpr int NW = C::ROWB / 4;
  if constexpr (C::BF16) {
    uint32_t lo0 = bf2_min(w[0], w[2]), hi0 = bf2_max(w[0], w[2]);
    uint32_t lo1 = bf2_min(w[1], w[3]), hi1 = bf2_max(w[1], w[3]);
#pragma unroll
    for (int j = 4; j < NW; j += 4) {
      lo0 = bf2_min(lo0, bf2_min(w[j], w[j + 2])); hi0 = bf2_max(hi0, bf2_max(w[j], w[j + 2]));
      lo1 = bf2_min(lo1, bf2_min(w[j + 1], w[j + 3])); hi1 = bf2_max(hi1, bf2_max(w[j + 1], w[j + 3]));
    }
    lo0 = bf2_min(lo0, lo1); hi0 = bf2_max(hi0, hi1);
    mn = fminf(__uint_as_float(lo0 << 16), __uint_as_float(lo0 & 0xffff0000u));
    mx = fmaxf(__uint_as_float(hi0 << 16), __uint_as_float(hi0 & 0xffff0000u));
  } else {
    float l0 = fminf(__uint_as_float(w[0]), __uint_as_float(w[2])), h0 = fmaxf(__uint_as_float(w[0]), __uint_as_float(w[2]));
    float l1 = fminf(__uint_as_float(w[1]), __uint_as_float(w[3])), h1 = fmaxf(__uint_as_float(w[1]), __uint_as_float(w[3]));
#pragma unroll
    for (int j = 4; j < NW; j += 4) {
      l0 = fminf(l0, fminf(__uint_as_float(w[j]), __uint_as_float(w[j + 2])));
      h0 = fmaxf(h0, fmaxf(__uint_as_float(w[j]), __uint_as_float(w[j + 2])));
      l1 = fminf(l1, fminf(__uint_as_float(w[j + 1]), __uint_as_float(w[j + 3])));
      h1 = fmaxf(h1, fmaxf(__uint_as_float(w[j + 1]), __uint_as_float(w[j + 3])));
    }
    mn = fminf(l0, l1);
    mx = fmaxf(h0, h1);
  }
}

// Sec. 3.3-3.4 for a row that is not transformed, straight from its raw words: zero-point and scale
// from the known range, codes (computed once), then the bit stream at the lane's own width.
// Returns the stored {scale, zero}.
template <class C>
__device__ __forceinline__ uint32_t encode_plain_words(const uint32_t (&w)[C::ROWB / 4], float mn, float mx,
                                                       uint32_t bits, uint32_t *dst) {
  const Quantiser q = make_quantiser(mn, mx, bits);
  const float ymin = (mn - q.z) * q.inv_s, ymax = (mx - q.z) * q.inv_s;
  const bool safe = ymin >= -0.4999f && ymax < q.qmax + 0.4999f;
  const float nz = -q.z;   // x + (-z) is x - z
  const float2 is = f2(q.inv_s), mg = f2(kMagic);
  float2 t[C::EPT / 2];
#pragma unroll
  for (int i = 0; i < C::EPT / 2; ++i) {
    float2 d;
    if constexpr (C::BF16) bf2_add_f32(w[i], nz, d.x, d.y);
    else d = add2(f2(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1])), f2(nz));
    t[i] = fma2(d, is, mg);
  }
  if (!__all_sync(__activemask(), safe)) {
#pragma unroll
    for (int i = 0; i < C::EPT / 2; ++i)
      t[i] = f2(fminf(fmaxf(t[i].x, kMagic), kMagic + q.qmax), fminf(fmaxf(t[i].y, kMagic), kMagic + q.qmax));
  }
  auto tk = [&](int k) { return (k & 1) ? t[k >> 1].y : t[k >> 1].x; };
  pack_row<C::EPT>(tk, bits, dst);
  return q.sz;
}

// Eq. 3-4 + Sec. 3.3-3.4 for a queued row (shared memory): exact pivot test, pivot swap, Hadamard,
// range, codes, bit stream, stores.
template <class C>
__device__ __noinline__ void encode_queued_row(float tau, float eps_ratio, uint8_t *queue, int row, uint32_t bits,
                                               uint32_t *dst, uint32_t *sz, uint8_t *pv) {
  float a1, a2;
  row_top2<C>(queue, row, a1, a2);
  const float t1 = a2 + eps_ratio;
  const float t2 = tau * t1;
  const bool flag = a1 > t2;   // Eq. 3
  int d = 0;
  if (flag) {   // Eq. 4: the pivot swap P_d, done in shared memory before the row is loaded
    d = row_first_index_of<C>(queue, row, a1);
    row_swap_0_d<C, !C::BF16>(queue, row, d);
    asm volatile("" ::: "memory");
  }
  float2 p[C::EPT / 2];
  load_row_pairs<C>(queue, row, p);
  if (flag) {   // Eq. 4: (1/sqrt G) H_G
    butterfly2<C::EPT / 2>(p);
#pragma unroll
    for (int i = 0; i < C::EPT / 2; ++i)   // scalar products: they are added to right after
      p[i] = f2(p[i].x * hadamard_scale<C>(), p[i].y * hadamard_scale<C>());
  }
  float mn = fminf(p[0].x, p[0].y), mx = fmaxf(p[0].x, p[0].y);
#pragma unroll
  for (int i = 1; i < C::EPT / 2; ++i) {
    mn = fminf(mn, fminf(p[i].x, p[i].y));
    mx = fmaxf(mx, fmaxf(p[i].x, p[i].y));
  }
  const Quantiser q = make_quantiser(mn, mx, bits);
  quantise_pairs<C::EPT / 2>(p, mn, mx, q);
  *sz = q.sz;
  *pv = flag ? (uint8_t)(0x80 | d) : (uint8_t)0;
  pack_row<C::EPT>([&](int k) { return (k & 1) ? p[k >> 1].y : p[k >> 1].x; }, bits, dst);
}

constexpr int kQueueCap = 64;   // tile indices a warp can hold back (32 left over + 32 of one unit)

template <class C, int NST>
__global__ void __launch_bounds__(kThreads, 2) quant_pack_stream_kernel(const Args a) {
  using S = StreamCfg<C>;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint32_t s_bm[kSegWords];    // bit-map words of the segment
  __shared__ uint32_t s_pre[kSegWords];   // higher-width tiles of the segment before each word
  __shared__ uint32_t s_wsum[kWarps];
  __shared__ uint32_t s_qtile[kWarps][kQueueCap];   // held-back tile: (tile - first tile of the CTA) * 2 + higher width
  __shared__ uint32_t s_qhib[kWarps][kQueueCap];    // held-back tile: higher-width tiles before it, from the CTA's first
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt = (1u << lane) - 1u;
  uint8_t *ring = smem + (size_t)warp * (NST + 1) * S::UNIT_BYTES;
  uint8_t *fstage = ring + (size_t)NST * S::UNIT_BYTES;   // rows fetched again for the flagged path
  uint32_t *sz32 = reinterpret_cast<uint32_t *>(a.packed + a.off_sz);
  uint8_t *pivot = a.packed + a.off_pivot;
  uint32_t *bitmap = reinterpret_cast<uint32_t *>(a.packed + a.off_bitmap);
  uint8_t *payload = a.packed + a.off_payload;

  const uint64_t n_units = (a.n_tiles + 31) / 32;
  const uint64_t u0 = n_units * blockIdx.x / gridDim.x, u1 = n_units * (blockIdx.x + 1ull) / gridDim.x;
  const uint64_t tile_cta = u0 * 32;

  // the first units of a segment start moving before anything else
  auto prime = [&](uint64_t s0, uint64_t s1) {
#pragma unroll
    for (int s = 0; s < NST; ++s) {
      const uint64_t u = s0 + warp + (uint64_t)s * kWarps;
      if (u < s1) warp_issue_unit<C>(a.in, a.n_tiles, u, ring + (size_t)s * S::UNIT_BYTES, lane);
      cp_async_commit();
    }
  };
  prime(u0, u0 + kSegWords < u1 ? u0 + kSegWords : u1);

  if (blockIdx.x == 0) {   // header and the zero padding behind every section
    if (threadIdx.x < 32) reinterpret_cast<uint32_t *>(a.packed)[threadIdx.x] = a.header[threadIdx.x];
    for (int s = 0; s < 4; ++s) {
      const uint64_t from = s == 0 ? a.off_bitmap + 4 * n_units : s == 1 ? a.off_sz + 4 * a.n_tiles
                          : s == 2 ? a.off_pivot + a.n_tiles : a.off_payload + a.payload_bytes;
      const uint64_t to = s == 0 ? a.off_sz : s == 1 ? a.off_pivot : s == 2 ? a.off_payload : a.total_bytes;
      for (uint64_t o = from + threadIdx.x; o < to; o += kThreads) a.packed[o] = 0;
    }
  }

  if (u0 == u1) {   // more CTAs than units: still take part in the look-back
    bool unused;
    if (a.mixed) cta_exclusive_prefix(a, 0, false, unused);
    cp_async_wait<0>();
    return;
  }
  const bool single = u1 - u0 <= (uint64_t)kSegWords;
  uint64_t counted = 0;
  if (a.mixed && !single) {   // long slices: count first, the look-back needs the CTA's total
    GroupCursor pc;
    pc.init(a, u0 * 32);
    const uint64_t t1 = u1 * 32 < a.n_tiles ? u1 * 32 : a.n_tiles;
    uint32_t n = 0;
    for (uint64_t tb = u0 * 32; tb < t1; tb += kThreads) {
      const uint64_t t = tb + threadIdx.x;
      if (t < t1) n += pc.is_hi(a, t, threadIdx.x) ? 1u : 0u;
      pc.advance(a, kThreads);
    }
    counted = block_sum(n);
  }

  uint64_t base_hi = 0;    // higher-width tiles before this CTA, over the whole tensor
  uint32_t seg_hi = 0;     // higher-width tiles of this CTA's earlier segments
  uint32_t qhead = 0, qn = 0;   // this warp's queue of held-back tiles (circular)
  uint32_t f_n = 0;             // rows on their way into (or waiting in) fstage
  uint32_t f_tile = 0, f_hib = 0;   // lane j's row of fstage
  const uint64_t row_bytes = (uint64_t)C::ROWB;

  // fetch the rows of the first n (<= 32) queued tiles again; lane j keeps the j-th tile's particulars
  auto gather = [&](uint32_t n) {
    f_tile = s_qtile[warp][(qhead + lane) & (kQueueCap - 1)];
    f_hib = s_qhib[warp][(qhead + lane) & (kQueueCap - 1)];
#pragma unroll
    for (int i = 0; i < C::CPR; ++i) {
      const int piece = i * 32 + lane, r = piece / C::CPR, q = piece % C::CPR;
      const uint32_t tr = __shfl_sync(kFull, f_tile, r) >> 1;
      const bool ok = (uint32_t)r < n;
      cp_async16(fstage + (size_t)phys_chunk<C>(r, q) * 16,
                 ok ? a.in + (tile_cta + tr) * row_bytes + (size_t)q * 16 : a.in, ok ? 16 : 0);
    }
    cp_async_commit();
    f_n = n;
    qhead = (qhead + n) & (kQueueCap - 1);
    qn -= n;
  };
  // Eq. 3-4 on the rows of fstage, lane j on row j
  auto run_flagged = [&]() {
    if ((uint32_t)lane < f_n) {
      const uint64_t tile = tile_cta + (f_tile >> 1);
      const uint64_t off = (uint64_t)(C::G / 8) * ((uint64_t)a.lo * tile + base_hi + f_hib);
      encode_queued_row<C>(a.tau, a.eps_ratio, fstage, lane, a.lo + (f_tile & 1u), reinterpret_cast<uint32_t *>(payload + off),
                           sz32 + tile, pivot + tile);
    }
    f_n = 0;
    __syncwarp();
  };

  for (uint64_t s0 = u0; s0 < u1; s0 += kSegWords) {
    const uint64_t s1 = s0 + kSegWords < u1 ? s0 + kSegWords : u1;
    const uint32_t nw = (uint32_t)(s1 - s0);
    if (s0 != u0) {
      __syncthreads();   // every warp is done with the previous segment's words
      prime(s0, s1);
    }
    // ---- bit-map words of the segment (Sec. 3.2), written to the packed buffer as they are formed
    if (a.mixed) {
      GroupCursor pc;
      pc.init(a, s0 * 32);
      for (uint64_t tb = s0 * 32; tb < s1 * 32; tb += kThreads) {
        const uint64_t t = tb + threadIdx.x;
        const bool hi = t < a.n_tiles && pc.is_hi(a, t, threadIdx.x);
        const unsigned word = __ballot_sync(kFull, hi);
        if (lane == 0 && (t >> 5) < s1) {
          s_bm[(t >> 5) - s0] = word;
          bitmap[t >> 5] = word;
        }
        pc.advance(a, kThreads);
      }
    } else {
      for (uint32_t i = threadIdx.x; i < nw; i += kThreads) {
        s_bm[i] = 0;
        bitmap[s0 + i] = 0;
      }
    }
    __syncthreads();
    // ---- exclusive running count of higher-width tiles over the segment's words
    uint32_t seg_total;
    {
      constexpr int PER = kSegWords / kThreads;
      uint32_t c[PER], mine = 0;
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const uint32_t i = threadIdx.x * PER + j;
        c[j] = i < nw ? (uint32_t)__popc(s_bm[i]) : 0u;
        mine += c[j];
      }
      uint32_t incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o *= 2) {
        const uint32_t v = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) s_wsum[warp] = incl;
      __syncthreads();
      uint32_t before = incl - mine, total = 0;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const uint32_t v = s_wsum[w];
        before += w < warp ? v : 0u;
        total += v;
      }
      seg_total = total;
      before += seg_hi;
#pragma unroll
      for (int j = 0; j < PER; ++j) {
        const uint32_t i = threadIdx.x * PER + j;
        if (i < nw) s_pre[i] = before;
        before += c[j];
      }
    }
    if (s0 == u0 && a.mixed) {   // Sec. 3.4: higher-width tiles of all CTAs before this one
      bool unused;
      base_hi = cta_exclusive_prefix(a, single ? (uint64_t)seg_total : counted, false, unused);
    }
    __syncthreads();

    // ---- the warp's units of this segment
    int slot = 0;
    for (uint64_t u = s0 + warp; u < s1; u += kWarps) {
      cp_async_wait<NST - 1>();   // this unit has landed, and so have the rows fetched again one round ago
      __syncwarp();
      if (f_n) run_flagged();
      if (qn >= 32u) gather(32u);

      uint8_t *stage = ring + (size_t)slot * S::UNIT_BYTES;
      uint32_t w[S::WORDS];
      row_load_words<C>(stage, lane, w);
      __syncwarp();
      {   // the slot is free again: fetch the unit that comes NST rounds later
        const uint64_t un = u + (uint64_t)NST * kWarps;
        if (un < s1) warp_issue_unit<C>(a.in, a.n_tiles, un, stage, lane);
        cp_async_commit();
      }
      slot = (slot + 1 == NST) ? 0 : slot + 1;

      const uint32_t word = s_bm[u - s0];
      const uint32_t hi = (word >> lane) & 1u;
      const uint64_t tile = u * 32 + lane;
      const bool live = tile < a.n_tiles;
      const uint32_t hib = s_pre[u - s0] + (uint32_t)__popc(word & lt);

      // Eq. 3, first look: the second-largest magnitude is at least the smaller of |min| and |max| (they
      // sit at different positions, or every element is equal), so a tile whose largest magnitude does
      // not exceed tau * (that + varrho) cannot be flagged.  The others are held back for the exact test.
      float mn, mx;
      words_minmax<C>(w, mn, mx);
      const float m_big = fmaxf(fabsf(mn), fabsf(mx)), m_small = fminf(fabsf(mn), fabsf(mx));
      const bool maybe = live && m_big > a.tau * (m_small + a.eps_ratio);
      const unsigned held = __ballot_sync(kFull, maybe);
      if (maybe) {
        const uint32_t e = (qhead + qn + (uint32_t)__popc(held & lt)) & (kQueueCap - 1);
        s_qtile[warp][e] = (uint32_t)((tile - tile_cta) << 1) | hi;
        s_qhib[warp][e] = hib;
      }
      qn += (uint32_t)__popc(held);
      if (live && !maybe) {
        const uint64_t off = (uint64_t)(C::G / 8) * ((uint64_t)a.lo * tile + base_hi + hib);
        sz32[tile] = encode_plain_words<C>(w, mn, mx, a.lo + hi, reinterpret_cast<uint32_t *>(payload + off));
        pivot[tile] = 0;
      }
      __syncwarp();
    }
    cp_async_wait<0>();
    __syncwarp();
    seg_hi += seg_total;
  }
  // ---- what is still held back
  if (f_n) run_flagged();
  while (qn) {
    gather(qn < 32u ? qn : 32u);
    cp_async_wait<0>();
    __syncwarp();
    run_flagged();
  }
}

}  // namespace tahq
