// Host side of the C ABI declared in include/tahq.h: parameter validation, layout of the packed
// buffer and of the workspace, kernel selection and launches on the caller's stream.
#include "../../include/tahq.h"

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <utility>
#include <vector>

#include "tahq_stream.cuh"
#include "qnaive.cuh"

namespace tahq {

static thread_local int g_launches = 0;

// Optional per-kernel timing (tahq_profile): every launch is bracketed by two events on its stream.
struct ProfRec { const char *name; cudaEvent_t e0, e1; };
static bool g_prof_on = false;
static std::vector<ProfRec> g_prof;

struct LaunchScope {
  cudaStream_t st;
  bool on;
  LaunchScope(const char *name, cudaStream_t s) : st(s), on(g_prof_on) {
    ++g_launches;
    if (on) {
      ProfRec r{name, nullptr, nullptr};
      cudaEventCreate(&r.e0);
      cudaEventCreate(&r.e1);
      cudaEventRecord(r.e0, st);
      g_prof.push_back(r);
    }
  }
  ~LaunchScope() {
    if (on) cudaEventRecord(g_prof.back().e1, st);
  }
};
#define TAHQ_LAUNCH(name, st, ...) do { LaunchScope scope_(name, st); __VA_ARGS__; } while (0)

struct Plan {
  tahq_layout L;
  uint32_t f;             // budget % 1000
  bool mixed;             // two widths in use (k_hi > 0)
  bool direct;            // small ranking groups: select straight from the scores
  uint32_t cpg, cand_cap, sel_m;
  uint32_t alloc_m;            // quantisation tiles per allocation tile (Sec. 3.2; 1 by default)
  uint64_t rank_per_group, rank_k;   // allocation tiles per ranking group, and how many of them get the higher width
  // workspace offsets
  uint64_t ws_flags, ws_ncand, ws_done, ws_nabove, ws_hist, ws_zero_end, ws_scores, ws_theta, ws_cand, ws_total;
};

static uint64_t up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// TAHQ_ENCODE_PATH=fused in the environment switches large-group encodes to the single cooperative kernel.
// It is off by default: measured on B200 it never beat the three-kernel path (equal encode time on the
// LLaMA-7B-shaped tensor, 7 % slower round trips because a cooperative launch does not overlap its
// neighbours' launch latency; 7-13 % slower on 320 MiB and 1 GiB tensors).
static bool fused_encode_wanted() {
  static const bool v = [] {
    const char *e = std::getenv("TAHQ_ENCODE_PATH");
    return e && std::strcmp(e, "fused") == 0;
  }();
  return v;
}


static tahq_status make_plan(const tahq_params *p, Plan *pl) {
  if (!p || p->struct_size != sizeof(tahq_params)) return TAHQ_ERR_INVALID_ARG;
  const uint32_t G = p->tile;
  if (G < 8 || G > 128 || (G & (G - 1))) return TAHQ_ERR_INVALID_ARG;
  if (p->dtype > 1 || p->rounding > 1) return TAHQ_ERR_INVALID_ARG;
  if (p->tokens == 0 || p->hidden == 0 || p->hidden % G) return TAHQ_ERR_INVALID_ARG;
  const uint64_t S = p->group_tokens ? p->group_tokens : p->tokens;
  if (p->tokens % S) return TAHQ_ERR_INVALID_ARG;
  const uint32_t beta = p->budget_millibits;
  if (beta < 2000 || beta > 8000) return TAHQ_ERR_INVALID_ARG;
  // varsigma must be a positive normal number: p + varsigma is split into exponent and mantissa
  if (!(p->tau >= 0.0f) || !(p->eps_l1 >= 0.0f) || !(p->eps_log >= 1.17549435e-38f) || !(p->eps_ratio >= 0.0f))
    return TAHQ_ERR_INVALID_ARG;
  const uint64_t M = p->hidden / G;
  if (p->tokens > (1ull << 40) / M) return TAHQ_ERR_INVALID_ARG;
  const uint32_t A = p->alloc_tile ? p->alloc_tile : G;   // allocation-tile width (Sec. 3.2)
  if (A % G || A > p->hidden || p->hidden % A) return TAHQ_ERR_INVALID_ARG;
  pl->alloc_m = A / G;
  tahq_layout &L = pl->L;
  L.n_tiles = p->tokens * M;
  L.tiles_per_group = S * M;
  L.n_groups = p->tokens / S;
  if (L.tiles_per_group >= (1ull << 32) || L.n_tiles >= (1ull << 36)) return TAHQ_ERR_INVALID_ARG;
  if (L.n_tiles > (uint64_t)kMaxGrid * kChunkCap * 128) return TAHQ_ERR_UNSUPPORTED;   // one call: up to 2^28 tiles
  pl->f = beta % 1000;
  L.lo_bits = beta / 1000;
  L.hi_bits = pl->f ? L.lo_bits + 1 : L.lo_bits;
  pl->rank_per_group = L.tiles_per_group / pl->alloc_m;
  pl->rank_k = pl->rank_per_group * (uint64_t)pl->f / 1000u;
  L.k_hi = pl->rank_k * pl->alloc_m;
  L.payload_bytes = L.n_groups * (uint64_t)(G / 8) * (L.tiles_per_group * L.lo_bits + L.k_hi);
  L.off_bitmap = 128;
  L.off_scale_zero = up(L.off_bitmap + (L.n_tiles + 7) / 8, 128);
  L.off_pivot = up(L.off_scale_zero + 4 * L.n_tiles, 128);
  L.off_payload = up(L.off_pivot + L.n_tiles, 128);
  L.total_bytes = up(L.off_payload + L.payload_bytes, 128);
  if (pl->alloc_m > 1 && A > 8192) return TAHQ_ERR_UNSUPPORTED;

  pl->mixed = L.k_hi > 0;
  pl->direct = pl->rank_per_group <= (uint64_t)kSortCap;
  pl->cpg = 1;
  pl->sel_m = 1;
  pl->cand_cap = 0;
  if (pl->mixed && !pl->direct) {
    // one CTA per slice of the group's scores, or several slices per CTA so that the grid stays near one wave
    const uint64_t slices = (pl->rank_per_group + kSelSlice - 1) / kSelSlice;
    uint64_t m = (slices * L.n_groups + 255) / 256;
    m = m < 1 ? 1 : m > 64 ? 64 : m;
    pl->sel_m = (uint32_t)m;
    pl->cpg = (uint32_t)((slices + m - 1) / m);
    // select_kernel copes with more candidates than the list holds; the single-launch encode does not, so
    // there the list holds a whole group (every tile is a candidate when all scores are equal)
    const uint64_t cap = fused_encode_wanted() ? 0xffffffffull : 32768ull;
    pl->cand_cap = (uint32_t)(pl->rank_per_group < cap ? pl->rank_per_group : cap);
  }
  const bool hist = pl->mixed && !pl->direct;
  uint64_t o = 256;                                         // status word and friends
  pl->ws_flags = o;  o += 8ull * kMaxGrid;
  pl->ws_ncand = o;  o = up(o + (hist ? 4 * L.n_groups : 0), 256);
  pl->ws_done = o;   o = up(o + (hist ? 4 * L.n_groups : 0), 256);
  pl->ws_nabove = o; o = up(o + (hist ? 4 * L.n_groups : 0), 256);
  pl->ws_hist = o;   o += hist ? 4ull * kBins * L.n_groups : 0;
  pl->ws_zero_end = o;                                      // [0, ws_zero_end) is cleared by every encode
  pl->ws_scores = o; o = up(o + (pl->mixed ? 4 * (L.n_tiles / pl->alloc_m) : 0), 256);
  pl->ws_theta = o;  o = up(o + (pl->mixed ? 8 * L.n_groups : 0), 256);
  pl->ws_cand = o;   o = up(o + 8ull * pl->cand_cap * L.n_groups, 256);
  pl->ws_total = o;
  return TAHQ_OK;
}

static void fill_header(const tahq_params *p, const Plan &pl, uint32_t *h) {
  std::memset(h, 0, 128);
  h[22] = pl.alloc_m > 1 ? pl.alloc_m * p->tile : 0u;   // allocation-tile width when it is not the tile
  auto f2u = [](float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; };
  auto put64 = [&](int w, uint64_t v) { h[w] = (uint32_t)v; h[w + 1] = (uint32_t)(v >> 32); };
  h[0] = 0x51484154u;  // "TAHQ"
  h[1] = 1;
  h[2] = p->dtype;
  h[3] = p->rounding;
  put64(4, p->tokens);
  h[6] = p->hidden;
  h[7] = p->tile;
  h[8] = (uint32_t)(pl.L.tiles_per_group / (p->hidden / p->tile));
  h[9] = p->budget_millibits;
  h[10] = f2u(p->tau);
  h[11] = f2u(p->eps_l1);
  h[12] = f2u(p->eps_log);
  h[13] = f2u(p->eps_ratio);
  put64(14, p->seed);
  put64(16, pl.L.n_tiles);
  put64(18, pl.L.payload_bytes);
  put64(20, pl.L.total_bytes);
}

static void fill_args(const tahq_params *p, const Plan &pl, uint8_t *ws, Args *a) {
  std::memset(a, 0, sizeof(*a));
  a->n_tiles = pl.L.n_tiles;
  a->tiles_per_group = pl.L.tiles_per_group;
  a->k_hi = pl.L.k_hi;
  a->rank_per_group = pl.rank_per_group;
  a->rank_k = pl.rank_k;
  a->alloc_m = pl.alloc_m;
  a->n_groups = pl.L.n_groups;
  a->lo = pl.L.lo_bits;
  a->mixed = pl.mixed;
  a->off_bitmap = pl.L.off_bitmap;
  a->off_sz = pl.L.off_scale_zero;
  a->off_pivot = pl.L.off_pivot;
  a->off_payload = pl.L.off_payload;
  a->payload_bytes = pl.L.payload_bytes;
  a->total_bytes = pl.L.total_bytes;
  a->tau = p->tau;
  a->eps_l1 = p->eps_l1;
  a->eps_log = p->eps_log;
  a->seed = p->seed;
  a->eps_ratio = p->eps_ratio;
  a->status = reinterpret_cast<uint32_t *>(ws);
  a->gbar = reinterpret_cast<uint32_t *>(ws) + 16;   // inside the status block, cleared with it
  a->ncand = reinterpret_cast<uint32_t *>(ws + pl.ws_ncand);
  a->hist = reinterpret_cast<uint32_t *>(ws + pl.ws_hist);
  a->scores = reinterpret_cast<float *>(ws + pl.ws_scores);
  a->done = reinterpret_cast<uint32_t *>(ws + pl.ws_done);
  a->nabove = reinterpret_cast<uint32_t *>(ws + pl.ws_nabove);
  a->bf16 = p->dtype == TAHQ_BF16;
  a->tile = p->tile;
  a->flags = reinterpret_cast<unsigned long long *>(ws + pl.ws_flags);
  a->theta = reinterpret_cast<unsigned long long *>(ws + pl.ws_theta);
  a->cand = reinterpret_cast<unsigned long long *>(ws + pl.ws_cand);
  a->cand_cap = pl.cand_cap;
  a->cpg = pl.cpg;
  a->sel_m = pl.sel_m;
  a->direct = pl.direct;
  // the screening score leaves varsigma out; its share of the score is below G * varsigma / ln 2
  a->exact_scores = pl.direct || pl.alloc_m > 1 || (double)p->tile * (double)p->eps_log > 1e-5;
  fill_header(p, pl, a->header);
}

// ---- launch helpers ----------------------------------------------------------------------

struct DevInfo { int dev, sms; };
static bool dev_info(DevInfo *d) {
  if (cudaGetDevice(&d->dev) != cudaSuccess) return false;
  return cudaDeviceGetAttribute(&d->sms, cudaDevAttrMultiProcessorCount, d->dev) == cudaSuccess;
}

// Opt a kernel into its dynamic shared memory once per device and return resident CTAs per SM.
template <class K>
static int prepare(K kernel, int smem, const DevInfo &d, std::atomic<int> *cache) {
  int v = cache[d.dev & 63].load(std::memory_order_acquire);
  if (v > 0) return v;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return 0;
  int occ = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kThreads, smem) != cudaSuccess || occ < 1)
    return 0;
  cache[d.dev & 63].store(occ, std::memory_order_release);
  return occ;
}

// Launch a kernel as a programmatic dependent of the kernel in front of it in the stream: the launch is set up
// while that kernel still runs (about 2 us less per kernel boundary, measured); the kernel starts with
// griddepcontrol.wait, so it reads nothing before that kernel is done.
template <class... P, class... A>
static cudaError_t launch_dependent(void (*kernel)(P...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                    A &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...);
  if (e == cudaErrorNotSupported || e == cudaErrorInvalidValue) {   // attribute refused: an ordinary launch does
    (void)cudaGetLastError();
    cfg.numAttrs = 0;
    e = cudaLaunchKernelEx(&cfg, kernel, args...);
  }
  return e;
}

// Zero the first `bytes` (a multiple of 16) of the workspace with a kernel, so that the call's next kernel can
// be its programmatic dependent.
static tahq_status clear_workspace(void *d_ws, uint64_t bytes, cudaStream_t st) {
  const uint64_t n16 = bytes / 16;
  const unsigned grid = (unsigned)std::min<uint64_t>((n16 + kThreads - 1) / kThreads, 592);
  TAHQ_LAUNCH("clear", st, clear_kernel<<<grid ? grid : 1, kThreads, 0, st>>>(static_cast<uint4 *>(d_ws), n16));
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

template <class C> struct Stages {
  static constexpr int STATS = 2;
  static constexpr int QUANT = (C::ROWB == 256) ? 2 : (C::ROWB == 128 ? 2 : 3);
};

// CTAs of a persistent tile kernel: every SM filled to the kernel's occupancy, never more than chunks.
static unsigned persistent_grid(uint64_t n_chunks, const DevInfo &d, int occ) {
  uint64_t cap = (uint64_t)d.sms * occ;
  if (cap > (uint64_t)kMaxGrid) cap = kMaxGrid;
  return (unsigned)(n_chunks < cap ? n_chunks : cap);
}

// Tensor map of the input seen as [n_tiles rows x 128 bytes] with boxes of 32 rows and the 128-byte
// swizzle, for the tiled TMA copies of the warp-streaming kernels.  The driver's encoder is looked up once
// through the runtime (no link-time dependency on libcuda).  Returns false when TMA cannot be used here
// (rows are not 128 bytes, too many rows for a 32-bit coordinate, or the encoder is unavailable).
template <class C>
static bool make_row_map(const void *in, uint64_t n_tiles, CUtensorMap *tm) {
  std::memset(tm, 0, sizeof(*tm));
  if (C::LPT != 1 || C::ROWB != 128 || n_tiles >= 0x7fffffe0ull) return false;
  typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn enc = [] {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<encode_fn>(f);
  }();
  if (!enc) { cudaGetLastError(); return false; }
  const cuuint64_t dims[2] = {(cuuint64_t)C::EPT, (cuuint64_t)n_tiles};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {(cuuint32_t)C::EPT, 32};
  const cuuint32_t estr[2] = {1, 1};
  return enc(tm, C::BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
             const_cast<void *>(in), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <class C, bool SR>
static tahq_status encode_t(const Plan &pl, const Args &a_in, cudaStream_t st) {
  DevInfo d;
  if (!dev_info(&d)) return TAHQ_ERR_CUDA;
  Args a = a_in;
  CUtensorMap tmap;
  a.use_tma = make_row_map<C>(a.in, a.n_tiles, &tmap) ? 1u : 0u;
  const uint64_t n_chunks = (a.n_tiles + C::TPC - 1) / C::TPC;
  static std::atomic<int> occ_stats[64], occ_quant[64], sel_ready[64], occ_fused[64];
  if constexpr (C::LPT == 1) {
    // large ranking groups, on request: the whole encode as one cooperative launch (grid-wide barriers
    // between scoring, the exact re-scoring near each group's threshold, and quantise + pack); if the device
    // cannot keep the grid resident the three-kernel path below does the same work
    if (pl.mixed && !pl.direct && pl.alloc_m == 1 && fused_encode_wanted()) {
      const int smem = StreamCfg<C>::smem_bytes(2);
      const int occ = prepare(encode_fused_kernel<C, SR>, smem, d, occ_fused);
      if (occ) {
        const uint64_t n_units = (a.n_tiles + 31) / 32;
        const unsigned grid = persistent_grid((n_units + kWarps - 1) / kWarps, d, occ);
        void *args[] = {&a, &tmap};
        cudaError_t e;
        {
          LaunchScope scope_("encode_fused", st);
          e = cudaLaunchCooperativeKernel(reinterpret_cast<void *>(encode_fused_kernel<C, SR>), dim3(grid),
                                          dim3(kThreads), args, (size_t)smem, st);
        }
        if (e == cudaSuccess) return TAHQ_OK;
        cudaGetLastError();   // not launched: fall through
        --g_launches;
      }
    }
  }
  if (pl.mixed && pl.alloc_m > 1) {   // Sec. 3.2 with A = m * G: one warp per allocation tile, exact scores
    const uint64_t n_alloc = a.n_tiles / pl.alloc_m;
    const uint64_t want = (n_alloc + kWarps - 1) / kWarps, cap = (uint64_t)d.sms * 8;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    TAHQ_LAUNCH("alloc_score", st, launch_dependent(alloc_score_kernel<C::BF16>, grid, kThreads, 0, st, a));
  }
  if (pl.mixed) {
    if (pl.alloc_m > 1) {
      // scores are in place
    } else if constexpr (C::LPT == 1) {
      constexpr int NS = C::ROWB <= 128 ? 3 : 2;
      const int smem = kWarps * NS * StreamCfg<C>::UNIT_BYTES + 256;   // ring slots, then the warps' mbarriers
      static std::atomic<int> occ_exact[64];
      const int occ = a.exact_scores ? prepare(stats_stream_kernel<C, NS, true>, smem, d, occ_exact)
                                     : prepare(stats_stream_kernel<C, NS, false>, smem, d, occ_stats);
      if (!occ) return TAHQ_ERR_CUDA;
      const uint64_t n_units = (a.n_tiles + 31) / 32;
      const unsigned grid = persistent_grid((n_units + kWarps - 1) / kWarps, d, occ);
      if (a.exact_scores)
        TAHQ_LAUNCH("stats", st, launch_dependent(stats_stream_kernel<C, NS, true>, grid, kThreads, smem, st, a, tmap));
      else
        TAHQ_LAUNCH("stats", st, launch_dependent(stats_stream_kernel<C, NS, false>, grid, kThreads, smem, st, a, tmap));
    } else {
      constexpr int NS = Stages<C>::STATS;
      const int smem = NS * C::STAGE_BYTES;
      const int occ = prepare(stats_kernel<C, NS>, smem, d, occ_stats);
      if (!occ) return TAHQ_ERR_CUDA;
      TAHQ_LAUNCH("stats", st,
                  launch_dependent(stats_kernel<C, NS>, persistent_grid(n_chunks, d, occ), kThreads, smem, st, a));
    }
    const int sel_smem = kSortCap * 8;
    if (!sel_ready[d.dev & 63].load(std::memory_order_acquire)) {
      if (cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sel_smem) != cudaSuccess)
        return TAHQ_ERR_CUDA;
      sel_ready[d.dev & 63].store(1, std::memory_order_release);
    }
    TAHQ_LAUNCH("select", st,
                launch_dependent(select_kernel, (unsigned)(a.n_groups * a.cpg), kSelThreads, sel_smem, st, a));
  }
  if constexpr (C::LPT == 1) {   // one lane per tile: warps stream units of 32 tiles independently
    constexpr int NQ = 2;
    const int smem = StreamCfg<C>::smem_bytes(NQ);
    static std::atomic<int> occ_wide[64];
    const bool narrow = a.lo + a.mixed <= 4u;   // no width above 4 bits: the kernel compiled for just that
    const int occ = narrow ? prepare(quant_pack_stream_kernel<C, NQ, SR, true>, smem, d, occ_quant)
                           : prepare(quant_pack_stream_kernel<C, NQ, SR, false>, smem, d, occ_wide);
    if (!occ) return TAHQ_ERR_CUDA;
    const uint64_t n_units = (a.n_tiles + 31) / 32;
    const unsigned grid = persistent_grid((n_units + kWarps - 1) / kWarps, d, occ);
    if (narrow)
      TAHQ_LAUNCH("quant_pack", st,
                  launch_dependent(quant_pack_stream_kernel<C, NQ, SR, true>, grid, kThreads, smem, st, a, tmap));
    else
      TAHQ_LAUNCH("quant_pack", st,
                  launch_dependent(quant_pack_stream_kernel<C, NQ, SR, false>, grid, kThreads, smem, st, a, tmap));
  } else {
    constexpr int NQ = Stages<C>::QUANT;
    const int smem = NQ * (C::STAGE_BYTES + C::TPC * 4);
    const int occ = prepare(quant_pack_kernel<C, NQ, SR>, smem, d, occ_quant);
    if (!occ) return TAHQ_ERR_CUDA;
    TAHQ_LAUNCH("quant_pack", st,
                launch_dependent(quant_pack_kernel<C, NQ, SR>, persistent_grid(n_chunks, d, occ), kThreads, smem, st, a));
  }
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

template <class C>
static tahq_status decode_t(const Plan &pl, const Args &a, cudaStream_t st) {
  DevInfo d;
  if (!dev_info(&d)) return TAHQ_ERR_CUDA;
  const uint64_t n_chunks = (a.n_tiles + C::TPC - 1) / C::TPC;
  static std::atomic<int> occ_dec[64];
  (void)pl;
  if constexpr (C::LPT == 1) {   // one lane per tile: warps stream units of 32 tiles independently
    const int smem = DecStreamCfg<C>::TOTAL;
    const int occ = prepare(decode_stream_kernel<C>, smem, d, occ_dec);
    if (!occ) return TAHQ_ERR_CUDA;
    const uint64_t n_units = (a.n_tiles + 31) / 32;
    TAHQ_LAUNCH("decode", st,
                launch_dependent(decode_stream_kernel<C>, persistent_grid((n_units + kWarps - 1) / kWarps, d, occ),
                                 kThreads, smem, st, a));
  } else {
    const int smem = DecSmem<C>::TOTAL;
    const int occ = prepare(decode_kernel<C>, smem, d, occ_dec);
    if (!occ) return TAHQ_ERR_CUDA;
    unsigned grid = persistent_grid(n_chunks, d, occ);
    const uint64_t need = (n_chunks + kChunkCap - 1) / kChunkCap;   // a CTA keeps its chunks' bit map in shared memory
    if (grid < need) grid = (unsigned)need;
    TAHQ_LAUNCH("decode", st, launch_dependent(decode_kernel<C>, grid, kThreads, smem, st, a));
  }
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Scratch for tahq_encode_noalloc: part of the library image, resident on every GPU that loads it.
// In host code this name is only a handle; the device address is looked up once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TAHQ_NOALLOC_SCRATCH_BYTES];
static void *g_noalloc_addr[64];
static std::atomic<int> g_noalloc_ready[64];

}  // namespace tahq

using namespace tahq;

extern "C" {

size_t tahq_packed_bound(const tahq_params *p) {
  Plan pl;
  return make_plan(p, &pl) == TAHQ_OK ? (size_t)pl.L.total_bytes : 0;
}

tahq_status tahq_packed_layout(const tahq_params *p, tahq_layout *out) {
  Plan pl;
  const tahq_status s = make_plan(p, &pl);
  if (s != TAHQ_OK) return s;
  if (!out) return TAHQ_ERR_INVALID_ARG;
  *out = pl.L;
  return TAHQ_OK;
}

size_t tahq_workspace_bound(const tahq_params *p) {
  Plan pl;
  return make_plan(p, &pl) == TAHQ_OK ? (size_t)pl.ws_total : 0;
}

tahq_status tahq_encode(const tahq_params *p, const void *d_in, void *d_packed, size_t packed_cap, void *d_ws,
                        size_t ws_cap, tahq_stream stream) {
  g_launches = 0;
  Plan pl;
  const tahq_status s = make_plan(p, &pl);
  if (s != TAHQ_OK) return s;
  if (!d_in || !d_packed || !d_ws) return TAHQ_ERR_INVALID_ARG;
  if (packed_cap < pl.L.total_bytes || ws_cap < pl.ws_total) return TAHQ_ERR_BUFFER_TOO_SMALL;
  if (!aligned16(d_in) || !aligned16(d_packed) || !aligned16(d_ws)) return TAHQ_ERR_MISALIGNED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  Args a;
  fill_args(p, pl, static_cast<uint8_t *>(d_ws), &a);
  a.in = static_cast<const uint8_t *>(d_in);
  a.packed = static_cast<uint8_t *>(d_packed);
  if (clear_workspace(d_ws, pl.ws_zero_end, st) != TAHQ_OK) return TAHQ_ERR_CUDA;
  const bool bf = p->dtype == TAHQ_BF16;
  if (p->rounding == 1) {   // stochastic rounding: kernels of their own, the default path carries none of it
    switch (p->tile) {
      case 8: return bf ? encode_t<Cfg<8, true>, true>(pl, a, st) : encode_t<Cfg<8, false>, true>(pl, a, st);
      case 16: return bf ? encode_t<Cfg<16, true>, true>(pl, a, st) : encode_t<Cfg<16, false>, true>(pl, a, st);
      case 32: return bf ? encode_t<Cfg<32, true>, true>(pl, a, st) : encode_t<Cfg<32, false>, true>(pl, a, st);
      case 64: return bf ? encode_t<Cfg<64, true>, true>(pl, a, st) : encode_t<Cfg<64, false>, true>(pl, a, st);
      default: return bf ? encode_t<Cfg<128, true>, true>(pl, a, st) : encode_t<Cfg<128, false>, true>(pl, a, st);
    }
  }
  switch (p->tile) {
    case 8: return bf ? encode_t<Cfg<8, true>, false>(pl, a, st) : encode_t<Cfg<8, false>, false>(pl, a, st);
    case 16: return bf ? encode_t<Cfg<16, true>, false>(pl, a, st) : encode_t<Cfg<16, false>, false>(pl, a, st);
    case 32: return bf ? encode_t<Cfg<32, true>, false>(pl, a, st) : encode_t<Cfg<32, false>, false>(pl, a, st);
    case 64: return bf ? encode_t<Cfg<64, true>, false>(pl, a, st) : encode_t<Cfg<64, false>, false>(pl, a, st);
    default: return bf ? encode_t<Cfg<128, true>, false>(pl, a, st) : encode_t<Cfg<128, false>, false>(pl, a, st);
  }
}

tahq_status tahq_decode(const tahq_params *p, const void *d_packed, size_t packed_bytes, void *d_out, void *d_ws,
                        size_t ws_cap, tahq_stream stream) {
  g_launches = 0;
  Plan pl;
  const tahq_status s = make_plan(p, &pl);
  if (s != TAHQ_OK) return s;
  if (!d_out || !d_packed || !d_ws) return TAHQ_ERR_INVALID_ARG;
  if (packed_bytes < pl.L.total_bytes || ws_cap < pl.ws_total) return TAHQ_ERR_BUFFER_TOO_SMALL;
  if (!aligned16(d_out) || !aligned16(d_packed) || !aligned16(d_ws)) return TAHQ_ERR_MISALIGNED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  Args a;
  fill_args(p, pl, static_cast<uint8_t *>(d_ws), &a);
  a.packed = const_cast<uint8_t *>(static_cast<const uint8_t *>(d_packed));
  a.out = static_cast<uint8_t *>(d_out);
  // Up to 65536 bit-map words (256 KiB) the streaming kernel needs no look-back and nothing cleared: one launch.
  a.own_prefix = p->tile != 128 && (pl.L.n_tiles + 31) / 32 <= 65536;
  if (!a.own_prefix && clear_workspace(d_ws, pl.ws_ncand, st) != TAHQ_OK) return TAHQ_ERR_CUDA;   // status + flags
  const bool bf = p->dtype == TAHQ_BF16;
  switch (p->tile) {
    case 8: return bf ? decode_t<Cfg<8, true>>(pl, a, st) : decode_t<Cfg<8, false>>(pl, a, st);
    case 16: return bf ? decode_t<Cfg<16, true>>(pl, a, st) : decode_t<Cfg<16, false>>(pl, a, st);
    case 32: return bf ? decode_t<Cfg<32, true>>(pl, a, st) : decode_t<Cfg<32, false>>(pl, a, st);
    case 64: return bf ? decode_t<Cfg<64, true>>(pl, a, st) : decode_t<Cfg<64, false>>(pl, a, st);
    default: return bf ? decode_t<Cfg<128, true>>(pl, a, st) : decode_t<Cfg<128, false>>(pl, a, st);
  }
}

tahq_status tahq_encode_noalloc(const tahq_params *p, const void *d_in, void *d_packed, size_t packed_cap,
                                tahq_stream stream) {
  g_launches = 0;
  Plan pl;
  const tahq_status s = make_plan(p, &pl);
  if (s != TAHQ_OK) return s;
  if (pl.ws_total > (uint64_t)TAHQ_NOALLOC_SCRATCH_BYTES) return TAHQ_ERR_TOO_LARGE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TAHQ_ERR_CUDA;
  if (!g_noalloc_ready[dev].load(std::memory_order_acquire)) {
    // set-up, once per device, with that device current: the device address behind the symbol
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return TAHQ_ERR_CUDA;
    g_noalloc_addr[dev] = ptr;
    g_noalloc_ready[dev].store(1, std::memory_order_release);
  }
  // tahq_encode clears the head of the workspace (status, flags, histograms, counters) on the stream
  return tahq_encode(p, d_in, d_packed, packed_cap, g_noalloc_addr[dev], TAHQ_NOALLOC_SCRATCH_BYTES, stream);
}

// ---- fixed-point gradient compressor -------------------------------------------------------------------
namespace {
struct QPlan { uint64_t n_scales, off_scales, off_payload, row_bytes, total_bytes; };
tahq_status q_plan(const tahq_qnaive_params *p, QPlan *q) {
  if (!p || p->struct_size != sizeof(tahq_qnaive_params)) return TAHQ_ERR_INVALID_ARG;
  if (p->dtype > 1 || p->per_tensor > 1) return TAHQ_ERR_INVALID_ARG;
  if (p->tokens == 0 || p->hidden == 0 || p->hidden % 8) return TAHQ_ERR_INVALID_ARG;
  if (p->bits < 2 || p->bits > 16) return TAHQ_ERR_INVALID_ARG;
  if (!(p->prescale > 0.0f) || p->prescale > 3.402823466e38f) return TAHQ_ERR_INVALID_ARG;
  q->n_scales = p->per_tensor ? 1 : p->tokens;
  q->row_bytes = up(((uint64_t)p->hidden * p->bits + 7) / 8, 16);
  q->off_scales = 128;
  q->off_payload = up(q->off_scales + 4 * q->n_scales, 128);
  q->total_bytes = up(q->off_payload + p->tokens * q->row_bytes, 128);
  return TAHQ_OK;
}
void q_args(const tahq_qnaive_params *p, const QPlan &q, QArgs *a, void *ws) {
  std::memset(a, 0, sizeof(*a));
  a->tokens = p->tokens; a->hidden = p->hidden; a->bits = p->bits; a->per_tensor = p->per_tensor;
  a->prescale = p->prescale;
  a->off_scales = q.off_scales; a->off_payload = q.off_payload; a->row_bytes = q.row_bytes; a->total_bytes = q.total_bytes;
  a->status = reinterpret_cast<uint32_t *>(ws);
  a->gmax = reinterpret_cast<uint32_t *>(ws) + 16;
  uint32_t *h = a->header;
  std::memcpy(h, "TAHN", 4);
  h[1] = 1; h[2] = p->dtype; h[3] = p->bits;
  h[4] = (uint32_t)p->tokens; h[5] = (uint32_t)(p->tokens >> 32);
  h[6] = p->hidden; h[7] = p->per_tensor;
  std::memcpy(&h[8], &p->prescale, 4);
  h[10] = (uint32_t)q.row_bytes; h[11] = (uint32_t)(q.row_bytes >> 32);
  h[12] = (uint32_t)q.total_bytes; h[13] = (uint32_t)(q.total_bytes >> 32);
}
unsigned q_grid(uint64_t tokens, const DevInfo &d) {
  const uint64_t want = (tokens + 7) / 8, cap = (uint64_t)d.sms * 8;
  return (unsigned)(want < cap ? want : cap);
}
}  // namespace

size_t tahq_qnaive_packed_bound(const tahq_qnaive_params *p) {
  QPlan q;
  return q_plan(p, &q) == TAHQ_OK ? (size_t)q.total_bytes : 0;
}

size_t tahq_qnaive_workspace_bound(const tahq_qnaive_params *p) {
  QPlan q;
  return q_plan(p, &q) == TAHQ_OK ? 256 : 0;
}

tahq_status tahq_qnaive_encode(const tahq_qnaive_params *p, const void *d_in, void *d_packed, size_t packed_cap,
                               void *d_ws, size_t ws_cap, tahq_stream stream) {
  QPlan q;
  g_launches = 0;
  if (tahq_status rc = q_plan(p, &q)) return rc;
  if (!d_in || !d_packed || !d_ws) return TAHQ_ERR_INVALID_ARG;
  if (packed_cap < q.total_bytes || ws_cap < 256) return TAHQ_ERR_BUFFER_TOO_SMALL;
  if (!aligned16(d_in) || !aligned16(d_packed) || !aligned16(d_ws)) return TAHQ_ERR_MISALIGNED;
  DevInfo d;
  if (!dev_info(&d)) return TAHQ_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  QArgs a;
  q_args(p, q, &a, d_ws);
  a.in = static_cast<const uint8_t *>(d_in);
  a.packed = static_cast<uint8_t *>(d_packed);
  if (clear_workspace(d_ws, 256, st) != TAHQ_OK) return TAHQ_ERR_CUDA;
  const bool bf = p->dtype == TAHQ_BF16;
  if (p->per_tensor) {
    if (bf) TAHQ_LAUNCH("qnaive_max", st, launch_dependent(qnaive_max_kernel<true>, d.sms * 4, kQThreads, 0, st, a));
    else TAHQ_LAUNCH("qnaive_max", st, launch_dependent(qnaive_max_kernel<false>, d.sms * 4, kQThreads, 0, st, a));
  }
  if (bf) TAHQ_LAUNCH("qnaive_encode", st, launch_dependent(qnaive_encode_kernel<true>, q_grid(p->tokens, d), kQThreads, 0, st, a));
  else TAHQ_LAUNCH("qnaive_encode", st, launch_dependent(qnaive_encode_kernel<false>, q_grid(p->tokens, d), kQThreads, 0, st, a));
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

tahq_status tahq_qnaive_decode(const tahq_qnaive_params *p, const void *d_packed, size_t packed_bytes, void *d_out,
                               void *d_ws, size_t ws_cap, tahq_stream stream) {
  QPlan q;
  g_launches = 0;
  if (tahq_status rc = q_plan(p, &q)) return rc;
  if (!d_packed || !d_out || !d_ws) return TAHQ_ERR_INVALID_ARG;
  if (packed_bytes < q.total_bytes || ws_cap < 256) return TAHQ_ERR_BUFFER_TOO_SMALL;
  if (!aligned16(d_packed) || !aligned16(d_out) || !aligned16(d_ws)) return TAHQ_ERR_MISALIGNED;
  DevInfo d;
  if (!dev_info(&d)) return TAHQ_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  QArgs a;
  q_args(p, q, &a, d_ws);
  a.packed = const_cast<uint8_t *>(static_cast<const uint8_t *>(d_packed));
  a.out = static_cast<uint8_t *>(d_out);
  if (clear_workspace(d_ws, 256, st) != TAHQ_OK) return TAHQ_ERR_CUDA;
  if (p->dtype == TAHQ_BF16)
    TAHQ_LAUNCH("qnaive_decode", st, launch_dependent(qnaive_decode_kernel<true>, q_grid(p->tokens, d), kQThreads, 0, st, a));
  else
    TAHQ_LAUNCH("qnaive_decode", st, launch_dependent(qnaive_decode_kernel<false>, q_grid(p->tokens, d), kQThreads, 0, st, a));
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

tahq_status tahq_selftest_wait_timeout(void *d_ws, size_t ws_cap, tahq_stream stream) {
  if (!d_ws) return TAHQ_ERR_INVALID_ARG;
  if (ws_cap < 256 + 8ull * kMaxGrid) return TAHQ_ERR_BUFFER_TOO_SMALL;
  if (!aligned16(d_ws)) return TAHQ_ERR_MISALIGNED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(d_ws, 0, 256 + 8ull * kMaxGrid, st) != cudaSuccess) return TAHQ_ERR_CUDA;
  Args a;
  std::memset(&a, 0, sizeof(a));
  a.status = reinterpret_cast<uint32_t *>(d_ws);
  a.flags = reinterpret_cast<unsigned long long *>(static_cast<uint8_t *>(d_ws) + 256);
  wait_selftest_kernel<<<2, kThreads, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? TAHQ_OK : TAHQ_ERR_CUDA;
}

const char *tahq_status_string(tahq_status s) {
  switch (s) {
    case TAHQ_OK: return "ok";
    case TAHQ_ERR_INVALID_ARG: return "invalid argument";
    case TAHQ_ERR_UNSUPPORTED: return "unsupported configuration";
    case TAHQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case TAHQ_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case TAHQ_ERR_CUDA: return "CUDA runtime error";
    case TAHQ_ERR_TOO_LARGE: return "tensor needs more scratch than the built-in buffer of tahq_encode_noalloc";
  }
  return "unknown status";
}

int tahq_last_launch_count(void) { return g_launches; }

void tahq_profile(int enable) {
  g_prof_on = enable != 0;
  if (g_prof_on) {
    for (auto &r : g_prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    g_prof.clear();
  }
}

int tahq_profile_read(char *names, float *ms, int max_records) {
  int n = 0;
  for (auto &r : g_prof) {
    if (n < max_records) {
      cudaEventSynchronize(r.e1);
      float t = 0.0f;
      cudaEventElapsedTime(&t, r.e0, r.e1);
      if (ms) ms[n] = t;
      if (names) { std::strncpy(names + 32 * n, r.name, 31); names[32 * n + 31] = 0; }
      ++n;
    }
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  g_prof.clear();
  return n;
}

}  // extern "C"
