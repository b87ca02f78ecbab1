// C-ABI of the CP-head log-likelihood library: validation, workspace layout and
// the launch sequence of each entry point.  See include/cpmtp.h for the contract.
#include "../../include/cpmtp.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "distill_epilogues.cuh"
#include "distill_kernels.cuh"
#include "epilogues.cuh"
#include "sampler_kernels.cuh"
#include "small_kernels.cuh"
#include "tc_gemm.cuh"
#include "tmap.cuh"

namespace cpmtp {
namespace {

constexpr int kBN = 256;
constexpr int kStages = 4;
constexpr size_t kAlign = 256;
// Bound on the chunk of recomputed logit gradients (bf16) that the backward holds at a time.  Large on
// purpose (the device has 180 GB): every chunk costs one read-modify-write of the fp32 dE accumulator and a
// partly filled last wave in each of its GEMMs, so few, long chunks are cheaper than many short ones.
constexpr size_t kLogitGradBudgetBytes = 16ull << 30;

using CfgKK = TileCfg<kBN, kStages, false, false>;   // A K-major, B K-major
constexpr int kWideStages = 3;                        // 64 KB per slot
constexpr int kWideBM = 2 * kBM;
using CfgKKSkinny = TileCfg<kBN, 5, false, false, 32>;   // <= 32 rows of A: bandwidth-bound draft scoring
using WideKK = TileCfg<kBN, kWideStages, false, false, kBM, 2>;   // 256 x 256 tiles, two row blocks share B
using CfgProj = TileCfg<kBN, kStages, false, false, kBM, 1, 2>;   // 128-row tiles, eight epilogue warps (head projection)

inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }

struct DeviceInfo {
  int sms = 0;
  int cc_major = 0;
  bool ok = false;
};

// One lock for the small per-process caches below (device properties, kernel attributes, tensor maps,
// the static scratch address).  Host-side only and held for microseconds; calls from several threads are safe.
std::mutex g_cache_mutex;

// Cached per device ordinal; filled on first use with that device current.
DeviceInfo* device_info() {
  static DeviceInfo infos[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  DeviceInfo& di = infos[dev];
  if (!di.ok) {
    if (cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&di.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return nullptr;
    di.ok = true;
  }
  return &di;
}

// Testing / tuning knobs from the environment, read once per process (and again by cpmtp_reload_knobs);
// 0 = not set.
struct Knobs {
  long long wide_min_k = 0, wide_min_rows = 0;
  long long lse_group_mb = 0, lse_splits = 0, lse_group_tiles = 0;
  long long bwd_chunk_rows = 0, bwd_chunk_heads = 0, gemm_group_rows = 0;
  long long kl_group_tiles = 0, kl_splits = 0;
  long long wait_limit_us = 0, test_skip_load = 0;
  long long proj_tiles = 0;
};
Knobs g_knobs;
std::once_flag g_knobs_once;

void read_knobs() {
  auto get = [](const char* name) -> long long {
    const char* v = std::getenv(name);
    return v != nullptr ? std::atoll(v) : 0;
  };
  Knobs k;
  k.wide_min_k = get("CPMTP_WIDE_MIN_K");
  k.wide_min_rows = get("CPMTP_WIDE_MIN_ROWS");
  k.lse_group_mb = get("CPMTP_LSE_GROUP_MB");
  k.lse_splits = get("CPMTP_LSE_SPLITS");
  k.lse_group_tiles = get("CPMTP_LSE_GROUP_TILES");
  k.bwd_chunk_rows = get("CPMTP_BWD_CHUNK_ROWS");
  k.bwd_chunk_heads = get("CPMTP_BWD_CHUNK_HEADS");
  k.gemm_group_rows = get("CPMTP_GEMM_GROUP_ROWS");
  k.kl_group_tiles = get("CPMTP_KL_GROUP_TILES");
  k.kl_splits = get("CPMTP_KL_SPLITS");
  k.wait_limit_us = get("CPMTP_WAIT_LIMIT_US");
  k.test_skip_load = get("CPMTP_TEST_SKIP_LOAD");
  k.proj_tiles = get("CPMTP_PROJ_TILE_ROWS");
  g_knobs = k;
}

const Knobs& knobs() {
  std::call_once(g_knobs_once, read_knobs);
  return g_knobs;
}

int sms_or_default() {
  DeviceInfo* di = device_info();
  return (di != nullptr && di->sms > 0) ? di->sms : 148;
}

int validate_shape(const cpmtp_shape* s) {
  if (s == nullptr) return CPMTP_ERR_NULL;
  if (s->N < 1 || s->d < 64 || s->V < 2 || s->n < 1 || s->r < 1) return CPMTP_ERR_SHAPE;
  if (s->d % 64 != 0 || s->r > CPMTP_MAX_R || s->n > CPMTP_MAX_N) return CPMTP_ERR_SHAPE;
  const double zsize = static_cast<double>(s->N) * s->n * s->r * s->d;
  if (zsize >= 1099511627776.0) return CPMTP_ERR_SHAPE;
  if (static_cast<double>(s->N) * s->n * s->r >= 2147483648.0) return CPMTP_ERR_SHAPE;
  return CPMTP_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Wide (256-row) tiles move a third fewer operand bytes per flop but cannot overlap their
// epilogue with the next tile's MMAs, so they pay when the contraction is long enough to
// amortise it; otherwise 128-row tiles with the double-buffered accumulator are used.
bool use_wide(long long rows, long long kdim) {
  long long min_k = 4096;
  if (knobs().wide_min_k >= 64) min_k = knobs().wide_min_k;   // tuning knob
  long long min_rows = 2 * kWideBM;
  if (knobs().wide_min_rows > kBM) min_rows = knobs().wide_min_rows;   // tuning knob
  return rows >= min_rows && kdim >= min_k;
}

// Column-split schedule of the fused unembedding: `group` row tiles x `splits`
// vocabulary ranges run concurrently, so the rows' z tiles stay L2-resident while
// each range of E is streamed once per group.  The split count minimises a simple
// time model: max(makespan of the tensor work, HBM traffic / bandwidth); ties go
// to the choice that keeps more SMs busy, then to fewer splits.
Sched sched_lse(int m_tiles, int n_tiles, int M, int V, int d, int bm, int slots) {
  // keep the concurrently swept z tiles (group * bm rows * d * 2 B) within a budget of L2
  // (bm = rows per row tile: 128 or 256; slots = tiles in flight = SMs)
  const int sms = slots;
  // L2 budget for the z tiles a group keeps re-reading.  Measured with DRAM-byte counters on
  // B200: with 256-row tiles at d = 4096 (2 MB per tile) 12 tiles x 12 vocabulary ranges gave the
  // least DRAM traffic and the best time at V = 32000 and V = 128256; larger groups start to
  // evict one another's z tiles and the E stream.  The 0.5 MB tiles at d = 2048 did best with 64 MB.
  long long l2_budget_mb = bm > kBM ? 24 : 64;
  if (knobs().lse_group_mb >= 1 && knobs().lse_group_mb <= 1024) l2_budget_mb = knobs().lse_group_mb;   // tuning knob
  int max_group = static_cast<int>((l2_budget_mb << 20) / (2ll * bm * d));
  if (max_group < 1) max_group = 1;
  const double tile_t = 2.0 * bm * kBN * d / (1.4e15 / 148.0);
  int best_s = 1, best_ctas = 0;
  double best_score = -1.0;
  const int s_max = n_tiles < sms ? n_tiles : sms;
  for (int s = 1; s <= s_max; ++s) {
    const int group = static_cast<long long>(m_tiles) * s >= sms ? (sms / s) : m_tiles;
    if (group < 1 || group > max_group) continue;
    const long long units = static_cast<long long>(m_tiles) * s;
    const double comp = static_cast<double>((units + sms - 1) / sms) * ((n_tiles + s - 1) / s) * tile_t;
    const double sweeps = (m_tiles + group - 1) / group;
    const double mem = (sweeps * V * d * 2.0 + static_cast<double>(M) * d * 2.0) / 6.0e12;
    const double score = (comp > mem ? comp : mem) + 0.1 * mem;
    const int ctas = units < sms ? static_cast<int>(units) : sms;
    if (best_score < 0 || score < best_score * 0.999 || (score <= best_score * 1.001 && ctas > best_ctas)) {
      best_score = score;
      best_s = s;
      best_ctas = ctas;
    }
  }
  if (knobs().lse_splits >= 1 && knobs().lse_splits <= s_max) best_s = static_cast<int>(knobs().lse_splits);   // tuning knob
  int group = static_cast<long long>(m_tiles) * best_s >= sms ? (sms / best_s) : m_tiles;
  if (bm > kBM && m_tiles >= 8) {
    // 256-row tiles (d >= 4096): measured on B200, short units in the raster of the plain GEMMs beat
    // the long lock-stepped sweeps above: 8 row tiles (2048 rows) x 125 vocabulary ranges ran the
    // unembedding 20 % faster at V = 128256 and 4-9 % faster at V = 32000 (A/B within one process).
    // Range counts that make a group a whole number of waves (e.g. 148) were clearly worse.
    group = 8;
    best_s = n_tiles < 125 ? n_tiles : 125;
    if ((static_cast<long long>(group) * best_s) % sms == 0 && best_s > 1) --best_s;
    if (knobs().lse_splits >= 1 && knobs().lse_splits <= n_tiles) best_s = static_cast<int>(knobs().lse_splits);
  }
  if (knobs().lse_group_tiles >= 1) group = static_cast<int>(knobs().lse_group_tiles);   // tuning knob: force the row group
  return make_sched(m_tiles, n_tiles, best_s, group < 1 ? 1 : group, d / kBK);
}

struct FwdLayout {
  size_t logw, q, wbar, lse, tgt, z, tgt_part, part_m, part_l, total;
  Sched lse_sched;
  int K, M;   // heads, rows of the unembedding GEMM
  bool wide;  // the unembedding runs on 256-row tiles
  int parts;  // (max, sum-exp) partials per logit row: one per vocabulary range
};

FwdLayout fwd_layout(const cpmtp_shape& s, int sms) {
  FwdLayout L;
  L.K = s.n * s.r;
  L.M = s.N * L.K;
  L.wide = use_wide(L.M, s.d);
  const int bm = L.wide ? kWideBM : kBM;
  const int m_tiles = (L.M + bm - 1) / bm;
  const int n_tiles = (s.V + kBN - 1) / kBN;
  L.lse_sched = sched_lse(m_tiles, n_tiles, L.M, s.V, s.d, bm, sms);
  L.parts = L.lse_sched.n_splits;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.logw = take(sizeof(float) * s.N * s.r);
  L.q = take(sizeof(float) * s.N * s.r);
  L.wbar = take(sizeof(float) * CPMTP_MAX_R);
  L.lse = take(sizeof(float) * L.M);
  L.tgt = take(sizeof(float) * L.M);
  L.z = take(2ull * L.M * s.d);
  L.tgt_part = take(sizeof(float) * static_cast<size_t>(L.M) * (s.d / 64));
  L.part_m = take(sizeof(float) * static_cast<size_t>(L.M) * L.parts);
  L.part_l = take(sizeof(float) * static_cast<size_t>(L.M) * L.parts);
  L.total = off;
  return L;
}

struct BwdLayout {
  size_t coef, dg, dz, zre, G, dE32, dwg_part, uk, total;
  int K, M, ldg, chunk_rows, chunks, dwg_slices, dwg_rows_per_slice;
};

// Group size of the distillation passes: r padded to a power of two (lanes of a warp).
inline int padded_rank(int r) {
  int R = 1;
  while (R < r) R <<= 1;
  return R;
}

// `quantum`: chunks of recomputed logit gradients hold a multiple of this many rows (whole row
// tiles: 128 rows, or 128 / R groups of r rows for the grouped distillation pass).
BwdLayout bwd_layout(const cpmtp_shape& s, int quantum = kBM, bool distill = false) {
  BwdLayout L;
  L.K = s.n * s.r;
  L.M = s.N * L.K;
  L.ldg = (s.V + 63) / 64 * 64;
  long long rows = static_cast<long long>(kLogitGradBudgetBytes / (2ull * L.ldg)) / quantum * quantum;
  if (rows < L.M) {
    // Several chunks: make a chunk a whole number of waves of the dz GEMM (row tiles x d/256 column tiles over
    // one CTA per SM), whose last wave would otherwise run partly empty in every chunk.
    const int sms = sms_or_default();
    const long long tile_rows = use_wide(rows, s.V) ? kWideBM : kBM;
    const long long col_tiles = (s.d + kBN - 1) / kBN;
    long long g = sms, b = col_tiles;
    while (b != 0) { const long long t = g % b; g = b; b = t; }
    const long long wave_rows = tile_rows * (sms / g);
    if (rows >= 2 * wave_rows) rows = rows / wave_rows * wave_rows / quantum * quantum;
  }
  if (knobs().bwd_chunk_rows >= quantum) rows = knobs().bwd_chunk_rows / quantum * quantum;   // testing knob
  if (rows < quantum) rows = quantum;
  const long long m_pad = (static_cast<long long>(L.M) + quantum - 1) / quantum * quantum;
  if (rows > m_pad) rows = m_pad;
  L.chunk_rows = static_cast<int>(rows);
  L.chunks = static_cast<int>((L.M + rows - 1) / rows);
  L.dwg_rows_per_slice = 256;
  L.dwg_slices = (s.N + L.dwg_rows_per_slice - 1) / L.dwg_rows_per_slice;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.coef = take(sizeof(float) * static_cast<size_t>(s.N) * L.K);
  L.dg = take(sizeof(float) * s.N * s.r);
  L.dz = take(2ull * L.M * s.d);
  L.zre = take((s.flags & CPMTP_FLAG_RECOMPUTE_Z) ? 2ull * L.M * s.d : 0);   // z recomputed instead of saved
  L.G = take(2ull * L.chunk_rows * L.ldg);
  L.dE32 = take(L.chunks > 1 ? sizeof(float) * static_cast<size_t>(s.V) * s.d : 0);
  L.dwg_part = take(sizeof(float) * static_cast<size_t>(L.dwg_slices) * s.r * s.d);
  L.uk = take(distill ? sizeof(float) * static_cast<size_t>(s.N) * s.n : 0);
  L.total = off;
  return L;
}

// Distillation forward: the plain forward pass, then the grouped KL pass over the vocabulary.
struct DistillLayout {
  FwdLayout fwd;
  size_t part, part_tm, part_tl, total;
  Sched sched;
  int R, gpt, groups;   // padded rank, groups per 128-row tile, N * n
};

DistillLayout distill_layout(const cpmtp_shape& s, int sms) {
  DistillLayout L;
  L.fwd = fwd_layout(s, sms);
  L.R = padded_rank(s.r);
  L.gpt = kBM / L.R;
  L.groups = s.N * s.n;
  const int m_tiles = (L.groups + L.gpt - 1) / L.gpt;
  const int n_tiles = (s.V + kBN - 1) / kBN;
  L.sched = sched_lse(m_tiles, n_tiles, m_tiles * kBM, s.V, s.d, kBM, sms);
  if (s.d >= 4096 && m_tiles >= 16) {
    // Long contractions: short units in the raster of the plain GEMMs (16 row tiles x up to 125 vocabulary
    // ranges) beat the long lock-stepped sweeps, as for the 256-row unembedding: measured 54.2 ms against
    // 57.6 ms at N = 8192, d = 4096, V = 32000, n = 4, r = 8 (interleaved A/B in one process); at d = 2048 the
    // sweeps of sched_lse stay ahead (6.8 ms against 7.2 ms at N = 4096, V = 32000, n = 2, r = 8).
    int sp = n_tiles < 125 ? n_tiles : 125;
    if ((16ll * sp) % sms == 0 && sp > 1) --sp;
    L.sched = make_sched(m_tiles, n_tiles, sp, 16, s.d / kBK);
  }
  {
    // tuning knobs for this sweep alone
    const int g = static_cast<int>(knobs().kl_group_tiles), sp = static_cast<int>(knobs().kl_splits);
    if (g >= 1 || sp >= 1)
      L.sched = make_sched(m_tiles, n_tiles, sp >= 1 ? sp : L.sched.n_splits, g >= 1 ? g : L.sched.m_group, s.d / kBK);
  }
  L.sched.a_groups = L.gpt;
  size_t off = align_up(L.fwd.total);
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.part = take(sizeof(float) * static_cast<size_t>(L.fwd.M) * L.sched.n_splits);
  L.part_tm = take(sizeof(float) * static_cast<size_t>(L.groups) * L.sched.n_splits);
  L.part_tl = take(sizeof(float) * static_cast<size_t>(L.groups) * L.sched.n_splits);
  L.total = off;
  return L;
}

// Optional per-stage timing: events bracket each launch while profiling is on.
struct Profiler {
  bool on = false;
  std::vector<cudaEvent_t> events;   // start/stop pairs
  std::vector<int> stages;
};
Profiler g_prof;

struct ProfScope {
  cudaStream_t st;
  bool active;
  ProfScope(int stage, cudaStream_t stream) : st(stream), active(g_prof.on) {
    if (!active) return;
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { active = false; return; }
    g_prof.events.push_back(a);
    g_prof.events.push_back(b);
    g_prof.stages.push_back(stage);
    cudaEventRecord(a, st);
  }
  ~ProfScope() {
    if (active) cudaEventRecord(g_prof.events.back(), st);
  }
};

// ---- full head (Eq. 6 as printed) ----
struct FullLayout {
  size_t logw, q, wbar, lse, tgt, part_m, part_l, total;
  Sched sched;
  int K, tph, sph;
  bool wide;
};

FullLayout full_layout(const cpmtp_shape& s, int sms) {
  FullLayout L;
  L.K = s.n * s.r;
  L.wide = use_wide(s.N, s.d);
  const int bm = L.wide ? kWideBM : kBM;
  const int m_tiles = (s.N + bm - 1) / bm;
  L.tph = (s.V + kBN - 1) / kBN;
  L.sph = (L.tph + 15) / 16;             // units of at most 16 column tiles
  int group = static_cast<int>(((L.wide ? 24ll : 64ll) << 20) / (2ll * bm * s.d));
  if (group < 1) group = 1;
  L.sched = make_sched(m_tiles, L.K * L.tph, L.K * L.sph, group, s.d / kBK);
  L.sched.seg_tiles = L.tph;
  L.sched.seg_stride = s.V;
  (void)sms;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.logw = take(sizeof(float) * s.N * s.r);
  L.q = take(sizeof(float) * s.N * s.r);
  L.wbar = take(sizeof(float) * CPMTP_MAX_R);
  L.lse = take(sizeof(float) * static_cast<size_t>(s.N) * L.K);
  L.tgt = take(sizeof(float) * static_cast<size_t>(s.N) * L.K);
  L.part_m = take(sizeof(float) * static_cast<size_t>(s.N) * L.K * L.sph);
  L.part_l = take(sizeof(float) * static_cast<size_t>(s.N) * L.K * L.sph);
  L.total = off;
  return L;
}

struct FullBwdLayout {
  size_t coef, dg, G, dh32, dwg_part, total;
  int K, ldv, heads_per_chunk, dwg_slices, dwg_rows_per_slice;
};

FullBwdLayout full_bwd_layout(const cpmtp_shape& s) {
  FullBwdLayout L;
  L.K = s.n * s.r;
  L.ldv = (s.V + 63) / 64 * 64;
  long long heads = static_cast<long long>(kLogitGradBudgetBytes / (2ull * s.N * L.ldv));
  if (knobs().bwd_chunk_heads >= 1) heads = knobs().bwd_chunk_heads;   // testing knob
  if (heads < 1) heads = 1;
  if (heads > L.K) heads = L.K;
  L.heads_per_chunk = static_cast<int>(heads);
  L.dwg_rows_per_slice = 256;
  L.dwg_slices = (s.N + L.dwg_rows_per_slice - 1) / L.dwg_rows_per_slice;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.coef = take(sizeof(float) * static_cast<size_t>(s.N) * L.K);
  L.dg = take(sizeof(float) * s.N * s.r);
  L.G = take(2ull * s.N * L.heads_per_chunk * L.ldv);
  L.dh32 = take(sizeof(float) * static_cast<size_t>(s.N) * s.d);
  L.dwg_part = take(sizeof(float) * static_cast<size_t>(L.dwg_slices) * s.r * s.d);
  L.total = off;
  return L;
}

struct SampleLayout {
  FwdLayout fwd;
  size_t logits, z32, lb, lb_exact, part_top, part_best, logp_tmp, done, cand, total;
  int lds, chunks;
};

SampleLayout sample_layout(const cpmtp_shape& s, int sms) {
  SampleLayout L;
  L.fwd = fwd_layout(s, sms);
  L.lds = (s.V + 31) / 32 * 32;
  L.chunks = (s.V + kSampleChunk - 1) / kSampleChunk;
  size_t off = align_up(L.fwd.total);
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.logits = take(sizeof(float) * static_cast<size_t>(L.fwd.M) * L.lds);
  L.z32 = take(sizeof(float) * static_cast<size_t>(L.fwd.M) * s.d);
  L.lb = take(sizeof(float) * static_cast<size_t>(s.n + 1) * s.N * s.r);   // expert weights before every step and after the last,
  L.lb_exact = take(sizeof(float) * static_cast<size_t>(s.n + 1) * s.N * s.r);   // as selected on, and exact
  L.part_top = take(sizeof(Cand) * static_cast<size_t>(s.N) * L.chunks * kMaxTopk);
  L.part_best = take(sizeof(Cand) * static_cast<size_t>(s.N) * L.chunks);
  L.logp_tmp = take(sizeof(float) * s.N);
  L.done = take(sizeof(unsigned int) * s.N);   // per-position count of finished blocks in a draft step
  L.cand = take(sizeof(int) * static_cast<size_t>(s.n) * s.N * (kMaxTopk + 1));   // candidate and chosen tokens of every step
  L.total = off;
  return L;
}

// Tensor maps depend only on (base address, extents, stride, box), so they are encoded once and kept:
// a decode loop that calls with the same buffers every step does no driver work on the host after the
// first call.  Small direct-mapped cache; a map never goes stale (it holds no more than its key).
struct TmapKey {
  const void* base;
  uint64_t rows, k, ld;
  uint32_t box_rows, groups;   // groups > 0: grouped-row 3-D map (box_rows = padded group size)
  uint32_t mn_major, group_rows;
  bool operator==(const TmapKey& o) const { return std::memcmp(this, &o, sizeof(TmapKey)) == 0; }
};
struct TmapSlot {
  TmapKey key;
  CUtensorMap map;
  bool used = false;
};
constexpr int kTmapSlots = 256;
TmapSlot g_tmaps[kTmapSlots];

bool cached_tmap(CUtensorMap* out, const TmapKey& key) {
  uint64_t hsh = reinterpret_cast<uintptr_t>(key.base) * 0x9E3779B97F4A7C15ull;
  hsh ^= (key.rows * 31 + key.k) * 0xC2B2AE3D27D4EB4Full + key.ld * 7 + key.box_rows * 131 + key.groups * 17 + key.mn_major;
  TmapSlot& slot = g_tmaps[(hsh >> 20) % kTmapSlots];
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  if (slot.used && slot.key == key) {
    *out = slot.map;
    return true;
  }
  CUtensorMap m;
  const bool ok = key.groups > 0
                      ? make_grouped_tmap_bf16(&m, key.base, key.k, key.group_rows, key.rows / key.group_rows, key.ld,
                                               key.box_rows, key.groups)
                      : make_operand_tmap(&m, key.base, key.mn_major != 0, key.rows, key.k, key.ld, key.box_rows);
  if (!ok) return false;
  slot.key = key;
  slot.map = m;
  slot.used = true;
  *out = m;
  return true;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while the one before it in
// the stream drains; it calls ptx::grid_dep_wait() before it touches anything that kernel produced.
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                       Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <class Cfg, class Epi>
cudaError_t launch_gemm(const void* A, uint64_t a_rows, uint64_t a_ld, const void* B, uint64_t b_rows,
                        uint64_t b_ld, uint64_t kdim, const Sched& sched_in, const typename Epi::Params& ep,
                        int* dev_status, int sms, cudaStream_t stream, int a_group_rows = 0) {
  static bool attr_set[64] = {};
  CUtensorMap tA, tB;
  TmapKey ka, kb;
  std::memset(&ka, 0, sizeof(ka));
  std::memset(&kb, 0, sizeof(kb));
  ka.base = A; ka.rows = a_rows; ka.k = kdim; ka.ld = a_ld;
  if (sched_in.a_groups > 0) {
    // grouped rows: a_rows = groups * a_group_rows, every group padded to 128 / a_groups tile rows
    if (Cfg::A_MN || Cfg::MB != 1 || Cfg::A_ROWS != kBM || a_group_rows < 1) return cudaErrorInvalidValue;
    ka.box_rows = kBM / sched_in.a_groups; ka.groups = sched_in.a_groups; ka.group_rows = a_group_rows;
  } else {
    ka.box_rows = Cfg::A_ROWS * Cfg::MB; ka.mn_major = Cfg::A_MN ? 1 : 0;
  }
  if (!cached_tmap(&tA, ka)) return cudaErrorInvalidValue;
  kb.base = B; kb.rows = b_rows; kb.k = kdim; kb.ld = b_ld; kb.box_rows = Cfg::BN; kb.mn_major = Cfg::B_MN ? 1 : 0;
  if (!cached_tmap(&tB, kb)) return cudaErrorInvalidValue;
  constexpr int smem = gemm_smem_bytes<Cfg, Epi>();
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64) {
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    if (!attr_set[dev]) {
      cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<Cfg, Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      attr_set[dev] = true;
    }
  }
  Sched sched = sched_in;
  // every wait inside the kernel gives up after this long (default 4 s; the knob exists so that a test can
  // watch the give-up path finish in milliseconds)
  sched.wait_limit_us = knobs().wait_limit_us > 0 ? static_cast<unsigned>(knobs().wait_limit_us) : 4000000u;
  sched.test_skip_load = static_cast<int>(knobs().test_skip_load);
  const int grid = sched.units < sms ? sched.units : sms;
  return launch_pdl(tc_gemm_kernel<Cfg, Epi>, dim3(grid), dim3(Cfg::THREADS), smem, stream, tA, tB, sched, ep,
                    dev_status);
}

// K-major x K-major launch on 128- or 256-row tiles.
template <class Epi>
cudaError_t launch_kk(bool wide, const void* A, uint64_t a_rows, uint64_t a_ld, const void* B, uint64_t b_rows,
                      uint64_t b_ld, uint64_t kdim, const Sched& sched, const typename Epi::Params& ep,
                      int* dev_status, int sms, cudaStream_t stream) {
  if (wide) return launch_gemm<WideKK, Epi>(A, a_rows, a_ld, B, b_rows, b_ld, kdim, sched, ep, dev_status, sms, stream);
  return launch_gemm<CfgKK, Epi>(A, a_rows, a_ld, B, b_rows, b_ld, kdim, sched, ep, dev_status, sms, stream);
}

// Tensor map of a row-major bf16 output [rows, cols] (row stride ld) written by the epilogues' TMA stores
// in boxes of 64 columns x 32 rows.
bool output_tmap(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
  TmapKey key;
  std::memset(&key, 0, sizeof(key));
  key.base = base; key.rows = rows; key.k = cols; key.ld = ld; key.box_rows = 32;
  return cached_tmap(out, key);
}

// A plain GEMM D[m_rows, n_cols] = A * B^T over `kdim`, every column tile its own unit, row tiles
// swept in groups of about `group_rows` rows; wide tiles when the problem is large enough.
template <bool A_MN, bool B_MN, class Epi>
cudaError_t gemm_auto(const void* A, uint64_t a_ld, const void* B, uint64_t b_ld, long long m_rows, int n_cols,
                      long long kdim, int group_rows, const typename Epi::Params& ep, int* dev_status, int sms,
                      cudaStream_t stream, int force_tile_rows = 0) {
  const int n_tiles = (n_cols + kBN - 1) / kBN;
  const int k_blocks = static_cast<int>((kdim + kBK - 1) / kBK);
  if (knobs().gemm_group_rows >= kWideBM) group_rows = static_cast<int>(knobs().gemm_group_rows);   // tuning knob
  const bool wide = force_tile_rows == kWideBM ? true : force_tile_rows == kBM ? false : use_wide(m_rows, kdim);
  if (wide) {
    const int m_tiles = static_cast<int>((m_rows + kWideBM - 1) / kWideBM);
    const Sched sc = make_sched(m_tiles, n_tiles, n_tiles, group_rows / kWideBM, k_blocks);
    return launch_gemm<TileCfg<kBN, kWideStages, A_MN, B_MN, kBM, 2>, Epi>(A, m_rows, a_ld, B, n_cols, b_ld, kdim, sc,
                                                                           ep, dev_status, sms, stream);
  }
  const int m_tiles = static_cast<int>((m_rows + kBM - 1) / kBM);
  const Sched sc = make_sched(m_tiles, n_tiles, n_tiles, group_rows / kBM, k_blocks);
  return launch_gemm<TileCfg<kBN, kStages, A_MN, B_MN>, Epi>(A, m_rows, a_ld, B, n_cols, b_ld, kdim, sc, ep,
                                                            dev_status, sms, stream);
}

#define CPMTP_TRY(expr)                         \
  do {                                          \
    if ((expr) != cudaSuccess) return CPMTP_ERR_LAUNCH; \
  } while (0)

// Forward pipeline shared by cpmtp_forward and cpmtp_score_draft.
int run_forward(const cpmtp_shape& s, const uint16_t* h, const uint16_t* W_head, const uint16_t* E,
                const uint16_t* W_g, const int32_t* x, float* logp, float* loss, const cpmtp_saved* saved,
                int32_t* counts, float* logp_prefix, uint8_t* ws, const FwdLayout& L, int* dev_status, int sms,
                cudaStream_t stream, float* logits = nullptr, int lds = 0, float* z32 = nullptr) {
  float* logw = saved ? saved->logw : reinterpret_cast<float*>(ws + L.logw);
  float* q = saved ? saved->q : reinterpret_cast<float*>(ws + L.q);
  float* wbar = saved ? saved->wbar : reinterpret_cast<float*>(ws + L.wbar);
  float* lse = saved ? saved->lse : reinterpret_cast<float*>(ws + L.lse);
  float* tgt = saved ? saved->tgt : reinterpret_cast<float*>(ws + L.tgt);
  const bool keep_z = saved != nullptr && !(s.flags & CPMTP_FLAG_RECOMPUTE_Z);
  uint16_t* z = keep_z ? static_cast<uint16_t*>(saved->z) : reinterpret_cast<uint16_t*>(ws + L.z);
  float* tgt_part = reinterpret_cast<float*>(ws + L.tgt_part);
  float* part_m = reinterpret_cast<float*>(ws + L.part_m);
  float* part_l = reinterpret_cast<float*>(ws + L.part_l);
  const int K = L.K;
  const int ncols = K * s.d;

  // head projection: z[N, K*d] = h[N, d] * W_cat[K*d, d]^T, plus the fp32 target-logit partials
  {
    ProfScope prof(CPMTP_STAGE_PROJ, stream);
    EpiProj<kBN>::Params ep{{}, z, tgt_part, E, x, z32, dev_status, s.N, ncols, s.d, s.V, s.n, s.r};
    if (!output_tmap(&ep.z_map, z, s.N, ncols, ncols)) return CPMTP_ERR_LAUNCH;
    if (s.N <= CfgKKSkinny::A_ROWS) {
      const int n_tiles = (ncols + kBN - 1) / kBN;
      const Sched sc = make_sched(1, n_tiles, n_tiles, 1, s.d / kBK);
      CPMTP_TRY((launch_gemm<CfgKKSkinny, EpiProj<kBN>>(h, s.N, s.d, W_head, ncols, s.d, s.d, sc, ep, dev_status, sms, stream)));
    } else if (knobs().proj_tiles == kBM || knobs().proj_tiles == kWideBM) {   // tuning knob: the plain tile shapes
      CPMTP_TRY((gemm_auto<false, false, EpiProj<kBN>>(h, s.d, W_head, s.d, s.N, ncols, s.d, 8192, ep, dev_status, sms, stream,
                                                      static_cast<int>(knobs().proj_tiles))));
    } else {
      // Its epilogue (bf16 slab stores, gathered rows of E, one partial per 64 columns) is a long dependent chain
      // per chunk: with one warp per scheduler it, not the MMAs, sets the pace of a tile.  Two warps per TMEM lane
      // quarter, each with half of the columns, on 128-row tiles whose accumulator is double-buffered.
      const int n_tiles = (ncols + kBN - 1) / kBN;
      const int m_tiles = (s.N + kBM - 1) / kBM;
      const Sched sc = make_sched(m_tiles, n_tiles, n_tiles, 8192 / kBM, s.d / kBK);
      CPMTP_TRY((launch_gemm<CfgProj, EpiProj<kBN>>(h, s.N, s.d, W_head, ncols, s.d, s.d, sc, ep, dev_status, sms, stream)));
    }
  }
  // unembedding fused with the vocabulary log-sum-exp (Eq. 6, Eq. 8)
  {
    ProfScope prof(CPMTP_STAGE_LSE, stream);
    if (logits != nullptr) {
      EpiLse<kBN, true>::Params ep{part_m, part_l, L.M, s.V, L.parts, logits, lds};
      if (L.M <= CfgKKSkinny::A_ROWS) {
        CPMTP_TRY((launch_gemm<CfgKKSkinny, EpiLse<kBN, true>>(z, L.M, s.d, E, s.V, s.d, s.d, L.lse_sched, ep, dev_status, sms, stream)));
      } else {
        CPMTP_TRY((launch_kk<EpiLse<kBN, true>>(L.wide, z, L.M, s.d, E, s.V, s.d, s.d, L.lse_sched, ep, dev_status, sms, stream)));
      }
    } else {
      EpiLse<kBN>::Params ep{part_m, part_l, L.M, s.V, L.parts, nullptr, 0};
      if (L.M <= CfgKKSkinny::A_ROWS) {
        CPMTP_TRY((launch_gemm<CfgKKSkinny, EpiLse<kBN>>(z, L.M, s.d, E, s.V, s.d, s.d, L.lse_sched, ep, dev_status, sms, stream)));
      } else {
        CPMTP_TRY((launch_kk<EpiLse<kBN>>(L.wide, z, L.M, s.d, E, s.V, s.d, s.d, L.lse_sched, ep, dev_status, sms, stream)));
      }
    }
  }
  // gate (Eq. 7) and mixture epilogue (Eq. 9)
  {
    ProfScope prof(CPMTP_STAGE_MIXTURE, stream);
    const int threads = s.N <= 256 ? 1024 : 256;
    CPMTP_TRY(launch_pdl(gate_mixture_kernel, dim3(s.N), dim3(threads), 0, stream, h, W_g, s.d, part_m, part_l, L.parts,
                         tgt_part, x != nullptr ? s.d / 64 : 0, logw, lse, tgt, q, logp, logp_prefix, s.N, s.n, s.r));
  }
  if (loss != nullptr || counts != nullptr || saved != nullptr) {
    ProfScope prof(CPMTP_STAGE_FINALIZE, stream);
    const float aux = (s.flags & CPMTP_FLAG_AUX) ? s.aux_coef : 0.f;
    finalize_kernel<<<1, kFinalizeThreads, 0, stream>>>(logp, logw, wbar, counts, loss, s.N, s.r, aux);
    CPMTP_TRY(cudaGetLastError());
  }
  return CPMTP_OK;
}

int check_common(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E, const void* W_g,
                 const void* x, const void* workspace, DeviceInfo** di_out) {
  const int vs = validate_shape(shape);
  if (vs != CPMTP_OK) return vs;
  if (!h || !W_head || !E || !W_g || !x || !workspace) return CPMTP_ERR_NULL;
  if (!aligned(h, 16) || !aligned(W_head, 16) || !aligned(E, 16) || !aligned(W_g, 16) || !aligned(x, 4) ||
      !aligned(workspace, kAlign))
    return CPMTP_ERR_ALIGN;
  DeviceInfo* di = device_info();
  if (di == nullptr) return CPMTP_ERR_LAUNCH;
  if (di->cc_major != 10) return CPMTP_ERR_ARCH;
  *di_out = di;
  return CPMTP_OK;
}

int check_saved(const cpmtp_saved* sv, bool need_z = true) {
  if (!sv->lse || !sv->tgt || !sv->logw || !sv->q || !sv->wbar || (need_z && !sv->z)) return CPMTP_ERR_NULL;
  if (!aligned(sv->z, 16) || !aligned(sv->lse, 4) || !aligned(sv->tgt, 4) || !aligned(sv->logw, 4) ||
      !aligned(sv->q, 4) || !aligned(sv->wbar, 4))
    return CPMTP_ERR_ALIGN;
  return CPMTP_OK;
}

}  // namespace
}  // namespace cpmtp

// Scratch of cpmtp_score_draft_static: lives in the library image, one copy per GPU.
// In host code this name is only a handle for cudaGetSymbolAddress, never a pointer
// a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[CPMTP_STATIC_SCRATCH_BYTES];

using namespace cpmtp;

// Device address of g_static_scratch on the current device, looked up once per device.
static unsigned char* static_scratch_ptr() {
  static unsigned char* ptrs[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  if (ptrs[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return nullptr;
    ptrs[dev] = static_cast<unsigned char*>(p);
  }
  return ptrs[dev];
}


// The two grouped passes, instantiated for every padded rank R (a power of two, 1..32).
template <template <int, int> class Epi, class Params>
static cudaError_t launch_grouped(int R, const uint16_t* z, long long rows, int d, const uint16_t* E, int V,
                                  const Sched& sc, const Params& ep, int r, int* dev_status, int sms,
                                  cudaStream_t st) {
  switch (R) {
    case 1: return launch_gemm<CfgKK, Epi<kBN, 1>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    case 2: return launch_gemm<CfgKK, Epi<kBN, 2>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    case 4: return launch_gemm<CfgKK, Epi<kBN, 4>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    case 8: return launch_gemm<CfgKK, Epi<kBN, 8>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    case 16: return launch_gemm<CfgKK, Epi<kBN, 16>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    case 32: return launch_gemm<CfgKK, Epi<kBN, 32>>(z, rows, d, E, V, d, d, sc, ep, dev_status, sms, st, r);
    default: return cudaErrorInvalidValue;
  }
}

// What the distillation objective adds to the backward pass (nullptr: plain log-likelihood).
struct DistillCtx {
  const uint16_t* teacher;          // [N, n, V] bf16
  const cpmtp_distill_saved* ds;
  const float* dloss_dkl;           // [N, n] or nullptr (weights of Eq. 14 from beta, gamma)
  float beta, gamma;
};

// Backward pipeline shared by cpmtp_backward and cpmtp_distill_backward.
static int backward_impl(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E, const void* W_g,
                         const int32_t* x, const cpmtp_saved* saved, const float* dloss_dlogp, void* dh,
                         void* dW_head, void* dE, void* dW_g, void* workspace, size_t workspace_bytes,
                         int32_t* dev_status, cpmtp_stream stream, const DistillCtx* dc) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, x, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (saved == nullptr) return CPMTP_ERR_NULL;
  if (!dh && !dW_head && !dE && !dW_g) return CPMTP_ERR_NULL;   // nothing asked for
  const bool recompute_z = (shape->flags & CPMTP_FLAG_RECOMPUTE_Z) != 0;
  const int rs = check_saved(saved, !recompute_z);
  if (rs != CPMTP_OK) return rs;
  if (!aligned(dh, 16) || !aligned(dW_head, 16) || !aligned(dE, 16) || !aligned(dW_g, 16)) return CPMTP_ERR_ALIGN;
  const bool need_dz = dh != nullptr || dW_head != nullptr;   // dz feeds only these two
  const cpmtp_shape& s = *shape;
  const int R = padded_rank(s.r);
  const int gpt = kBM / R;   // groups per row tile of the grouped pass
  const BwdLayout L = dc != nullptr ? bwd_layout(s, gpt * s.r, true) : bwd_layout(s);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* coef = reinterpret_cast<float*>(ws + L.coef);
  float* dg = reinterpret_cast<float*>(ws + L.dg);
  uint16_t* dz = reinterpret_cast<uint16_t*>(ws + L.dz);
  uint16_t* G = reinterpret_cast<uint16_t*>(ws + L.G);
  float* dE32 = reinterpret_cast<float*>(ws + L.dE32);
  float* dwg_part = reinterpret_cast<float*>(ws + L.dwg_part);
  const uint16_t* z = recompute_z ? reinterpret_cast<const uint16_t*>(ws + L.zre)
                                  : static_cast<const uint16_t*>(saved->z);
  const uint16_t* Eb = static_cast<const uint16_t*>(E);
  const int sms = di->sms;
  const int K = L.K, d = s.d, V = s.V;
  const int ncols = K * d;
  const float aux = (s.flags & CPMTP_FLAG_AUX) ? s.aux_coef : 0.f;
  const int per_token = (s.flags & CPMTP_FLAG_PER_TOKEN) ? 1 : 0;
  const int accum = (s.flags & CPMTP_FLAG_ACCUM_GRADS) ? 1 : 0;   // outputs += instead of =
  if (per_token && dloss_dlogp == nullptr && dc == nullptr) return CPMTP_ERR_NULL;
  float* uk = reinterpret_cast<float*>(ws + L.uk);

  if (recompute_z) {   // z[N, K*d] = h W_cat^T again: the same MMAs and the same rounding as in the forward pass
    ProfScope prof(CPMTP_STAGE_PROJ, st);
    EpiStoreBf16<kBN, false>::Params ep{reinterpret_cast<uint16_t*>(ws + L.zre), nullptr, nullptr, s.N, ncols, ncols, 0};
    CPMTP_TRY((gemm_auto<false, false, EpiStoreBf16<kBN, false>>(h, d, W_head, d, s.N, ncols, d, 8192, ep, dev_status, sms, st)));
  }
  {
    ProfScope prof(CPMTP_STAGE_COEFF, st);
    if (dc != nullptr) {
      distill_coeff_kernel<<<(s.N + 127) / 128, 128, 0, st>>>(saved->logw, saved->wbar, saved->lse, saved->tgt,
                                                             dc->ds->logpi, dc->ds->pm, dc->ds->kl, dloss_dlogp,
                                                             dc->dloss_dkl, dc->beta, dc->gamma, coef, dg, uk, s.N,
                                                             s.n, s.r, aux);
    } else {
      coeff_kernel<<<(s.N + 127) / 128, 128, 0, st>>>(saved->q, saved->logw, saved->wbar, saved->lse, saved->tgt,
                                                     dloss_dlogp, per_token, coef, dg, s.N, s.n, s.r, aux);
    }
    CPMTP_TRY(cudaGetLastError());
  }

  for (int c = 0; c < L.chunks; ++c) {
    const long long row0 = static_cast<long long>(c) * L.chunk_rows;
    const int rows = static_cast<int>((L.M - row0) < L.chunk_rows ? (L.M - row0) : L.chunk_rows);
    const uint16_t* zc = z + row0 * d;
    // recompute logits tile by tile -> G = dloss/dS (bf16), never more than one chunk
    if (dc != nullptr && (need_dz || dE != nullptr)) {
      ProfScope prof(CPMTP_STAGE_LOGIT_GRAD, st);
      const int groups = rows / s.r;   // chunks hold whole groups
      Sched sc = make_sched((groups + gpt - 1) / gpt, (V + kBN - 1) / kBN, (V + kBN - 1) / kBN, 2048 / kBM, d / kBK);
      sc.a_groups = gpt;
      // the column tiles that cover V also cover the padding columns [V, ldg), which are written as zero
      const DistillGradParams ep{G, saved->lse, coef, dc->ds->logpi, dc->ds->pm, uk, dc->ds->lse_t, dc->teacher, x,
                                 row0 / s.r, groups, s.r, V, L.ldg, V % 8 == 0 ? 1 : 0};
      CPMTP_TRY((launch_grouped<EpiDistillGrad>(R, zc, rows, d, Eb, V, sc, ep, s.r, dev_status, sms, st)));
    } else if (dc == nullptr && (need_dz || dE != nullptr)) {
      ProfScope prof(CPMTP_STAGE_LOGIT_GRAD, st);
      EpiLogitGrad<kBN>::Params ep{{}, G, saved->lse, coef, x, row0, rows, L.ldg, V, K, s.n, s.r};
      if (!output_tmap(&ep.G_map, G, rows, L.ldg, L.ldg)) return CPMTP_ERR_LAUNCH;
      CPMTP_TRY((gemm_auto<false, false, EpiLogitGrad<kBN>>(zc, d, Eb, d, rows, V, d, 2048, ep, dev_status, sms, st)));
    }
    // dz[rows, d] = G[rows, V] * E[V, d]
    if (need_dz) {
      ProfScope prof(CPMTP_STAGE_DZ, st);
      EpiStoreBf16<kBN, false>::Params ep{dz + row0 * d, nullptr, nullptr, rows, d, d, 0};
      CPMTP_TRY((gemm_auto<false, true, EpiStoreBf16<kBN, false>>(G, L.ldg, Eb, d, rows, d, V, 2048, ep, dev_status, sms, st)));
    }
    // dE[V, d] (+)= G^T[V, rows] * z[rows, d]
    if (dE != nullptr) {
      ProfScope prof(CPMTP_STAGE_DE, st);
      if (L.chunks == 1) {
        EpiStoreBf16<kBN, false>::Params ep{static_cast<uint16_t*>(dE), nullptr, nullptr, V, d, d, 0, accum};
        CPMTP_TRY((gemm_auto<true, true, EpiStoreBf16<kBN, false>>(G, L.ldg, zc, d, V, d, rows, 2048, ep, dev_status, sms, st)));
      } else {
        EpiAccumF32<kBN>::Params ep{dE32, V, d, d, c > 0 ? 1 : 0};
        CPMTP_TRY((gemm_auto<true, true, EpiAccumF32<kBN>>(G, L.ldg, zc, d, V, d, rows, 2048, ep, dev_status, sms, st)));
      }
    }
  }
  if (L.chunks > 1 && dE != nullptr) {
    ProfScope prof(CPMTP_STAGE_DE_CONVERT, st);
    f32_to_bf16_kernel<<<sms * 8, 256, 0, st>>>(dE32, static_cast<uint16_t*>(dE), static_cast<size_t>(V) * d, accum);
    CPMTP_TRY(cudaGetLastError());
  }
  // dW_head[K*d, d] = dz^T[K*d, N] * h[N, d]
  if (dW_head != nullptr) {
    ProfScope prof(CPMTP_STAGE_DW_HEAD, st);
    EpiStoreBf16<kBN, false>::Params ep{static_cast<uint16_t*>(dW_head), nullptr, nullptr, ncols, d, d, 0, accum};
    CPMTP_TRY((gemm_auto<true, true, EpiStoreBf16<kBN, false>>(dz, ncols, h, d, ncols, d, s.N, 2048, ep, dev_status, sms, st)));
  }
  // dh[N, d] = dz[N, K*d] * W_cat[K*d, d] + dg * W_g
  if (dh != nullptr) {
    ProfScope prof(CPMTP_STAGE_DH, st);
    EpiStoreBf16<kBN, true>::Params ep{static_cast<uint16_t*>(dh), dg, static_cast<const uint16_t*>(W_g), s.N, d, d, s.r, accum};
    CPMTP_TRY((gemm_auto<false, true, EpiStoreBf16<kBN, true>>(dz, ncols, W_head, d, s.N, d, ncols, 2048, ep, dev_status, sms, st)));
  }
  // dW_g[r, d] = dg^T * h
  if (dW_g != nullptr) {
    ProfScope prof(CPMTP_STAGE_DW_G, st);
    dim3 grid((d + 127) / 128, L.dwg_slices);
    dwg_partial_kernel<CPMTP_MAX_R><<<grid, 128, 0, st>>>(dg, static_cast<const uint16_t*>(h), dwg_part, s.N, d, s.r,
                                                          L.dwg_rows_per_slice);
    CPMTP_TRY(cudaGetLastError());
    dwg_reduce_kernel<<<(s.r * d + 255) / 256, 256, 0, st>>>(dwg_part, static_cast<uint16_t*>(dW_g), L.dwg_slices,
                                                            s.r, d, accum);
    CPMTP_TRY(cudaGetLastError());
  }
  return CPMTP_OK;
}


extern "C" {

int cpmtp_version(void) { return 120; }   // 1.2: gradient accumulation flag, knob reload

int cpmtp_reload_knobs(void) {
  knobs();   // make sure the one-time read has happened, then read again
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  read_knobs();
  return CPMTP_OK;
}

int cpmtp_debug_status(void) {
#ifdef CPMTP_DEBUG
  int seen = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return CPMTP_ERR_LAUNCH;
  if (cudaMemcpyFromSymbol(&seen, g_debug_status, sizeof(int)) != cudaSuccess) return CPMTP_ERR_LAUNCH;
  return seen;
#else
  return -1;   // not a checked build
#endif
}

int cpmtp_profile_begin(void) {
  for (cudaEvent_t e : g_prof.events) cudaEventDestroy(e);
  g_prof.events.clear();
  g_prof.stages.clear();
  g_prof.on = true;
  return CPMTP_OK;
}

int cpmtp_profile_end(float* stage_ms, int32_t* stage_launches, int count) {
  g_prof.on = false;
  if (count < 0 || count > CPMTP_STAGE_COUNT) return CPMTP_ERR_SHAPE;
  if (cudaDeviceSynchronize() != cudaSuccess) return CPMTP_ERR_LAUNCH;
  for (int i = 0; i < count; ++i) {
    if (stage_ms) stage_ms[i] = 0.f;
    if (stage_launches) stage_launches[i] = 0;
  }
  const int total = static_cast<int>(g_prof.stages.size());
  for (int j = 0; j < total; ++j) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, g_prof.events[2 * j], g_prof.events[2 * j + 1]);
    const int stg = g_prof.stages[j];
    if (stg < count) {
      if (stage_ms) stage_ms[stg] += ms;
      if (stage_launches) stage_launches[stg] += 1;
    }
  }
  for (cudaEvent_t e : g_prof.events) cudaEventDestroy(e);
  g_prof.events.clear();
  g_prof.stages.clear();
  return total;
}

const char* cpmtp_status_string(int status) {
  switch (status) {
    case CPMTP_OK: return "ok";
    case CPMTP_ERR_NULL: return "a required pointer is NULL";
    case CPMTP_ERR_SHAPE: return "shape outside the supported limits (d % 64 == 0, r <= 32, n <= 8, sizes >= 1)";
    case CPMTP_ERR_ALIGN: return "a pointer is not aligned as required";
    case CPMTP_ERR_WORKSPACE: return "workspace too small";
    case CPMTP_ERR_ARCH: return "current device is not compute capability 10.x";
    case CPMTP_ERR_LAUNCH: return "a CUDA call failed";
    case CPMTP_ERR_LIMIT: return "size beyond a fixed built-in capacity";
    default: return "unknown status";
  }
}

size_t cpmtp_workspace_bytes(const cpmtp_shape* shape, int op) {
  if (validate_shape(shape) != CPMTP_OK) return 0;
  const int sms = sms_or_default();
  switch (op) {
    case CPMTP_OP_FORWARD:
    case CPMTP_OP_SCORE: return fwd_layout(*shape, sms).total;
    case CPMTP_OP_BACKWARD: return bwd_layout(*shape).total;
    case CPMTP_OP_SAMPLE: return sample_layout(*shape, sms).total;
    case CPMTP_OP_FORWARD_FULL: return full_layout(*shape, sms).total;
    case CPMTP_OP_BACKWARD_FULL: return full_bwd_layout(*shape).total;
    case CPMTP_OP_DISTILL_FORWARD: return distill_layout(*shape, sms).total;
    case CPMTP_OP_DISTILL_BACKWARD:
      return bwd_layout(*shape, kBM / padded_rank(shape->r) * shape->r, true).total;
    default: return 0;
  }
}

size_t cpmtp_host_staging_bytes(const cpmtp_shape* shape) {
  if (validate_shape(shape) != CPMTP_OK) return 0;
  return align_up(2ull * shape->N * shape->d) + align_up(4ull * shape->N * shape->n) +
         align_up(4ull * shape->N) + align_up(4);
}

int cpmtp_forward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E, const void* W_g,
                  const int32_t* x, float* logp, float* loss, const cpmtp_saved* saved, int32_t* expert_counts,
                  void* workspace, size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, x, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (logp == nullptr) return CPMTP_ERR_NULL;
  if (saved != nullptr) {
    const int rs = check_saved(saved, !(shape->flags & CPMTP_FLAG_RECOMPUTE_Z));
    if (rs != CPMTP_OK) return rs;
  }
  const FwdLayout L = fwd_layout(*shape, di->sms);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  return run_forward(*shape, static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_head),
                     static_cast<const uint16_t*>(E), static_cast<const uint16_t*>(W_g), x, logp, loss, saved,
                     expert_counts, nullptr, static_cast<uint8_t*>(workspace), L, dev_status, di->sms,
                     reinterpret_cast<cudaStream_t>(stream));
}

int cpmtp_score_draft(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                      const void* W_g, const int32_t* draft, float* logp_joint, float* logp_prefix,
                      void* workspace, size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, draft, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (logp_joint == nullptr) return CPMTP_ERR_NULL;
  const FwdLayout L = fwd_layout(*shape, di->sms);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  return run_forward(*shape, static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_head),
                     static_cast<const uint16_t*>(E), static_cast<const uint16_t*>(W_g), draft, logp_joint,
                     nullptr, nullptr, nullptr, logp_prefix, static_cast<uint8_t*>(workspace), L, dev_status,
                     di->sms, reinterpret_cast<cudaStream_t>(stream));
}

int cpmtp_sample_draft(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                       const void* W_g, const float* uniform, float temperature, int32_t topk,
                       const int32_t* forced, int32_t* draft, float* logp_joint, int32_t* topk_tokens,
                       float* topk_logp, void* workspace,
                       size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, /*x=*/h, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (draft == nullptr) return CPMTP_ERR_NULL;
  if (topk < 1 || topk > kMaxTopk || topk > shape->V) return CPMTP_ERR_SHAPE;
  if (shape->N > 65535) return CPMTP_ERR_LIMIT;   // positions ride on gridDim.y
  if (uniform != nullptr && !(temperature > 0.f)) return CPMTP_ERR_SHAPE;
  const cpmtp_shape& s = *shape;
  const SampleLayout L = sample_layout(s, di->sms);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* logits = reinterpret_cast<float*>(ws + L.logits);
  float* lb = reinterpret_cast<float*>(ws + L.lb);
  float* z32 = reinterpret_cast<float*>(ws + L.z32);
  Cand* part_top = reinterpret_cast<Cand*>(ws + L.part_top);
  Cand* part_best = reinterpret_cast<Cand*>(ws + L.part_best);
  float* logp_tmp = reinterpret_cast<float*>(ws + L.logp_tmp);
  float* logw = reinterpret_cast<float*>(ws + L.fwd.logw);
  float* lse = reinterpret_cast<float*>(ws + L.fwd.lse);
  // projection, unembedding (logits kept) and gate: the forward pipeline without targets
  const int rf = run_forward(s, static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_head),
                             static_cast<const uint16_t*>(E), static_cast<const uint16_t*>(W_g), nullptr, logp_tmp,
                             nullptr, nullptr, nullptr, nullptr, ws, L.fwd, dev_status, di->sms, st, logits, L.lds, z32);
  if (rf != CPMTP_OK) return rf;
  float* lb_exact = reinterpret_cast<float*>(ws + L.lb_exact);
  CPMTP_TRY(cudaMemcpyAsync(lb, logw, sizeof(float) * s.N * s.r, cudaMemcpyDeviceToDevice, st));   // b = w
  CPMTP_TRY(cudaMemcpyAsync(lb_exact, logw, sizeof(float) * s.N * s.r, cudaMemcpyDeviceToDevice, st));
  const float inv_temp = uniform != nullptr ? 1.0f / temperature : 1.0f;
  unsigned int* done = reinterpret_cast<unsigned int*>(ws + L.done);
  int* cand = reinterpret_cast<int*>(ws + L.cand);
  CPMTP_TRY(cudaMemsetAsync(done, 0, sizeof(unsigned int) * s.N, st));
  for (int step = 0; step < s.n; ++step) {
    ProfScope prof(CPMTP_STAGE_DRAFT_STEP, st);
    CPMTP_TRY(launch_pdl(draft_step_kernel, dim3(L.chunks, s.N), dim3(kSampleThreads), 0, st, logits, L.lds, z32,
                         static_cast<const uint16_t*>(E), s.d, lse, lb, lb_exact, uniform, inv_temp, step, s.N, s.V, s.n,
                         s.r, topk, forced, part_top, part_best, done, cand, dev_status, draft, logp_joint, topk_tokens,
                         topk_logp));
  }
  if (topk_logp != nullptr || logp_joint != nullptr) {
    // the last step's exact values (those of the earlier steps rode on the next step's launch)
    ProfScope prof(CPMTP_STAGE_DRAFT_STEP, st);
    CPMTP_TRY(launch_pdl(draft_tail_kernel, dim3(topk + 1, s.N), dim3(kSampleThreads), 0, st, z32,
                         static_cast<const uint16_t*>(E), s.d, lse, lb_exact, cand, s.N, s.V, s.n, s.r, topk, topk_logp,
                         logp_joint));
  }
  return CPMTP_OK;
}

int cpmtp_forward_full(const cpmtp_shape* shape, const void* h, const void* W_full, const void* W_g,
                       const int32_t* x, float* logp, float* loss, float* logp_prefix, const cpmtp_saved* saved,
                       int32_t* expert_counts, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                       cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_full, W_full, W_g, x, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (logp == nullptr) return CPMTP_ERR_NULL;
  if (static_cast<double>(shape->n) * shape->r * shape->V >= 2147483648.0) return CPMTP_ERR_SHAPE;
  if (saved != nullptr && (!saved->lse || !saved->tgt || !saved->logw || !saved->q || !saved->wbar))
    return CPMTP_ERR_NULL;
  const cpmtp_shape& s = *shape;
  const FullLayout L = full_layout(s, di->sms);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* logw = saved ? saved->logw : reinterpret_cast<float*>(ws + L.logw);
  float* q = saved ? saved->q : reinterpret_cast<float*>(ws + L.q);
  float* wbar = saved ? saved->wbar : reinterpret_cast<float*>(ws + L.wbar);
  float* lse = saved ? saved->lse : reinterpret_cast<float*>(ws + L.lse);
  float* tgt = saved ? saved->tgt : reinterpret_cast<float*>(ws + L.tgt);
  float* part_m = reinterpret_cast<float*>(ws + L.part_m);
  float* part_l = reinterpret_cast<float*>(ws + L.part_l);
  {
    ProfScope prof(CPMTP_STAGE_LSE, st);
    EpiLseFull<kBN>::Params ep{part_m, part_l, tgt, x, dev_status, s.N, s.V, L.K, s.n, s.r, L.tph, L.K * L.sph};
    const uint64_t b_rows = static_cast<uint64_t>(L.K) * s.V;
    CPMTP_TRY((launch_kk<EpiLseFull<kBN>>(L.wide, h, s.N, s.d, W_full, b_rows, s.d, s.d, L.sched, ep, dev_status, di->sms, st)));
  }
  {
    ProfScope prof(CPMTP_STAGE_MIXTURE, st);
    const int threads = s.N <= 256 ? 1024 : 256;
    // the target logits are complete already: handed over as one "partial" per head
    gate_mixture_kernel<<<s.N, threads, 0, st>>>(static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_g),
                                                s.d, part_m, part_l, L.sph, tgt, 1, logw, lse, nullptr, q, logp,
                                                logp_prefix, s.N, s.n, s.r);
    CPMTP_TRY(cudaGetLastError());
  }
  if (loss != nullptr || expert_counts != nullptr || saved != nullptr) {
    ProfScope prof(CPMTP_STAGE_FINALIZE, st);
    const float aux = (s.flags & CPMTP_FLAG_AUX) ? s.aux_coef : 0.f;
    finalize_kernel<<<1, kFinalizeThreads, 0, st>>>(logp, logw, wbar, expert_counts, loss, s.N, s.r, aux);
    CPMTP_TRY(cudaGetLastError());
  }
  return CPMTP_OK;
}

int cpmtp_backward_full(const cpmtp_shape* shape, const void* h, const void* W_full, const void* W_g,
                        const int32_t* x, const cpmtp_saved* saved, const float* dloss_dlogp, void* dh,
                        void* dW_full, void* dW_g, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                        cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_full, W_full, W_g, x, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (saved == nullptr || !saved->lse || !saved->logw || !saved->q || !saved->wbar || !dh || !dW_full || !dW_g)
    return CPMTP_ERR_NULL;
  if (!aligned(dh, 16) || !aligned(dW_full, 16) || !aligned(dW_g, 16)) return CPMTP_ERR_ALIGN;
  if (static_cast<double>(shape->n) * shape->r * shape->V >= 2147483648.0) return CPMTP_ERR_SHAPE;
  const cpmtp_shape& s = *shape;
  const FullBwdLayout L = full_bwd_layout(s);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* coef = reinterpret_cast<float*>(ws + L.coef);
  float* dg = reinterpret_cast<float*>(ws + L.dg);
  uint16_t* G = reinterpret_cast<uint16_t*>(ws + L.G);
  float* dh32 = reinterpret_cast<float*>(ws + L.dh32);
  float* dwg_part = reinterpret_cast<float*>(ws + L.dwg_part);
  const uint16_t* Wf = static_cast<const uint16_t*>(W_full);
  const uint16_t* hb = static_cast<const uint16_t*>(h);
  const int sms = di->sms;
  const int K = L.K, d = s.d, V = s.V;
  const float aux = (s.flags & CPMTP_FLAG_AUX) ? s.aux_coef : 0.f;
  const int per_token = (s.flags & CPMTP_FLAG_PER_TOKEN) ? 1 : 0;
  const int accum = (s.flags & CPMTP_FLAG_ACCUM_GRADS) ? 1 : 0;
  if (per_token && (dloss_dlogp == nullptr || saved->tgt == nullptr)) return CPMTP_ERR_NULL;
  {
    ProfScope prof(CPMTP_STAGE_COEFF, st);
    coeff_kernel<<<(s.N + 127) / 128, 128, 0, st>>>(saved->q, saved->logw, saved->wbar, saved->lse, saved->tgt,
                                                   dloss_dlogp, per_token, coef, dg, s.N, s.n, s.r, aux);
    CPMTP_TRY(cudaGetLastError());
  }
  const bool wide = use_wide(s.N, d);
  const int bm = wide ? kWideBM : kBM;
  const int tph = (V + kBN - 1) / kBN;
  for (int k0 = 0; k0 < K; k0 += L.heads_per_chunk) {
    const int heads = (K - k0) < L.heads_per_chunk ? (K - k0) : L.heads_per_chunk;
    const int ldg = L.heads_per_chunk * L.ldv;
    // recompute the logits of these heads -> G (bf16)
    {
      ProfScope prof(CPMTP_STAGE_LOGIT_GRAD, st);
      EpiLogitGradFull<kBN>::Params ep{{}, G, saved->lse, coef, x, s.N, V, K, s.n, s.r, tph, L.ldv, ldg, k0};
      if (!output_tmap(&ep.G_map, G, s.N, ldg, ldg)) return CPMTP_ERR_LAUNCH;
      Sched sc = make_sched((s.N + bm - 1) / bm, heads * tph, heads * tph, 2048 / bm, d / kBK);
      sc.seg_tiles = tph;
      sc.seg_stride = V;
      const uint16_t* Wc = Wf + static_cast<size_t>(k0) * V * d;
      const uint64_t b_rows = static_cast<uint64_t>(heads) * V;
      CPMTP_TRY((launch_kk<EpiLogitGradFull<kBN>>(wide, hb, s.N, d, Wc, b_rows, d, d, sc, ep, dev_status, sms, st)));
    }
    for (int k = k0; k < k0 + heads; ++k) {
      const uint16_t* Gk = G + static_cast<size_t>(k - k0) * L.ldv;
      const uint16_t* Wk = Wf + static_cast<size_t>(k) * V * d;
      // dW_full[k][V, d] = G_k^T[V, N] * h[N, d]
      {
        ProfScope prof(CPMTP_STAGE_DE, st);
        EpiStoreBf16<kBN, false>::Params ep{static_cast<uint16_t*>(dW_full) + static_cast<size_t>(k) * V * d, nullptr,
                                            nullptr, V, d, d, 0, accum};
        CPMTP_TRY((gemm_auto<true, true, EpiStoreBf16<kBN, false>>(Gk, ldg, hb, d, V, d, s.N, 2048, ep, dev_status, sms, st)));
      }
      // dh (+)= G_k[N, V] * W_full[k][V, d]
      {
        ProfScope prof(CPMTP_STAGE_DH, st);
        EpiAccumF32<kBN>::Params ep{dh32, s.N, d, d, k > 0 ? 1 : 0};
        CPMTP_TRY((gemm_auto<false, true, EpiAccumF32<kBN>>(Gk, ldg, Wk, d, s.N, d, V, 2048, ep, dev_status, sms, st)));
      }
    }
  }
  {
    ProfScope prof(CPMTP_STAGE_DE_CONVERT, st);
    const size_t total = static_cast<size_t>(s.N) * d;
    dh_finish_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(
        dh32, dg, static_cast<const uint16_t*>(W_g), static_cast<uint16_t*>(dh), s.N, d, s.r, accum);
    CPMTP_TRY(cudaGetLastError());
  }
  {
    ProfScope prof(CPMTP_STAGE_DW_G, st);
    dim3 grid((d + 127) / 128, L.dwg_slices);
    dwg_partial_kernel<CPMTP_MAX_R><<<grid, 128, 0, st>>>(dg, hb, dwg_part, s.N, d, s.r, L.dwg_rows_per_slice);
    CPMTP_TRY(cudaGetLastError());
    dwg_reduce_kernel<<<(s.r * d + 255) / 256, 256, 0, st>>>(dwg_part, static_cast<uint16_t*>(dW_g), L.dwg_slices, s.r, d, accum);
    CPMTP_TRY(cudaGetLastError());
  }
  return CPMTP_OK;
}

int cpmtp_verify_draft(int32_t N, int32_t n, const int32_t* draft, const int32_t* base_tokens,
                       const float* logp_prefix, const float* logp_base, const float* uniform, int32_t* accepted,
                       cpmtp_stream stream) {
  if (N < 1 || n < 1 || n > CPMTP_MAX_N) return CPMTP_ERR_SHAPE;
  if (accepted == nullptr) return CPMTP_ERR_NULL;
  if (base_tokens != nullptr) {
    if (draft == nullptr) return CPMTP_ERR_NULL;
  } else if (!logp_prefix || !logp_base || !uniform) {
    return CPMTP_ERR_NULL;
  }
  verify_draft_kernel<<<(N + 127) / 128, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      draft, base_tokens, logp_prefix, logp_base, uniform, accepted, N, n);
  CPMTP_TRY(cudaGetLastError());
  return CPMTP_OK;
}

int cpmtp_score_draft_static(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                             const void* W_g, const int32_t* draft, float* logp_joint, float* logp_prefix,
                             int32_t* dev_status, cpmtp_stream stream) {
  const int vs = validate_shape(shape);
  if (vs != CPMTP_OK) return vs;
  // architecture first: on a device without an sm_100a image the symbol lookup below would fail
  // with a less telling error
  DeviceInfo* dinfo = device_info();
  if (dinfo == nullptr) return CPMTP_ERR_LAUNCH;
  if (dinfo->cc_major != 10) return CPMTP_ERR_ARCH;
  unsigned char* scratch = static_scratch_ptr();
  if (scratch == nullptr) return CPMTP_ERR_LAUNCH;
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, draft, scratch, &di);
  if (rc != CPMTP_OK) return rc;
  if (logp_joint == nullptr) return CPMTP_ERR_NULL;
  const FwdLayout L = fwd_layout(*shape, di->sms);
  if (L.total > CPMTP_STATIC_SCRATCH_BYTES) return CPMTP_ERR_LIMIT;
  return run_forward(*shape, static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_head),
                     static_cast<const uint16_t*>(E), static_cast<const uint16_t*>(W_g), draft, logp_joint,
                     nullptr, nullptr, nullptr, logp_prefix, scratch, L, dev_status, di->sms,
                     reinterpret_cast<cudaStream_t>(stream));
}

int cpmtp_forward_host(const cpmtp_shape* shape, const void* h_host, const void* W_head, const void* E,
                       const void* W_g, const int32_t* x_host, float* logp_host, float* loss_host,
                       const cpmtp_saved* saved, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                       cpmtp_stream stream) {
  if (validate_shape(shape) != CPMTP_OK) return validate_shape(shape);
  if (!h_host || !x_host || !workspace) return CPMTP_ERR_NULL;
  if (!aligned(workspace, kAlign)) return CPMTP_ERR_ALIGN;
  const size_t fwd_bytes = cpmtp_workspace_bytes(shape, CPMTP_OP_FORWARD);
  if (workspace_bytes < fwd_bytes + cpmtp_host_staging_bytes(shape)) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* stage = static_cast<uint8_t*>(workspace) + align_up(fwd_bytes);
  const size_t h_bytes = 2ull * shape->N * shape->d, x_bytes = 4ull * shape->N * shape->n;
  uint8_t* h_dev = stage;
  uint8_t* x_dev = h_dev + align_up(h_bytes);
  uint8_t* logp_dev = x_dev + align_up(x_bytes);
  uint8_t* loss_dev = logp_dev + align_up(4ull * shape->N);
  {
    // everything cpmtp_forward would refuse is refused here, before anything is enqueued
    DeviceInfo* di = nullptr;
    const int rc = check_common(shape, h_dev, W_head, E, W_g, x_dev, workspace, &di);
    if (rc != CPMTP_OK) return rc;
    if (saved != nullptr) {
      const int rs = check_saved(saved, !(shape->flags & CPMTP_FLAG_RECOMPUTE_Z));
      if (rs != CPMTP_OK) return rs;
    }
  }
  CPMTP_TRY(cudaMemcpyAsync(h_dev, h_host, h_bytes, cudaMemcpyHostToDevice, st));
  CPMTP_TRY(cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, st));
  const int rc = cpmtp_forward(shape, h_dev, W_head, E, W_g, reinterpret_cast<const int32_t*>(x_dev),
                               reinterpret_cast<float*>(logp_dev), reinterpret_cast<float*>(loss_dev), saved,
                               nullptr, workspace, fwd_bytes, dev_status, stream);
  if (rc != CPMTP_OK) return rc;
  if (logp_host != nullptr)
    CPMTP_TRY(cudaMemcpyAsync(logp_host, logp_dev, 4ull * shape->N, cudaMemcpyDeviceToHost, st));
  if (loss_host != nullptr) CPMTP_TRY(cudaMemcpyAsync(loss_host, loss_dev, 4, cudaMemcpyDeviceToHost, st));
  return CPMTP_OK;
}

int cpmtp_distill_forward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                          const void* W_g, const int32_t* x, const void* teacher, float beta, float gamma,
                          float* logp, float* logp_prefix, float* loss, const cpmtp_saved* saved,
                          const cpmtp_distill_saved* dsaved, void* workspace, size_t workspace_bytes,
                          int32_t* dev_status, cpmtp_stream stream) {
  DeviceInfo* di = nullptr;
  const int rc = check_common(shape, h, W_head, E, W_g, x, workspace, &di);
  if (rc != CPMTP_OK) return rc;
  if (!teacher || !logp || !logp_prefix || !saved || !dsaved) return CPMTP_ERR_NULL;
  if (!dsaved->lse_t || !dsaved->logpi || !dsaved->pm || !dsaved->kl) return CPMTP_ERR_NULL;
  if (!aligned(teacher, 16)) return CPMTP_ERR_ALIGN;
  const cpmtp_shape& s = *shape;
  const bool recompute_z = (s.flags & CPMTP_FLAG_RECOMPUTE_Z) != 0;
  const int rs = check_saved(saved, !recompute_z);
  if (rs != CPMTP_OK) return rs;
  const DistillLayout L = distill_layout(s, di->sms);
  if (workspace_bytes < L.total) return CPMTP_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const uint16_t* Tb = static_cast<const uint16_t*>(teacher);
  // Eq. 9 with the prefix scores (the cross-entropy part of Eq. 14), lse / tgt / logw / wbar / z kept
  const int rf = run_forward(s, static_cast<const uint16_t*>(h), static_cast<const uint16_t*>(W_head),
                             static_cast<const uint16_t*>(E), static_cast<const uint16_t*>(W_g), x, logp, nullptr, saved,
                             nullptr, logp_prefix, ws, L.fwd, dev_status, di->sms, st);
  if (rf != CPMTP_OK) return rf;
  const uint16_t* z = recompute_z ? reinterpret_cast<const uint16_t*>(ws + L.fwd.z)
                                  : static_cast<const uint16_t*>(saved->z);
  {
    ProfScope prof(CPMTP_STAGE_TEACHER_LSE, st);   // expert weights per token; the teacher's normaliser comes out of the KL sweep
    distill_pi_kernel<<<(s.N + 127) / 128, 128, 0, st>>>(saved->logw, saved->lse, saved->tgt, dsaved->logpi, s.N, s.n,
                                                        s.r);
    CPMTP_TRY(cudaGetLastError());
  }
  float* part = reinterpret_cast<float*>(ws + L.part);
  float* part_tm = reinterpret_cast<float*>(ws + L.part_tm);
  float* part_tl = reinterpret_cast<float*>(ws + L.part_tl);
  {
    ProfScope prof(CPMTP_STAGE_KL, st);
    const KlParams ep{part, part_tm, part_tl, saved->lse, dsaved->logpi, Tb, L.groups, s.r, s.V, L.sched.n_splits,
                      s.V % 8 == 0 ? 1 : 0};
    CPMTP_TRY((launch_grouped<EpiKl>(L.R, z, L.fwd.M, s.d, static_cast<const uint16_t*>(E), s.V, L.sched, ep, s.r,
                                     dev_status, di->sms, st)));
  }
  {
    ProfScope prof(CPMTP_STAGE_FINALIZE, st);
    distill_merge_kernel<<<(L.groups + 3) / 4, 128, 0, st>>>(part, part_tm, part_tl, dsaved->logpi, L.sched.n_splits,
                                                            dsaved->lse_t, dsaved->pm, dsaved->kl, L.groups, s.r);
    CPMTP_TRY(cudaGetLastError());
    if (loss != nullptr) {
      const float aux = (s.flags & CPMTP_FLAG_AUX) ? s.aux_coef : 0.f;
      distill_loss_kernel<<<1, kDistillLossThreads, 0, st>>>(logp_prefix, dsaved->kl, saved->wbar, nullptr, nullptr,
                                                            beta, gamma, aux, s.N, s.n, s.r, loss);
      CPMTP_TRY(cudaGetLastError());
    }
  }
  return CPMTP_OK;
}

int cpmtp_distill_backward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E,
                           const void* W_g, const int32_t* x, const void* teacher, const cpmtp_saved* saved,
                           const cpmtp_distill_saved* dsaved, float beta, float gamma, const float* dloss_dprefix,
                           const float* dloss_dkl, void* dh, void* dW_head, void* dE, void* dW_g, void* workspace,
                           size_t workspace_bytes, int32_t* dev_status, cpmtp_stream stream) {
  if (!teacher || !dsaved) return CPMTP_ERR_NULL;
  if (!dsaved->lse_t || !dsaved->logpi || !dsaved->pm || !dsaved->kl) return CPMTP_ERR_NULL;
  if (!aligned(teacher, 16)) return CPMTP_ERR_ALIGN;
  DistillCtx dc{static_cast<const uint16_t*>(teacher), dsaved, dloss_dkl, beta, gamma};
  return backward_impl(shape, h, W_head, E, W_g, x, saved, dloss_dprefix, dh, dW_head, dE, dW_g, workspace,
                       workspace_bytes, dev_status, stream, &dc);
}

int cpmtp_backward(const cpmtp_shape* shape, const void* h, const void* W_head, const void* E, const void* W_g,
                   const int32_t* x, const cpmtp_saved* saved, const float* dloss_dlogp, void* dh, void* dW_head,
                   void* dE, void* dW_g, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                   cpmtp_stream stream) {
  return backward_impl(shape, h, W_head, E, W_g, x, saved, dloss_dlogp, dh, dW_head, dE, dW_g, workspace,
                       workspace_bytes, dev_status, stream, nullptr);
}

}  // extern "C"
