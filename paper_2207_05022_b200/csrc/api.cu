// Host runtime behind the C ABI: contexts, plans, the preload buffer, the pinned arena, the ring of
// streamed-layer slots, tile-job tables, and the layerwise copy/compute pipeline (Sections 3.1, 5.5).
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <chrono>
#include <string>
#include <thread>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/sti.h"
#include "retile.h"
#include "sti_kernels.h"

using namespace sti;

namespace {

constexpr int kMaxLayersStats = 64;
constexpr size_t kMaxSmem = 227 * 1024;
// Guard words around the preload buffer and around every ring slot: nothing may ever write them (only the layer
// copies and the upload write those buffers), sti_plan_check_guards reads them back.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardPattern = 0xA5;
constexpr int kStampKernels = 8;       // per layer: cast, QKV, attention, O projection, LayerNorm 1, FFN1, FFN2, LayerNorm 2
constexpr int kStampRecord = 8;        // 64-bit words per kernel launch (kStampWords of the device code)

inline size_t align16(size_t v) { return (v + 15) & ~static_cast<size_t>(15); }
inline size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

struct MatrixInfo {
  uint32_t rows, kc;
  uint32_t flat_base;   // first weight's flat offset in the unit
};

struct Tuning {
  int qkv_n = 32, f1_n = 64, o_n = 64, o_group = 4, f2_n = 64, f2_group = 2;
  int cta_budget = 148;                // (replaced by the device's SM count in parse_tuning) CTAs a GEMM launch may use when it splits the token tiles over CTAs
  int pair_min_tiles = 8;              // two-CTA GEMM from this many 128-token tiles on (0 = never)
  int f2_kacc_min_tokens = 4096;       // FFN2 through the K-accumulating kernel (one output plane) from this many tokens on (0 = never)
  int f2_kacc_k = 512;                 // columns per K group there
  int f2_kacc_bps = 2;                 // boxes of 64 columns per ring stage there (1 or 2)
  int attn_tc_min_items = 96;          // tensor-core attention from this many (sequence, kept head) pairs on, seq >= 256 (0 = never)
  int ln1_ctas = -1, ln2_ctas = -1;    // LayerNorm CTA counts: -1 = chosen per launch (see ln_ctas_hint), 0 = one row per CTA
};

struct Unit {
  sti_shard_cfg cfg{};
  bool uploaded = false;
  std::vector<uint8_t> codes;          // re-tiled (or raw fp32), until finalize moves it into an arena
  std::vector<float> table;
  std::vector<uint32_t> out_off;
  std::vector<float> out_val;
  size_t off_codes = 0, off_table = 0, off_ooff = 0, off_oval = 0, bytes = 0;   // inside the layer part
  uint8_t* dev = nullptr;              // where the unit's region starts in device memory
  size_t codes_bytes = 0;              // size of the index stream (known even when the bytes are not on the host)
  // Back-to-back executions (Section 3.2): a unit another plan already holds in device memory is taken over with
  // a device-to-device copy instead of an upload; a streamed unit can be kept after a run for the next plan.
  const uint8_t* adopt_src = nullptr;  // device address of the whole unit region in the plan it is adopted from
  bool retain = false;                 // copy this streamed unit out of its ring slot during the next forward
  uint8_t* retained = nullptr;         // where that copy lives (retained arena), valid once retained_done
  bool retained_done = false;
};

struct GemmTable {
  Job* jobs = nullptr;
  Seg* segs = nullptr;
  int n_jobs = 0;
  size_t smem = 0;
  uint32_t w_bytes = 0, n_stages = 0, bps = 1, k_max = 0, hdr_bytes = 0, seg_stride = 0;
  bool pair_ok = false;                // consecutive jobs can share two-CTA MMAs (64-row tiles, same K range)
  int n_split = 0;
};

struct Layer {
  std::vector<Unit> attn, ffn;
  std::vector<int> kept_heads, kept_slices;
  size_t res_bytes = 0, str_bytes = 0;
  uint8_t* res_dev = nullptr;          // in the preload buffer
  uint8_t* str_host = nullptr;         // in the pinned arena
  int slot = -1;                       // ring slot of the streamed part
  size_t tables_off = 0, tables_bytes = 0;   // this layer's tile-job descriptors inside the plan's table buffer
  GemmTable qkv, o, f1, f2;
  GemmTable f2k;                       // FFN2 again, cut for the K-accumulating kernel (plans made for many tokens only)
  cudaEvent_t ev_loaded = nullptr, ev_done = nullptr, ev_copy_start = nullptr, ev_comp_start = nullptr;
  cudaEvent_t g_ev_loaded = nullptr;   // the same role inside graph capture (captured events cannot be reused outside)
  cudaEvent_t ev_k[8] = {};           // boundaries of the seven kernels (kernel-level profiling)
  bool k_ran[7] = {};
};

}  // namespace

struct sti_ctx {
  sti_model_desc desc{};
  int device = 0;
  cudaStream_t compute = nullptr, copy = nullptr;
  bool own_compute = false;
  float* dense = nullptr;              // [n_layers][dense_stride]
  size_t dense_stride = 0;
  size_t off_bq = 0, off_bk = 0, off_bv = 0, off_bo = 0, off_b1 = 0, off_b2 = 0, off_ln1g = 0, off_ln1b = 0,
         off_ln2g = 0, off_ln2b = 0;
  int* err_dev = nullptr;
  uint64_t launches = 0;
  bool simt_debug = false;
  bool pdl = true;                     // programmatic dependent launch between the kernels of a layer
  int sm_count = 0;
  sti_status async_error = STI_OK;
  MatrixInfo attn_m[4]{}, ffn_m[2]{};
  uint32_t attn_weights = 0, ffn_weights = 0;
};

struct ForwardKey {
  const void* x = nullptr; void* y = nullptr;            // device buffers (device variant)
  const void* x_host = nullptr; void* y_host = nullptr;  // host buffers (host variant)
  const int32_t* lens = nullptr;                         // device
  int batch = 0, seq = 0;
  int layer = -1;                                        // >= 0: a single layer (sti_layer_forward)
  bool stamps = false;                                   // kernels write profiling stamps (profiling level 3)
  bool operator==(const ForwardKey& o) const {
    return stamps == o.stamps && layer == o.layer && x == o.x && y == o.y && x_host == o.x_host && y_host == o.y_host && lens == o.lens && batch == o.batch &&
           seq == o.seq;
  }
};

struct sti_plan {
  sti_ctx* ctx = nullptr;
  std::vector<Layer> layers;
  int ring_slots = 2;
  bool finalized = false;
  bool attempted = false;
  int profiling = 0;                   // 0 off, 1 per layer, 2 per kernel
  Tuning tune;
  uint8_t* preload = nullptr;  size_t preload_bytes = 0;
  uint8_t* pinned = nullptr;   size_t pinned_bytes = 0;
  uint8_t* ring = nullptr;     size_t slot_bytes = 0;      // a slot = its data followed by kGuardBytes of guard pattern
  uint8_t* ring_alloc = nullptr; uint8_t* preload_alloc = nullptr;   // the allocations: a leading guard, then `ring` / `preload`
  uint8_t* tables = nullptr;   size_t tables_bytes = 0;       // job/segment descriptors
  std::vector<cudaEvent_t> slot_free, g_slot_free;   // direct launches / graph capture
  cudaEvent_t ev_copy_tail = nullptr, ev_begin = nullptr, ev_end = nullptr, ev_fork = nullptr, g_ev_join = nullptr;
  struct CachedGraph { ForwardKey key; cudaGraphExec_t exec = nullptr; uint64_t launches = 0; uint64_t last_use = 0; };
  std::vector<CachedGraph> graphs;     // captured forwards, a few most recently used (buffers + shape + layer)
  uint64_t graph_clock = 0;
  bool graph_off = false;
  bool copy_tail_valid = false;
  // activation scratch
  uint16_t* qkv = nullptr; uint16_t* attn_out = nullptr; float* partial = nullptr;
  float* h1_f32 = nullptr; uint16_t* h1_bf16 = nullptr; uint16_t* u = nullptr;
  uint16_t* x_bf16 = nullptr;          // bf16 copy of fp32 layer inputs (the GEMM operand)
  void* buf[2] = {nullptr, nullptr};
  void* x_in = nullptr; void* y_out = nullptr; int32_t* lens_dev = nullptr;
  int max_partial = 1;
  float* zero_bias = nullptr;          // all-zero bias vector of sti_gemm_probe (allocated by its first call)
  uint8_t* rate_tables = nullptr;      // every layer's FFN1 tile jobs in one table (sti_decode_rate_probe, built by its first call)
  int rate_jobs = 0; uint32_t rate_seg_stride = 0; uint64_t rate_packed_bytes = 0;
  unsigned long long* stamps = nullptr;   // [layer][kStampKernels][kStampWords] device, profiling level 3
  bool stamping = false;               // the forward being enqueued writes stamps
  bool overlap = true;                 // false: load every streamed layer, then execute (Load&Exec)
  uint8_t* retain_arena = nullptr; size_t retain_bytes = 0;   // streamed units kept for the next plan
  bool retain_pending = false;         // the next model forward copies the units marked `retain` out of the ring
  uint64_t finalize_h2d_bytes = 0, finalize_d2d_bytes = 0;    // how the preload buffer was filled
  int slow_copy_layer = -1;            // host-made faults (sti_plan_inject): sleep before enqueueing this layer's copy ...
  unsigned slow_copy_us = 0;           // ... for this long
  bool fail_pinned_alloc = false;      // make the pinned-arena allocation of sti_plan_finalize fail
  int n_streamed_layers = 0;
  bool stats_valid = false;
};

namespace {

#define CUDA_TRY(expr)                          \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) {                   \
      if (e__ == cudaErrorMemoryAllocation) {   \
        (void)cudaGetLastError();               \
        return STI_ERR_OOM;                     \
      }                                         \
      return STI_ERR_CUDA;                      \
    }                                           \
  } while (0)

size_t act_size(const sti_ctx* c) { return c->desc.act_dtype == STI_BF16 ? 2 : 4; }

const MatrixInfo* unit_matrices(const sti_ctx* c, sti_kind kind, int* n) {
  *n = kind == STI_ATTN ? 4 : 2;
  return kind == STI_ATTN ? c->attn_m : c->ffn_m;
}

size_t matrix_code_bytes(const MatrixInfo& m, int bits) {
  return static_cast<size_t>(m.rows) * m.kc * bits / 8;
}

void parse_tuning(Tuning* t, int tmax, const sti_model_desc& d, int sm_count) {
  t->cta_budget = sm_count;
  // few tokens: K groups of 8 heads / 2 FFN slices, one CTA per token tile (the decode is spread over the SMs, MMA
  // chains stay short); many tokens: wide K groups, each CTA walks many token tiles with its decoded weights
  if (tmax > 1024) {
    t->qkv_n = 64; t->f1_n = 64; t->o_n = 64; t->o_group = 16; t->f2_n = 64; t->f2_group = 4;
  } else {
    t->qkv_n = 64; t->f1_n = 64; t->o_n = 64; t->o_group = 8; t->f2_n = 64; t->f2_group = 2;
  }
  const char* env = getenv("STI_TUNE");     // debugging aid: "qkv_n=32,o_group=4,..."
  if (env) {
    std::string s(env);
    size_t pos = 0;
    while (pos < s.size()) {
      size_t end = s.find(',', pos);
      if (end == std::string::npos) end = s.size();
      const std::string kv = s.substr(pos, end - pos);
      const size_t eq = kv.find('=');
      if (eq != std::string::npos) {
        const std::string k = kv.substr(0, eq);
        const int v = atoi(kv.c_str() + eq + 1);
        if (k == "qkv_n") t->qkv_n = v;
        else if (k == "f1_n") t->f1_n = v;
        else if (k == "o_n") t->o_n = v;
        else if (k == "o_group") t->o_group = v;
        else if (k == "f2_n") t->f2_n = v;
        else if (k == "f2_group") t->f2_group = v;
        else if (k == "pair_min_tiles") t->pair_min_tiles = v;
        else if (k == "f2_kacc_min_tokens") t->f2_kacc_min_tokens = std::max(0, v);
        else if (k == "f2_kacc_k") t->f2_kacc_k = std::max(64, std::min(v, 1024));
        else if (k == "f2_kacc_bps") t->f2_kacc_bps = v == 1 ? 1 : 2;
        else if (k == "attn_tc_min_items") t->attn_tc_min_items = std::max(0, v);
        else if (k == "cta_budget") t->cta_budget = std::max(1, v);
        else if (k == "ln1_ctas") t->ln1_ctas = std::max(-1, v);
        else if (k == "ln2_ctas") t->ln2_ctas = std::max(-1, v);
      }
      pos = end + 1;
    }
  }
  auto pow2_tile = [](int v, int lo) { return (v == 32 || v == 64 || v == 128) && v >= lo ? v : lo; };
  t->qkv_n = std::min(pow2_tile(t->qkv_n, 32), 64);
  const int f = d.ffn / d.n_ffn_slices;
  t->f1_n = pow2_tile(t->f1_n, 32);
  while (f % t->f1_n) t->f1_n /= 2;
  t->o_n = pow2_tile(t->o_n, 64);
  t->f2_n = pow2_tile(t->f2_n, 32);
  while (d.hidden % t->o_n) t->o_n /= 2;
  while (d.hidden % t->f2_n) t->f2_n /= 2;
  t->o_group = std::max(1, std::min(t->o_group, 16));
  t->f2_group = std::max(1, std::min(t->f2_group, 16));
  // keep every weight tile inside shared memory
  auto fits = [](int n, int k) {
    uint32_t st = 0, bp = 0;
    return gemm_pick_ring(static_cast<uint32_t>(gemm_weight_bytes(n, k)), k, gemm_header_bytes(), &st, &bp) && st * bp >= 4;
  };
  while (t->qkv_n > 32 && !fits(t->qkv_n, d.hidden)) t->qkv_n /= 2;
  while (t->f1_n > 32 && !fits(t->f1_n, d.hidden)) t->f1_n /= 2;
  while (t->o_group > 1 && !fits(t->o_n, t->o_group * 64)) --t->o_group;
  while (t->f2_group > 1 && !fits(t->f2_n, t->f2_group * f)) --t->f2_group;
}

Unit* find_unit(sti_plan* p, int layer, sti_kind kind, int index) {
  if (layer < 0 || layer >= static_cast<int>(p->layers.size())) return nullptr;
  auto& v = kind == STI_ATTN ? p->layers[layer].attn : p->layers[layer].ffn;
  if (index < 0 || index >= static_cast<int>(v.size())) return nullptr;
  return &v[index];
}

// Segment for rows [row0, row0 + n_rows) of matrix `m` of `u`.
Seg make_seg(const sti_ctx* c, const Unit& u, sti_kind kind, int m, uint32_t row0, uint32_t n_rows, uint32_t koff) {
  int nm;
  const MatrixInfo* mi = unit_matrices(c, kind, &nm);
  const int bits = u.cfg.bits;
  size_t mat_off = 0;
  for (int i = 0; i < m; ++i) mat_off += matrix_code_bytes(mi[i], bits);
  Seg s{};
  s.codes = reinterpret_cast<const uint4*>(u.dev + u.off_codes + mat_off +
                                           static_cast<size_t>(row0) * mi[m].kc * bits / 8);
  s.table = reinterpret_cast<const float*>(u.dev + u.off_table);
  s.flat_base = mi[m].flat_base + row0 * mi[m].kc;
  const uint32_t flat_end = s.flat_base + n_rows * mi[m].kc;
  const size_t lo = std::lower_bound(u.out_off.begin(), u.out_off.end(), s.flat_base) - u.out_off.begin();
  const size_t hi = std::lower_bound(u.out_off.begin(), u.out_off.end(), flat_end) - u.out_off.begin();
  s.out_off = reinterpret_cast<const uint32_t*>(u.dev + u.off_ooff) + lo;
  s.out_val = reinterpret_cast<const float*>(u.dev + u.off_oval) + lo;
  s.n_out = static_cast<uint32_t>(hi - lo);
  s.bits = bits;
  s.kc = mi[m].kc;
  s.koff = koff;
  return s;
}

struct TableBuilder {
  std::vector<Job> jobs;
  std::vector<std::vector<Seg>> job_segs;
  std::vector<Seg> segs;               // filled by finish(): job j's segments start at j * seg_stride
  uint32_t w_bytes = 0, k_max = 0, seg_stride = 0;
  void add(Job j, const std::vector<Seg>& ss) {
    j.n_seg = static_cast<uint32_t>(ss.size());
    jobs.push_back(j);
    job_segs.push_back(ss);
    w_bytes = std::max(w_bytes, static_cast<uint32_t>(gemm_weight_bytes(j.n_rows, j.k_total)));
    k_max = std::max(k_max, j.k_total);
    seg_stride = std::max(seg_stride, j.n_seg);
  }
  // A fixed stride lets a CTA fetch its job and its segments in the same memory round trip.
  void finish() {
    segs.assign(jobs.size() * seg_stride, Seg{});
    for (size_t j = 0; j < jobs.size(); ++j) {
      jobs[j].seg_begin = static_cast<uint32_t>(j * seg_stride);
      std::copy(job_segs[j].begin(), job_segs[j].end(), segs.begin() + j * seg_stride);
    }
  }
};

void build_layer_tables(sti_plan* p, Layer& L, TableBuilder tb[5]) {
  const sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  const Tuning& t = p->tune;
  const uint32_t f = d.ffn / d.n_ffn_slices;
  // QKV: one job per (kept head, matrix, row tile); full K
  for (size_t hi = 0; hi < L.kept_heads.size(); ++hi) {
    const int h = L.kept_heads[hi];
    for (int which = 0; which < 3; ++which)
      for (uint32_t r0 = 0; r0 < 64; r0 += t.qkv_n) {
        Job j{};
        j.n_rows = t.qkv_n; j.k_total = d.hidden; j.x_koff = 0;
        j.out_mat = static_cast<uint32_t>(hi * 3 + which); j.out_col = r0;
        j.bias_off = which * d.n_heads * 64 + h * 64 + static_cast<int>(r0);
        tb[0].add(j, {make_seg(c, L.attn[h], STI_ATTN, which, r0, t.qkv_n, 0)});
      }
  }
  // O projection: K is split over groups of kept heads, each group writes its own partial sum
  const int nh = static_cast<int>(L.kept_heads.size());
  L.o.n_split = (nh + t.o_group - 1) / t.o_group;
  for (int sp = 0; sp < L.o.n_split; ++sp) {
    const int first = sp * t.o_group, cnt = std::min(t.o_group, nh - first);
    for (uint32_t n0 = 0; n0 < static_cast<uint32_t>(d.hidden); n0 += t.o_n) {
      Job j{};
      j.n_rows = t.o_n; j.k_total = cnt * 64; j.x_koff = first * 64;
      j.out_mat = sp; j.out_col = n0; j.bias_off = -1;
      std::vector<Seg> ss;
      for (int i = 0; i < cnt; ++i)
        ss.push_back(make_seg(c, L.attn[L.kept_heads[first + i]], STI_ATTN, 3, n0, t.o_n, i * 64));
      tb[1].add(j, ss);
    }
  }
  // FFN1: one job per (kept slice, row tile); full K
  for (size_t ji = 0; ji < L.kept_slices.size(); ++ji) {
    const int s = L.kept_slices[ji];
    for (uint32_t r0 = 0; r0 < f; r0 += t.f1_n) {
      Job j{};
      j.n_rows = t.f1_n; j.k_total = d.hidden; j.x_koff = 0;
      j.out_mat = 0; j.out_col = static_cast<uint32_t>(ji * f + r0);
      j.bias_off = s * static_cast<int>(f) + static_cast<int>(r0);
      tb[2].add(j, {make_seg(c, L.ffn[s], STI_FFN, 0, r0, t.f1_n, 0)});
    }
  }
  // FFN2: K split over groups of kept slices
  const int ns = static_cast<int>(L.kept_slices.size());
  L.f2.n_split = (ns + t.f2_group - 1) / t.f2_group;
  for (int sp = 0; sp < L.f2.n_split; ++sp) {
    const int first = sp * t.f2_group, cnt = std::min(t.f2_group, ns - first);
    for (uint32_t n0 = 0; n0 < static_cast<uint32_t>(d.hidden); n0 += t.f2_n) {
      Job j{};
      j.n_rows = t.f2_n; j.k_total = cnt * f; j.x_koff = first * f;
      j.out_mat = sp; j.out_col = n0; j.bias_off = -1;
      std::vector<Seg> ss;
      for (int i = 0; i < cnt; ++i)
        ss.push_back(make_seg(c, L.ffn[L.kept_slices[first + i]], STI_FFN, 1, n0, t.f2_n, i * f));
      tb[3].add(j, ss);
    }
  }
  // FFN2 for the K-accumulating kernel: 64-row tiles, K groups of at most 512 columns, group-major order
  const int kacc_group = static_cast<int>(t.f2_kacc_k / f);      // whole slices per K group (0: a slice does not fit)
  L.f2k.n_split = 0;
  if (kacc_group > 0 && ns > 0 && d.hidden % 128 == 0 && t.f2_kacc_min_tokens > 0 &&
      static_cast<long long>(d.max_batch) * d.max_seq >= t.f2_kacc_min_tokens) {
    L.f2k.n_split = (ns + kacc_group - 1) / kacc_group;
    for (int sp = 0; sp < L.f2k.n_split; ++sp) {
      const int first = sp * kacc_group, cnt = std::min(kacc_group, ns - first);
      for (uint32_t n0 = 0; n0 < static_cast<uint32_t>(d.hidden); n0 += 64) {
        Job j{};
        j.n_rows = 64; j.k_total = cnt * f; j.x_koff = first * f;
        j.out_mat = 0; j.out_col = n0; j.bias_off = -1;
        std::vector<Seg> ss;
        for (int i = 0; i < cnt; ++i)
          ss.push_back(make_seg(c, L.ffn[L.kept_slices[first + i]], STI_FFN, 1, n0, 64, i * f));
        tb[4].add(j, ss);
      }
    }
  }
}

sti_status check_async(sti_ctx* c) {
  int flag = 0;
  if (cudaMemcpy(&flag, c->err_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return STI_ERR_CUDA;
  if (flag != ERR_NONE) {
    int zero = 0;
    (void)cudaMemcpy(c->err_dev, &zero, sizeof(int), cudaMemcpyHostToDevice);
    if (getenv("STI_VERBOSE")) fprintf(stderr, "sti: device status word 0x%08x\n", static_cast<unsigned>(flag));
    return (flag & 0xff) == ERR_WAIT_TIMEOUT ? STI_ERR_TIMEOUT : STI_ERR_ARG;
  }
  return STI_OK;
}

// cuTensorMapEncodeTiled is a driver entry point; it is looked up through the runtime so that the
// library does not link against libcuda directly.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// TMA view of a bf16 activation matrix [rows, ld]: boxes of 128 rows x 64 columns, 128-byte swizzle,
// rows past `rows` read as zeros.
bool make_xmap(CUtensorMap* map, const void* base, int ld, int rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || (reinterpret_cast<uintptr_t>(base) & 15) || (ld % 8) != 0) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(ld), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int m_ctas_for(int n_jobs, int T, int cta_budget) {
  const int n_mtiles = (T + 127) / 128;
  int m = n_jobs > 0 ? cta_budget / n_jobs : 1;
  return std::max(1, std::min(m, n_mtiles));
}

// The packed shards of layer `li` as (address, bytes) ranges: its part of the preload buffer and its ring slot.
void layer_ranges(const sti_plan* p, int li, const uint8_t* ptr[4], uint32_t bytes[4]) {
  for (int r = 0; r < 4; ++r) { ptr[r] = nullptr; bytes[r] = 0; }
  if (li < 0 || li >= static_cast<int>(p->layers.size())) return;
  const Layer& L = p->layers[li];
  if (L.res_bytes) { ptr[0] = L.res_dev; bytes[0] = static_cast<uint32_t>(L.res_bytes); }
  if (L.str_bytes) { ptr[1] = p->ring + static_cast<size_t>(L.slot) * p->slot_bytes; bytes[1] = static_cast<uint32_t>(L.str_bytes); }
  ptr[2] = p->tables + L.tables_off; bytes[2] = static_cast<uint32_t>(L.tables_bytes);
  ptr[3] = reinterpret_cast<const uint8_t*>(p->ctx->dense + static_cast<size_t>(li) * p->ctx->dense_stride);
  bytes[3] = static_cast<uint32_t>(p->ctx->dense_stride * sizeof(float));
}

// `force_pair`: -1 = the two-CTA kernel from pair_min_tiles token tiles on, 0 = never, 1 = always (the table must allow it).
sti_status run_gemm(sti_plan* p, GemmKind kind, const GemmTable& tab, const void* x, int ldx, int T, void* out,
                    int ldo, const float* bias, int prefetch_layer = -1, int force_pair = -1,
                    unsigned long long* stamps = nullptr) {
  if (tab.n_jobs == 0) return STI_OK;
  GemmLaunch g{};
  g.stamps = stamps;
  g.jobs = tab.jobs; g.segs = tab.segs; g.n_jobs = tab.n_jobs; g.m_ctas = m_ctas_for(tab.n_jobs, T, p->tune.cta_budget);
  const int n_mtiles = (T + 127) / 128;
  g.pair = tab.pair_ok && p->tune.pair_min_tiles > 0 && n_mtiles >= p->tune.pair_min_tiles;
  if (force_pair == 0) g.pair = false;
  if (force_pair == 1) {
    if (!tab.pair_ok) return STI_ERR_STATE;
    g.pair = true;
  }
  if (g.pair) {      // a pair of CTAs takes two token tiles at a time
    const int n_mpairs = (n_mtiles + 1) / 2;
    g.m_ctas = std::max(1, std::min(n_mpairs, p->tune.cta_budget / tab.n_jobs));
  }
  if (!make_xmap(&g.xmap, x, ldx, T)) return STI_ERR_CUDA;
  layer_ranges(p, prefetch_layer, g.pf_ptr, g.pf_bytes);
  g.x = x; g.ldx = ldx; g.T = T; g.out = out; g.ldo = ldo; g.bias = bias; g.err = p->ctx->err_dev;
  g.smem_bytes = tab.smem; g.n_stages = tab.n_stages; g.bps = tab.bps; g.w_bytes = tab.w_bytes; g.hdr_bytes = tab.hdr_bytes; g.seg_stride = tab.seg_stride; g.simt_debug = p->ctx->simt_debug; g.pdl = p->ctx->pdl;
  CUDA_TRY(launch_gemm(kind, g, p->ctx->compute));
  p->ctx->launches++;
  return STI_OK;
}

// FFN2 through the K-accumulating kernel: one complete fp32 plane [T][ldo] instead of one plane per K group.
sti_status run_gemm_kacc(sti_plan* p, const GemmTable& tab, const void* x, int ldx, int T, float* out, int ldo,
                         unsigned long long* stamps) {
  if (tab.n_jobs == 0 || tab.n_split == 0) return STI_ERR_STATE;
  KaccLaunch g{};
  g.jobs = tab.jobs; g.segs = tab.segs; g.n_groups = tab.n_split; g.n_cols64 = tab.n_jobs / tab.n_split;
  const int n_mpairs = ((T + 127) / 128 + 1) / 2;
  g.m_ctas = std::max(1, std::min(n_mpairs, p->tune.cta_budget / g.n_cols64));
  if (!make_xmap(&g.xmap, x, ldx, T)) return STI_ERR_CUDA;
  // an operand that does not fit L2 (126 MB, shared with everything else in flight) is prefetched by idle warps;
  // measured: 32 x 512 tokens (134 MB) 159 -> 149 us per launch, 8,192 tokens (67 MB) 79 -> 81
  g.x = static_cast<size_t>(T) * ldx * 2 > (100u << 20) ? x : nullptr; g.ldx = ldx;
  g.T = T; g.out = out; g.ldo = ldo; g.err = p->ctx->err_dev;
  g.n_stages = tab.n_stages; g.bps = tab.bps; g.hdr_bytes = tab.hdr_bytes; g.seg_stride = tab.seg_stride; g.k_group = tab.k_max;
  g.pdl = p->ctx->pdl; g.stamps = stamps;
  CUDA_TRY(launch_gemm_kacc(g, p->ctx->compute));
  p->ctx->launches++;
  return STI_OK;
}

// How many CTAs a LayerNorm launch should use, given the GEMM that follows it.  A GEMM CTA needs a whole SM and its
// CTAs are launched while the LayerNorm runs (they decode their weights meanwhile) - on SMs that hold no LayerNorm
// CTA.  With one row per CTA the LayerNorm of a few hundred tokens spreads over about 64 SMs; when the next GEMM
// wants more than the SMs it leaves free (84 of a B200's 148), its last CTAs start late and their decode lands on the critical path.  Then the
// rows are packed into fewer CTAs (measured: 54.6 -> 50.5 us per BERT-large layer at 256 tokens; at 512 tokens
// packing loses 1-3 us, at BERT-base sizes it changes nothing).  Otherwise one row per CTA.
int ln_ctas_hint(int tuned, int T, int next_gemm_ctas, int sm_count) {
  if (tuned >= 0) return tuned;
  if (T > 256 || next_gemm_ctas <= sm_count - 64) return 0;      // at 512 tokens the packed LayerNorm itself costs more than it frees
  return std::max(32, sm_count - next_gemm_ctas);
}

// The seven kernels of one layer on the compute stream.
// `x_ready_bf16`: the bf16 copy of x already sits in p->x_bf16 (written by the previous layer's LayerNorm);
// `want_next_bf16`: this layer's last kernel also writes y as bf16 into p->x_bf16 for the next layer.
sti_status enqueue_layer(sti_plan* p, int li, const void* x, void* y, int batch, int seq, const int32_t* lens,
                         bool x_ready_bf16, bool want_next_bf16, int next_layer = -1) {
  sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  Layer& L = p->layers[li];
  const int T = batch * seq;
  const float* dense = c->dense + static_cast<size_t>(li) * c->dense_stride;
  const bool bf16_act = d.act_dtype == STI_BF16;
  const int nh = static_cast<int>(L.kept_heads.size()), ns = static_cast<int>(L.kept_slices.size());
  const int f = d.ffn / d.n_ffn_slices;
  sti_status st;
  const bool kprof = p->profiling >= 2;
  auto mark = [&](int i) -> cudaError_t { return kprof ? cudaEventRecord(L.ev_k[i], c->compute) : cudaSuccess; };
  for (bool& r : L.k_ran) r = false;
  auto stamp = [&](int kernel) -> unsigned long long* {
    return p->stamping ? p->stamps + (static_cast<size_t>(li) * kStampKernels + kernel) * kStampRecord : nullptr;
  };
  CUDA_TRY(mark(0));
  if (nh > 0) {
    const void* xq = x;
    if (!bf16_act) {
      // the GEMMs take bf16 operands: fp32 activations are rounded once (round-to-nearest-even)
      if (!x_ready_bf16) {
        CUDA_TRY(launch_cast_bf16(static_cast<const float*>(x), p->x_bf16, static_cast<size_t>(T) * d.hidden,
                                  c->compute, c->pdl, stamp(0)));
        c->launches++;
      }
      xq = p->x_bf16;
    }
    st = run_gemm(p, GEMM_BF16_TO_BF16, L.qkv, xq, d.hidden, T, p->qkv, 64, dense + c->off_bq, next_layer, -1, stamp(1));
    if (st != STI_OK) return st;
    CUDA_TRY(mark(1));
    if (p->tune.attn_tc_min_items > 0 && seq >= 256 && batch * nh >= p->tune.attn_tc_min_items && !c->simt_debug) {
      // many (sequence, head) pairs: one CTA each on the tensor cores, K and V of the sequence resident in shared memory
      CUtensorMap qmap;
      if (!make_xmap(&qmap, p->qkv, 64, 3 * nh * T)) return STI_ERR_CUDA;
      CUDA_TRY(launch_attention_tc(qmap, p->attn_out, nh, batch, seq, lens, c->err_dev, c->compute, c->pdl, stamp(2)));
    } else {
      CUDA_TRY(launch_attention(p->qkv, p->attn_out, nh, batch, seq, lens, c->sm_count, c->compute, c->pdl, stamp(2)));
    }
    c->launches++;
    CUDA_TRY(mark(2));
    st = run_gemm(p, GEMM_BF16_TO_F32, L.o, p->attn_out, nh * 64, T, p->partial, d.hidden, nullptr, -1, -1, stamp(3));
    if (st != STI_OK) return st;
    L.k_ran[0] = L.k_ran[1] = L.k_ran[2] = true;
  } else {
    CUDA_TRY(mark(1));
    CUDA_TRY(mark(2));
  }
  CUDA_TRY(mark(3));
  {
    LnLaunch ln{};
    ln.partial = p->partial; ln.n_partial = nh > 0 ? L.o.n_split : 0;
    ln.bias = dense + c->off_bo; ln.resid = x; ln.resid_bf16 = bf16_act ? 1 : 0;
    ln.gamma = dense + c->off_ln1g; ln.beta = dense + c->off_ln1b; ln.eps = d.ln_eps; ln.T = T; ln.d = d.hidden;
    // With bf16 activations every activation that crosses a kernel boundary is bf16 (the layer's input and output are):
    // the second LayerNorm then takes its residual from the bf16 copy the FFN reads, and no fp32 copy is written.
    ln.out_f32 = bf16_act ? nullptr : p->h1_f32; ln.out_bf16 = p->h1_bf16;
    ln.ctas_hint = ln_ctas_hint(p->tune.ln1_ctas, T, ns > 0 ? L.f1.n_jobs * m_ctas_for(L.f1.n_jobs, T, p->tune.cta_budget) : 0, c->sm_count);
    ln.stamps = stamp(4);
    CUDA_TRY(launch_layernorm(ln, c->compute, c->pdl));
    c->launches++;
    L.k_ran[3] = true;
  }
  CUDA_TRY(mark(4));
  bool f2_kacc = false;
  if (ns > 0) {
    st = run_gemm(p, GEMM_BF16_TO_BF16_GELU, L.f1, p->h1_bf16, d.hidden, T, p->u, ns * f, dense + c->off_b1, -1, -1, stamp(5));
    if (st != STI_OK) return st;
    CUDA_TRY(mark(5));
    f2_kacc = L.f2k.n_jobs > 0 && T >= p->tune.f2_kacc_min_tokens && !c->simt_debug;
    if (f2_kacc)
      st = run_gemm_kacc(p, L.f2k, p->u, ns * f, T, p->partial, d.hidden, stamp(6));
    else
      st = run_gemm(p, GEMM_BF16_TO_F32, L.f2, p->u, ns * f, T, p->partial, d.hidden, nullptr, -1, -1, stamp(6));
    if (st != STI_OK) return st;
    L.k_ran[4] = L.k_ran[5] = true;
  } else {
    CUDA_TRY(mark(5));
  }
  CUDA_TRY(mark(6));
  LnLaunch l2{};
  l2.partial = p->partial; l2.n_partial = ns > 0 ? (f2_kacc ? 1 : L.f2.n_split) : 0;
  l2.bias = dense + c->off_b2;
  l2.resid = bf16_act ? static_cast<const void*>(p->h1_bf16) : static_cast<const void*>(p->h1_f32);
  l2.resid_bf16 = bf16_act ? 1 : 0;
  l2.gamma = dense + c->off_ln2g; l2.beta = dense + c->off_ln2b; l2.eps = d.ln_eps; l2.T = T; l2.d = d.hidden;
  l2.out_f32 = bf16_act ? nullptr : static_cast<float*>(y);
  l2.out_bf16 = bf16_act ? static_cast<uint16_t*>(y) : (want_next_bf16 ? p->x_bf16 : nullptr);
  {
    int next_ctas = 0;
    if (next_layer >= 0 && next_layer < static_cast<int>(p->layers.size())) {
      const GemmTable& q = p->layers[next_layer].qkv;
      next_ctas = q.n_jobs * m_ctas_for(q.n_jobs, T, p->tune.cta_budget);
    }
    l2.ctas_hint = ln_ctas_hint(p->tune.ln2_ctas, T, next_ctas, c->sm_count);
    l2.stamps = stamp(7);
  }
  CUDA_TRY(launch_layernorm(l2, c->compute, c->pdl));
  c->launches++;
  L.k_ran[6] = true;
  CUDA_TRY(mark(7));
  return STI_OK;
}

sti_status check_forward_args(sti_plan* p, const void* x, void* y, int batch, int seq, bool device_buffers = true) {
  if (!p || !x || !y) return STI_ERR_ARG;
  // device activations are read through TMA descriptors and vector loads: 16-byte alignment
  if (device_buffers && ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15)) return STI_ERR_ARG;
  const sti_model_desc& d = p->ctx->desc;
  if (batch < 1 || seq < 1 || seq > d.max_seq) return STI_ERR_SHAPE;
  if (static_cast<long long>(batch) * seq > static_cast<long long>(d.max_batch) * d.max_seq) return STI_ERR_SHAPE;
  return STI_OK;
}

// Copy of layer li's streamed part into its ring slot, on stream `s`.
sti_status enqueue_layer_copy(sti_plan* p, int li, cudaStream_t s) {
  Layer& L = p->layers[li];
  if (L.str_bytes == 0) return STI_OK;
  if (li == p->slow_copy_layer && p->slow_copy_us)      // injected slow IO: the job reaches the copy engine late
    std::this_thread::sleep_for(std::chrono::microseconds(p->slow_copy_us));
  CUDA_TRY(cudaMemcpyAsync(p->ring + static_cast<size_t>(L.slot) * p->slot_bytes, L.str_host, L.str_bytes,
                           cudaMemcpyHostToDevice, s));
  return STI_OK;
}

// Enqueues one whole forward: per layer the shard copy on the copy stream and the seven kernels on the
// compute stream, ordered by events.  With `capturing` the same calls are recorded into a CUDA graph:
// the copy stream is forked from and joined back into the compute stream, and a ring slot's "free" event
// is only waited for when it was recorded inside this forward (stream order covers earlier forwards).
sti_status enqueue_forward(sti_plan* p, const void* x, void* y, int batch, int seq, const int32_t* lens,
                           bool capturing) {
  sti_ctx* c = p->ctx;
  const int n = static_cast<int>(p->layers.size());
  const bool prof = p->profiling && !capturing;
  bool any_streamed = false;
  for (auto& L : p->layers) any_streamed |= L.str_bytes > 0;
  std::vector<char> slot_used(p->ring_slots, 0);
  if (prof) CUDA_TRY(cudaEventRecord(p->ev_begin, c->compute));
  if (capturing && any_streamed) {
    CUDA_TRY(cudaEventRecord(p->ev_fork, c->compute));
    CUDA_TRY(cudaStreamWaitEvent(c->copy, p->ev_fork, 0));
  }
  if (!p->overlap && any_streamed) {
    // load-then-execute: every IO job first (each layer has its own slot), compute waits for the last one
    cudaEvent_t last = nullptr;
    for (int li = 0; li < n; ++li) {
      Layer& L = p->layers[li];
      if (L.str_bytes == 0) continue;
      if (!capturing) CUDA_TRY(cudaStreamWaitEvent(c->copy, p->slot_free[L.slot], 0));
      if (prof) CUDA_TRY(cudaEventRecord(L.ev_copy_start, c->copy));
      sti_status st = enqueue_layer_copy(p, li, c->copy);
      if (st != STI_OK) return st;
      last = capturing ? L.g_ev_loaded : L.ev_loaded;
      CUDA_TRY(cudaEventRecord(last, c->copy));
    }
    CUDA_TRY(cudaStreamWaitEvent(c->compute, last, 0));
  }
  const void* cur = x;
  for (int li = 0; li < n; ++li) {
    Layer& L = p->layers[li];
    if (L.str_bytes > 0 && p->overlap) {
      // one IO job per layer (Section 3.1); the slot is reused only after its previous layer finished
      if (!capturing) CUDA_TRY(cudaStreamWaitEvent(c->copy, p->slot_free[L.slot], 0));
      else if (slot_used[L.slot]) CUDA_TRY(cudaStreamWaitEvent(c->copy, p->g_slot_free[L.slot], 0));
      if (prof) CUDA_TRY(cudaEventRecord(L.ev_copy_start, c->copy));
      sti_status st = enqueue_layer_copy(p, li, c->copy);
      if (st != STI_OK) return st;
      cudaEvent_t loaded = capturing ? L.g_ev_loaded : L.ev_loaded;
      CUDA_TRY(cudaEventRecord(loaded, c->copy));
      // a layer starts only when its own shards (and, by stream order, all earlier ones) are loaded
      CUDA_TRY(cudaStreamWaitEvent(c->compute, loaded, 0));
    }
    if (prof) CUDA_TRY(cudaEventRecord(L.ev_comp_start, c->compute));
    void* nxt = (li == n - 1) ? y : p->buf[li & 1];
    // the layer's first GEMM also pulls the next layer's packed shards into L2 (if they are on the device yet)
    sti_status st = enqueue_layer(p, li, cur, nxt, batch, seq, lens, li > 0, li + 1 < n, li + 1 < n ? li + 1 : -1);
    if (st != STI_OK) return st;
    if (p->retain_pending && !capturing && L.str_bytes > 0) {
      // keep what this run loaded (Section 3.2): the marked units leave their ring slot for the retained arena
      // before the slot is handed back to the copy stream
      const uint8_t* slot = p->ring + static_cast<size_t>(L.slot) * p->slot_bytes;
      auto keep_unit = [&](Unit& u) -> cudaError_t {
        if (!u.retain || u.retained_done || u.cfg.resident) return cudaSuccess;
        u.retained_done = true;
        return cudaMemcpyAsync(u.retained, slot + u.off_codes, u.bytes, cudaMemcpyDeviceToDevice, c->compute);
      };
      for (auto& u : L.attn) CUDA_TRY(keep_unit(u));
      for (auto& u : L.ffn) CUDA_TRY(keep_unit(u));
    }
    if (prof) CUDA_TRY(cudaEventRecord(L.ev_done, c->compute));
    if (L.str_bytes > 0) {
      CUDA_TRY(cudaEventRecord(capturing ? p->g_slot_free[L.slot] : p->slot_free[L.slot], c->compute));
      slot_used[L.slot] = 1;
    }
    cur = nxt;
  }
  if (!capturing) {
    CUDA_TRY(cudaEventRecord(p->ev_copy_tail, c->copy));
    p->copy_tail_valid = true;
  } else if (any_streamed) {
    CUDA_TRY(cudaEventRecord(p->g_ev_join, c->copy));
    CUDA_TRY(cudaStreamWaitEvent(c->compute, p->g_ev_join, 0));   // join the copy stream back
  }
  if (prof) {
    CUDA_TRY(cudaEventRecord(p->ev_end, c->compute));
    p->stats_valid = true;
  }
  return STI_OK;
}

// Body of a forward with optional host staging of x and y (all on the compute stream around the layers).
sti_status enqueue_forward_io(sti_plan* p, const ForwardKey& k, bool capturing) {
  sti_ctx* c = p->ctx;
  const size_t bytes = static_cast<size_t>(k.batch) * k.seq * c->desc.hidden * act_size(c);
  const void* x = k.x;
  void* y = k.y;
  if (k.x_host) {
    CUDA_TRY(cudaMemcpyAsync(p->x_in, k.x_host, bytes, cudaMemcpyHostToDevice, c->compute));
    x = p->x_in;
    y = p->y_out;
  }
  p->stamping = k.stamps;
  if (k.stamps)
    CUDA_TRY(cudaMemsetAsync(p->stamps, 0xff, p->layers.size() * kStampKernels * kStampRecord * sizeof(unsigned long long), c->compute));
  sti_status st;
  if (k.layer >= 0) {
    // a single layer: its IO job (if it has streamed units) runs on the compute stream, not overlapped
    Layer& L = p->layers[k.layer];
    if (L.str_bytes > 0) {
      if (!capturing && p->copy_tail_valid) CUDA_TRY(cudaStreamWaitEvent(c->compute, p->ev_copy_tail, 0));
      if ((st = enqueue_layer_copy(p, k.layer, c->compute)) != STI_OK) return st;
    }
    st = enqueue_layer(p, k.layer, x, y, k.batch, k.seq, k.lens, false, false);
    if (st == STI_OK && L.str_bytes > 0 && !capturing) CUDA_TRY(cudaEventRecord(p->slot_free[L.slot], c->compute));
  } else {
    st = enqueue_forward(p, x, y, k.batch, k.seq, k.lens, capturing);
  }
  if (st != STI_OK) return st;
  if (k.y_host) CUDA_TRY(cudaMemcpyAsync(k.y_host, p->y_out, bytes, cudaMemcpyDeviceToHost, c->compute));
  return STI_OK;
}

// A forward with the same buffers and shape as the previous one replays its CUDA graph (one launch instead of
// ~7 per layer, no per-kernel host work); anything else is captured anew.  Profiling runs ungraphed.
sti_status model_forward_impl(sti_plan* p, const ForwardKey& k) {
  sti_ctx* c = p->ctx;
  if ((p->profiling && p->profiling < 3) || p->graph_off) return enqueue_forward_io(p, k, false);
  if (p->retain_pending && k.layer < 0) {
    // one forward launched kernel by kernel: it also moves the shards to keep out of the ring slots
    const sti_status st = enqueue_forward_io(p, k, false);
    if (st == STI_OK) p->retain_pending = false;
    return st;
  }
  sti_plan::CachedGraph* hit = nullptr;
  for (auto& g : p->graphs) if (g.exec && g.key == k) hit = &g;
  if (!hit) {
    const uint64_t launches_before = c->launches;
    cudaGraph_t graph = nullptr;
    if (cudaStreamBeginCapture(c->compute, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
      (void)cudaGetLastError();
      p->graph_off = true;
      return enqueue_forward_io(p, k, false);
    }
    const sti_status st = enqueue_forward_io(p, k, true);
    const cudaError_t ce = cudaStreamEndCapture(c->compute, &graph);
    const uint64_t n_launches = c->launches - launches_before;
    c->launches = launches_before;
    if (st != STI_OK || ce != cudaSuccess || !graph) {
      (void)cudaGetLastError();
      if (graph) cudaGraphDestroy(graph);
      // an argument or shape error of this call says nothing about later, valid calls: only a failure of the
      // capture itself switches the plan to plain stream launches
      if (st == STI_ERR_ARG || st == STI_ERR_SHAPE || st == STI_ERR_STATE) return st;
      p->graph_off = true;
      return st != STI_OK ? st : enqueue_forward_io(p, k, false);
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess || !exec) {
      (void)cudaGetLastError();
      p->graph_off = true;
      return enqueue_forward_io(p, k, false);
    }
    constexpr size_t kMaxGraphs = 8;
    if (p->graphs.size() < kMaxGraphs) {
      p->graphs.emplace_back();
      hit = &p->graphs.back();
    } else {                          // replace the least recently used one
      hit = &p->graphs[0];
      for (auto& g : p->graphs) if (g.last_use < hit->last_use) hit = &g;
      (void)cudaStreamSynchronize(c->compute);      // it may still be running
      cudaGraphExecDestroy(hit->exec);
    }
    hit->key = k; hit->exec = exec; hit->launches = n_launches;
  }
  hit->last_use = ++p->graph_clock;
  CUDA_TRY(cudaGraphLaunch(hit->exec, c->compute));
  // later ungraphed work (profiled forwards, single layers) must not reuse a ring slot before this graph is done
  for (auto e : p->slot_free) CUDA_TRY(cudaEventRecord(e, c->compute));
  c->launches += hit->launches;
  p->copy_tail_valid = false;
  return STI_OK;
}

void free_plan_device(sti_plan* p) {
  if (!p) return;
  cudaFree(p->preload_alloc); cudaFree(p->ring_alloc); cudaFree(p->tables); cudaFree(p->retain_arena);
  if (p->pinned) cudaFreeHost(p->pinned);
  cudaFree(p->qkv); cudaFree(p->attn_out); cudaFree(p->partial); cudaFree(p->h1_f32); cudaFree(p->h1_bf16);
  cudaFree(p->u); cudaFree(p->x_bf16); cudaFree(p->buf[0]); cudaFree(p->buf[1]); cudaFree(p->x_in); cudaFree(p->y_out);
  cudaFree(p->lens_dev);
  cudaFree(p->stamps);
  cudaFree(p->zero_bias);
  cudaFree(p->rate_tables);
  for (auto& L : p->layers) {
    if (L.ev_loaded) cudaEventDestroy(L.ev_loaded);
    if (L.g_ev_loaded) cudaEventDestroy(L.g_ev_loaded);
    if (L.ev_done) cudaEventDestroy(L.ev_done);
    if (L.ev_copy_start) cudaEventDestroy(L.ev_copy_start);
    if (L.ev_comp_start) cudaEventDestroy(L.ev_comp_start);
    for (auto e : L.ev_k) if (e) cudaEventDestroy(e);
  }
  for (auto e : p->slot_free) cudaEventDestroy(e);
  for (auto e : p->g_slot_free) cudaEventDestroy(e);
  if (p->g_ev_join) cudaEventDestroy(p->g_ev_join);
  if (p->ev_copy_tail) cudaEventDestroy(p->ev_copy_tail);
  if (p->ev_fork) cudaEventDestroy(p->ev_fork);
  for (auto& g : p->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
  if (p->ev_begin) cudaEventDestroy(p->ev_begin);
  if (p->ev_end) cudaEventDestroy(p->ev_end);
}

}  // namespace

extern "C" {

const char* sti_strerror(sti_status s) {
  switch (s) {
    case STI_OK: return "ok";
    case STI_ERR_ARG: return "invalid argument";
    case STI_ERR_BITS: return "unsupported or mismatched bitwidth";
    case STI_ERR_SHAPE: return "unsupported shape";
    case STI_ERR_SIZE: return "blob size does not match the unit";
    case STI_ERR_STATE: return "call not allowed in this state";
    case STI_ERR_SHARD_MISSING: return "a kept shard unit was never uploaded";
    case STI_ERR_OOM: return "out of memory";
    case STI_ERR_CUDA: return "CUDA runtime error";
    case STI_ERR_TIMEOUT: return "a bounded device-side wait ran out";
  }
  return "unknown status";
}

sti_status sti_ctx_create(const sti_model_desc* desc, int device, void* compute_stream, sti_ctx** out) {
  if (!desc || !out) return STI_ERR_ARG;
  const sti_model_desc& d = *desc;
  if (d.n_layers < 1 || d.n_layers > kMaxLayersStats || d.n_heads < 1 || d.n_ffn_slices < 1 || d.max_batch < 1 ||
      d.max_seq < 1)
    return STI_ERR_SHAPE;
  if (d.head_dim != 64 || d.hidden < 128 || d.hidden % 128 != 0 || d.hidden > 2048 || d.ffn % d.n_ffn_slices != 0 ||
      (d.ffn / d.n_ffn_slices) % 128 != 0 || d.max_seq > 512 || d.n_heads * 64 > 16 * 128)
    return STI_ERR_SHAPE;
  if (d.act_dtype != STI_F32 && d.act_dtype != STI_BF16) return STI_ERR_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) {
    (void)cudaGetLastError();
    return STI_ERR_CUDA;      // no usable CUDA device: there is no other execution path
  }
  CUDA_TRY(cudaSetDevice(device));
  sti_ctx* c = new (std::nothrow) sti_ctx();
  if (!c) return STI_ERR_OOM;
  c->desc = d;
  c->device = device;
  const uint32_t dd = d.hidden, f = d.ffn / d.n_ffn_slices;
  c->attn_m[0] = {64, dd, 0};
  c->attn_m[1] = {64, dd, 64 * dd};
  c->attn_m[2] = {64, dd, 2 * 64 * dd};
  c->attn_m[3] = {dd, 64, 3 * 64 * dd};
  c->attn_weights = 4 * 64 * dd;
  c->ffn_m[0] = {f, dd, 0};
  c->ffn_m[1] = {dd, f, f * dd};
  c->ffn_weights = 2 * f * dd;
  const size_t hq = static_cast<size_t>(d.n_heads) * 64;
  size_t o = 0;
  c->off_bq = o; o += hq;
  c->off_bk = o; o += hq;
  c->off_bv = o; o += hq;
  c->off_bo = o; o += dd;
  c->off_b1 = o; o += d.ffn;
  c->off_b2 = o; o += dd;
  c->off_ln1g = o; o += dd;
  c->off_ln1b = o; o += dd;
  c->off_ln2g = o; o += dd;
  c->off_ln2b = o; o += dd;
  c->dense_stride = (o + 63) / 64 * 64;
  auto fail = [&](sti_status s) { sti_ctx_destroy(c); return s; };
  if (compute_stream) {
    c->compute = static_cast<cudaStream_t>(compute_stream);
  } else {
    if (cudaStreamCreateWithFlags(&c->compute, cudaStreamNonBlocking) != cudaSuccess) return fail(STI_ERR_CUDA);
    c->own_compute = true;
  }
  if (cudaStreamCreateWithFlags(&c->copy, cudaStreamNonBlocking) != cudaSuccess) return fail(STI_ERR_CUDA);
  if (cudaMalloc(&c->dense, c->dense_stride * d.n_layers * sizeof(float)) != cudaSuccess) return fail(STI_ERR_OOM);
  if (cudaMemset(c->dense, 0, c->dense_stride * d.n_layers * sizeof(float)) != cudaSuccess) return fail(STI_ERR_CUDA);
  if (cudaMalloc(&c->err_dev, sizeof(int)) != cudaSuccess) return fail(STI_ERR_OOM);
  if (cudaMemset(c->err_dev, 0, sizeof(int)) != cudaSuccess) return fail(STI_ERR_CUDA);
  if (gemm_configure() != cudaSuccess || gemm_kacc_configure() != cudaSuccess || attention_configure() != cudaSuccess ||
      attention_tc_configure() != cudaSuccess)
    return fail(STI_ERR_CUDA);
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || c->sm_count < 1)
    return fail(STI_ERR_CUDA);
  const char* dbg = getenv("STI_DEBUG_SIMT");
  c->simt_debug = dbg && dbg[0] == '1';
  const char* nopdl = getenv("STI_NO_PDL");
  c->pdl = !(nopdl && nopdl[0] == '1');
  *out = c;
  return STI_OK;
}

void sti_ctx_destroy(sti_ctx* c) {
  if (!c) return;
  cudaSetDevice(c->device);
  if (c->compute) cudaStreamSynchronize(c->compute);
  if (c->copy) cudaStreamSynchronize(c->copy);
  cudaFree(c->dense);
  cudaFree(c->err_dev);
  if (c->own_compute && c->compute) cudaStreamDestroy(c->compute);
  if (c->copy) cudaStreamDestroy(c->copy);
  delete c;
}

sti_status sti_ctx_set_layer_params(sti_ctx* c, int layer, const float* bq, const float* bk, const float* bv,
                                    const float* bo, const float* b1, const float* b2, const float* ln1_g,
                                    const float* ln1_b, const float* ln2_g, const float* ln2_b) {
  if (!c || !bq || !bk || !bv || !bo || !b1 || !b2 || !ln1_g || !ln1_b || !ln2_g || !ln2_b) return STI_ERR_ARG;
  if (layer < 0 || layer >= c->desc.n_layers) return STI_ERR_ARG;
  CUDA_TRY(cudaSetDevice(c->device));
  std::vector<float> h(c->dense_stride, 0.f);
  const size_t hq = static_cast<size_t>(c->desc.n_heads) * 64, d = c->desc.hidden;
  memcpy(&h[c->off_bq], bq, hq * 4); memcpy(&h[c->off_bk], bk, hq * 4); memcpy(&h[c->off_bv], bv, hq * 4);
  memcpy(&h[c->off_bo], bo, d * 4); memcpy(&h[c->off_b1], b1, static_cast<size_t>(c->desc.ffn) * 4);
  memcpy(&h[c->off_b2], b2, d * 4);
  memcpy(&h[c->off_ln1g], ln1_g, d * 4); memcpy(&h[c->off_ln1b], ln1_b, d * 4);
  memcpy(&h[c->off_ln2g], ln2_g, d * 4); memcpy(&h[c->off_ln2b], ln2_b, d * 4);
  CUDA_TRY(cudaStreamSynchronize(c->compute));
  CUDA_TRY(cudaMemcpy(c->dense + static_cast<size_t>(layer) * c->dense_stride, h.data(), h.size() * 4,
                      cudaMemcpyHostToDevice));
  return STI_OK;
}

sti_status sti_plan_create(sti_ctx* c, const sti_shard_cfg* attn, const sti_shard_cfg* ffn, int ring_slots,
                           sti_plan** out) {
  if (!c || !attn || !ffn || !out) return STI_ERR_ARG;
  if (ring_slots < 2 || ring_slots > 64) return STI_ERR_ARG;
  const sti_model_desc& d = c->desc;
  auto ok_bits = [](int b) { return (b >= 2 && b <= 6) || b == 32; };
  for (int i = 0; i < d.n_layers * d.n_heads; ++i)
    if (attn[i].keep && !ok_bits(attn[i].bits)) return STI_ERR_BITS;
  for (int i = 0; i < d.n_layers * d.n_ffn_slices; ++i)
    if (ffn[i].keep && !ok_bits(ffn[i].bits)) return STI_ERR_BITS;
  sti_plan* p = new (std::nothrow) sti_plan();
  if (!p) return STI_ERR_OOM;
  p->ctx = c;
  p->ring_slots = ring_slots;
  p->layers.resize(d.n_layers);
  for (int l = 0; l < d.n_layers; ++l) {
    Layer& L = p->layers[l];
    L.attn.resize(d.n_heads);
    L.ffn.resize(d.n_ffn_slices);
    for (int h = 0; h < d.n_heads; ++h) {
      L.attn[h].cfg = attn[l * d.n_heads + h];
      if (L.attn[h].cfg.keep) L.kept_heads.push_back(h);
    }
    for (int s = 0; s < d.n_ffn_slices; ++s) {
      L.ffn[s].cfg = ffn[l * d.n_ffn_slices + s];
      if (L.ffn[s].cfg.keep) L.kept_slices.push_back(s);
    }
  }
  parse_tuning(&p->tune, d.max_batch * d.max_seq, d, c->sm_count);
  *out = p;
  return STI_OK;
}

void sti_plan_destroy(sti_plan* p) {
  if (!p) return;
  cudaSetDevice(p->ctx->device);
  cudaStreamSynchronize(p->ctx->compute);
  cudaStreamSynchronize(p->ctx->copy);
  free_plan_device(p);
  delete p;
}

sti_status sti_shard_upload(sti_plan* p, int layer, sti_kind kind, int index, const sti_shard_blob* blob) {
  if (!p || !blob || (kind != STI_ATTN && kind != STI_FFN)) return STI_ERR_ARG;
  if (p->finalized) return STI_ERR_STATE;
  Unit* u = find_unit(p, layer, kind, index);
  if (!u) return STI_ERR_ARG;
  if (!u->cfg.keep) return STI_ERR_STATE;
  if (blob->bits != u->cfg.bits) return STI_ERR_BITS;
  if (!blob->codes) return STI_ERR_ARG;
  const sti_ctx* c = p->ctx;
  int nm;
  const MatrixInfo* mi = unit_matrices(c, kind, &nm);
  const uint32_t n_weights = kind == STI_ATTN ? c->attn_weights : c->ffn_weights;
  const int bits = blob->bits;
  if (blob->n_code_words != static_cast<size_t>(n_weights) * bits / 32) return STI_ERR_SIZE;
  if (bits != 32 && !blob->centroids) return STI_ERR_ARG;
  if (blob->n_outliers && (!blob->outlier_off || !blob->outlier_val)) return STI_ERR_ARG;
  if (bits == 32 && blob->n_outliers) return STI_ERR_ARG;
  for (size_t i = 0; i < blob->n_outliers; ++i) {
    if (blob->outlier_off[i] >= n_weights) return STI_ERR_SIZE;
    if (i && blob->outlier_off[i] <= blob->outlier_off[i - 1]) return STI_ERR_ARG;
  }
  u->adopt_src = nullptr;
  u->codes_bytes = blob->n_code_words * 4;
  u->codes.assign(blob->n_code_words * 4, 0);
  const uint8_t* src = reinterpret_cast<const uint8_t*>(blob->codes);
  if (bits == 32) {
    memcpy(u->codes.data(), src, u->codes.size());
  } else {
    size_t off = 0;
    for (int m = 0; m < nm; ++m) {
      retile_matrix(src + off, u->codes.data() + off, mi[m].rows, mi[m].kc, bits);
      off += matrix_code_bytes(mi[m], bits);
    }
  }
  u->table.clear();
  if (bits != 32) u->table.assign(blob->centroids, blob->centroids + (1u << bits));
  u->out_off.assign(blob->outlier_off, blob->outlier_off + blob->n_outliers);
  u->out_val.assign(blob->outlier_val, blob->outlier_val + blob->n_outliers);
  u->uploaded = true;
  return STI_OK;
}

sti_status sti_plan_finalize(sti_plan* p) {
  if (!p) return STI_ERR_ARG;
  if (p->finalized) return STI_OK;
  if (p->attempted) return STI_ERR_STATE;    // an earlier attempt failed half-way; the plan is unusable
  sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  CUDA_TRY(cudaSetDevice(c->device));
  // 1. every kept unit must have its blob; lay units out inside their layer's resident / streamed part
  size_t preload_total = 0, pinned_total = 0, slot_bytes = 0;
  int n_streamed = 0, max_heads = 0, max_slices = 0;
  for (auto& L : p->layers) {
    L.res_bytes = L.str_bytes = 0;
    auto place = [&](Unit& u) -> bool {
      if (!u.cfg.keep) return true;
      if (!u.uploaded) return false;
      size_t& cursor = u.cfg.resident ? L.res_bytes : L.str_bytes;
      const size_t start = cursor;
      u.off_codes = cursor; cursor += align16(u.codes_bytes);
      u.off_table = cursor; cursor += align16(u.table.size() * 4);
      u.off_ooff = cursor; cursor += align16(u.out_off.size() * 4);
      u.off_oval = cursor; cursor += align16(u.out_val.size() * 4);
      u.bytes = cursor - start;
      return true;
    };
    for (auto& u : L.attn) if (!place(u)) return STI_ERR_SHARD_MISSING;
    for (auto& u : L.ffn) if (!place(u)) return STI_ERR_SHARD_MISSING;
    preload_total += align256(L.res_bytes);
    pinned_total += align256(L.str_bytes);
    if (L.str_bytes) slot_bytes = std::max(slot_bytes, align256(L.str_bytes) + kGuardBytes);
    if (L.str_bytes) L.slot = (n_streamed++) % p->ring_slots;
    p->n_streamed_layers = n_streamed;
    max_heads = std::max<int>(max_heads, L.kept_heads.size());
    max_slices = std::max<int>(max_slices, L.kept_slices.size());
  }
  p->attempted = true;
  p->preload_bytes = preload_total; p->pinned_bytes = pinned_total; p->slot_bytes = slot_bytes;
  if (preload_total) {
    CUDA_TRY(cudaMalloc(&p->preload_alloc, preload_total + 2 * kGuardBytes));
    CUDA_TRY(cudaMemset(p->preload_alloc, kGuardPattern, preload_total + 2 * kGuardBytes));
    p->preload = p->preload_alloc + kGuardBytes;
  }
  if (pinned_total) {
    if (p->fail_pinned_alloc) return STI_ERR_OOM;          // injected allocation failure
    CUDA_TRY(cudaMallocHost(&p->pinned, pinned_total));
  }
  if (slot_bytes) {
    CUDA_TRY(cudaMalloc(&p->ring_alloc, kGuardBytes + slot_bytes * p->ring_slots));
    CUDA_TRY(cudaMemset(p->ring_alloc, kGuardPattern, kGuardBytes + slot_bytes * p->ring_slots));
    p->ring = p->ring_alloc + kGuardBytes;
  }
  // 2. fill the preload buffer (device) and the pinned arena (host), one contiguous blob per layer
  size_t pre_cur = 0, pin_cur = 0;
  std::vector<uint8_t> staging;
  for (auto& L : p->layers) {
    L.res_dev = p->preload ? p->preload + pre_cur : nullptr;
    L.str_host = p->pinned ? p->pinned + pin_cur : nullptr;
    pre_cur += align256(L.res_bytes);
    pin_cur += align256(L.str_bytes);
    if (L.str_bytes) memset(L.str_host, 0, L.str_bytes);
    cudaError_t unit_err = cudaSuccess;
    auto emit = [&](Unit& u) {
      if (!u.cfg.keep || unit_err != cudaSuccess) return;
      if (u.adopt_src) {
        // already in device memory (another plan's preload buffer or retained shards): no host traffic
        u.dev = L.res_dev;
        unit_err = cudaMemcpyAsync(L.res_dev + u.off_codes, u.adopt_src, u.bytes, cudaMemcpyDeviceToDevice, c->compute);
        p->finalize_d2d_bytes += u.bytes;
        return;
      }
      // resident units go up one by one (nothing is uploaded for the units adopted above)
      staging.assign(u.cfg.resident ? u.bytes : 0, 0);
      // a resident unit's region is built in `staging` (its first byte = off_codes), a streamed one in the pinned blob
      auto at = [&](size_t off) { return u.cfg.resident ? staging.data() + (off - u.off_codes) : L.str_host + off; };
      memcpy(at(u.off_codes), u.codes.data(), u.codes.size());
      if (!u.table.empty()) memcpy(at(u.off_table), u.table.data(), u.table.size() * 4);
      if (!u.out_off.empty()) {
        memcpy(at(u.off_ooff), u.out_off.data(), u.out_off.size() * 4);
        memcpy(at(u.off_oval), u.out_val.data(), u.out_val.size() * 4);
      }
      u.dev = u.cfg.resident ? L.res_dev : p->ring + static_cast<size_t>(L.slot) * p->slot_bytes;
      if (u.cfg.resident) {
        unit_err = cudaMemcpy(L.res_dev + u.off_codes, staging.data(), u.bytes, cudaMemcpyHostToDevice);
        p->finalize_h2d_bytes += u.bytes;
      }
      std::vector<uint8_t>().swap(u.codes);     // the arenas now hold the only copy
    };
    for (auto& u : L.attn) emit(u);
    for (auto& u : L.ffn) emit(u);
    CUDA_TRY(unit_err);
  }
  CUDA_TRY(cudaStreamSynchronize(c->compute));   // adopted units are in place before their source plan may go away
  // 3. tile-job tables
  std::vector<uint8_t> host_tables;
  struct Fix { GemmTable* t; size_t jobs_off, segs_off; };
  std::vector<Fix> fixes;
  p->max_partial = 1;
  for (auto& L : p->layers) {
    TableBuilder tb[5];
    L.tables_off = align16(host_tables.size());
    build_layer_tables(p, L, tb);
    GemmTable* gt[5] = {&L.qkv, &L.o, &L.f1, &L.f2, &L.f2k};
    for (int i = 0; i < 5; ++i) {
      tb[i].finish();
      gt[i]->seg_stride = tb[i].seg_stride;
      gt[i]->n_jobs = static_cast<int>(tb[i].jobs.size());
      gt[i]->w_bytes = tb[i].w_bytes;
      gt[i]->n_stages = 2; gt[i]->bps = 1;
      gt[i]->hdr_bytes = gemm_header_bytes();
      gt[i]->pair_ok = !tb[i].jobs.empty() && tb[i].jobs.size() % 2 == 0;
      for (size_t j = 0; gt[i]->pair_ok && j < tb[i].jobs.size(); j += 2) {
        const Job &a = tb[i].jobs[j], &b = tb[i].jobs[j + 1];
        gt[i]->pair_ok = a.n_rows == 64 && b.n_rows == 64 && a.k_total == b.k_total && a.x_koff == b.x_koff;
      }
      if (i == 4) {                 // two weight buffers, the rest of the shared memory is the ring of single boxes
        gt[i]->k_max = tb[i].k_max;
        gt[i]->bps = p->tune.f2_kacc_bps;
        for (const Job& j : tb[i].jobs)
          if (j.k_total % (128 * gt[i]->bps / 2) != 0) gt[i]->bps = 1;      // an odd number of boxes somewhere
        gt[i]->n_stages = gemm_kacc_stages(gt[i]->hdr_bytes, tb[i].k_max, gt[i]->bps, kMaxSmem);
        gt[i]->smem = gemm_kacc_smem_bytes(gt[i]->hdr_bytes, gt[i]->n_stages, gt[i]->bps, tb[i].k_max);
        if (!tb[i].jobs.empty() && (gt[i]->n_stages < 2 || gt[i]->smem > kMaxSmem)) return STI_ERR_SHAPE;
      } else {
      if (!tb[i].jobs.empty() &&
          !gemm_pick_ring(tb[i].w_bytes, tb[i].k_max, gt[i]->hdr_bytes, &gt[i]->n_stages, &gt[i]->bps))
        return STI_ERR_SHAPE;
      gt[i]->smem = gemm_smem_bytes(tb[i].w_bytes, gt[i]->n_stages, gt[i]->bps, gt[i]->hdr_bytes);
      }
      if (gt[i]->smem > kMaxSmem && !tb[i].jobs.empty()) return STI_ERR_SHAPE;
      Fix fx{gt[i], 0, 0};
      fx.jobs_off = align16(host_tables.size());
      host_tables.resize(fx.jobs_off + tb[i].jobs.size() * sizeof(Job));
      if (!tb[i].jobs.empty()) memcpy(host_tables.data() + fx.jobs_off, tb[i].jobs.data(), tb[i].jobs.size() * sizeof(Job));
      fx.segs_off = align16(host_tables.size());
      host_tables.resize(fx.segs_off + tb[i].segs.size() * sizeof(Seg));
      if (!tb[i].segs.empty()) memcpy(host_tables.data() + fx.segs_off, tb[i].segs.data(), tb[i].segs.size() * sizeof(Seg));
      fixes.push_back(fx);
    }
    L.tables_bytes = host_tables.size() - L.tables_off;
    p->max_partial = std::max(p->max_partial, std::max(L.o.n_split, L.f2.n_split));
  }
  p->tables_bytes = std::max<size_t>(host_tables.size(), 16);
  CUDA_TRY(cudaMalloc(&p->tables, p->tables_bytes));
  if (!host_tables.empty())
    CUDA_TRY(cudaMemcpy(p->tables, host_tables.data(), host_tables.size(), cudaMemcpyHostToDevice));
  for (auto& fx : fixes) {
    fx.t->jobs = reinterpret_cast<Job*>(p->tables + fx.jobs_off);
    fx.t->segs = reinterpret_cast<Seg*>(p->tables + fx.segs_off);
  }
  // 4. activation scratch for max_batch * max_seq tokens
  const size_t Tmax = static_cast<size_t>(d.max_batch) * d.max_seq;
  const size_t f = d.ffn / d.n_ffn_slices;
  CUDA_TRY(cudaMalloc(&p->qkv, std::max<size_t>(1, 3 * max_heads) * Tmax * 64 * 2));
  CUDA_TRY(cudaMalloc(&p->attn_out, std::max<size_t>(1, max_heads) * Tmax * 64 * 2));
  CUDA_TRY(cudaMalloc(&p->partial, static_cast<size_t>(p->max_partial) * Tmax * d.hidden * 4));
  CUDA_TRY(cudaMalloc(&p->h1_f32, Tmax * d.hidden * 4));
  CUDA_TRY(cudaMalloc(&p->h1_bf16, Tmax * d.hidden * 2));
  CUDA_TRY(cudaMalloc(&p->u, std::max<size_t>(1, max_slices) * Tmax * f * 2));
  CUDA_TRY(cudaMalloc(&p->x_bf16, Tmax * d.hidden * 2));
  CUDA_TRY(cudaMalloc(&p->buf[0], Tmax * d.hidden * act_size(c)));
  CUDA_TRY(cudaMalloc(&p->buf[1], Tmax * d.hidden * act_size(c)));
  CUDA_TRY(cudaMalloc(&p->x_in, Tmax * d.hidden * act_size(c)));
  CUDA_TRY(cudaMalloc(&p->y_out, Tmax * d.hidden * act_size(c)));
  CUDA_TRY(cudaMalloc(&p->lens_dev, static_cast<size_t>(d.max_batch) * 4));
  CUDA_TRY(cudaMalloc(&p->stamps, static_cast<size_t>(d.n_layers) * kStampKernels * kStampRecord * sizeof(unsigned long long)));
  // 5. events
  const unsigned flags = cudaEventDefault;     // timing-capable; only recorded when profiling
  for (auto& L : p->layers) {
    CUDA_TRY(cudaEventCreateWithFlags(&L.ev_loaded, flags));
    CUDA_TRY(cudaEventCreateWithFlags(&L.g_ev_loaded, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&L.ev_done, flags));
    CUDA_TRY(cudaEventCreateWithFlags(&L.ev_copy_start, flags));
    CUDA_TRY(cudaEventCreateWithFlags(&L.ev_comp_start, flags));
    for (auto& e : L.ev_k) CUDA_TRY(cudaEventCreateWithFlags(&e, flags));
  }
  p->slot_free.resize(p->ring_slots);
  for (auto& e : p->slot_free) {
    CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    CUDA_TRY(cudaEventRecord(e, c->compute));
  }
  CUDA_TRY(cudaEventCreateWithFlags(&p->ev_copy_tail, cudaEventDisableTiming));
  CUDA_TRY(cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming));
  CUDA_TRY(cudaEventCreateWithFlags(&p->g_ev_join, cudaEventDisableTiming));
  p->g_slot_free.resize(p->ring_slots);
  for (auto& e : p->g_slot_free) CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  { const char* ng = getenv("STI_NO_GRAPH"); p->graph_off = ng && ng[0] == '1'; }
  CUDA_TRY(cudaEventCreateWithFlags(&p->ev_begin, flags));
  CUDA_TRY(cudaEventCreateWithFlags(&p->ev_end, flags));
  p->finalized = true;
  return STI_OK;
}

sti_status sti_layer_forward(sti_plan* p, int layer, const void* x, void* y, int batch, int seq,
                             const int32_t* lens) {
  sti_status st = check_forward_args(p, x, y, batch, seq);
  if (st != STI_OK) return st;
  if (layer < 0 || layer >= static_cast<int>(p->layers.size())) return STI_ERR_ARG;
  if ((st = sti_plan_finalize(p)) != STI_OK) return st;
  sti_ctx* c = p->ctx;
  CUDA_TRY(cudaSetDevice(c->device));
  if (p->copy_tail_valid) {       // an ungraphed forward may still have copies in flight on the copy stream
    CUDA_TRY(cudaStreamWaitEvent(c->compute, p->ev_copy_tail, 0));
    p->copy_tail_valid = false;
  }
  ForwardKey k;
  k.x = x; k.y = y; k.lens = lens; k.batch = batch; k.seq = seq; k.layer = layer;
  k.stamps = p->profiling == 3;
  return model_forward_impl(p, k);
}

sti_status sti_model_forward(sti_plan* p, const void* x, void* y, int batch, int seq, const int32_t* lens) {
  sti_status st = check_forward_args(p, x, y, batch, seq);
  if (st != STI_OK) return st;
  if ((st = sti_plan_finalize(p)) != STI_OK) return st;
  CUDA_TRY(cudaSetDevice(p->ctx->device));
  ForwardKey k;
  k.x = x; k.y = y; k.lens = lens; k.batch = batch; k.seq = seq;
  k.stamps = p->profiling == 3;
  return model_forward_impl(p, k);
}

sti_status sti_model_forward_host(sti_plan* p, const void* x_host, void* y_host, int batch, int seq,
                                  const int32_t* lens_host) {
  sti_status st = check_forward_args(p, x_host, y_host, batch, seq, false);
  if (st != STI_OK) return st;
  if ((st = sti_plan_finalize(p)) != STI_OK) return st;
  sti_ctx* c = p->ctx;
  CUDA_TRY(cudaSetDevice(c->device));
  ForwardKey k;
  k.x_host = x_host; k.y_host = y_host; k.batch = batch; k.seq = seq;
  if (lens_host) {
    // sequence lengths change from call to call: staged outside the graph
    CUDA_TRY(cudaMemcpyAsync(p->lens_dev, lens_host, static_cast<size_t>(batch) * 4, cudaMemcpyHostToDevice, c->compute));
    k.lens = p->lens_dev;
  }
  k.stamps = p->profiling == 3;
  return model_forward_impl(p, k);
}

sti_status sti_sync(sti_ctx* c) {
  if (!c) return STI_ERR_ARG;
  if (cudaSetDevice(c->device) != cudaSuccess) return STI_ERR_CUDA;
  cudaError_t e1 = cudaStreamSynchronize(c->copy);
  cudaError_t e2 = cudaStreamSynchronize(c->compute);
  if (e1 != cudaSuccess || e2 != cudaSuccess) return STI_ERR_CUDA;
  return check_async(c);
}

sti_status sti_shard_decode(sti_plan* p, int layer, sti_kind kind, int index, int matrix, float* w_dev,
                            uint8_t* codes_dev, uint16_t* wbf16_dev) {
  if (!p || (kind != STI_ATTN && kind != STI_FFN)) return STI_ERR_ARG;
  Unit* u = find_unit(p, layer, kind, index);
  if (!u || !u->cfg.keep) return STI_ERR_ARG;
  sti_status st = sti_plan_finalize(p);
  if (st != STI_OK) return st;
  sti_ctx* c = p->ctx;
  int nm;
  const MatrixInfo* mi = unit_matrices(c, kind, &nm);
  if (matrix < 0 || matrix >= nm) return STI_ERR_ARG;
  CUDA_TRY(cudaSetDevice(c->device));
  Layer& L = p->layers[layer];
  if (!u->cfg.resident) {
    if (p->copy_tail_valid) CUDA_TRY(cudaStreamWaitEvent(c->compute, p->ev_copy_tail, 0));
    if ((st = enqueue_layer_copy(p, layer, c->compute)) != STI_OK) return st;
  }
  const Seg s = make_seg(c, *u, kind, matrix, 0, mi[matrix].rows, 0);
  DecodeLaunch dl{};
  dl.codes = s.codes; dl.table = s.table; dl.out_off = s.out_off; dl.out_val = s.out_val; dl.n_out = s.n_out;
  dl.flat_base = s.flat_base; dl.bits = s.bits; dl.rows = mi[matrix].rows; dl.kc = mi[matrix].kc;
  dl.w = w_dev; dl.codes_out = codes_dev; dl.wbf16 = wbf16_dev;
  CUDA_TRY(launch_decode(dl, c->compute));
  c->launches += (s.bits == 32 || s.n_out == 0) ? 1 : 2;
  if (!u->cfg.resident) CUDA_TRY(cudaEventRecord(p->slot_free[L.slot], c->compute));
  return STI_OK;
}

sti_status sti_gemm_probe(sti_plan* p, int layer, int gemm, const void* x_bf16_dev, int tokens, void* out_dev,
                          size_t out_capacity_bytes, int variant, int32_t* n_partials) {
  if (!p || !x_bf16_dev || !out_dev || gemm < 0 || gemm > 3 || variant < 0 || variant > 3) return STI_ERR_ARG;
  if (variant == 3 && gemm != 3) return STI_ERR_ARG;       // the K-accumulating kernel exists for FFN2 only
  if (layer < 0 || layer >= static_cast<int>(p->layers.size())) return STI_ERR_ARG;
  if (tokens < 1 || tokens > 65536) return STI_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x_bf16_dev) & 15) || (reinterpret_cast<uintptr_t>(out_dev) & 15)) return STI_ERR_ARG;
  sti_status st = sti_plan_finalize(p);
  if (st != STI_OK) return st;
  sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  CUDA_TRY(cudaSetDevice(c->device));
  Layer& L = p->layers[layer];
  const int nh = static_cast<int>(L.kept_heads.size()), ns = static_cast<int>(L.kept_slices.size());
  const int f = d.ffn / d.n_ffn_slices;
  const GemmTable* tabs[4] = {&L.qkv, &L.o, &L.f1, &L.f2};
  const GemmTable& tab = *tabs[gemm];
  if (tab.n_jobs == 0) return STI_ERR_STATE;               // no kept unit feeds this GEMM
  const int ldx[4] = {d.hidden, nh * 64, d.hidden, ns * f};
  const int ldo[4] = {64, d.hidden, ns * f, d.hidden};
  const int parts[4] = {1, tabs[1]->n_split, 1, variant == 3 ? 1 : tabs[3]->n_split};
  if (variant == 3 && L.f2k.n_jobs == 0) return STI_ERR_STATE;   // the plan was not made for many tokens
  const size_t out_elems[4] = {static_cast<size_t>(3) * nh * tokens * 64, static_cast<size_t>(parts[1]) * tokens * d.hidden,
                               static_cast<size_t>(tokens) * ns * f, static_cast<size_t>(parts[3]) * tokens * d.hidden};
  const size_t need = out_elems[gemm] * ((gemm == 1 || gemm == 3) ? 4 : 2);
  if (out_capacity_bytes < need) return STI_ERR_SIZE;
  if (!p->zero_bias) {
    const size_t n = static_cast<size_t>(3) * d.n_heads * 64 + d.ffn;
    CUDA_TRY(cudaMalloc(&p->zero_bias, n * sizeof(float)));
    CUDA_TRY(cudaMemset(p->zero_bias, 0, n * sizeof(float)));
  }
  if (L.str_bytes > 0) {           // a streamed layer is brought into its ring slot first (not overlapped)
    if (p->copy_tail_valid) CUDA_TRY(cudaStreamWaitEvent(c->compute, p->ev_copy_tail, 0));
    if ((st = enqueue_layer_copy(p, layer, c->compute)) != STI_OK) return st;
  }
  const GemmKind kind = (gemm == 1 || gemm == 3) ? GEMM_BF16_TO_F32 : GEMM_BF16_TO_BF16;
  if (variant == 3)
    st = run_gemm_kacc(p, L.f2k, x_bf16_dev, ldx[3], tokens, static_cast<float*>(out_dev), ldo[3], nullptr);
  else
  st = run_gemm(p, kind, tab, x_bf16_dev, ldx[gemm], tokens, out_dev, ldo[gemm], p->zero_bias, -1,
                variant == 0 ? -1 : variant - 1);
  if (st != STI_OK) return st;
  if (L.str_bytes > 0) CUDA_TRY(cudaEventRecord(p->slot_free[L.slot], c->compute));
  if (n_partials) *n_partials = parts[gemm];
  return STI_OK;
}

sti_status sti_decode_rate_probe(sti_plan* p, const void* x_bf16_dev, int tokens, void* out_dev, size_t out_capacity_bytes,
                                 uint64_t* packed_bytes, int32_t* n_tiles) {
  if (!p || !x_bf16_dev || !out_dev) return STI_ERR_ARG;
  if (tokens < 1 || tokens > 128) return STI_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x_bf16_dev) & 15) || (reinterpret_cast<uintptr_t>(out_dev) & 15)) return STI_ERR_ARG;
  sti_status st = sti_plan_finalize(p);
  if (st != STI_OK) return st;
  sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  CUDA_TRY(cudaSetDevice(c->device));
  const int f = d.ffn / d.n_ffn_slices;
  for (auto& L : p->layers) if (L.str_bytes) return STI_ERR_STATE;       // every shard must sit in device memory
  if (!p->rate_tables) {
    // one table with the FFN1 tile jobs of all layers; layer l's tiles write output columns l * ffn + ...
    std::vector<Job> jobs;
    std::vector<Seg> segs;
    uint32_t stride = 0;
    for (auto& L : p->layers) stride = std::max(stride, L.f1.seg_stride);
    if (stride == 0) return STI_ERR_STATE;                               // no FFN slice kept anywhere
    std::vector<Job> hj;
    std::vector<Seg> hs;
    uint64_t bytes = 0;
    for (size_t l = 0; l < p->layers.size(); ++l) {
      Layer& L = p->layers[l];
      if (L.f1.n_jobs == 0) continue;
      hj.resize(L.f1.n_jobs);
      hs.resize(static_cast<size_t>(L.f1.n_jobs) * L.f1.seg_stride);
      CUDA_TRY(cudaMemcpy(hj.data(), L.f1.jobs, hj.size() * sizeof(Job), cudaMemcpyDeviceToHost));
      CUDA_TRY(cudaMemcpy(hs.data(), L.f1.segs, hs.size() * sizeof(Seg), cudaMemcpyDeviceToHost));
      for (int j = 0; j < L.f1.n_jobs; ++j) {
        Job job = hj[j];
        job.seg_begin = static_cast<uint32_t>(jobs.size()) * stride;
        job.out_col += static_cast<uint32_t>(l) * d.ffn;
        job.bias_off = -1;
        jobs.push_back(job);
        for (uint32_t k = 0; k < stride; ++k) segs.push_back(k < job.n_seg ? hs[static_cast<size_t>(j) * L.f1.seg_stride + k] : Seg{});
      }
      for (int sl : L.kept_slices) {
        const int bits = L.ffn[sl].cfg.bits;
        bytes += static_cast<uint64_t>(f) * d.hidden * bits / 8 + (bits == 32 ? 0 : (4ull << bits));
      }
    }
    const size_t jb = align16(jobs.size() * sizeof(Job)), sb = segs.size() * sizeof(Seg);
    CUDA_TRY(cudaMalloc(&p->rate_tables, jb + sb));
    CUDA_TRY(cudaMemcpy(p->rate_tables, jobs.data(), jobs.size() * sizeof(Job), cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(p->rate_tables + jb, segs.data(), sb, cudaMemcpyHostToDevice));
    p->rate_jobs = static_cast<int>(jobs.size());
    p->rate_seg_stride = stride;
    p->rate_packed_bytes = bytes;
  }
  const int ldo = static_cast<int>(p->layers.size()) * d.ffn;
  if (out_capacity_bytes < static_cast<size_t>(tokens) * ldo * 2) return STI_ERR_SIZE;
  const GemmTable& ref = p->layers[0].f1.n_jobs ? p->layers[0].f1 : p->layers.back().f1;
  GemmTable tab = ref;                                                   // same tile shape, ring and shared memory
  tab.jobs = reinterpret_cast<Job*>(p->rate_tables);
  tab.segs = reinterpret_cast<Seg*>(p->rate_tables + align16(static_cast<size_t>(p->rate_jobs) * sizeof(Job)));
  tab.n_jobs = p->rate_jobs;
  tab.seg_stride = p->rate_seg_stride;
  tab.pair_ok = false;
  for (auto& L : p->layers) {                                            // the widest tile decides the shared-memory shape
    if (L.f1.n_jobs && L.f1.smem > tab.smem) { tab.smem = L.f1.smem; tab.w_bytes = L.f1.w_bytes; tab.n_stages = L.f1.n_stages; tab.bps = L.f1.bps; }
  }
  st = run_gemm(p, GEMM_BF16_TO_BF16, tab, x_bf16_dev, d.hidden, tokens, out_dev, ldo, nullptr, -1, 0);
  if (st != STI_OK) return st;
  if (packed_bytes) *packed_bytes = p->rate_packed_bytes;
  if (n_tiles) *n_tiles = p->rate_jobs;
  return STI_OK;
}

sti_status sti_plan_set_profiling(sti_plan* p, int enabled) {
  if (!p) return STI_ERR_ARG;
  p->profiling = enabled < 0 ? 0 : (enabled > 3 ? 3 : enabled);
  p->stats_valid = false;
  return STI_OK;
}

sti_status sti_get_stats(sti_plan* p, sti_stats* out) {
  if (!p || !out) return STI_ERR_ARG;
  if (!p->finalized || !p->stats_valid) return STI_ERR_STATE;
  sti_ctx* c = p->ctx;
  CUDA_TRY(cudaSetDevice(c->device));
  CUDA_TRY(cudaStreamSynchronize(c->copy));
  CUDA_TRY(cudaStreamSynchronize(c->compute));
  sti_stats s;
  memset(&s, 0, sizeof(s));
  const int n = static_cast<int>(p->layers.size());
  s.n_layers = n;
  float prev_done = 0.f;
  for (int l = 0; l < n; ++l) {
    Layer& L = p->layers[l];
    float t_start = 0.f, t_done = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&t_start, p->ev_begin, L.ev_comp_start));
    CUDA_TRY(cudaEventElapsedTime(&t_done, p->ev_begin, L.ev_done));
    s.compute_us[l] = (t_done - t_start) * 1e3f;
    if (L.str_bytes) {
      float ms = 0.f, t_loaded = 0.f;
      CUDA_TRY(cudaEventElapsedTime(&ms, L.ev_copy_start, L.ev_loaded));
      s.copy_us[l] = ms * 1e3f;
      CUDA_TRY(cudaEventElapsedTime(&t_loaded, p->ev_begin, L.ev_loaded));
      s.stall_us[l] = std::max(0.f, t_loaded - prev_done) * 1e3f;
    }
    if (p->profiling >= 2) {
      float k[7] = {};
      for (int i = 0; i < 7; ++i)
        if (L.k_ran[i]) CUDA_TRY(cudaEventElapsedTime(&k[i], L.ev_k[i], L.ev_k[i + 1]));
      s.gemm_us[l] = (k[0] + k[2] + k[4] + k[5]) * 1e3f;
      s.attn_us[l] = k[1] * 1e3f;
      s.ln_us[l] = (k[3] + k[6]) * 1e3f;
      s.gemm_launches += (L.k_ran[0] ? 2 : 0) + (L.k_ran[4] ? 2 : 0);
    }
    s.streamed_bytes[l] = L.str_bytes;
    s.resident_bytes[l] = L.res_bytes;
    prev_done = t_done;
  }
  float tot = 0.f;
  CUDA_TRY(cudaEventElapsedTime(&tot, p->ev_begin, p->ev_end));
  s.total_us = tot * 1e3f;
  *out = s;
  return STI_OK;
}

sti_status sti_get_kernel_stamps(sti_plan* p, uint64_t* out, size_t capacity_words, int32_t* n_layers) {
  if (!p || !out) return STI_ERR_ARG;
  if (!p->finalized) return STI_ERR_STATE;
  const size_t n = p->layers.size() * kStampKernels * kStampRecord;
  if (capacity_words < n) return STI_ERR_SIZE;
  sti_ctx* c = p->ctx;
  CUDA_TRY(cudaSetDevice(c->device));
  CUDA_TRY(cudaStreamSynchronize(c->copy));
  CUDA_TRY(cudaStreamSynchronize(c->compute));
  std::vector<unsigned long long> raw(n);
  CUDA_TRY(cudaMemcpy(raw.data(), p->stamps, n * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  for (size_t i = 0; i < n; ++i) {
    const size_t slot = i % kStampRecord;
    const bool is_min = slot == 0 || slot == 1;          // the other slots hold complemented maxima
    const unsigned long long v = raw[i];
    out[i] = v == ~0ull ? 0 : (is_min ? v : ~v);
  }
  if (n_layers) *n_layers = static_cast<int32_t>(p->layers.size());
  return STI_OK;
}

sti_status sti_plan_retain(sti_plan* p, const uint8_t* attn_keep, const uint8_t* ffn_keep, uint64_t* retained_bytes) {
  if (!p || !attn_keep || !ffn_keep) return STI_ERR_ARG;
  sti_status st = sti_plan_finalize(p);
  if (st != STI_OK) return st;
  if (p->retain_arena) return STI_ERR_STATE;               // one retained set per plan
  sti_ctx* c = p->ctx;
  const sti_model_desc& d = c->desc;
  CUDA_TRY(cudaSetDevice(c->device));
  size_t total = 0;
  for (int l = 0; l < d.n_layers; ++l) {
    Layer& L = p->layers[l];
    for (int h = 0; h < d.n_heads; ++h)
      if (attn_keep[l * d.n_heads + h] && !L.attn[h].cfg.keep) return STI_ERR_ARG;     // cannot keep what the plan dropped
    for (int j = 0; j < d.n_ffn_slices; ++j)
      if (ffn_keep[l * d.n_ffn_slices + j] && !L.ffn[j].cfg.keep) return STI_ERR_ARG;
  }
  for (int l = 0; l < d.n_layers; ++l) {
    Layer& L = p->layers[l];
    auto mark = [&](Unit& u, bool keep) {
      u.retain = keep && u.cfg.keep && !u.cfg.resident;    // resident units are on the device anyway
      if (u.retain) total += align256(u.bytes);
    };
    for (int h = 0; h < d.n_heads; ++h) mark(L.attn[h], attn_keep[l * d.n_heads + h] != 0);
    for (int j = 0; j < d.n_ffn_slices; ++j) mark(L.ffn[j], ffn_keep[l * d.n_ffn_slices + j] != 0);
  }
  if (total) {
    CUDA_TRY(cudaMalloc(&p->retain_arena, total));
    size_t cur = 0;
    for (auto& L : p->layers) {
      auto bind = [&](Unit& u) { if (u.retain) { u.retained = p->retain_arena + cur; cur += align256(u.bytes); } };
      for (auto& u : L.attn) bind(u);
      for (auto& u : L.ffn) bind(u);
    }
    p->retain_pending = true;
  }
  p->retain_bytes = total;
  if (retained_bytes) *retained_bytes = total;
  return STI_OK;
}

sti_status sti_shard_adopt(sti_plan* p, const sti_plan* from, int layer, sti_kind kind, int index) {
  if (!p || !from || p == from || (kind != STI_ATTN && kind != STI_FFN)) return STI_ERR_ARG;
  if (p->ctx != from->ctx) return STI_ERR_ARG;             // same device, same streams
  if (p->finalized || !from->finalized) return STI_ERR_STATE;
  Unit* u = find_unit(p, layer, kind, index);
  const Unit* src = find_unit(const_cast<sti_plan*>(from), layer, kind, index);
  if (!u || !src) return STI_ERR_ARG;
  if (!u->cfg.keep || !u->cfg.resident || !src->cfg.keep) return STI_ERR_STATE;   // adopted units live in the preload buffer
  if (u->cfg.bits != src->cfg.bits) return STI_ERR_BITS;                          // a shard is cached at the version it was loaded with
  const uint8_t* where = nullptr;
  if (src->cfg.resident) where = src->dev + src->off_codes;
  else if (src->retained && src->retained_done) where = src->retained;
  if (!where) return STI_ERR_STATE;                        // not in device memory: it has to be uploaded
  u->table = src->table;                                   // host-side metadata the tile tables are built from
  u->out_off = src->out_off;
  u->out_val = src->out_val;
  u->codes.clear();
  u->codes_bytes = src->codes_bytes;
  u->adopt_src = where;
  u->uploaded = true;
  return STI_OK;
}

sti_status sti_plan_fill_stats(sti_plan* p, uint64_t* uploaded_bytes, uint64_t* adopted_bytes, uint64_t* retained_bytes) {
  if (!p) return STI_ERR_ARG;
  if (!p->finalized) return STI_ERR_STATE;
  if (uploaded_bytes) *uploaded_bytes = p->finalize_h2d_bytes;
  if (adopted_bytes) *adopted_bytes = p->finalize_d2d_bytes;
  if (retained_bytes) *retained_bytes = p->retain_bytes;
  return STI_OK;
}

sti_status sti_plan_inject(sti_plan* p, int what, int layer, unsigned value) {
  if (!p) return STI_ERR_ARG;
  switch (what) {
    case STI_INJECT_NONE:
      p->slow_copy_layer = -1; p->slow_copy_us = 0; p->fail_pinned_alloc = false;
      return STI_OK;
    case STI_INJECT_SLOW_COPY:
      if (layer < 0 || layer >= static_cast<int>(p->layers.size()) || value > 1000000u) return STI_ERR_ARG;
      p->slow_copy_layer = layer; p->slow_copy_us = value;
      return STI_OK;
    case STI_INJECT_PINNED_ALLOC_FAILURE:
      if (p->finalized || p->attempted) return STI_ERR_STATE;
      p->fail_pinned_alloc = value != 0;
      return STI_OK;
    default:
      return STI_ERR_ARG;
  }
}

sti_status sti_plan_memory(sti_plan* p, uint64_t* preload_bytes, uint64_t* pinned_bytes, uint64_t* ring_bytes) {
  if (!p) return STI_ERR_ARG;
  if (!p->finalized) return STI_ERR_STATE;
  if (preload_bytes) *preload_bytes = p->preload_bytes;
  if (pinned_bytes) *pinned_bytes = p->pinned_bytes;
  if (ring_bytes) *ring_bytes = p->slot_bytes * p->ring_slots;
  return STI_OK;
}

sti_status sti_plan_check_guards(sti_plan* p, int32_t* damaged) {
  if (!p || !damaged) return STI_ERR_ARG;
  if (!p->finalized) return STI_ERR_STATE;
  sti_ctx* c = p->ctx;
  CUDA_TRY(cudaSetDevice(c->device));
  CUDA_TRY(cudaStreamSynchronize(c->copy));
  CUDA_TRY(cudaStreamSynchronize(c->compute));
  std::vector<const uint8_t*> guards;
  if (p->preload_alloc) {
    guards.push_back(p->preload_alloc);
    guards.push_back(p->preload + p->preload_bytes);
  }
  if (p->ring_alloc) {
    guards.push_back(p->ring_alloc);
    for (int i = 1; i <= p->ring_slots; ++i) guards.push_back(p->ring + static_cast<size_t>(i) * p->slot_bytes - kGuardBytes);
  }
  uint8_t host[kGuardBytes];
  int bad = 0;
  for (const uint8_t* g : guards) {
    CUDA_TRY(cudaMemcpy(host, g, kGuardBytes, cudaMemcpyDeviceToHost));
    bool ok = true;
    for (size_t i = 0; i < kGuardBytes; ++i) ok = ok && host[i] == static_cast<uint8_t>(kGuardPattern);
    if (!ok) ++bad;
  }
  *damaged = bad;
  return STI_OK;
}

sti_status sti_plan_set_overlap(sti_plan* p, int overlap) {
  if (!p) return STI_ERR_ARG;
  if (!overlap) {
    sti_status st = sti_plan_finalize(p);
    if (st != STI_OK) return st;
    if (p->n_streamed_layers > p->ring_slots) return STI_ERR_STATE;
  }
  const bool want = overlap != 0;
  if (want != p->overlap) {
    // captured forwards encode the old order
    cudaSetDevice(p->ctx->device);
    cudaStreamSynchronize(p->ctx->compute);
    for (auto& g : p->graphs) if (g.exec) { cudaGraphExecDestroy(g.exec); g.exec = nullptr; }
    p->graphs.clear();
    p->overlap = want;
  }
  return STI_OK;
}

uint64_t sti_ctx_launch_count(sti_ctx* c) { return c ? c->launches : 0; }

sti_status sti_host_retile(const uint8_t* src, uint8_t* dst, uint32_t rows, uint32_t cols, uint32_t bits) {
  if (!src || !dst) return STI_ERR_ARG;
  if (bits < 2 || bits > 6) return STI_ERR_BITS;
  if (cols == 64 ? rows % 64 != 0 : (cols % 128 != 0 || rows % 32 != 0)) return STI_ERR_SHAPE;
  retile_matrix(src, dst, rows, cols, bits);
  return STI_OK;
}

}  // extern "C"
