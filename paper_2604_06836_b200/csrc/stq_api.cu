// C-ABI host layer of libstq: argument validation, tensor-table and tile-map upload, launches.
// No arithmetic of the method lives here; every step of the path runs in stq_kernels.cu.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include <cuda.h>   // types of the one driver query below; the entry point is fetched at run time, nothing links libcuda

#include "../../include/stq.h"
#include "stq_internal.h"

using stq::TensorDesc;
static_assert(STQ_TILE_ELEMS == stq::kTile, "the tile size promised in the header");

struct stq_handle {
  int device = 0;
  int sm_count = 0;
  int grid = 0;
  uint64_t launches = 0;
  std::string cuda_err;

  // cached caller table (to skip re-uploads) and its device image
  std::vector<stq_tensor> cached;
  int cached_kind = -1;          // which entry point built the device table
  std::vector<uint64_t> cached_sig;   // numel | wide<<63 per tensor: decides the tile map
  TensorDesc* d_table = nullptr;
  size_t d_table_cap = 0;
  // tile -> tensor index; order: fast tiles, then the remaining narrow tiles, then wide ones
  uint32_t* d_tile_map = nullptr;
  size_t d_tile_cap = 0;
  uint32_t n_tiles = 0, n_fast = 0, n_narrow = 0;   // n_narrow counts fast + remaining narrow
  uint32_t n_main = 0, n_var_end = 0;               // fast tiles: [0, n_main) fused bodies, [n_main, n_var_end) fused bodies
                                                    // of the "sr" / "ts" codes, [n_var_end, n_fast) change width
  int fast_grid = 0;
  bool any_lp = false;              // some tensor of the current table wants a low-precision copy
  bool any_variant = false;         // some tensor's second moment uses a code only the generic kernel serves
  int* d_err = nullptr;         // [0] raised by a kernel whose bounded wait ran out; [1] non-zero if the last call
                                // that carried statistics really produced them (a skipped step does not)
  float* d_scalars = nullptr;   // {step_size, rsqrt_bc2, lr} when the step count lives on the device
  stq::FastSched* d_sched = nullptr;   // two work lists of the main step kernel (fused bodies, width changes)

  // pinned staging for uploads
  void* h_stage = nullptr;
  size_t h_stage_cap = 0;
  cudaEvent_t stage_ev = nullptr;
  // the generic kernel's share of a step (ragged tails, 32-bit states) runs beside the main kernel:
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool stage_busy = false;

  // statistics
  double* d_partials = nullptr;
  size_t d_partials_cap = 0;
  double* d_stats = nullptr;
  size_t d_stats_cap = 0;
  uint32_t* d_seg_map = nullptr;   // statistics segment -> tensor
  size_t d_seg_map_cap = 0;
  double* d_seg_sums = nullptr;
  size_t d_seg_sums_cap = 0;
  uint32_t n_seg = 0;
  double* h_stats = nullptr;
  size_t h_stats_cap = 0;
  int stats_L = 0;            // > 0: partials of a table with this many tensors are pending

  // device arena, streams and events of stq_step_host
  uint8_t* d_arena = nullptr;
  size_t d_arena_cap = 0;
  cudaStream_t host_streams[3] = {nullptr, nullptr, nullptr};
  std::vector<cudaEvent_t> host_events;
};

namespace {

enum Kind { kKindStep = 0, kKindRepack = 1, kKindInit = 2, kKindStats = 3 };

bool width_ok(int b) { return b == 2 || b == 3 || b == 4 || b == 8 || b == 16 || b == 32; }
bool block_ok(uint32_t b) { return b >= (uint32_t)stq::kMinBlock && b <= (uint32_t)stq::kMaxBlock && (b & (b - 1)) == 0; }
bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int fail_cuda(stq_handle* h, cudaError_t e) {
  h->cuda_err = cudaGetErrorString(e);
  return STQ_E_CUDA;
}
#define STQ_CUDA(h, call)                                   \
  do {                                                      \
    cudaError_t e__ = (call);                               \
    if (e__ != cudaSuccess) return fail_cuda((h), e__);     \
  } while (0)

template <class T>
int grow(stq_handle* h, T*& p, size_t& cap, size_t need) {
  if (need <= cap) return STQ_OK;
  if (p) cudaFree(p);
  p = nullptr;
  cap = 0;
  size_t want = need + need / 4 + 256;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&p), want * sizeof(T));
  if (e != cudaSuccess) { h->cuda_err = cudaGetErrorString(e); p = nullptr; return STQ_E_WORKSPACE; }
  cap = want;
  return STQ_OK;
}

int grow_stage(stq_handle* h, size_t bytes) {
  if (bytes <= h->h_stage_cap) return STQ_OK;
  if (h->stage_busy) { cudaEventSynchronize(h->stage_ev); h->stage_busy = false; }
  if (h->h_stage) cudaFreeHost(h->h_stage);
  h->h_stage = nullptr;
  h->h_stage_cap = 0;
  size_t want = bytes + bytes / 4 + 4096;
  cudaError_t e = cudaMallocHost(&h->h_stage, want);
  if (e != cudaSuccess) { h->cuda_err = cudaGetErrorString(e); h->h_stage = nullptr; return STQ_E_WORKSPACE; }
  h->h_stage_cap = want;
  return STQ_OK;
}

// True if [p, p + len) lies inside ONE allocation known to the driver.  Buffers that are neighbours in
// the address space may still be separate allocations, and a copy must not span two of them.
bool one_allocation(const void* p, size_t len) {
  typedef CUresult (*get_attr_t)(void*, CUpointer_attribute, CUdeviceptr);
  static const get_attr_t get = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuPointerGetAttribute", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    (void)cudaGetLastError();
    return reinterpret_cast<get_attr_t>(f);
  }();
  if (!get) return false;
  CUdeviceptr base = 0;
  size_t size = 0;
  const CUdeviceptr q = reinterpret_cast<CUdeviceptr>(p);
  if (get(&base, CU_POINTER_ATTRIBUTE_RANGE_START_ADDR, q) != CUDA_SUCCESS) return false;
  if (get(&size, CU_POINTER_ATTRIBUTE_RANGE_SIZE, q) != CUDA_SUCCESS) return false;
  return q >= base && q + len <= base + size;
}

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + nb && y < x + na;
}

// Host-side validation of one row for the given entry point.
int validate_row(const stq_tensor& t, int kind) {
  if (t.numel == 0 || t.numel > (1ull << 40)) return STQ_E_NUMEL;
  if (t.lp_dtype > STQ_LP_F16) return STQ_E_ARG;
  if (t.v_log > STQ_VLOG_TS) return STQ_E_ARG;
  if (t.v_log != STQ_VLOG_SR && t.sr_id != 0) return STQ_E_ARG;
  if (kind == kKindStep && t.lp_dtype != STQ_LP_NONE) {
    if (!t.param_lp) return STQ_E_NULL;
    if (!aligned(t.param_lp, 8)) return STQ_E_ALIGN;
  }
  if (kind == kKindStats) {
    if (!t.grad) return STQ_E_NULL;
    if (!aligned(t.grad, 16)) return STQ_E_ALIGN;
    return STQ_OK;
  }
  if (!block_ok(t.block)) return STQ_E_BLOCK;
  if (!width_ok(t.bits_m_out) || !width_ok(t.bits_v_out)) return STQ_E_BITS;
  if (!t.m_codes_out || !t.v_codes_out) return STQ_E_NULL;
  if (t.bits_m_out != 32 && !t.m_scales_out) return STQ_E_NULL;
  if (t.bits_v_out != 32 && !t.v_scales_out) return STQ_E_NULL;
  if (!aligned(t.m_codes_out, 16) || !aligned(t.v_codes_out, 16)) return STQ_E_ALIGN;
  if (!aligned(t.m_scales_out, 4) || !aligned(t.v_scales_out, 4)) return STQ_E_ALIGN;
  if (kind == kKindInit) return STQ_OK;

  if (!width_ok(t.bits_m) || !width_ok(t.bits_v)) return STQ_E_BITS;
  if (!t.m_codes_in || !t.v_codes_in) return STQ_E_NULL;
  if (t.bits_m != 32 && !t.m_scales_in) return STQ_E_NULL;
  if (t.bits_v != 32 && !t.v_scales_in) return STQ_E_NULL;
  if (!aligned(t.m_codes_in, 16) || !aligned(t.v_codes_in, 16)) return STQ_E_ALIGN;
  if (!aligned(t.m_scales_in, 4) || !aligned(t.v_scales_in, 4)) return STQ_E_ALIGN;
  if (kind == kKindStep) {
    if (!t.param || !t.grad) return STQ_E_NULL;
    if (!aligned(t.param, 16) || !aligned(t.grad, 16)) return STQ_E_ALIGN;
  }
  // in-place is allowed only for identical pointer and identical width
  const size_t mi = stq_codes_bytes(t.numel, t.bits_m), mo = stq_codes_bytes(t.numel, t.bits_m_out);
  const size_t vi = stq_codes_bytes(t.numel, t.bits_v), vo = stq_codes_bytes(t.numel, t.bits_v_out);
  if (overlap(t.m_codes_in, mi, t.m_codes_out, mo) &&
      !(t.m_codes_in == t.m_codes_out && t.bits_m == t.bits_m_out))
    return STQ_E_ALIAS;
  if (overlap(t.v_codes_in, vi, t.v_codes_out, vo) &&
      !(t.v_codes_in == t.v_codes_out && t.bits_v == t.bits_v_out))
    return STQ_E_ALIAS;
  if (overlap(t.m_codes_out, mo, t.v_codes_out, vo) || overlap(t.m_codes_in, mi, t.v_codes_out, vo) ||
      overlap(t.v_codes_in, vi, t.m_codes_out, mo))
    return STQ_E_ALIAS;
  const size_t sb = stq_scales_bytes(t.numel, t.block), sbv = stq_v_scales_bytes(t.numel, t.block, t.v_log);
  if (t.bits_m != 32 && t.bits_m_out != 32 && t.m_scales_in != t.m_scales_out &&
      overlap(t.m_scales_in, sb, t.m_scales_out, sb))
    return STQ_E_ALIAS;
  if (t.bits_v != 32 && t.bits_v_out != 32 && t.v_scales_in != t.v_scales_out &&
      overlap(t.v_scales_in, sbv, t.v_scales_out, sbv))
    return STQ_E_ALIAS;
  return STQ_OK;
}

// Tensors with the same key run the same specialised body of the main kernel: the two widths, and
// for v at 8 or 16 bits the variant of its quantizer.  Ordered from cheap to expensive v codes.
// Relative time per tile of the fused bodies, from the measured throughput of each on one large tensor
// (rows: m at 2, 3, 4, 8, 16 bits; columns: v at 2, 3, 4, 8, 16 bits, then 8 and 16 bits in the
// piecewise-linear variant; 1.0 = the 4/4-bit body).  Only the initial spread of the CTAs over the
// groups uses it; the balance itself is dynamic.
double body_cost(const stq_tensor& t) {
  static const double kRate[5][7] = {
      {581, 550, 564, 488, 445, 480, 430},
      {550, 523, 540, 454, 417, 450, 400},
      {567, 536, 551, 488, 439, 480, 425},
      {531, 520, 510, 471, 414, 465, 405},
      {458, 450, 443, 414, 369, 410, 360},
  };
  auto idx = [](int b) { return b == 2 ? 0 : b == 3 ? 1 : b == 4 ? 2 : b == 8 ? 3 : 4; };
  int iv = idx(t.bits_v);
  if (t.v_log == STQ_VLOG_PL && iv >= 3) iv += 2;
  if (t.v_log >= STQ_VLOG_SR) return 1.2;      // (their own launch: only the spread among themselves matters)
  return 551.0 / kRate[idx(t.bits_m)][iv];
}

constexpr int kSplitKey = 1 << 20, kVariantKey = 1 << 19;
int body_key(const stq_tensor& t) {
  if (t.bits_m != t.bits_m_out || t.bits_v != t.bits_v_out) return kSplitKey;   // one runtime-width body for all of them
  if (t.v_log >= STQ_VLOG_SR) return kVariantKey + ((int)t.v_log * 32 + t.bits_v) * 64 + t.bits_m;
  const int pl = t.v_log == STQ_VLOG_PL && (t.bits_v == 8 || t.bits_v == 16) ? 1 : 0;
  return (t.bits_v * 2 + (1 - pl)) * 64 + t.bits_m;
}

bool row_is_wide(const stq_tensor& t, int kind) {
  if (kind == kKindStats) return false;
  if (t.bits_m_out == 32 || t.bits_v_out == 32) return true;
  if (kind != kKindInit && (t.bits_m == 32 || t.bits_v == 32)) return true;
  return false;
}

// Builds (or reuses) the device table and tile map for `tensors`.
int prepare(stq_handle* h, const stq_tensor* tensors, int L, int kind, cudaStream_t stream) {
  if (!h || !tensors) return STQ_E_NULL;
  if (L <= 0 || L > (1 << 20)) return STQ_E_NUMEL;
  STQ_CUDA(h, cudaSetDevice(h->device));
  // the same table as last time (the usual case between decision steps) was validated and uploaded then
  const bool same = h->cached_kind == kind && (int)h->cached.size() == L &&
                    std::memcmp(h->cached.data(), tensors, sizeof(stq_tensor) * (size_t)L) == 0;
  if (same) return STQ_OK;
  // Pending statistics belong to the table they were taken with (its tile map and segment map finish the
  // reduction): a call with another table drops them, and stq_layer_stats then reports STQ_E_STATE.
  h->stats_L = 0;
  for (int l = 0; l < L; ++l) {
    int rc = validate_row(tensors[l], kind);
    if (rc != STQ_OK) return rc;
  }

  // Tile classes.  "Fast": full tiles of a step whose widths do not change (2..16 bits); they go to
  // the main kernel.  The rest (ragged last tile, width change, 32-bit state, other entry points)
  // goes to the generic kernel: narrow tiles first, wide (any 32-bit state) after.
  std::vector<uint32_t> nfast(L), nslow(L);
  std::vector<uint64_t> sig(L);
  uint64_t total = 0, fast = 0, slow_narrow = 0;
  for (int l = 0; l < L; ++l) {
    const stq_tensor& t = tensors[l];
    const uint64_t nt = (t.numel + stq::kTile - 1) / stq::kTile;
    const bool wide = row_is_wide(t, kind);
    // (the main kernel moves the scales with 16-byte bulk copies as well)
    // (a tensor whose widths change inside the step takes the main kernel's runtime-width body)
    const bool changes = t.bits_m != t.bits_m_out || t.bits_v != t.bits_v_out;
    const bool fast_ok = kind == kKindStep && !wide && !(t.v_log >= STQ_VLOG_SR && changes) &&
                         t.numel < (1ull << 32) && aligned(t.m_scales_in, 16) && aligned(t.v_scales_in, 16) &&
                         t.block >= 128 && t.block <= (uint32_t)stq::kFastMaxBlock;   // (one or two rows of a warp)
    const uint64_t nf = fast_ok ? t.numel / stq::kTile : 0;
    nfast[l] = (uint32_t)nf;
    nslow[l] = (uint32_t)(nt - nf);
    total += nt;
    fast += nf;
    if (!wide) slow_narrow += nt - nf;
    sig[l] = t.numel | (wide ? 1ull << 63 : 0ull) | (fast_ok ? 1ull << 62 : 0ull) |
             ((uint64_t)t.bits_m << 56) | ((uint64_t)t.bits_v << 48) |
             ((uint64_t)(t.v_log & 1u) << 47) | ((uint64_t)(t.v_log >> 1) << 45) |
             ((uint64_t)(t.bits_m != t.bits_m_out || t.bits_v != t.bits_v_out) << 46);   // numel <= 2^40
  }
  if (total > 0xFFFFFFF0ull) return STQ_E_NUMEL;
  // the tile map depends only on sizes and classes: skip it when unchanged
  const bool same_map = h->cached_kind >= 0 && sig == h->cached_sig && h->n_tiles == (uint32_t)total;
  // from here on the device image is being rewritten: a failure below must not leave the old table looking current
  h->cached_kind = -1;

  const size_t bytes_table = sizeof(TensorDesc) * (size_t)L;
  const size_t bytes_map = sizeof(uint32_t) * (size_t)total;
  const size_t off_map = (bytes_table + 255) & ~size_t(255);
  const size_t off_sched = (off_map + bytes_map + 255) & ~size_t(255);
  uint64_t n_seg = 0;
  for (int l = 0; l < L; ++l) n_seg += ((uint64_t)nfast[l] + nslow[l] + stq::kStatSegTiles - 1) / stq::kStatSegTiles;
  const size_t off_seg = (off_sched + 3 * sizeof(stq::FastSched) + 255) & ~size_t(255);
  int rc;
  if ((rc = grow_stage(h, off_seg + sizeof(uint32_t) * (size_t)n_seg)) != STQ_OK) return rc;
  if ((rc = grow(h, h->d_seg_map, h->d_seg_map_cap, (size_t)n_seg)) != STQ_OK) return rc;
  if ((rc = grow(h, h->d_table, h->d_table_cap, (size_t)L)) != STQ_OK) return rc;
  if ((rc = grow(h, h->d_tile_map, h->d_tile_cap, (size_t)total)) != STQ_OK) return rc;
  if (h->stage_busy) { STQ_CUDA(h, cudaEventSynchronize(h->stage_ev)); h->stage_busy = false; }

  uint8_t* st = static_cast<uint8_t*>(h->h_stage);
  TensorDesc* ht = reinterpret_cast<TensorDesc*>(st);
  uint32_t* hm = reinterpret_cast<uint32_t*>(st + off_map);
  // Fast tiles are laid out grouped by body (width pair, variant of the v code): the main kernel runs
  // one specialised body per group, and a change of body costs an instruction-cache refill on every
  // SM, so tensors that share a body are made neighbours in the tile order (at most 35 changes per
  // launch).  The order of the table itself is untouched.
  std::vector<int> order(L);
  for (int l = 0; l < L; ++l) order[l] = l;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    return body_key(tensors[a]) < body_key(tensors[b]);
  });
  std::vector<uint32_t> fast0(L);
  // three work lists: hs[0] for the fused bodies of the default and "pl" codes, hs[1] for the fused bodies of
  // the "sr" and "ts" codes (its own launch: its own register allocation), hs[2] (one group) for the tensors
  // that change width in this step
  stq::FastSched* hs = reinterpret_cast<stq::FastSched*>(st + off_sched);
  std::memset(hs, 0, 3 * sizeof(*hs));
  uint32_t list_begin[4] = {0, 0, 0, 0};
  {
    // groups of equal body, and an estimate of their cost for the initial spread of the CTAs
    // (relative cost per tile from measurement: 8- and 16-bit log codes and 3-bit packing cost more;
    // the estimate only decides where CTAs start, the balance itself is dynamic)
    double cost[2][stq::kFastMaxGroups] = {{0.0}, {0.0}};
    uint32_t next_fast = 0;
    int last_key = -1, cur = 0;
    for (int i = 0; i < L; ++i) {
      const int l = order[i];
      fast0[l] = next_fast;
      if (nfast[l] == 0) continue;
      const stq_tensor& t = tensors[l];
      const int key = body_key(t);
      const int list = key == kSplitKey ? 2 : key >= kVariantKey ? 1 : 0;     // (keys are sorted: lists follow one another)
      while (cur < list) list_begin[++cur] = next_fast;
      if (list < 2) {
        stq::FastSched* q = hs + list;
        if (key != last_key && q->ng < (uint32_t)stq::kFastMaxGroups) {
          q->grp_begin[q->ng++] = next_fast;
          last_key = key;
        }
        cost[list][q->ng - 1] += body_cost(t) * nfast[l];
      }
      if (!same_map)
        for (uint32_t k = 0; k < nfast[l]; ++k) hm[next_fast + k] = (uint32_t)l;
      next_fast += nfast[l];
    }
    while (cur < 3) list_begin[++cur] = next_fast;
    // chunk size: the usual one when every CTA gets several chunks, down to single tiles for small launches
    auto chunk_for = [&](uint64_t tiles) {
      const uint64_t per_cta = tiles / (uint64_t)std::max(1, h->fast_grid);
      return (uint32_t)std::min<uint64_t>(stq::kFastChunk, std::max<uint64_t>(1, per_cta / 4));
    };
    for (int list = 0; list < 3; ++list) hs[list].chunk = chunk_for(list_begin[list + 1] - list_begin[list]);
    hs[0].grp_begin[hs[0].ng] = list_begin[1];
    hs[1].grp_begin[hs[1].ng] = list_begin[2];
    hs[2].ng = 1;
    hs[2].grp_begin[0] = list_begin[2];
    hs[2].grp_begin[1] = list_begin[3];                   // (cta_group stays 0: every CTA starts in the one group)
    // CTAs per group in proportion to cost (largest remainders), at least one each
    const int G = h->fast_grid;
    for (int list = 0; list < 2; ++list) {
      stq::FastSched* q = hs + list;
      if (q->ng == 0) continue;
      double total_cost = 0.0;
      for (uint32_t g = 0; g < q->ng; ++g) total_cost += cost[list][g];
      std::vector<int> share(q->ng, 0);
      std::vector<std::pair<double, int>> rem;
      int given = 0;
      for (uint32_t g = 0; g < q->ng; ++g) {
        const double exact = total_cost > 0 ? cost[list][g] / total_cost * G : 0.0;
        share[g] = std::max(1, (int)exact);
        given += share[g];
        rem.push_back({exact - (int)exact, (int)g});
      }
      std::sort(rem.begin(), rem.end(), [](const std::pair<double, int>& a, const std::pair<double, int>& b) {
        return a.first > b.first;
      });
      for (size_t k = 0; given < G && !rem.empty(); ++k, ++given) share[rem[k % rem.size()].second]++;
      // Groups are ordered by v width, i.e. from memory-bound bodies to instruction-bound ones.  CTA c
      // and CTA c + (number of SMs) tend to share an SM, so the second wave is handed out in reverse:
      // an SM then hosts one CTA from either end, and the issue slots the memory-bound one leaves idle
      // serve the other.
      std::vector<uint16_t> glist;
      for (uint32_t g = 0; g < q->ng; ++g)
        for (int k = 0; k < share[g] && (int)glist.size() < G; ++k) glist.push_back((uint16_t)g);
      while ((int)glist.size() < G) glist.push_back((uint16_t)(glist.size() % q->ng));
      const int wave = std::min(G, h->sm_count);
      for (int c = 0; c < G; ++c) q->cta_group[c] = c < wave ? glist[c] : glist[G - 1 - (c - wave)];
    }
  }
  uint32_t next_narrow = (uint32_t)fast, next_wide = (uint32_t)(fast + slow_narrow);
  uint32_t* hseg = reinterpret_cast<uint32_t*>(st + off_seg);
  uint32_t next_seg = 0;
  for (int l = 0; l < L; ++l) {
    const stq_tensor& t = tensors[l];
    TensorDesc d;
    std::memset(&d, 0, sizeof(d));
    d.seg0 = next_seg;
    for (uint32_t k = 0; k < (nfast[l] + nslow[l] + stq::kStatSegTiles - 1) / stq::kStatSegTiles; ++k)
      hseg[next_seg++] = (uint32_t)l;
    d.tile0 = fast0[l];
    d.nfast = nfast[l];
    uint32_t& next = row_is_wide(t, kind) ? next_wide : next_narrow;
    d.tile0s = next;
    d.nslow = nslow[l];
    if (!same_map)
      for (uint32_t i = 0; i < nslow[l]; ++i) hm[next + i] = (uint32_t)l;
    next += nslow[l];
    d.param = t.param;
    d.grad = t.grad;
    d.mc_in = static_cast<const uint8_t*>(t.m_codes_in);
    d.ms_in = t.m_scales_in;
    d.vc_in = static_cast<const uint8_t*>(t.v_codes_in);
    d.vs_in = t.v_scales_in;
    d.mc_out = static_cast<uint8_t*>(t.m_codes_out);
    d.ms_out = t.m_scales_out;
    d.vc_out = static_cast<uint8_t*>(t.v_codes_out);
    d.vs_out = t.v_scales_out;
    d.numel = t.numel;
    d.block = kind == kKindStats ? 128u : t.block;
    d.bm_in = t.bits_m; d.bv_in = t.bits_v; d.bm_out = t.bits_m_out; d.bv_out = t.bits_v_out;
    d.wd = t.weight_decay;
    d.lp_dtype = kind == kKindStep ? t.lp_dtype : 0u;
    d.v_mode = kind != kKindStats ? t.v_log : 0u;
    d.sr_id = t.sr_id;
    d.param_lp = kind == kKindStep && t.lp_dtype != STQ_LP_NONE ? t.param_lp : nullptr;
    ht[l] = d;
  }
  STQ_CUDA(h, cudaMemcpyAsync(h->d_table, ht, bytes_table, cudaMemcpyHostToDevice, stream));
  if (!same_map)
    STQ_CUDA(h, cudaMemcpyAsync(h->d_tile_map, hm, bytes_map, cudaMemcpyHostToDevice, stream));
  STQ_CUDA(h, cudaMemcpyAsync(h->d_sched, hs, 3 * sizeof(stq::FastSched), cudaMemcpyHostToDevice, stream));
  if (!same_map)
    STQ_CUDA(h, cudaMemcpyAsync(h->d_seg_map, hseg, sizeof(uint32_t) * (size_t)n_seg, cudaMemcpyHostToDevice, stream));
  h->n_seg = (uint32_t)n_seg;
  STQ_CUDA(h, cudaEventRecord(h->stage_ev, stream));
  h->stage_busy = true;
  h->cached.assign(tensors, tensors + L);
  h->cached_kind = kind;
  h->cached_sig.swap(sig);
  h->any_lp = false;
  h->any_variant = false;
  for (int l = 0; l < L; ++l) h->any_variant = h->any_variant || (kind != kKindStats && tensors[l].v_log >= STQ_VLOG_SR);
  for (int l = 0; l < L; ++l) h->any_lp = h->any_lp || (kind == kKindStep && tensors[l].lp_dtype != STQ_LP_NONE);
  h->n_tiles = (uint32_t)total;
  h->n_fast = (uint32_t)fast;
  h->n_main = list_begin[1];
  h->n_var_end = list_begin[2];
  h->n_narrow = (uint32_t)(fast + slow_narrow);
  return STQ_OK;
}

int run(stq_handle* h, stq::Mode mode, int grad_dtype, bool stats, const stq::StepConsts& sc,
        cudaStream_t stream) {
  double* partials = nullptr;
  if (stats) {
    int rc = grow(h, h->d_partials, h->d_partials_cap, (size_t)h->n_tiles * 3 * (stq::kThreads / 32));
    if (rc != STQ_OK) return rc;
    partials = h->d_partials;
  }
  // The tiles of the generic kernel are independent of the main kernel's.  When a step has both, the
  // generic launches go to a side stream forked from the caller's and joined back into it, so that they
  // fill the SMs the persistent CTAs leave free at the ends of the main kernel instead of waiting for it.
  const bool both = h->n_fast > 0 && h->n_tiles > h->n_fast && h->side != nullptr;
  cudaStream_t gs = stream;
  if (both) {
    STQ_CUDA(h, cudaEventRecord(h->ev_fork, stream));
    STQ_CUDA(h, cudaStreamWaitEvent(h->side, h->ev_fork, 0));
    gs = h->side;
  }
  if (h->n_narrow > h->n_fast) {
    STQ_CUDA(h, stq::launch_tiles(mode, false, h->any_variant, grad_dtype, stats, h->d_table, h->d_tile_map, h->n_fast,
                                  h->n_narrow, sc, partials, h->grid, gs));
    h->launches++;
  }
  if (h->n_tiles > h->n_narrow) {
    STQ_CUDA(h, stq::launch_tiles(mode, true, h->any_variant, grad_dtype, stats, h->d_table, h->d_tile_map, h->n_narrow,
                                  h->n_tiles, sc, partials, h->grid, gs));
    h->launches++;
  }
  if (both) STQ_CUDA(h, cudaEventRecord(h->ev_join, h->side));
  if (h->n_main > 0) {   // only a step table has fast tiles
    const bool amp = h->any_lp || sc.inv_scale != nullptr || sc.dev_scalars != nullptr;
    STQ_CUDA(h, stq::launch_step_fast(grad_dtype, stats, amp, 0, h->d_table, h->d_tile_map, h->d_sched, sc,
                                      partials, h->d_err, h->fast_grid, stream));
    h->launches++;
  }
  if (h->n_var_end > h->n_main) {   // tensors whose second moment uses the "sr" or the "ts" code
    const int grid = (int)std::min<uint32_t>((uint32_t)h->fast_grid, h->n_var_end - h->n_main);
    STQ_CUDA(h, stq::launch_step_fast(grad_dtype, stats, true, 1, h->d_table, h->d_tile_map, h->d_sched + 1, sc,
                                      partials, h->d_err, grid, stream));
    h->launches++;
  }
  if (h->n_fast > h->n_var_end) {   // tensors that change width inside this step
    const int grid = (int)std::min<uint32_t>((uint32_t)h->fast_grid, h->n_fast - h->n_var_end);
    STQ_CUDA(h, stq::launch_step_fast(grad_dtype, stats, true, 2, h->d_table, h->d_tile_map, h->d_sched + 2, sc,
                                      partials, h->d_err, grid, stream));
    h->launches++;
  }
  if (both) STQ_CUDA(h, cudaStreamWaitEvent(stream, h->ev_join, 0));
  return STQ_OK;
}

int check_hparams(const stq_hparams* hp, unsigned flags) {
  if (!hp) return STQ_E_NULL;
  if (hp->step < 1) return STQ_E_ARG;
  if (hp->grad_dtype < STQ_GRAD_F32 || hp->grad_dtype > STQ_GRAD_F16) return STQ_E_ARG;
  if (flags & ~(unsigned)STQ_WITH_STATS) return STQ_E_ARG;
  if (!aligned(hp->inv_grad_scale, 4) || !aligned(hp->found_inf, 4)) return STQ_E_ALIGN;
  if (!aligned(hp->step_dev, 8) || !aligned(hp->lr_dev, 4)) return STQ_E_ALIGN;
  if (!(hp->beta1 >= 0.0 && hp->beta1 < 1.0 && hp->beta2 >= 0.0 && hp->beta2 < 1.0)) return STQ_E_ARG;
  return STQ_OK;
}

stq::StepConsts make_consts(const stq_hparams* hp) {
  stq::StepConsts sc;
  sc.b1 = (float)hp->beta1;
  sc.c1 = (float)(1.0 - hp->beta1);
  sc.b2 = (float)hp->beta2;
  sc.c2 = (float)(1.0 - hp->beta2);
  const double bc1 = 1.0 - std::pow(hp->beta1, (double)hp->step);
  const double bc2 = 1.0 - std::pow(hp->beta2, (double)hp->step);
  sc.step_size = (float)(hp->lr / bc1);
  sc.rsqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
  sc.eps = (float)hp->eps;
  sc.one = 1.0f;
  {   // stochastic rounding: the word every tensor's key is mixed from (seed and step; see include/stq.h)
    auto mix32 = [](uint32_t h) { h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16; return h; };
    const uint64_t step = (uint64_t)hp->step, seed = hp->sr_seed;
    uint32_t h = mix32((uint32_t)(step >> 32) ^ 0x9E3779B9u);
    h = mix32((uint32_t)step ^ h);
    h = mix32((uint32_t)(seed >> 32) ^ h);
    sc.sr_h = mix32((uint32_t)seed ^ h);
  }
  sc.l2_mode = hp->decoupled_wd ? 0 : 1;
  sc.lr = hp->lr;
  sc.inv_scale = hp->inv_grad_scale;
  sc.found_inf = hp->found_inf;
  sc.dev_scalars = nullptr;
  return sc;
}

}  // namespace

extern "C" {

int stq_create(stq_handle** out, int device) {
  if (!out) return STQ_E_NULL;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return STQ_E_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return STQ_E_CUDA;
  stq_handle* h = new (std::nothrow) stq_handle();
  if (!h) return STQ_E_WORKSPACE;
  h->device = device;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->stage_ev, cudaEventDisableTiming) != cudaSuccess) {
    delete h;
    return STQ_E_CUDA;
  }
  h->sm_count = prop.multiProcessorCount;
  h->grid = h->sm_count * stq::step_ctas_per_sm();
  h->fast_grid = h->sm_count * stq::fast_ctas_per_sm();
  if (h->fast_grid > stq::kFastMaxGrid) h->fast_grid = stq::kFastMaxGrid;
  if (cudaMalloc(reinterpret_cast<void**>(&h->d_err), 2 * sizeof(int)) != cudaSuccess ||
      cudaMemset(h->d_err, 0, 2 * sizeof(int)) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&h->d_scalars), 4 * sizeof(float)) != cudaSuccess ||
      cudaMalloc(reinterpret_cast<void**>(&h->d_sched), 3 * sizeof(stq::FastSched)) != cudaSuccess) {
    cudaEventDestroy(h->stage_ev);
    delete h;
    return STQ_E_WORKSPACE;
  }
  // (without the side stream everything simply runs in order on the caller's stream)
  if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess) {
    (void)cudaGetLastError();
    if (h->side) cudaStreamDestroy(h->side);
    h->side = nullptr;
  }
  *out = h;
  return STQ_OK;
}

int stq_destroy(stq_handle* h) {
  if (!h) return STQ_E_NULL;
  cudaSetDevice(h->device);
  if (h->stage_busy) cudaEventSynchronize(h->stage_ev);
  cudaFree(h->d_table);
  cudaFree(h->d_tile_map);
  cudaFree(h->d_err);
  cudaFree(h->d_sched);
  cudaFree(h->d_scalars);
  cudaFree(h->d_partials);
  cudaFree(h->d_stats);
  cudaFree(h->d_seg_map);
  cudaFree(h->d_seg_sums);
  cudaFree(h->d_arena);
  for (cudaStream_t st : h->host_streams)
    if (st) cudaStreamDestroy(st);
  for (cudaEvent_t e : h->host_events) cudaEventDestroy(e);
  if (h->h_stage) cudaFreeHost(h->h_stage);
  if (h->h_stats) cudaFreeHost(h->h_stats);
  if (h->stage_ev) cudaEventDestroy(h->stage_ev);
  if (h->side) cudaStreamDestroy(h->side);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  delete h;
  return STQ_OK;
}

size_t stq_codes_bytes(uint64_t numel, int bits) {
  const uint64_t by = (numel * (uint64_t)bits + 7) / 8;
  return (size_t)((by + 15) / 16 * 16);
}

size_t stq_scales_bytes(uint64_t numel, uint32_t block) {
  if (block == 0) return 0;
  return (size_t)((numel + block - 1) / block * 4);
}

size_t stq_v_scales_bytes(uint64_t numel, uint32_t block, uint32_t v_log) {
  return stq_scales_bytes(numel, block) * (v_log == STQ_VLOG_TS ? 2 : 1);
}

int stq_init_state(stq_handle* h, const stq_tensor* tensors, int L, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(h, tensors, L, kKindInit, s);
  if (rc != STQ_OK) return rc;
  stq::StepConsts sc;
  std::memset(&sc, 0, sizeof(sc));
  return run(h, stq::kInit, 0, false, sc, s);
}

int stq_step(stq_handle* h, const stq_tensor* tensors, int L, const stq_hparams* hp, unsigned flags,
             void* stream) {
  if (!h) return STQ_E_NULL;
  int rc = check_hparams(hp, flags);
  if (rc != STQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rc = prepare(h, tensors, L, kKindStep, s);
  if (rc != STQ_OK) return rc;
  const bool stats = (flags & STQ_WITH_STATS) != 0;
  stq::StepConsts sc = make_consts(hp);
  if (hp->step_dev != nullptr || hp->lr_dev != nullptr) {
    // step count and / or learning rate on the device: a one-thread kernel derives the step's scalars
    // ahead of the step kernels, which then read them instead of their launch parameters
    if (hp->step_dev == nullptr) return STQ_E_ARG;       // (a device learning rate comes with a device step count)
    for (int l = 0; l < L; ++l)                          // (the random words are keyed on the host's step count)
      if (tensors[l].v_log == STQ_VLOG_SR) return STQ_E_ARG;
    STQ_CUDA(h, stq::launch_step_scalars(reinterpret_cast<const long long*>(hp->step_dev), hp->lr_dev, hp->lr,
                                         hp->beta1, hp->beta2, h->d_scalars, s));
    h->launches++;
    sc.dev_scalars = h->d_scalars;
  }
  if (stats) {   // a step skipped through found_inf writes no partial sums: record whether this one will
    STQ_CUDA(h, stq::launch_stats_valid(hp->found_inf, h->d_err + 1, s));
    h->launches++;
  }
  rc = run(h, stq::kStep, hp->grad_dtype, stats, sc, s);
  if (rc == STQ_OK && stats) h->stats_L = L;
  return rc;
}

int stq_grad_stats(stq_handle* h, const stq_tensor* tensors, int L, int grad_dtype, void* stream) {
  if (!h) return STQ_E_NULL;
  if (grad_dtype < STQ_GRAD_F32 || grad_dtype > STQ_GRAD_F16) return STQ_E_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(h, tensors, L, kKindStats, s);
  if (rc != STQ_OK) return rc;
  stq::StepConsts sc;
  std::memset(&sc, 0, sizeof(sc));
  STQ_CUDA(h, stq::launch_stats_valid(nullptr, h->d_err + 1, s));
  h->launches++;
  rc = run(h, stq::kStatsOnly, grad_dtype, true, sc, s);
  if (rc == STQ_OK) h->stats_L = L;
  return rc;
}

int stq_layer_stats(stq_handle* h, double* out, int L, void* stream) {
  if (!h || !out) return STQ_E_NULL;
  if (h->stats_L <= 0 || L != h->stats_L) return STQ_E_STATE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  STQ_CUDA(h, cudaSetDevice(h->device));
  int rc = grow(h, h->d_stats, h->d_stats_cap, (size_t)L * 4);
  if (rc != STQ_OK) return rc;
  if ((size_t)L * 4 > h->h_stats_cap) {
    if (h->h_stats) cudaFreeHost(h->h_stats);
    h->h_stats = nullptr;
    h->h_stats_cap = 0;
    // (one more slot: the "statistics were produced" word travels with the sums)
    cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&h->h_stats), sizeof(double) * (4 * (size_t)L + 1));
    if (e != cudaSuccess) { h->cuda_err = cudaGetErrorString(e); return STQ_E_WORKSPACE; }
    h->h_stats_cap = (size_t)L * 4;
  }
  rc = grow(h, h->d_seg_sums, h->d_seg_sums_cap, (size_t)h->n_seg * 3);
  if (rc != STQ_OK) return rc;
  STQ_CUDA(h, stq::launch_stats_finish(h->d_table, L, h->d_seg_map, h->n_seg, h->d_partials, h->d_seg_sums,
                                       h->d_stats, s));
  h->launches += 2;
  STQ_CUDA(h, cudaMemcpyAsync(h->h_stats, h->d_stats, sizeof(double) * 4 * (size_t)L, cudaMemcpyDeviceToHost, s));
  int* h_valid = reinterpret_cast<int*>(h->h_stats + 4 * (size_t)L);
  STQ_CUDA(h, cudaMemcpyAsync(h_valid, h->d_err + 1, sizeof(int), cudaMemcpyDeviceToHost, s));
  STQ_CUDA(h, cudaStreamSynchronize(s));
  if (*h_valid == 0) {        // the step that was to carry the sums was skipped (found_inf): nothing to report
    h->stats_L = 0;
    return STQ_E_STATE;
  }
  std::memcpy(out, h->h_stats, sizeof(double) * 4 * (size_t)L);
  return STQ_OK;
}

int stq_device_status(stq_handle* h, void* stream) {
  if (!h) return STQ_E_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  STQ_CUDA(h, cudaSetDevice(h->device));
  int flag = 0;
  STQ_CUDA(h, cudaMemcpyAsync(&flag, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, s));
  STQ_CUDA(h, cudaStreamSynchronize(s));
  return flag ? STQ_E_TIMEOUT : STQ_OK;
}

int stq_repack(stq_handle* h, const stq_tensor* tensors, int L, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = prepare(h, tensors, L, kKindRepack, s);
  if (rc != STQ_OK) return rc;
  stq::StepConsts sc;
  std::memset(&sc, 0, sizeof(sc));
  return run(h, stq::kRepack, 0, false, sc, s);
}

int stq_step_host(stq_handle* h, const stq_tensor* tensors, int L, const stq_hparams* hp, unsigned flags,
                  uint64_t* bytes_h2d, uint64_t* bytes_d2h) {
  if (!h || !tensors) return STQ_E_NULL;
  int rc = check_hparams(hp, flags);
  if (rc != STQ_OK) return rc;
  if (L <= 0 || L > (1 << 20)) return STQ_E_NUMEL;
  STQ_CUDA(h, cudaSetDevice(h->device));
  // validate with the host pointers (same rules: alignment, widths, aliasing)
  for (int l = 0; l < L; ++l) {
    rc = validate_row(tensors[l], kKindStep);
    if (rc != STQ_OK) return rc;
  }
  // lay the device arena out: every buffer 256-byte aligned
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  const size_t gsz = hp->grad_dtype == STQ_GRAD_F32 ? 4 : 2;
  size_t need = 0;
  for (int l = 0; l < L; ++l) {
    const stq_tensor& t = tensors[l];
    const size_t sb = stq_scales_bytes(t.numel, t.block);
    need += up(t.numel * 4) + up(t.numel * gsz);
    need += up(stq_codes_bytes(t.numel, t.bits_m)) + up(stq_codes_bytes(t.numel, t.bits_v)) + up(sb) +
            up(stq_v_scales_bytes(t.numel, t.block, t.v_log));
    if (t.bits_m_out != t.bits_m) need += up(stq_codes_bytes(t.numel, t.bits_m_out));
    if (t.bits_v_out != t.bits_v) need += up(stq_codes_bytes(t.numel, t.bits_v_out));
    if (t.lp_dtype != STQ_LP_NONE) need += up(t.numel * 2);
    need += 6 * (4096 + 512);   // padding carried along when buffers travel as one run
  }
  if (hp->inv_grad_scale || hp->found_inf || hp->step_dev || hp->lr_dev)
    return STQ_E_ARG;   // device pointers have no place in the host-buffer call
  rc = grow(h, h->d_arena, h->d_arena_cap, need);
  if (rc != STQ_OK) return rc;

  // Chunks of consecutive tensors are pipelined over three streams: copies in, the step, copies out.
  // With pinned host buffers the two copy directions and the kernels overlap; pageable buffers make
  // the copies synchronous but stay correct.  A step with statistics needs one table, hence one chunk.
  if (!h->host_streams[0]) {
    for (int k = 0; k < 3; ++k) STQ_CUDA(h, cudaStreamCreateWithFlags(&h->host_streams[k], cudaStreamNonBlocking));
  }
  cudaStream_t s_in = h->host_streams[0], s_run = h->host_streams[1], s_out = h->host_streams[2];
  STQ_CUDA(h, cudaDeviceSynchronize());   // earlier work on other streams may still use the arena or the buffers
  std::vector<stq_tensor> dev(tensors, tensors + L);
  uint64_t h2d = 0, d2h = 0;
  size_t off = 0;
  auto place = [&](size_t bytes) { uint8_t* p = h->d_arena + off; off += up(bytes); return p; };
  const size_t chunk_bytes = (flags & STQ_WITH_STATS) ? ~size_t(0) : (size_t(256) << 20);
  size_t n_events = 0;
  auto next_event = [&](cudaEvent_t* ev) -> cudaError_t {
    if (n_events == h->host_events.size()) {
      cudaEvent_t e;
      cudaError_t rc2 = cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
      if (rc2 != cudaSuccess) return rc2;
      h->host_events.push_back(e);
    }
    *ev = h->host_events[n_events++];
    return cudaSuccess;
  };
  // Buffers of one kind (parameters, gradients, codes or scales of one state) that lie back to back in
  // host memory over the tensors of a chunk, with nothing but alignment padding between them, travel
  // as ONE copy into a device image of the whole run: under a concurrent copy in the other direction
  // every separate host-to-device copy costs tens of microseconds of start-up, which a table of
  // hundreds of tensors cannot afford.  Callers that keep each kind in one flat pinned buffer get this
  // path; separately allocated buffers (even when they happen to be neighbours) are copied one by one.
  constexpr size_t kMaxGap = 4096;
  struct Run { const uint8_t* lo; size_t len; uint8_t* dev; };
  enum { kParam, kGrad, kMc, kVc, kMs, kVs, kKinds };
  auto in_ptr = [&](const stq_tensor& t, int kind) -> const uint8_t* {
    switch (kind) {
      case kParam: return reinterpret_cast<const uint8_t*>(t.param);
      case kGrad: return static_cast<const uint8_t*>(t.grad);
      case kMc: return static_cast<const uint8_t*>(t.m_codes_in);
      case kVc: return static_cast<const uint8_t*>(t.v_codes_in);
      case kMs: return reinterpret_cast<const uint8_t*>(t.m_scales_in);
      default: return reinterpret_cast<const uint8_t*>(t.v_scales_in);
    }
  };
  auto in_size = [&](const stq_tensor& t, int kind) -> size_t {
    switch (kind) {
      case kParam: return t.numel * 4;
      case kGrad: return t.numel * gsz;
      case kMc: return stq_codes_bytes(t.numel, t.bits_m);
      case kVc: return stq_codes_bytes(t.numel, t.bits_v);
      case kMs: return t.bits_m != 32 ? stq_scales_bytes(t.numel, t.block) : 0;
      default: return t.bits_v != 32 ? stq_v_scales_bytes(t.numel, t.block, t.v_log) : 0;
    }
  };
  // the run of kind `kind` over tensors [a, b), or len 0 if the buffers do not lie back to back
  auto find_run = [&](int a, int b, int kind) -> Run {
    Run r{nullptr, 0, nullptr};
    if (b - a < 2) return r;
    const uint8_t* end = nullptr;
    for (int l = a; l < b; ++l) {
      const uint8_t* p = in_ptr(tensors[l], kind);
      const size_t n = in_size(tensors[l], kind);
      if (!p || n == 0) return r;
      if (l == a) r.lo = p;
      else if (p < end || (size_t)(p - end) > kMaxGap) return r;
      end = p + n;
    }
    r.len = (size_t)(end - r.lo);
    if (!one_allocation(r.lo, r.len)) r.len = 0;
    return r;
  };
  int a = 0;
  while (a < L) {
    // ---- the chunk: consecutive tensors up to the byte budget ----
    size_t moved = 0;
    int b = a;
    for (; b < L && (b == a || moved < chunk_bytes); ++b)
      for (int k = 0; k < kKinds; ++k) moved += in_size(tensors[b], k);
    // ---- copies in (stream s_in) ----
    Run run[kKinds];
    for (int k = 0; k < kKinds; ++k) {
      run[k] = find_run(a, b, k);
      if (run[k].len) {
        // the image keeps the host run's offset inside a 256-byte line, so every buffer keeps its alignment
        uint8_t* base = place(run[k].len + 256);
        run[k].dev = base + (reinterpret_cast<uintptr_t>(run[k].lo) & 255u);
        STQ_CUDA(h, cudaMemcpyAsync(run[k].dev, run[k].lo, run[k].len, cudaMemcpyHostToDevice, s_in));
        h2d += run[k].len;
      }
    }
    auto dev_in = [&](const stq_tensor& t, int kind, size_t always_bytes) -> uint8_t* {
      const size_t n = in_size(t, kind);
      if (run[kind].len) return run[kind].dev + (in_ptr(t, kind) - run[kind].lo);
      uint8_t* p = place(n ? n : always_bytes);
      if (n) {
        cudaError_t e = cudaMemcpyAsync(p, in_ptr(t, kind), n, cudaMemcpyHostToDevice, s_in);
        if (e != cudaSuccess) { h->cuda_err = cudaGetErrorString(e); return nullptr; }
        h2d += n;
      }
      return p;
    };
    // which outputs may go back as one copy of the run they came in with: written in place on the host too
    bool out_run[kKinds];
    for (int k = 0; k < kKinds; ++k) out_run[k] = run[k].len != 0;
    out_run[kGrad] = false;
    for (int l = a; l < b; ++l) {
      const stq_tensor& t = tensors[l];
      if (t.bits_m_out != t.bits_m || t.m_codes_out != t.m_codes_in) out_run[kMc] = false;
      if (t.bits_v_out != t.bits_v || t.v_codes_out != t.v_codes_in) out_run[kVc] = false;
      if (t.bits_m_out == 32 || t.m_scales_out != t.m_scales_in) out_run[kMs] = false;
      if (t.bits_v_out == 32 || t.v_scales_out != t.v_scales_in) out_run[kVs] = false;
    }
    for (int l = a; l < b; ++l) {
      const stq_tensor& t = tensors[l];
      stq_tensor& d = dev[l];
      const size_t sb = stq_scales_bytes(t.numel, t.block);
      d.param = reinterpret_cast<float*>(dev_in(t, kParam, 0));
      d.grad = dev_in(t, kGrad, 0);
      d.m_codes_in = dev_in(t, kMc, 0);
      d.v_codes_in = dev_in(t, kVc, 0);
      d.m_scales_in = reinterpret_cast<float*>(dev_in(t, kMs, sb));   // placed even at 32 bits: the step may write scales
      d.v_scales_in = reinterpret_cast<float*>(dev_in(t, kVs, stq_v_scales_bytes(t.numel, t.block, t.v_log)));
      if (!d.param || !d.grad || !d.m_codes_in || !d.v_codes_in || !d.m_scales_in || !d.v_scales_in) {
        cudaDeviceSynchronize();
        return STQ_E_CUDA;
      }
      d.m_codes_out = t.bits_m_out != t.bits_m ? place(stq_codes_bytes(t.numel, t.bits_m_out))
                                               : const_cast<void*>(d.m_codes_in);
      d.v_codes_out = t.bits_v_out != t.bits_v ? place(stq_codes_bytes(t.numel, t.bits_v_out))
                                               : const_cast<void*>(d.v_codes_in);
      d.m_scales_out = const_cast<float*>(d.m_scales_in);
      d.v_scales_out = const_cast<float*>(d.v_scales_in);
      if (t.lp_dtype != STQ_LP_NONE) d.param_lp = place(t.numel * 2);
    }
    cudaEvent_t ev_in, ev_run;
    STQ_CUDA(h, next_event(&ev_in));
    STQ_CUDA(h, next_event(&ev_run));
    STQ_CUDA(h, cudaEventRecord(ev_in, s_in));
    // ---- the step on this chunk (stream s_run) ----
    STQ_CUDA(h, cudaStreamWaitEvent(s_run, ev_in, 0));
    rc = stq_step(h, dev.data() + a, b - a, hp, flags, s_run);
    if (rc != STQ_OK) { cudaDeviceSynchronize(); return rc; }
    STQ_CUDA(h, cudaEventRecord(ev_run, s_run));
    // ---- copies out (stream s_out) ----
    STQ_CUDA(h, cudaStreamWaitEvent(s_out, ev_run, 0));
    for (int k = 0; k < kKinds; ++k) {
      if (!out_run[k]) continue;
      // (the padding between the buffers goes back as it came)
      STQ_CUDA(h, cudaMemcpyAsync(const_cast<uint8_t*>(run[k].lo), run[k].dev, run[k].len, cudaMemcpyDeviceToHost, s_out));
      d2h += run[k].len;
    }
    for (int l = a; l < b; ++l) {
      const stq_tensor& t = tensors[l];
      const stq_tensor& d = dev[l];
      const size_t sb = stq_scales_bytes(t.numel, t.block);
      const size_t mo = stq_codes_bytes(t.numel, t.bits_m_out), vo = stq_codes_bytes(t.numel, t.bits_v_out);
      if (!out_run[kParam]) {
        STQ_CUDA(h, cudaMemcpyAsync(t.param, d.param, t.numel * 4, cudaMemcpyDeviceToHost, s_out));
        d2h += t.numel * 4;
      }
      if (!out_run[kMc]) {
        STQ_CUDA(h, cudaMemcpyAsync(t.m_codes_out, d.m_codes_out, mo, cudaMemcpyDeviceToHost, s_out));
        d2h += mo;
      }
      if (!out_run[kVc]) {
        STQ_CUDA(h, cudaMemcpyAsync(t.v_codes_out, d.v_codes_out, vo, cudaMemcpyDeviceToHost, s_out));
        d2h += vo;
      }
      if (t.lp_dtype != STQ_LP_NONE) {
        STQ_CUDA(h, cudaMemcpyAsync(t.param_lp, d.param_lp, t.numel * 2, cudaMemcpyDeviceToHost, s_out));
        d2h += t.numel * 2;
      }
      if (t.bits_m_out != 32 && !out_run[kMs]) {
        STQ_CUDA(h, cudaMemcpyAsync(t.m_scales_out, d.m_scales_out, sb, cudaMemcpyDeviceToHost, s_out));
        d2h += sb;
      }
      if (t.bits_v_out != 32 && !out_run[kVs]) {
        const size_t sbv = stq_v_scales_bytes(t.numel, t.block, t.v_log);
        STQ_CUDA(h, cudaMemcpyAsync(t.v_scales_out, d.v_scales_out, sbv, cudaMemcpyDeviceToHost, s_out));
        d2h += sbv;
      }
    }
    a = b;
  }
  STQ_CUDA(h, cudaStreamSynchronize(s_out));
  STQ_CUDA(h, cudaStreamSynchronize(s_run));
  // the cached table now refers to arena addresses; drop it so a later device call re-uploads
  h->cached_kind = -1;
  if (bytes_h2d) *bytes_h2d = h2d;
  if (bytes_d2h) *bytes_d2h = d2h;
  return STQ_OK;
}

int stq_selftest_wait_timeout(stq_handle* h, void* stream) {
  if (!h) return STQ_E_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  STQ_CUDA(h, cudaSetDevice(h->device));
  STQ_CUDA(h, stq::launch_wait_timeout_selftest(h->d_err, s));
  h->launches++;
  return STQ_OK;
}

uint64_t stq_launch_count(const stq_handle* h) { return h ? h->launches : 0; }
int stq_grid_size(const stq_handle* h) { return h ? h->fast_grid : 0; }
int stq_sm_count(const stq_handle* h) { return h ? h->sm_count : 0; }

const char* stq_strerror(int code) {
  switch (code) {
    case STQ_OK: return "ok";
    case STQ_E_NULL: return "a required pointer is NULL";
    case STQ_E_BITS: return "bit-width not in {2,3,4,8,16,32}";
    case STQ_E_BLOCK: return "block is not a power of two in 32..1024";
    case STQ_E_ALIGN: return "buffer not aligned (16 bytes for param/grad/codes, 4 for scales)";
    case STQ_E_ALIAS: return "in/out buffers overlap (in-place needs the same pointer and width)";
    case STQ_E_NUMEL: return "numel is 0, or the table is empty or too large";
    case STQ_E_CUDA: return "CUDA runtime error";
    case STQ_E_WORKSPACE: return "could not allocate library workspace";
    case STQ_E_ARG: return "invalid scalar argument";
    case STQ_E_STATE: return "no statistics pending for this table (none requested, another table since, or the step was skipped)";
    case STQ_E_TIMEOUT: return "a bounded wait inside a kernel ran out (results of that launch are invalid)";
    case STQ_E_TOO_LARGE: return "tensor larger than the fixed capacity of this non-allocating entry point";
    default: return "unknown error";
  }
}

const char* stq_last_cuda_error(const stq_handle* h) { return h ? h->cuda_err.c_str() : ""; }

}  // extern "C"
