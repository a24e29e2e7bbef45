// Host side of the C ABI: argument checks, the registry of packed buffers, path selection.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "lqer_common.cuh"

namespace lqer {

static std::atomic<unsigned long long> g_launches{0};

// Optional per-family kernel timing: pairs of events recorded around each launch while enabled.
struct TimedLaunch { int family; int n_kernels; cudaEvent_t start, stop; };
static std::mutex g_prof_mu;
static std::atomic<int> g_prof_on{0};
static std::vector<TimedLaunch> g_prof_records;
static std::vector<cudaEvent_t> g_prof_free;

static cudaEvent_t prof_event() {
  if (!g_prof_free.empty()) { cudaEvent_t e = g_prof_free.back(); g_prof_free.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}

LaunchScope::LaunchScope(int family, cudaStream_t s, int n_kernels) : stream_(s), stop_(nullptr) {
  g_launches.fetch_add((unsigned long long)n_kernels, std::memory_order_relaxed);
  if (g_prof_on.load(std::memory_order_relaxed) == 0) return;
  std::lock_guard<std::mutex> lock(g_prof_mu);
  TimedLaunch r{family, n_kernels, prof_event(), prof_event()};
  if (r.start == nullptr || r.stop == nullptr) return;
  cudaEventRecord(r.start, s);
  stop_ = r.stop;
  g_prof_records.push_back(r);
}
LaunchScope::~LaunchScope() {
  if (stop_ != nullptr) cudaEventRecord(stop_, stream_);
}

static std::mutex g_mu;
static std::unordered_map<const void*, PackedMeta> g_registry;
static std::atomic<int> g_path{0};
static std::atomic<long long> g_wait_limit{4000000000LL};      // about two seconds of SM clock
static std::atomic<int> g_stall_family{-1};

long long wait_limit_cycles() { return g_wait_limit.load(std::memory_order_relaxed); }
static std::atomic<size_t> g_y_shrink{0};                      // checked build only: see lqer_debug_bounds_shrink
size_t debug_y_shrink() { return g_y_shrink.load(std::memory_order_relaxed); }

bool take_stall(int family) {
  int want = family;
  return g_stall_family.compare_exchange_strong(want, -1);
}

int sm_count() {
  static std::mutex mu;
  static int count_of[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  std::lock_guard<std::mutex> lock(mu);
  if (count_of[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    count_of[dev] = n;
  }
  return count_of[dev];
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static lqer_status_t check_config(const lqer_config_t* cfg) {
  if (cfg == nullptr) return LQER_ERR_NULL;
  // activations (and T) take 3 to 8 mantissa bits (Section 4.3 compares W4A8 and W4A6); weights 4 or 2 (Section 4.4: W2A8)
  if ((cfg->w_bits != 4 && cfg->w_bits != 2) || cfg->a_bits < 3 || cfg->a_bits > 8 || cfg->lr_bits != 8 || cfg->block != 16) return LQER_ERR_CONFIG;
  // every dequantised value must be a normal bf16 and every product a normal fp32
  if (cfg->exp_min < -56 || cfg->exp_max > 55 || cfg->exp_min > cfg->exp_max) return LQER_ERR_CONFIG;
  if (cfg->w_exp_min < -56 || cfg->w_exp_max > 55 || cfg->w_exp_min > cfg->w_exp_max) return LQER_ERR_CONFIG;
  if (cfg->deterministic != 0 && cfg->deterministic != 1) return LQER_ERR_CONFIG;
  return LQER_OK;
}

static lqer_status_t check_shape(int K, int N, int k) {
  if (K <= 0 || N <= 0 || k < 0) return LQER_ERR_SHAPE;
  if (K % 16 != 0 || N % 8 != 0) return LQER_ERR_SHAPE;
  if (k > 256 || k > K || k > N) return LQER_ERR_SHAPE;
  if ((long long)K > (1 << 20) || (long long)N > (1 << 22)) return LQER_ERR_SHAPE;
  return LQER_OK;
}

static void fill_meta(PackedMeta& m, int K, int N, int k, const lqer_config_t& c) {
  std::memset(&m, 0, sizeof(m));
  m.magic = kMagic; m.version = kVersion;
  m.K = K; m.N = N; m.k = k; m.k_pad = (k + 15) / 16 * 16;
  m.K64 = (K + 63) / 64 * 64;
  m.n_tiles = (N + kTileN - 1) / kTileN;
  m.k_slabs = m.K64 / kSlabK;
  m.r_blocks = m.k_pad / 16;
  m.w_bits = c.w_bits; m.a_bits = c.a_bits; m.lr_bits = c.lr_bits; m.block = c.block;
  m.exp_min = c.exp_min; m.exp_max = c.exp_max; m.deterministic = 1;
  m.w_exp_min = c.w_exp_min; m.w_exp_max = c.w_exp_max;
  m.off_w = kHeaderBytes;
  m.off_b = align_up(m.off_w + (size_t)m.n_tiles * m.k_slabs * w_tile_bytes(m.w_bits), 256);
  m.off_a = align_up(m.off_b + (size_t)m.n_tiles * b_tile_bytes(m), 256);
  m.total_bytes = align_up(m.off_a + (size_t)(K / 16) * m.k_pad * 17, 256);
  m.checksum = meta_checksum(m);
}

static bool meta_valid(const PackedMeta& m) {
  if (m.magic != kMagic || m.version != kVersion || m.checksum != meta_checksum(m)) return false;
  lqer_config_t c{m.w_bits, m.a_bits, m.lr_bits, m.block, m.exp_min, m.exp_max, m.deterministic, m.w_exp_min, m.w_exp_max};
  if (check_config(&c) != LQER_OK || check_shape(m.K, m.N, m.k) != LQER_OK) return false;
  PackedMeta ref;
  fill_meta(ref, m.K, m.N, m.k, c);
  return std::memcmp(&ref, &m, sizeof(m)) == 0;
}

// The shape and formats of a packed buffer live in its 256-byte header.  The host keeps a copy per buffer address so
// that a call costs no device read; a buffer the host has not seen yet (one that was copied to a new address, or
// loaded from a file) has its header read back from the device once, checked, and remembered.  That first call
// synchronises with the device (cudaMemcpy); lqer_attach_packed does the same ahead of time.
static lqer_status_t lookup(const void* packed, PackedMeta& out) {
  if (packed == nullptr) return LQER_ERR_NULL;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_registry.find(packed);
    if (it != g_registry.end()) { out = it->second; return LQER_OK; }
  }
  if ((reinterpret_cast<uintptr_t>(packed) & 255u) != 0) return LQER_ERR_BAD_PACKED;
  cudaPointerAttributes pa;
  if (cudaPointerGetAttributes(&pa, packed) != cudaSuccess) { cudaGetLastError(); return LQER_ERR_BAD_PACKED; }
  if (pa.type != cudaMemoryTypeDevice && pa.type != cudaMemoryTypeManaged) return LQER_ERR_BAD_PACKED;
  PackedMeta m;
  if (cudaMemcpy(&m, packed, sizeof(m), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return LQER_ERR_BAD_PACKED; }
  if (!meta_valid(m)) return LQER_ERR_BAD_PACKED;
  std::lock_guard<std::mutex> lock(g_mu);
  g_registry[packed] = m;
  out = m;
  return LQER_OK;
}

static lqer_status_t check_arch() {
  static std::mutex mu;
  static std::unordered_map<int, int> major_of;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LQER_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  auto it = major_of.find(dev);
  if (it == major_of.end()) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return LQER_ERR_CUDA;
    it = major_of.emplace(dev, major).first;
  }
  return it->second == 10 ? LQER_OK : LQER_ERR_ARCH;
}

static size_t xcat_bytes(const PackedMeta& m, int M) { return align_up((size_t)M * xcat_cols(m) * 2, 256); }
// Scratch of one small-batch call behind the head: Xcat, the prologue's partial sums of T, the GEMM's partial sums of Y.
// The activations of a small-batch call: Xcat, or (register-operand GEMM) the fragment order of 16 rows.
static size_t small_xcat_bytes(const PackedMeta& m, int M) {
  const size_t a = xcat_bytes(m, M), b = small_takes_mma(m, M) ? align_up(frag_bytes(m), 256) : 0;
  return a > b ? a : b;
}
static size_t small_slice_bytes(const PackedMeta& m, int M) {
  return small_xcat_bytes(m, M) + align_up(prologue_small_slot_bytes(m, M), 256) + align_up(small_gemm_partial_bytes(m, M), 256);
}
// A call of up to kSmallMaxM rows runs the column-owner decode kernel (M <= 4 where the layer fits it) or the small
// prologue and the small-batch GEMM; either finds its scratch behind the head.
static size_t small_bytes(const PackedMeta& m, int M) {
  const size_t a = small_slice_bytes(m, M), b = decode_cols_slot_bytes(m);
  return a > b ? a : b;
}
// Bytes a call with M rows needs: the persistent head plus the scratch of the path it takes.
static size_t call_bytes(const PackedMeta& m, int M, bool small) {
  return align_up(persist_bytes(m), 256) +
         (small ? small_bytes(m, M)
                : xcat_bytes(m, M) + align_up(prologue_tc_scratch_bytes(m, M), 256) + gemm_splitk_bytes(m, M));
}
// Whether a call with M rows takes the small-batch kernels under the current path setting.
static bool takes_small_path(int path, int M) {
  return (path == 0 || path == 2 || path == 5 || path == 7) && M <= kSmallMaxM;
}
// The same for a registered packed buffer, on the path lqer_linear_stream takes for M rows right now.
lqer_status_t call_workspace_bytes(const void* packed, int M, size_t* bytes) {
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  if (M <= 0 || M > (1 << 24)) return LQER_ERR_SHAPE;
  *bytes = call_bytes(m, M, takes_small_path(g_path.load(), M));
  return LQER_OK;
}
// Bytes that fit every call of up to M_max rows, whichever path it takes.
static size_t workspace_total(const PackedMeta& m, int M_max) {
  const size_t a = xcat_bytes(m, M_max) + align_up(prologue_tc_scratch_bound(m, M_max), 256) + gemm_splitk_bound(m, M_max);
  const size_t b = small_bytes(m, M_max < kSmallMaxM ? M_max : kSmallMaxM);
  return align_up(persist_bytes(m), 256) + (a > b ? a : b);
}

// Element types of X and Y (Section 2.1: the layer sits between 16-bit activations in the w-only setting).
struct IoTypes {
  int x_type = kXF32;          // kXF32, kXBF16 or kXMXINT8
  int y_type = kYF32;          // kYF32, kYBF16 or kYMXINT8
};

// n small-batch layers with one M (n == 1: a single call): one launch of the small prologue for all of them, then one
// launch of the GEMM over the work items of all of them.  Layer g finds its scratch at slices[g], its tile counters
// at tile_counts[g] and its row-group counters at row_counts[g].
static cudaError_t run_small(const lqer_call_t* calls, const PackedMeta* metas, int n, uint8_t* const* slices,
                             int* const* tile_counts, int* const* row_counts, DeviceStatus* dst, IoTypes io,
                             int8_t* Tm, uint8_t* Te, bool project_only, cudaStream_t s) {
  const int M = calls[0].M;
  SmallPrologueLayer pl[16];
  SmallGemmLayer gl[16];
  for (int g = 0; g < n; ++g) {
    const PackedMeta& m = metas[g];
    uint8_t* xcat = slices[g];
    uint8_t* slots = xcat + small_xcat_bytes(m, M);
    uint8_t* partials = slots + align_up(prologue_small_slot_bytes(m, M), 256);
    int* flags = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(dst) + kFlagAreaOffset) + 2 * g;
    pl[g] = SmallPrologueLayer{calls[g].X, calls[g].packed, &metas[g], xcat, reinterpret_cast<double*>(slots), row_counts[g],
                               n == 1 ? Tm : nullptr, n == 1 ? Te : nullptr, flags};
    gl[g] = SmallGemmLayer{xcat, calls[g].packed, &metas[g], calls[g].Y, reinterpret_cast<float*>(partials), tile_counts[g], flags};
  }
  // a number for the flags of this pair of launches that no earlier pair on any workspace used (never zero)
  static std::atomic<unsigned> epochs{0};
  const int epoch = (int)(epochs.fetch_add(1) & 0x3FFFFFFFu) + 1;
  // the register-operand GEMM reads the activations in fragment order and follows the prologue's flags
  // (a call on its own is a chain of latencies that the tensor-memory kernel gets through sooner: measured 23.6 against
  // 26.6 us on a 4096 x 4096 layer; the register-operand kernel serves launches that several layers share, and single
  // calls where path 5 is forced)
  const int path = g_path.load();
  const bool tmem_form = path == 7 || ((path == 0 || path == 2) && n == 1);
  const bool frag = !project_only && !tmem_form && small_takes_mma(metas[0], M);
  cudaError_t err = launch_prologue_small(pl, n, M, io.x_type, frag, epoch, dst, s);
  if (err == cudaSuccess && !project_only) err = launch_gemm_small(gl, n, M, io.y_type, tmem_form, epoch, dst, s);
  return err;
}

static lqer_status_t run_linear(const void* X, int M, const void* packed, void* Y, void* workspace,
                                size_t workspace_bytes, cudaStream_t s, int8_t* Tm, uint8_t* Te, bool project_only,
                                IoTypes io = IoTypes()) {
  if (X == nullptr || packed == nullptr || workspace == nullptr || (Y == nullptr && !project_only)) return LQER_ERR_NULL;
  if (M <= 0 || M > (1 << 24)) return LQER_ERR_SHAPE;
  if (!aligned16(X) || (Y != nullptr && !aligned16(Y)) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return LQER_ERR_ALIGN;
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  if (io.y_type == kYMXINT8 && m.N % 16 != 0) return LQER_ERR_SHAPE;     // whole 16-blocks of Y along N
  int path = g_path.load();
  if ((path == 2 || path == 5 || path == 7) && M > kSmallMaxM) return LQER_ERR_SHAPE;
  const bool small = takes_small_path(path, M);
  if (project_only && !small) path = 3;
  // Paths 1 and 3 keep the SIMT-style prologue at every batch size; the others take the tensor-core one where it fits.
  const bool tc_prologue = path != 1 && path != 3 && prologue_tc_fits(m, M, X, path == 6);
  if (path == 6) path = 4;
  if (workspace_bytes < call_bytes(m, M, small)) return LQER_ERR_BUFFER_TOO_SMALL;
  if ((st = check_arch()) != LQER_OK) return st;
  DeviceStatus* dst = static_cast<DeviceStatus*>(workspace);
  uint8_t* wsb = static_cast<uint8_t*>(workspace);
  void* xcat = wsb + align_up(persist_bytes(m), 256);
  cudaError_t err;
  if (small) {
    if (path != 5 && path != 7 && !project_only && decode_cols_fits(m, M)) {
      err = launch_decode_cols(X, io.x_type, M, m, packed, Y, io.y_type, workspace, s);
    } else {
      const lqer_call_t one = {static_cast<const float*>(X), M, packed, static_cast<float*>(Y)};
      uint8_t* slice = static_cast<uint8_t*>(xcat);
      int* tiles = reinterpret_cast<int*>(wsb + kStatusBytes);
      int* rows = reinterpret_cast<int*>(wsb + pcount_offset(m));
      err = run_small(&one, &m, 1, &slice, &tiles, &rows, dst, io, Tm, Te, project_only, s);
    }
  } else {
    if (path == 1 && (M > 65535 || io.y_type != kYF32)) return LQER_ERR_SHAPE;   // the checking kernel writes fp32 only
    err = tc_prologue ? launch_prologue_tc(X, io.x_type, M, m, packed, xcat, Tm, Te, dst,
                                           reinterpret_cast<double*>(static_cast<uint8_t*>(xcat) + xcat_bytes(m, M)),
                                           reinterpret_cast<int*>(wsb + pcount_offset(m)), kChainAlone, s)
                      : launch_prologue(X, io.x_type, M, m, packed, xcat, Tm, Te, dst, s);
    if (err == cudaSuccess && !project_only)
      err = (path == 1) ? launch_gemm_simt(xcat, M, m, packed, static_cast<float*>(Y), s)
                        : launch_gemm_tc2_splitk(xcat, M, m, packed, Y, io.y_type,
                                                 reinterpret_cast<float*>(static_cast<uint8_t*>(xcat) + xcat_bytes(m, M) +
                                                                          align_up(prologue_tc_scratch_bytes(m, M), 256)),
                                                 dst, s);
  }
  return err == cudaSuccess ? LQER_OK : LQER_ERR_CUDA;
}

// Scratch one layer of a grouped prefill launch needs: its own Xcat and its own prologue partial sums.
static size_t group_slice_bytes(const PackedMeta& m, int M) {
  return xcat_bytes(m, M) + align_up(prologue_tc_scratch_bytes(m, M), 256);
}
// Consecutive prefill calls from `first` on that may share a GEMM launch with it (auto path only): the same M > 256,
// the same formats, any shapes; at most `limit`, and only as many as the workspace has slices for.
static bool same_formats(const PackedMeta& a, const PackedMeta& b) {
  return a.w_bits == b.w_bits && a.a_bits == b.a_bits && a.lr_bits == b.lr_bits && a.exp_min == b.exp_min &&
         a.exp_max == b.exp_max && a.block == b.block;
}
static int prefill_run(const lqer_call_t* calls, int first, int n_calls, int limit, size_t workspace_bytes,
                       PackedMeta* metas, size_t* need) {
  const int M = calls[first].M;
  size_t head = 0, slices = 0;
  int n = 0;
  while (first + n < n_calls && n < limit) {
    PackedMeta m;
    if (calls[first + n].M != M || lookup(calls[first + n].packed, m) != LQER_OK) break;
    if (n > 0 && !same_formats(metas[0], m)) break;
    const size_t h = std::max(head, align_up(persist_bytes(m), 256));
    const size_t sl = slices + group_slice_bytes(m, M);
    if (n > 0 && h + sl > workspace_bytes) break;
    metas[n] = m; head = h; slices = sl;
    ++n;
  }
  if (need != nullptr) *need = head + slices;
  return n;
}
// Consecutive small-batch calls from `first` on that may share the two launches of the small-batch path (auto path only):
// the same M <= kSmallMaxM, the same formats, any shapes, none of them served by the column-owner decode kernel; at most
// `limit`, only as many as the workspace has slices for, and tile counters for.
constexpr size_t kGroupRowCountOffset = 256 + 32768 * 4 + 16 * 256 * 8;   // the row-tile counter area at its highest position
static int small_run(const lqer_call_t* calls, int first, int n_calls, int limit, size_t workspace_bytes, bool cols_ok,
                     PackedMeta* metas, size_t* need) {
  const int M = calls[first].M;
  const size_t head = align_up(kPersistMaxBytes, 256);
  size_t slices = 0;
  int n = 0, tiles = 0;
  while (first + n < n_calls && n < limit) {
    PackedMeta m;
    if (calls[first + n].M != M || lookup(calls[first + n].packed, m) != LQER_OK || (cols_ok && decode_cols_fits(m, M))) break;
    if (n > 0 && !same_formats(metas[0], m)) break;
    if (tiles + m.n_tiles > 32768) break;
    const size_t sl = slices + small_slice_bytes(m, M);
    if (n > 0 && head + sl > workspace_bytes) break;
    metas[n] = m; slices = sl; tiles += m.n_tiles;
    ++n;
  }
  if (need != nullptr) *need = head + slices;
  return n;
}
static lqer_status_t run_small_group(const lqer_call_t* calls, int n, const PackedMeta* metas, void* workspace, IoTypes io,
                                     cudaStream_t s) {
  uint8_t* wsb = static_cast<uint8_t*>(workspace);
  uint8_t* slices[16];
  int* tile_counts[16];
  int* row_counts[16];
  size_t off = align_up(kPersistMaxBytes, 256);
  int tiles = 0;
  for (int g = 0; g < n; ++g) {
    slices[g] = wsb + off;
    off += small_slice_bytes(metas[g], calls[0].M);
    tile_counts[g] = reinterpret_cast<int*>(wsb + kStatusBytes) + tiles;
    tiles += metas[g].n_tiles;
    row_counts[g] = reinterpret_cast<int*>(wsb + kGroupRowCountOffset) + 8 * g;
  }
  return run_small(calls, metas, n, slices, tile_counts, row_counts, static_cast<DeviceStatus*>(workspace), io, nullptr,
                   nullptr, false, s) == cudaSuccess ? LQER_OK : LQER_ERR_CUDA;
}
// Three or four rows in many layers at once: the register-operand GEMM's launches take less per layer than the
// column-owner kernel's (measured on 4096 x 4096 layers: from 6 layers on at 4 rows, 5.7 against 6.9 us, and from 12 on
// at 3 rows, 4.4 against 4.6 us; with fewer layers the column-owner kernel's shorter chain wins).  The length of such
// a run from calls[first] on, or 0.
static int many_small_rows(const lqer_call_t* calls, int first, int n_calls, size_t workspace_bytes, const PackedMeta& m0,
                           PackedMeta* metas, size_t* need) {
  const int M = calls[first].M;
  if (M < 3 || m0.w_bits != 4 || !decode_cols_fits(m0, M) || !small_takes_mma(m0, M)) return 0;     // measured on 4-bit weights only
  const int lim = std::min(gemm_small_max_layers(), prologue_small_max_layers());
  const int n = small_run(calls, first, n_calls, lim, workspace_bytes, false, metas, need);
  return n >= (M == 4 ? 6 : 12) ? n : 0;
}
// The run of decode calls from calls[first] on that may share one launch of the column-owner kernel: one M, one set of
// formats, each fitting the kernel, at least 32 columns, and a slot for each layer's partial sums of T in the workspace.
static int decode_run(const lqer_call_t* calls, int first, int n_calls, int max_group, size_t workspace_bytes,
                      PackedMeta* metas, size_t* need) {
  PackedMeta m0;
  if (lookup(calls[first].packed, m0) != LQER_OK || !decode_cols_fits(m0, calls[first].M)) return 0;
  metas[0] = m0;
  const size_t head = align_up(kPersistMaxBytes, 256);   // one bound for all layers, so that consecutive groups agree on it
  size_t slots = decode_cols_slot_bytes(m0);
  int n = 1;
  while (first + n < n_calls && n < max_group) {
    PackedMeta m1;
    if (calls[first + n].M != calls[first].M || lookup(calls[first + n].packed, m1) != LQER_OK ||
        !same_formats(m0, m1) || !decode_cols_fits(m1, calls[first].M) || m1.N < 32 || m0.N < 32)
      break;
    if (head + 2 * (slots + decode_cols_slot_bytes(m1)) > workspace_bytes) break;   // two sets: see launch_decode_cols_group
    slots += decode_cols_slot_bytes(m1);
    metas[n++] = m1;
  }
  if (need != nullptr) *need = head + 2 * slots;
  return n;
}
// The stretch of calls from calls[first] on that run as shared decode launches (decode_run after decode_run), and the
// bytes that their quantised activations and T_q take when computed ahead; offsets[i - first] is call i's place
// behind `base`.
static int decode_stretch(const lqer_call_t* calls, int first, int n_calls, size_t workspace_bytes,
                          std::vector<PackedMeta>* metas_out, std::vector<size_t>* offsets, size_t* bytes) {
  int j = first;
  size_t total = 0;
  while (j < n_calls) {
    PackedMeta metas[16];
    const int n = decode_run(calls, j, n_calls, decode_cols_max_group(), workspace_bytes, metas, nullptr);
    if (n < 2) break;
    for (int g = 0; g < n; ++g) {
      if (metas_out != nullptr) metas_out->push_back(metas[g]);
      if (offsets != nullptr) offsets->push_back(total);
      total += decode_pre_bytes(metas[g], calls[j + g].M);
    }
    j += n;
  }
  if (bytes != nullptr) *bytes = total;
  return j - first;
}
// CTAs a tensor-core prologue launch may have: one per SM (its CTAs wait for one another), within what the scratch is sized for.
static int prologue_max_ctas() {
  const int sms = sm_count();
  return sms > 0 && sms < kPrologueMaxCtas ? sms : kPrologueMaxCtas;
}
// n prefill layers with one M: each layer's prologue into its own slice of the workspace, then ONE GEMM launch over
// the tiles of all of them.
static lqer_status_t run_prefill_group(const lqer_call_t* calls, int n, const PackedMeta* metas, void* workspace,
                                       IoTypes io, cudaStream_t s) {
  const int M = calls[0].M;
  uint8_t* wsb = static_cast<uint8_t*>(workspace);
  DeviceStatus* dst = static_cast<DeviceStatus*>(workspace);
  size_t head = 0;
  for (int g = 0; g < n; ++g) head = std::max(head, align_up(persist_bytes(metas[g]), 256));
  const void* xcats[8];
  const void* packed[8];
  void* Ys[8];
  // The prologues of the group share nothing but the status word: each has its slice of the workspace, and, while the
  // counter pairs last, its own range of them, so that each may overlap the tail of the one before.
  size_t count_base = 0;
  for (int g = 0; g < n; ++g) count_base = std::max(count_base, pcount_offset(metas[g]));
  const int row_tiles = (M + 127) / 128;
  const bool own_counters = (long long)row_tiles * n <= kPrologueRowTiles;
  size_t off = head;
  for (int g = 0; g < n; ++g) {
    xcats[g] = wsb + off;
    off += group_slice_bytes(metas[g], M);
    packed[g] = calls[g].packed; Ys[g] = calls[g].Y;
  }
  // One launch for the prologues of all layers, if every one takes the tensor-core prologue with the same rank padding:
  // a CTA then carries a whole row tile of a layer, or a long K range of it, instead of a ninth.
  bool together = own_counters && n > 1;
  for (int g = 0; g < n && together; ++g)
    together = prologue_tc_fits(metas[g], M, calls[g].X, false) && metas[g].k_pad == metas[0].k_pad;
  if (together) {
    // Layers whose K is so long that the CTAs of the whole group would carry unequal work get a launch of their own
    // (as many K ranges as fit the SMs); the launches share no buffer, so a later one overlaps the tail of the one before.
    bool alone[8] = {false, false, false, false, false, false, false, false};
    int splits[8];
    const long long row_tiles_ll = row_tiles;
    for (;;) {
      PackedMeta sub[8];
      int idx[8], ns = 0;
      for (int g = 0; g < n; ++g)
        if (!alone[g]) { sub[ns] = metas[g]; idx[ns++] = g; }
      if (ns == 0) break;
      int sp[8];
      const bool squeezed = prologue_tc_group_splits(sub, ns, M, prologue_max_ctas(), sp);
      long long total = 0;
      double longest = 0.0;
      int worst = 0;
      for (int q = 0; q < ns; ++q) {
        const int panels = (sub[q].K64 + 127) / 128;
        total += row_tiles_ll * panels;
        const double len = (double)panels / sp[q];
        if (len > longest) { longest = len; worst = q; }
      }
      for (int q = 0; q < ns; ++q) splits[idx[q]] = sp[q];
      if (ns == 1 || !squeezed || longest <= 1.35 * (double)total / prologue_max_ctas()) break;
      alone[idx[worst]] = true;
    }
    const void* Xs[8];
    const void* pk[8];
    void* xc[8];
    double* parts[8];
    int* counts[8];
    PackedMeta ms[8];
    int sp[8];
    int launches = 0, planned = 0;
    for (int g = 0, rest = 0; g < n; ++g) {
      if (alone[g]) ++planned;
      else if (rest++ == 0) ++planned;
    }
    for (int pass = 0; pass < 1 + n; ++pass) {                  // pass 0: the layers that stay together; then each loner
      int cnt = 0;
      for (int g = 0; g < n; ++g) {
        const bool take = pass == 0 ? !alone[g] : (alone[g] && g == pass - 1);
        if (!take) continue;
        Xs[cnt] = calls[g].X;
        pk[cnt] = packed[g];
        xc[cnt] = const_cast<void*>(xcats[g]);
        parts[cnt] = reinterpret_cast<double*>(static_cast<uint8_t*>(xc[cnt]) + xcat_bytes(metas[g], M));
        counts[cnt] = reinterpret_cast<int*>(wsb + count_base) + (size_t)g * row_tiles * 2;
        ms[cnt] = metas[g];
        sp[cnt] = pass == 0 ? splits[g] : prologue_tc_splits(metas[g], M, prologue_max_ctas());
        ++cnt;
      }
      if (cnt == 0) continue;
      const int order = planned == 1 ? kChainAlone : launches == 0 ? kChainFirst : kChainLater;
      if (launch_prologue_tc_group(Xs, io.x_type, M, ms, pk, xc, parts, counts, sp, cnt, nullptr, nullptr, dst, order, s) != cudaSuccess)
        return LQER_ERR_CUDA;
      ++launches;
    }
  } else {
    for (int g = 0; g < n; ++g) {
      const PackedMeta& m = metas[g];
      uint8_t* xcat = static_cast<uint8_t*>(const_cast<void*>(xcats[g]));
      const float* X = calls[g].X;
      int* counters = reinterpret_cast<int*>(wsb + count_base) + (own_counters ? (size_t)g * row_tiles * 2 : 0);
      const int order = !own_counters ? kChainAlone : g == 0 ? kChainFirst : kChainLater;
      cudaError_t err = prologue_tc_fits(m, M, X, false)
                            ? launch_prologue_tc(X, io.x_type, M, m, calls[g].packed, xcat, nullptr, nullptr, dst,
                                                 reinterpret_cast<double*>(xcat + xcat_bytes(m, M)), counters, order, s)
                            : launch_prologue(X, io.x_type, M, m, calls[g].packed, xcat, nullptr, nullptr, dst, s);
      if (err != cudaSuccess) return LQER_ERR_CUDA;
    }
  }
  return launch_gemm_tc2_group(xcats, packed, Ys, io.y_type, metas, n, M, dst, s) == cudaSuccess ? LQER_OK : LQER_ERR_CUDA;
}

}  // namespace lqer

using namespace lqer;

extern "C" {

const char* lqer_status_string(lqer_status_t status) {
  switch (status) {
    case LQER_OK: return "ok";
    case LQER_ERR_NULL: return "null pointer";
    case LQER_ERR_SHAPE: return "unsupported shape";
    case LQER_ERR_ALIGN: return "misaligned pointer";
    case LQER_ERR_CONFIG: return "unsupported configuration";
    case LQER_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case LQER_ERR_BAD_PACKED: return "unknown or corrupt packed buffer";
    case LQER_ERR_ARCH: return "device is not compute capability 10.x";
    case LQER_ERR_CUDA: return "CUDA call failed";
    case LQER_ERR_TIMEOUT: return "device-side wait timed out";
    case LQER_ERR_BOUNDS: return "device-side bounds check failed";
    case LQER_ERR_STATIC_SCRATCH: return "problem too large for the library's fixed scratch array";
  }
  return "unknown status";
}

lqer_status_t lqer_default_config(lqer_config_t* cfg) {
  if (cfg == nullptr) return LQER_ERR_NULL;
  *cfg = lqer_config_t{4, 8, 8, 16, -56, 55, 1, -56, 55};
  return LQER_OK;
}

lqer_status_t lqer_packed_bytes(int K, int N, int k, const lqer_config_t* cfg, size_t* bytes) {
  if (bytes == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if ((st = check_shape(K, N, k)) != LQER_OK) return st;
  PackedMeta m;
  fill_meta(m, K, N, k, *cfg);
  *bytes = (size_t)m.total_bytes;
  return LQER_OK;
}

lqer_status_t lqer_workspace_bytes(int M_max, int K, int N, int k, const lqer_config_t* cfg, size_t* bytes) {
  if (bytes == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if ((st = check_shape(K, N, k)) != LQER_OK) return st;
  if (M_max <= 0 || M_max > (1 << 24)) return LQER_ERR_SHAPE;
  PackedMeta m;
  fill_meta(m, K, N, k, *cfg);
  *bytes = workspace_total(m, M_max);
  return LQER_OK;
}

lqer_status_t lqer_call_workspace_bytes(int M, int K, int N, int k, const lqer_config_t* cfg, size_t* bytes) {
  if (bytes == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if ((st = check_shape(K, N, k)) != LQER_OK) return st;
  if (M <= 0 || M > (1 << 24)) return LQER_ERR_SHAPE;
  PackedMeta m;
  fill_meta(m, K, N, k, *cfg);
  *bytes = call_bytes(m, M, M <= kSmallMaxM);
  return LQER_OK;
}

lqer_status_t lqer_prepare_weights(const float* W, const float* A, const float* B, int K, int N, int k,
                                   const lqer_config_t* cfg, void* packed, size_t packed_bytes, void* stream) {
  if (W == nullptr || packed == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if ((st = check_shape(K, N, k)) != LQER_OK) return st;
  if (k > 0 && (A == nullptr || B == nullptr)) return LQER_ERR_NULL;
  if (!aligned16(W) || (k > 0 && (!aligned16(A) || !aligned16(B))) || (reinterpret_cast<uintptr_t>(packed) & 255u) != 0)
    return LQER_ERR_ALIGN;
  PackedMeta m;
  fill_meta(m, K, N, k, *cfg);
  if (packed_bytes < m.total_bytes) return LQER_ERR_BUFFER_TOO_SMALL;
  if ((st = check_arch()) != LQER_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    // the header travels with the buffer; the registry keeps a stable host copy for the async copy
    std::lock_guard<std::mutex> lock(g_mu);
    PackedMeta& slot = g_registry[packed];
    slot = m;
    if (cudaMemcpyAsync(packed, &slot, sizeof(PackedMeta), cudaMemcpyHostToDevice, s) != cudaSuccess) {
      g_registry.erase(packed);
      return LQER_ERR_CUDA;
    }
  }
  if (launch_pack(W, A, B, m, packed, s) != cudaSuccess) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_registry.erase(packed);
    return LQER_ERR_CUDA;
  }
  return LQER_OK;
}

lqer_status_t lqer_factor_sketch_columns(int K, int N, int k, int* columns) {
  if (columns == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_shape(K, N, k);
  if (st != LQER_OK) return st;
  if (k < 1) return LQER_ERR_SHAPE;
  *columns = factor_sketch_rank(K, N, k);
  return LQER_OK;
}

lqer_status_t lqer_prepare_workspace_bytes(int K, int N, int k, size_t* bytes) {
  if (bytes == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_shape(K, N, k);
  if (st != LQER_OK) return st;
  if (k < 1) return LQER_ERR_SHAPE;
  *bytes = factor_workspace_bytes(K, N, k, 0);
  return LQER_OK;
}

lqer_status_t lqer_prepare_from_calibration(const float* W, const float* const* samples, const int* sample_rows, int n_samples,
                                            const float* omega, int K, int N, int k, const lqer_config_t* cfg, void* packed,
                                            size_t packed_bytes, float* A_out, float* B_out, void* workspace,
                                            size_t workspace_bytes, void* stream) {
  if (W == nullptr || omega == nullptr || packed == nullptr || workspace == nullptr) return LQER_ERR_NULL;
  if (n_samples < 0 || n_samples > 4096 || (n_samples > 0 && (samples == nullptr || sample_rows == nullptr))) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if ((st = check_shape(K, N, k)) != LQER_OK) return st;
  if (k < 1) return LQER_ERR_SHAPE;
  for (int i = 0; i < n_samples; ++i) {
    if (samples[i] == nullptr) return LQER_ERR_NULL;
    if (sample_rows[i] < 1) return LQER_ERR_SHAPE;
  }
  if (!aligned16(W) || !aligned16(omega) || (A_out != nullptr && !aligned16(A_out)) || (B_out != nullptr && !aligned16(B_out)) ||
      (reinterpret_cast<uintptr_t>(packed) & 255u) != 0 || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return LQER_ERR_ALIGN;
  PackedMeta m;
  fill_meta(m, K, N, k, *cfg);
  if (packed_bytes < m.total_bytes || workspace_bytes < factor_workspace_bytes(K, N, k, 0)) return LQER_ERR_BUFFER_TOO_SMALL;
  if ((st = check_arch()) != LQER_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* A = nullptr;
  float* B = nullptr;
  if (launch_factorize(W, samples, sample_rows, n_samples, omega, K, N, k, cfg->w_bits, cfg->w_exp_min, cfg->w_exp_max, A_out, B_out,
                       workspace, nullptr, &A, &B, s) != cudaSuccess)
    return LQER_ERR_CUDA;
  return lqer_prepare_weights(W, A, B, K, N, k, cfg, packed, packed_bytes, stream);
}

lqer_status_t lqer_prepare_status(const void* workspace, int K, int N, int k, void* stream, int* code) {
  if (workspace == nullptr || code == nullptr) return LQER_ERR_NULL;
  lqer_status_t st = check_shape(K, N, k);
  if (st != LQER_OK) return st;
  if (k < 1) return LQER_ERR_SHAPE;
  // the status word sits behind the fixed-size pieces of the workspace, in front of the internal A and B
  auto al = [](size_t v) { return (v + 255) & ~(size_t)255; };
  const size_t off = factor_workspace_bytes(K, N, k, 0) - al((size_t)K * k * 4) - al((size_t)k * N * 4) - 256;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(code, static_cast<const uint8_t*>(workspace) + off, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return LQER_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? LQER_OK : LQER_ERR_CUDA;
}

lqer_status_t lqer_attach_packed(const void* packed, size_t packed_bytes, void* stream) {
  if (packed == nullptr) return LQER_ERR_NULL;
  if (packed_bytes < (size_t)kHeaderBytes) return LQER_ERR_BUFFER_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(packed) & 255u) != 0) return LQER_ERR_ALIGN;
  PackedMeta m;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&m, packed, sizeof(m), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LQER_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return LQER_ERR_CUDA;
  if (!meta_valid(m)) return LQER_ERR_BAD_PACKED;
  if (packed_bytes < m.total_bytes) return LQER_ERR_BUFFER_TOO_SMALL;
  std::lock_guard<std::mutex> lock(g_mu);
  g_registry[packed] = m;
  return LQER_OK;
}

lqer_status_t lqer_release_packed(const void* packed) {
  if (packed == nullptr) return LQER_ERR_NULL;
  std::lock_guard<std::mutex> lock(g_mu);
  return g_registry.erase(packed) ? LQER_OK : LQER_ERR_BAD_PACKED;
}

lqer_status_t lqer_packed_shape(const void* packed, int* K, int* N, int* k, int* k_pad) {
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  if (K) *K = m.K;
  if (N) *N = m.N;
  if (k) *k = m.k;
  if (k_pad) *k_pad = m.k_pad;
  return LQER_OK;
}

lqer_status_t lqer_export_weights(const void* packed, int8_t* Wm, uint8_t* We, int8_t* Am, uint8_t* Ae,
                                  int8_t* Bm, uint8_t* Be, void* stream) {
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  if ((st = check_arch()) != LQER_OK) return st;
  return launch_export(m, packed, Wm, We, Am, Ae, Bm, Be, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LQER_OK : LQER_ERR_CUDA;
}

lqer_status_t lqer_quantize_activations(const float* X, int M, int K, const lqer_config_t* cfg, int8_t* Xm,
                                        uint8_t* Xe, void* stream) {
  if (X == nullptr || (Xm == nullptr && Xe == nullptr)) return LQER_ERR_NULL;
  lqer_status_t st = check_config(cfg);
  if (st != LQER_OK) return st;
  if (M <= 0 || K <= 0 || K % 16 != 0 || M > (1 << 24) || K > (1 << 20)) return LQER_ERR_SHAPE;
  if (!aligned16(X) || (Xm != nullptr && (reinterpret_cast<uintptr_t>(Xm) & 3u) != 0)) return LQER_ERR_ALIGN;
  if ((st = check_arch()) != LQER_OK) return st;
  return launch_quantize_x(X, M, K, cfg->a_bits, cfg->exp_min, cfg->exp_max, Xm, Xe,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess ? LQER_OK : LQER_ERR_CUDA;
}

lqer_status_t lqer_project_lowrank(const float* X, int M, const void* packed, int8_t* Tm, uint8_t* Te,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  if (Tm == nullptr && Te == nullptr) return LQER_ERR_NULL;
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  if (m.k == 0) return LQER_ERR_SHAPE;
  return run_linear(X, M, packed, nullptr, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), Tm, Te, true);
}

lqer_status_t lqer_linear_stream(const float* X, int M, const void* packed, float* Y, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  return run_linear(X, M, packed, Y, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), nullptr,
                    nullptr, false);
}

lqer_status_t lqer_linear(const float* X, int M, const void* packed, float* Y, void* workspace,
                          size_t workspace_bytes) {
  return lqer_linear_stream(X, M, packed, Y, workspace, workspace_bytes, nullptr);
}

}  // extern "C"

// The batched entry points: independent calls share launches where the path is left at 0.
static lqer_status_t linear_batched(const lqer_call_t* calls, int n_calls, void* workspace, size_t workspace_bytes,
                                    void* stream, IoTypes io) {
  const bool cols_ok = true;
  if (calls == nullptr) return LQER_ERR_NULL;
  if (n_calls < 0) return LQER_ERR_SHAPE;
  // validate everything before the first launch
  for (int i = 0; i < n_calls; ++i) {
    const lqer_call_t& c = calls[i];
    if (c.X == nullptr || c.packed == nullptr || c.Y == nullptr || workspace == nullptr) return LQER_ERR_NULL;
    if (c.M <= 0 || c.M > (1 << 24)) return LQER_ERR_SHAPE;
    if (!aligned16(c.X) || !aligned16(c.Y)) return LQER_ERR_ALIGN;
    PackedMeta m;
    lqer_status_t st = lookup(c.packed, m);
    if (st != LQER_OK) return st;
    const int path = g_path.load();
    if ((path == 2 || path == 5 || path == 7) && c.M > kSmallMaxM) return LQER_ERR_SHAPE;
    if (io.y_type == kYMXINT8 && m.N % 16 != 0) return LQER_ERR_SHAPE;
    if (workspace_bytes < call_bytes(m, c.M, takes_small_path(path, c.M))) return LQER_ERR_BUFFER_TOO_SMALL;
  }
  const bool may_group = g_path.load() == 0;   // a forced path runs every call on its own
  // Decode launches that follow one another are independent too (no buffer in common: two sets of slots and counters
  // in turn), so a launch need not wait for the one before it, as long as that one had a CTA on every SM.
  bool chain_open = false;
  int chain_set = 0;
  // The quantised activations and T_q of a stretch of several decode launches are computed ahead, one CTA per call, if
  // the workspace has room for them behind its head: the decode launches then stream weights from their first
  // instruction.
  const size_t pre_base = align_up(kPersistMaxBytes, 256);
  int pre_first = 0, pre_end = 0;               // calls [pre_first, pre_end): the stretch looked at last
  std::vector<size_t> pre_off;                  // its offsets behind pre_base; empty: nothing computed ahead
  for (int i = 0; i < n_calls;) {
    // The calls are independent, so consecutive calls of one shape (the q, k, v projections of a layer, or its gate
    // and up projections) share launches: decode calls one launch of the column-owner kernel (a slot of the workspace per
    // layer for the partial sums of T), prefill calls one GEMM launch after their prologues, if the workspace has a
    // slice for each.
    int n = 1;
    PackedMeta m0, metas[16];
    bool decode_group = false, small_group = false;
    if (may_group && lookup(calls[i].packed, m0) == LQER_OK) {
      const int many = cols_ok ? many_small_rows(calls, i, n_calls, workspace_bytes, m0, metas, nullptr) : 0;
      if (many > 0) {
        n = many;
        small_group = true;
      } else if (cols_ok && decode_cols_fits(m0, calls[i].M)) {
        n = decode_run(calls, i, n_calls, decode_cols_max_group(), workspace_bytes, metas, nullptr);
        if (n < 1) n = 1;
        decode_group = n > 1;
      } else if (calls[i].M <= kSmallMaxM) {
        const int lim = std::min(gemm_small_max_layers(), prologue_small_max_layers());
        n = small_run(calls, i, n_calls, lim, workspace_bytes, cols_ok, metas, nullptr);
        if (n < 1) n = 1;
        small_group = n > 1;
      } else if (calls[i].M > kGemmSplitMaxM) {   // batches in between run split K, each on its own
        n = prefill_run(calls, i, n_calls, gemm_tc2_max_group(), workspace_bytes, metas, nullptr);
        if (n < 1) n = 1;
      }
    }
    if (n > 1) {
      lqer_status_t st = check_arch();
      if (st != LQER_OK) return st;
      if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LQER_ERR_ALIGN;
      if (decode_group) {
        cudaStream_t cs = static_cast<cudaStream_t>(stream);
        if (i >= pre_end) {
          std::vector<PackedMeta> pm;
          size_t bytes = 0;
          pre_off.clear();
          pre_first = i;
          pre_end = i + decode_stretch(calls, i, n_calls, workspace_bytes, &pm, &pre_off, &bytes);
          if (pre_base + bytes > workspace_bytes || pre_end - i <= decode_cols_max_group()) {   // no room, or a single launch: it does the work itself
            pre_off.clear();
          } else {
            std::vector<uint8_t*> outs(pm.size());
            for (size_t q = 0; q < pm.size(); ++q) outs[q] = static_cast<uint8_t*>(workspace) + pre_base + pre_off[q];
            const int step = decode_pre_max_calls();
            for (int q = 0; q < (int)pm.size(); q += step) {
              const int cnt = std::min(step, (int)pm.size() - q);
              if (launch_decode_pre(calls + i + q, pm.data() + q, outs.data() + q, cnt, q == 0 ? kChainFirst : kChainLater,
                                    io.x_type, cs) != cudaSuccess)
                return LQER_ERR_CUDA;
            }
          }
        }
        const uint8_t* pres[16];
        const bool ahead = !pre_off.empty();
        for (int g = 0; g < n; ++g)
          pres[g] = ahead ? static_cast<const uint8_t*>(workspace) + pre_base + pre_off[i + g - pre_first] : nullptr;
        const int set = chain_open ? 1 - chain_set : 0;
        bool fills = false;
        if (launch_decode_cols_group(calls + i, metas, n, workspace, workspace_bytes, chain_open ? kChainLater : kChainFirst,
                                     set, &fills, ahead ? pres : nullptr, io.x_type, io.y_type, cs) != cudaSuccess)
          return LQER_ERR_CUDA;
        chain_open = fills;
        chain_set = set;
      } else if (small_group) {
        chain_open = false;
        if ((st = run_small_group(calls + i, n, metas, workspace, io, static_cast<cudaStream_t>(stream))) != LQER_OK) return st;
      } else {
        chain_open = false;
        if ((st = run_prefill_group(calls + i, n, metas, workspace, io, static_cast<cudaStream_t>(stream))) != LQER_OK) return st;
      }
    } else {
      chain_open = false;
      lqer_status_t st = run_linear(calls[i].X, calls[i].M, calls[i].packed, calls[i].Y, workspace, workspace_bytes,
                                    static_cast<cudaStream_t>(stream), nullptr, nullptr, false, io);
      if (st != LQER_OK) return st;
    }
    i += n;
  }
  return LQER_OK;
}

static lqer_status_t io_types(lqer_dtype_t x_dtype, lqer_dtype_t y_dtype, IoTypes* io) {
  if ((x_dtype != LQER_F32 && x_dtype != LQER_BF16 && x_dtype != LQER_MXINT8) ||
      (y_dtype != LQER_F32 && y_dtype != LQER_BF16 && y_dtype != LQER_MXINT8))
    return LQER_ERR_CONFIG;
  io->x_type = x_dtype == LQER_BF16 ? kXBF16 : x_dtype == LQER_MXINT8 ? kXMXINT8 : kXF32;
  io->y_type = y_dtype == LQER_BF16 ? kYBF16 : y_dtype == LQER_MXINT8 ? kYMXINT8 : kYF32;
  return LQER_OK;
}

extern "C" {

lqer_status_t lqer_linear_batched(const lqer_call_t* calls, int n_calls, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  return linear_batched(calls, n_calls, workspace, workspace_bytes, stream, IoTypes());
}

lqer_status_t lqer_linear_batched_ex(const lqer_call_t* calls, int n_calls, lqer_dtype_t x_dtype, lqer_dtype_t y_dtype,
                                     void* workspace, size_t workspace_bytes, void* stream) {
  IoTypes io;
  lqer_status_t st = io_types(x_dtype, y_dtype, &io);
  if (st != LQER_OK) return st;
  return linear_batched(calls, n_calls, workspace, workspace_bytes, stream, io);
}

lqer_status_t lqer_linear_ex(const void* X, lqer_dtype_t x_dtype, int M, const void* packed, void* Y, lqer_dtype_t y_dtype,
                             void* workspace, size_t workspace_bytes, void* stream) {
  IoTypes io;
  lqer_status_t st = io_types(x_dtype, y_dtype, &io);
  if (st != LQER_OK) return st;
  return run_linear(X, M, packed, Y, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), nullptr, nullptr, false, io);
}

lqer_status_t lqer_batched_workspace_bytes(const lqer_call_t* calls, int n_calls, size_t* bytes) {
  if (calls == nullptr || bytes == nullptr) return LQER_ERR_NULL;
  if (n_calls < 0) return LQER_ERR_SHAPE;
  int stretch_end = 0;
  size_t need = kStatusBytes;
  for (int i = 0; i < n_calls; ++i) {           // every call on its own
    const lqer_call_t& c = calls[i];
    if (c.packed == nullptr) return LQER_ERR_NULL;
    if (c.M <= 0 || c.M > (1 << 24)) return LQER_ERR_SHAPE;
    PackedMeta m;
    lqer_status_t st = lookup(c.packed, m);
    if (st != LQER_OK) return st;
    need = std::max(need, workspace_total(m, c.M));
  }
  for (int i = 0; i < n_calls;) {               // the launches that calls may share
    const lqer_call_t& c = calls[i];
    PackedMeta m;
    lookup(c.packed, m);
    PackedMeta many_metas[16];
    size_t many_need = 0;
    const int many = many_small_rows(calls, i, n_calls, ~(size_t)0, m, many_metas, &many_need);
    int n = 1;
    if (many > 0) {
      n = many;
      need = std::max(need, many_need);
    } else if (decode_cols_fits(m, c.M)) {
      PackedMeta metas[16];
      size_t group_need = 0, ahead = 0;
      n = decode_run(calls, i, n_calls, decode_cols_max_group(), ~(size_t)0, metas, &group_need);
      if (n < 1) n = 1;
      need = std::max(need, group_need);
      if (n > 1 && i >= stretch_end) {          // room to compute a whole stretch's activations ahead
        stretch_end = i + decode_stretch(calls, i, n_calls, ~(size_t)0, nullptr, nullptr, &ahead);
        need = std::max(need, align_up(kPersistMaxBytes, 256) + ahead);
      }
    } else if (c.M <= kSmallMaxM) {
      PackedMeta metas[16];
      size_t group_need = 0;
      n = small_run(calls, i, n_calls, std::min(gemm_small_max_layers(), prologue_small_max_layers()), ~(size_t)0, true, metas, &group_need);
      if (n < 1) n = 1;
      if (n > 1) need = std::max(need, group_need);
    } else if (c.M > kGemmSplitMaxM) {
      PackedMeta metas[8];
      size_t group_need = 0;
      n = prefill_run(calls, i, n_calls, gemm_tc2_max_group(), ~(size_t)0, metas, &group_need);
      if (n < 1) n = 1;
      need = std::max(need, group_need);
    }
    i += n;
  }
  *bytes = need;
  return LQER_OK;
}

lqer_status_t lqer_linear_host(const float* X_host, int M, const void* packed, float* Y_host, void* workspace,
                               size_t workspace_bytes, void* stream) {
  if (X_host == nullptr || Y_host == nullptr || workspace == nullptr) return LQER_ERR_NULL;
  if (M <= 0 || M > (1 << 24)) return LQER_ERR_SHAPE;
  PackedMeta m;
  lqer_status_t st = lookup(packed, m);
  if (st != LQER_OK) return st;
  const size_t core = workspace_total(m, M);
  const size_t xb = align_up((size_t)M * m.K * 4, 256), yb = align_up((size_t)M * m.N * 4, 256);
  if (workspace_bytes < core + xb + yb) return LQER_ERR_BUFFER_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* Xd = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + core);
  float* Yd = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + core + xb);
  if (cudaMemcpyAsync(Xd, X_host, (size_t)M * m.K * 4, cudaMemcpyHostToDevice, s) != cudaSuccess) return LQER_ERR_CUDA;
  if ((st = lqer_linear_stream(Xd, M, packed, Yd, workspace, core, stream)) != LQER_OK) return st;
  if (cudaMemcpyAsync(Y_host, Yd, (size_t)M * m.N * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LQER_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return LQER_ERR_CUDA;
  return LQER_OK;
}

// Streams and events of lqer_linear_host_batched, made once per device.
namespace {
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, in_done[2] = {}, comp_done[2] = {}, out_done[2] = {};
};
HostPipe g_pipes[64];

HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_mu);
  HostPipe& hp = g_pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess;
    for (int b = 0; b < 2 && ok; ++b)
      ok = cudaEventCreateWithFlags(&hp.in_done[b], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.comp_done[b], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.out_done[b], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    hp.ready = true;
  }
  return &hp;
}
}  // namespace

lqer_status_t lqer_linear_host_batched_bytes(const lqer_call_t* calls, int n_calls, size_t* bytes) {
  if (calls == nullptr || bytes == nullptr) return LQER_ERR_NULL;
  if (n_calls < 0) return LQER_ERR_SHAPE;
  size_t core = kStatusBytes, xb = 0, yb = 0;
  for (int i = 0; i < n_calls; ++i) {
    const lqer_call_t& c = calls[i];
    if (c.packed == nullptr) return LQER_ERR_NULL;
    if (c.M <= 0 || c.M > (1 << 24)) return LQER_ERR_SHAPE;
    PackedMeta m;
    lqer_status_t st = lookup(c.packed, m);
    if (st != LQER_OK) return st;
    core = std::max(core, workspace_total(m, c.M));
    xb = std::max(xb, align_up((size_t)c.M * m.K * 4, 256));
    yb = std::max(yb, align_up((size_t)c.M * m.N * 4, 256));
  }
  *bytes = align_up(core, 256) + 2 * xb + 2 * yb;
  return LQER_OK;
}

}  // extern "C"

static lqer_status_t linear_host_batched(const lqer_call_t* calls, int n_calls, void* workspace, size_t workspace_bytes,
                                         void* stream, IoTypes io) {
  if (calls == nullptr || workspace == nullptr) return LQER_ERR_NULL;
  if (n_calls < 0) return LQER_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LQER_ERR_ALIGN;
  size_t core = kStatusBytes, xb = 0, yb = 0;
  for (int i = 0; i < n_calls; ++i) {
    const lqer_call_t& c = calls[i];
    if (c.X == nullptr || c.Y == nullptr || c.packed == nullptr) return LQER_ERR_NULL;
    if (c.M <= 0 || c.M > (1 << 24)) return LQER_ERR_SHAPE;
    PackedMeta m;
    lqer_status_t st = lookup(c.packed, m);
    if (st != LQER_OK) return st;
    if (io.y_type == kYMXINT8 && m.N % 16 != 0) return LQER_ERR_SHAPE;
    core = std::max(core, workspace_total(m, c.M));
    xb = std::max(xb, align_up((size_t)c.M * m.K * 4, 256));
    yb = std::max(yb, align_up((size_t)c.M * m.N * 4, 256));
  }
  core = align_up(core, 256);
  if (workspace_bytes < core + 2 * xb + 2 * yb) return LQER_ERR_BUFFER_TOO_SMALL;
  if (n_calls == 0) return LQER_OK;
  HostPipe* hp = host_pipe();
  if (hp == nullptr) return LQER_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* Xd[2] = {reinterpret_cast<float*>(ws + core), reinterpret_cast<float*>(ws + core + xb)};
  float* Yd[2] = {reinterpret_cast<float*>(ws + core + 2 * xb), reinterpret_cast<float*>(ws + core + 2 * xb + yb)};
  bool ok = cudaEventRecord(hp->start, s) == cudaSuccess &&          // earlier work on `stream` may still use the workspace
            cudaStreamWaitEvent(hp->in, hp->start, 0) == cudaSuccess &&
            cudaStreamWaitEvent(hp->out, hp->start, 0) == cudaSuccess;
  lqer_status_t result = ok ? LQER_OK : LQER_ERR_CUDA;
  for (int i = 0; i < n_calls && result == LQER_OK; ++i) {
    const lqer_call_t& c = calls[i];
    const int b = i & 1;
    PackedMeta m;
    lookup(c.packed, m);
    // copy in: the buffer is free once the layer two calls back has run
    ok = (i < 2 || cudaStreamWaitEvent(hp->in, hp->comp_done[b], 0) == cudaSuccess) &&
         cudaMemcpyAsync(Xd[b], c.X, x_bytes(io.x_type, (size_t)c.M, (size_t)m.K), cudaMemcpyHostToDevice, hp->in) == cudaSuccess &&
         cudaEventRecord(hp->in_done[b], hp->in) == cudaSuccess &&
         // the layer: after its X has landed and after the Y buffer's previous contents have left
         cudaStreamWaitEvent(s, hp->in_done[b], 0) == cudaSuccess &&
         (i < 2 || cudaStreamWaitEvent(s, hp->out_done[b], 0) == cudaSuccess);
    if (!ok) { result = LQER_ERR_CUDA; break; }
    result = run_linear(Xd[b], c.M, c.packed, Yd[b], workspace, core, s, nullptr, nullptr, false, io);
    if (result != LQER_OK) break;
    ok = cudaEventRecord(hp->comp_done[b], s) == cudaSuccess &&
         cudaStreamWaitEvent(hp->out, hp->comp_done[b], 0) == cudaSuccess &&
         cudaMemcpyAsync(c.Y, Yd[b], y_bytes(io.y_type, (size_t)c.M, (size_t)m.N), cudaMemcpyDeviceToHost, hp->out) == cudaSuccess &&
         cudaEventRecord(hp->out_done[b], hp->out) == cudaSuccess;
    if (!ok) result = LQER_ERR_CUDA;
  }
  // nothing of this call is in flight when it returns, whatever happened
  const bool drained = cudaStreamSynchronize(hp->in) == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess &&
                       cudaStreamSynchronize(hp->out) == cudaSuccess;
  if (result == LQER_OK && !drained) result = LQER_ERR_CUDA;
  return result;
}

extern "C" {

lqer_status_t lqer_linear_host_batched(const lqer_call_t* calls, int n_calls, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  return linear_host_batched(calls, n_calls, workspace, workspace_bytes, stream, IoTypes());
}

lqer_status_t lqer_linear_host_batched_ex(const lqer_call_t* calls, int n_calls, lqer_dtype_t x_dtype, lqer_dtype_t y_dtype,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  IoTypes io;
  lqer_status_t st = io_types(x_dtype, y_dtype, &io);
  if (st != LQER_OK) return st;
  return linear_host_batched(calls, n_calls, workspace, workspace_bytes, stream, io);
}

lqer_status_t lqer_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (workspace == nullptr) return LQER_ERR_NULL;
  if (workspace_bytes < (size_t)kStatusBytes) return LQER_ERR_BUFFER_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return LQER_ERR_ALIGN;
  const size_t n = workspace_bytes < kPersistMaxBytes ? workspace_bytes : kPersistMaxBytes;
  return cudaMemsetAsync(workspace, 0, n, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LQER_OK : LQER_ERR_CUDA;
}

lqer_status_t lqer_poll_status(const void* workspace, void* stream, lqer_status_t* device_status) {
  if (workspace == nullptr || device_status == nullptr) return LQER_ERR_NULL;
  DeviceStatus h;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LQER_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return LQER_ERR_CUDA;
  *device_status = (h.code >= 0 && h.code <= LQER_ERR_BOUNDS) ? (lqer_status_t)h.code : LQER_ERR_CUDA;
  return LQER_OK;
}

lqer_status_t lqer_debug_bounds_shrink(long long bytes) {
  if (!kDebugBounds) return LQER_ERR_CONFIG;          // the ordinary build has no checks to trip
  if (bytes < 0 || bytes > (1LL << 40)) return LQER_ERR_CONFIG;
  g_y_shrink.store((size_t)bytes);
  return LQER_OK;
}

lqer_status_t lqer_set_wait_limit_cycles(long long cycles) {
  if (cycles < 1000 || cycles > (1LL << 40)) return LQER_ERR_CONFIG;
  g_wait_limit.store(cycles);
  return LQER_OK;
}

lqer_status_t lqer_inject_stall(int kernel_family) {
  if (kernel_family < -1 || kernel_family >= LQER_NUM_KERNEL_FAMILIES) return LQER_ERR_CONFIG;
  g_stall_family.store(kernel_family);
  return LQER_OK;
}

lqer_status_t lqer_set_path(int path) {
  if (path < 0 || path > 7) return LQER_ERR_CONFIG;
  g_path.store(path);
  return LQER_OK;
}

unsigned long long lqer_launch_count(void) { return g_launches.load(); }

lqer_status_t lqer_profile_enable(int on) {
  if (on != 0 && on != 1) return LQER_ERR_CONFIG;
  g_prof_on.store(on);
  return LQER_OK;
}

lqer_status_t lqer_profile_collect(lqer_kernel_times_t* out) {
  if (out == nullptr) return LQER_ERR_NULL;
  std::memset(out, 0, sizeof(*out));
  std::lock_guard<std::mutex> lock(g_prof_mu);
  lqer_status_t st = LQER_OK;
  for (const TimedLaunch& r : g_prof_records) {
    float ms = 0.0f;
    if (cudaEventSynchronize(r.stop) != cudaSuccess || cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) {
      st = LQER_ERR_CUDA;
    } else if (r.family >= 0 && r.family < LQER_NUM_KERNEL_FAMILIES) {
      out->launches[r.family] += (unsigned long long)r.n_kernels;
      out->milliseconds[r.family] += (double)ms;
    }
    g_prof_free.push_back(r.start);
    g_prof_free.push_back(r.stop);
  }
  g_prof_records.clear();
  return st;
}

}  // extern "C"
