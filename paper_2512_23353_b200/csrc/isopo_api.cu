// C-ABI entry points of libisopo: argument validation, workspace layout, path choice, dispatch.
// Every step of the path runs in the CUDA kernels launched from here; there is no host arithmetic
// on the data and no CPU fallback.
#include <cstdio>
#include <cstring>
#include <algorithm>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "isopo_internal.h"

namespace isopo {

// NVTX range named after the entry point, open for the duration of the host call (the kernels it
// enqueues appear under it in a profiler's timeline; without a profiler attached this is a no-op).
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
};

static thread_local char g_cuda_err[256] = "no error";

void set_cuda_error(cudaError_t e, const char* where) {
  if (e == cudaSuccess)
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s", where);  // a plain explanation, no CUDA error behind it
  else
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e), where);
}

static bool g_deterministic = false;
bool deterministic_mode() { return g_deterministic; }
static isopo_store_format g_store_format = ISOPO_STORE_BF16;

// The split store lives in the 2-CTA gradient GEMM and sums the diagonal of K with float atomics: layers that
// take the 1-CTA kernel, and everything in deterministic mode, keep the bf16 store.
bool use_split_store(const WsLayout& L, int B) {
  return g_store_format == ISOPO_STORE_E4M3_SPLIT && !g_deterministic && B <= 256 && (L.tiles_m % 2 == 0 || L.tiles_m >= 7);
}
StoreFmt store_fmt(const WsLayout& L, int B, void* ws) {
  float* aux = (float*)((char*)ws + L.off_aux);
  return StoreFmt{use_split_store(L, B) ? 1 : 0, aux, aux + B};
}

// ---- measurement hooks ----
struct ProfRecord { int id; cudaEvent_t a, b; };
static bool g_prof_on = false;
static std::vector<ProfRecord> g_prof;
static std::vector<cudaEvent_t> g_event_pool;
static int64_t g_launches[kIdCount] = {};

static cudaEvent_t take_event() {
  if (!g_event_pool.empty()) {
    cudaEvent_t e = g_event_pool.back();
    g_event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

LaunchScope::LaunchScope(int id, cudaStream_t st) : slot_(-1), st_(st) {
  ++g_launches[id];
  if (!g_prof_on) return;
  ProfRecord r{id, take_event(), take_event()};
  if (!r.a || !r.b) return;
  cudaEventRecord(r.a, st);
  slot_ = (int)g_prof.size();
  g_prof.push_back(r);
}

LaunchScope::~LaunchScope() {
  if (slot_ >= 0) cudaEventRecord(g_prof[slot_].b, st_);
}

ProfilingPause::ProfilingPause() : was_on_(g_prof_on) { g_prof_on = false; }
ProfilingPause::~ProfilingPause() { g_prof_on = was_on_; }

WsLayout ws_layout(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, isopo_path resolved) {
  WsLayout L{};
  size_t p = 0;
  L.off_tag = p;
  p = align_up(p + sizeof(WsTag), 1024);
  L.off_aux = p;
  if (dtype == ISOPO_BF16 && resolved == ISOPO_PATH_MATERIALISE) p = align_up(p + 2 * sizeof(float) * (size_t)B, 1024);
  L.off_offsets = p;
  p = align_up(p + sizeof(int64_t) * (size_t)(B + 1), 1024);
  L.off_order = p;
  p = align_up(p + sizeof(int32_t) * (size_t)B, 1024);
  L.off_tokseq = p;
  p = align_up(p + sizeof(int32_t) * (size_t)T, 1024);
  L.off_kacc = p;
  if (dtype == ISOPO_F32) p = align_up(p + sizeof(double) * (size_t)B * (size_t)B, 1024);
  L.off_scaled = p;
  if (dtype == ISOPO_BF16 && resolved == ISOPO_PATH_GRAM)
    p = align_up(p + (size_t)2 * (size_t)T * (size_t)std::min(d_in, d_out), 1024);
  L.off_G = p;
  if (dtype == ISOPO_BF16) {
    L.tiles_m = (d_out + kTileM - 1) / kTileM;
    L.tiles_n = (d_in + kTileN - 1) / kTileN;
    L.n_pad = (int64_t)L.tiles_m * L.tiles_n * kTileElems;
    if (resolved == ISOPO_PATH_MATERIALISE) p = align_up(p + (size_t)2 * (size_t)B * (size_t)L.n_pad, 1024);
    L.off_kpart = p;
    if (resolved == ISOPO_PATH_MATERIALISE && deterministic_mode())
      p = align_up(p + sizeof(float) * (size_t)kNtkMaxPartials * (size_t)B * (size_t)B, 1024);
  } else {
    L.tiles_m = L.tiles_n = 0;
    L.off_kpart = p;
    L.n_pad = (int64_t)d_in * d_out;
    if (resolved == ISOPO_PATH_MATERIALISE) p = align_up(p + (size_t)4 * (size_t)B * (size_t)L.n_pad, 1024);
  }
  L.total = p;
  return L;
}

WsTag make_ws_tag(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, const int64_t* off_host) {
  uint64_t h = 1469598103934665603ull;  // FNV-1a over the offsets' bytes
  for (int i = 0; i <= B; ++i) {
    uint64_t w = (uint64_t)off_host[i];
    for (int b = 0; b < 8; ++b) { h ^= w & 0xffu; h *= 1099511628211ull; w >>= 8; }
  }
  WsTag t{};
  t.v[0] = 0x49534f504f5f4753ll;
  t.v[1] = (int64_t)dtype; t.v[2] = T; t.v[3] = d_in; t.v[4] = d_out; t.v[5] = B; t.v[6] = (int64_t)h;
  if (dtype == ISOPO_BF16) {  // the format the stored gradients of this shape are kept in right now
    const WsLayout L = ws_layout(dtype, T, d_in, d_out, B, ISOPO_PATH_MATERIALISE);
    t.v[7] = use_split_store(L, B) ? 1 : 0;
  }
  return t;
}

static bool sizes_ok(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B) {
  if (dtype != ISOPO_F32 && dtype != ISOPO_BF16) return false;
  if (T < 1 || B < 1 || d_in < 1 || d_out < 1 || (int64_t)B > T) return false;
  if (T > ((int64_t)1 << 31) - 1024) return false;  // token coordinates are 32-bit in the tensor maps
  return true;
}

static isopo_status check_layer_args(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                                     const int64_t* off, int B, isopo_path path, const void* ws) {
  if (!X || !dY || !off || !ws) return ISOPO_ERR_INVALID_ARG;
  if (!sizes_ok(dtype, T, d_in, d_out, B)) return ISOPO_ERR_INVALID_ARG;
  if (path != ISOPO_PATH_AUTO && path != ISOPO_PATH_GRAM && path != ISOPO_PATH_MATERIALISE)
    return ISOPO_ERR_INVALID_ARG;
  if (((uintptr_t)X & 15) || ((uintptr_t)dY & 15) || ((uintptr_t)ws & 1023)) return ISOPO_ERR_INVALID_ARG;
  if (off[0] != 0 || off[B] != T) return ISOPO_ERR_INVALID_ARG;
  for (int i = 0; i < B; ++i)
    if (off[i + 1] <= off[i]) return ISOPO_ERR_INVALID_ARG;
  if (dtype == ISOPO_BF16 && ((d_in & 7) || (d_out & 7))) return ISOPO_ERR_UNSUPPORTED;
  return ISOPO_OK;
}

static isopo_path resolve_path(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, isopo_path path) {
  return path == ISOPO_PATH_AUTO ? isopo_choose_path(dtype, T, d_in, d_out, B) : path;
}

}  // namespace isopo

using namespace isopo;

extern "C" {

const char* isopo_status_string(isopo_status s) {
  switch (s) {
    case ISOPO_OK: return "ISOPO_OK";
    case ISOPO_ERR_INVALID_ARG: return "ISOPO_ERR_INVALID_ARG";
    case ISOPO_ERR_UNSUPPORTED: return "ISOPO_ERR_UNSUPPORTED";
    case ISOPO_ERR_WORKSPACE: return "ISOPO_ERR_WORKSPACE";
    case ISOPO_ERR_CUDA: return "ISOPO_ERR_CUDA";
  }
  return "ISOPO_ERR_UNKNOWN";
}

const char* isopo_last_cuda_error(void) { return g_cuda_err; }

void isopo_profile_enable(int on) { g_prof_on = on != 0; }

void isopo_set_deterministic(int on) { g_deterministic = on != 0; }
isopo_status isopo_set_store_format(isopo_store_format f) {
  if (f != ISOPO_STORE_BF16 && f != ISOPO_STORE_E4M3_SPLIT) return ISOPO_ERR_INVALID_ARG;
  g_store_format = f;
  return ISOPO_OK;
}
isopo_store_format isopo_get_store_format(void) { return g_store_format; }
int isopo_get_deterministic(void) { return g_deterministic ? 1 : 0; }
int isopo_debug_build(void) {
#ifdef ISOPO_DEBUG
  return 1;
#else
  return 0;
#endif
}

isopo_status isopo_profile_collect(double* ms_by_kernel, int64_t* launches_by_kernel) {
  if (!ms_by_kernel || !launches_by_kernel) return ISOPO_ERR_INVALID_ARG;
  for (int k = 0; k < kIdCount; ++k) { ms_by_kernel[k] = 0.0; launches_by_kernel[k] = g_launches[k]; g_launches[k] = 0; }
  isopo_status rc = ISOPO_OK;
  for (const ProfRecord& r : g_prof) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(r.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.a, r.b);
    if (e != cudaSuccess) { set_cuda_error(e, "isopo_profile_collect"); rc = ISOPO_ERR_CUDA; }
    ms_by_kernel[r.id] += ms;
    g_event_pool.push_back(r.a);
    g_event_pool.push_back(r.b);
  }
  g_prof.clear();
  return rc;
}

const char* isopo_kernel_name(int id) {
  static const char* names[kIdCount] = {"k_tokseq", "k_bf16_seq_grad", "k_bf16_ntk", "k_bf16_gram", "k_bf16_weight_grad",
                                        "k_bf16_combine", "k_transform", "k_mirror_upper", "k_f32_seq_grad",
                                        "k_f32_ntk", "k_f32_gram", "k_f32_weight_grad", "k_f32_combine",
                                        "k_sampled", "k_sampled_aux", "k_scale_rows", "k_wait_probe"};
  return id >= 0 && id < kIdCount ? names[id] : "unknown";
}

isopo_path isopo_choose_path(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B) {
  if (!sizes_ok(dtype, T, d_in, d_out, B)) return ISOPO_PATH_GRAM;
  if (dtype == ISOPO_BF16 && B > 256) return ISOPO_PATH_GRAM;  // stored-gradient kernels hold all B rows on chip
  // Modelled extra time over the plain dW GEMM (which both routes pay once).
  const double peak = dtype == ISOPO_BF16 ? 1.39e15 : 4.0e13;  // flop/s: tcgen05 bf16 vs SIMT fp32
  const double bw = 6.5e12;                                     // HBM bytes/s
  const double elt = dtype == ISOPO_BF16 ? 2.0 : 4.0;
  const double N = (double)d_in * (double)d_out;
  const double t_gram = (double)(d_in + d_out) * (double)T * (double)T / peak;
  const double t_mat = (double)B * (double)B * N / peak + 3.0 * elt * (double)B * N / bw;
  return t_gram < t_mat ? ISOPO_PATH_GRAM : ISOPO_PATH_MATERIALISE;
}

size_t isopo_workspace_bytes(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, isopo_path path) {
  if (!sizes_ok(dtype, T, d_in, d_out, B)) return 0;
  if (path != ISOPO_PATH_AUTO && path != ISOPO_PATH_GRAM && path != ISOPO_PATH_MATERIALISE) return 0;
  return ws_layout(dtype, T, d_in, d_out, B, resolve_path(dtype, T, d_in, d_out, B, path)).total;
}

isopo_status isopo_layer_gram(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                              const int64_t* seq_offsets_host, int B, isopo_path path, float* K, void* ws,
                              size_t ws_bytes, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_layer_gram");
  if (!K || !info) return ISOPO_ERR_INVALID_ARG;
  isopo_status s = check_layer_args(X, dY, dtype, T, d_in, d_out, seq_offsets_host, B, path, ws);
  if (s != ISOPO_OK) return s;
  const isopo_path rp = resolve_path(dtype, T, d_in, d_out, B, path);
  if (dtype == ISOPO_BF16 && rp == ISOPO_PATH_MATERIALISE && B > 256) return ISOPO_ERR_UNSUPPORTED;
  const WsLayout L = ws_layout(dtype, T, d_in, d_out, B, rp);
  if (ws_bytes < L.total) return ISOPO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* w = (char*)ws;
  int64_t* off_dev = (int64_t*)(w + L.off_offsets);
  int32_t* tokseq = (int32_t*)(w + L.off_tokseq);
  WsTag* tag_dev = (WsTag*)(w + L.off_tag);
  if (dtype == ISOPO_BF16 && rp == ISOPO_PATH_MATERIALISE) {
    // the stored-gradient kernels need the offsets and the longest-first order, not the token map
    void* G = w + L.off_G;
    int32_t* order = (int32_t*)(w + L.off_order);
    s = launch_prep_stored(seq_offsets_host, B, make_ws_tag(dtype, T, d_in, d_out, B, seq_offsets_host), off_dev, order,
                           tag_dev, K, st);
    if (s != ISOPO_OK) return s;
    const StoreFmt fmt = store_fmt(L, B, ws);
    if (fmt.split) {
      s = launch_seq_scales(X, dY, d_in, d_out, off_dev, B, (float*)fmt.scales, fmt.kdiag, st);
      if (s != ISOPO_OK) return s;
    }
    s = bf16_seq_grad(X, dY, T, d_in, d_out, seq_offsets_host, off_dev, order, B, L, G, fmt, info, st);
    if (s != ISOPO_OK) return s;
    return bf16_ntk(G, L, B, K, /*k_is_zero=*/true, deterministic_mode() ? (float*)(w + L.off_kpart) : nullptr, fmt, info, st);
  }
  s = launch_prep(seq_offsets_host, B, T, off_dev, tokseq, st);
  if (s != ISOPO_OK) return s;
  if (dtype == ISOPO_F32) {
    if (rp == ISOPO_PATH_GRAM)
      return f32_gram((const float*)X, (const float*)dY, T, d_in, d_out, tokseq, B, (double*)(w + L.off_kacc), K, st);
    s = store_tag(make_ws_tag(dtype, T, d_in, d_out, B, seq_offsets_host), tag_dev, st);
    if (s != ISOPO_OK) return s;
    float* G = (float*)(w + L.off_G);
    s = f32_seq_grad((const float*)X, (const float*)dY, d_in, d_out, off_dev, B, G, st);
    if (s != ISOPO_OK) return s;
    return f32_ntk(G, L.n_pad, B, K, st);
  }
  return bf16_gram(X, dY, T, d_in, d_out, tokseq, B, K, info, st);
}

isopo_status isopo_layer_gram_shared_x(const void* X, int n_proj, const void* const* dY, const int* d_out, isopo_dtype dtype,
                                       int64_t T, int d_in, const int64_t* seq_offsets_host, int B, float* const* K,
                                       void* ws, size_t ws_bytes, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_layer_gram_shared_x");
  if (!dY || !d_out || !K || !info || n_proj < 1 || n_proj > 3) return ISOPO_ERR_INVALID_ARG;
  if (dtype != ISOPO_BF16) return ISOPO_ERR_UNSUPPORTED;
  int d_max = 0;
  for (int h = 0; h < n_proj; ++h) {
    if (!K[h]) return ISOPO_ERR_INVALID_ARG;
    isopo_status s = check_layer_args(X, dY[h], dtype, T, d_in, d_out[h], seq_offsets_host, B, ISOPO_PATH_GRAM, ws);
    if (s != ISOPO_OK) return s;
    d_max = std::max(d_max, d_out[h]);
  }
  const WsLayout L = ws_layout(dtype, T, d_in, d_max, B, ISOPO_PATH_GRAM);
  if (ws_bytes < L.total) return ISOPO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* w = (char*)ws;
  int32_t* tokseq = (int32_t*)(w + L.off_tokseq);
  isopo_status s = launch_prep(seq_offsets_host, B, T, (int64_t*)(w + L.off_offsets), tokseq, st);
  if (s != ISOPO_OK) return s;
  return bf16_gram_shared(X, dY, T, d_in, d_out, n_proj, tokseq, B, K, info, st);
}

isopo_status isopo_layer_gram_shared_x_stored(const void* X, int n_proj, const void* const* dY, const int* d_out,
                                              isopo_dtype dtype, int64_t T, int d_in, const int64_t* seq_offsets_host, int B,
                                              float* const* K, void* const* ws, const size_t* ws_bytes, int32_t* info,
                                              void* cuda_stream) {
  ApiRange nvtx_range("isopo_layer_gram_shared_x_stored");
  if (!dY || !d_out || !K || !ws || !ws_bytes || !info || n_proj < 1 || n_proj > 3) return ISOPO_ERR_INVALID_ARG;
  if (dtype != ISOPO_BF16 || B > 256) return ISOPO_ERR_UNSUPPORTED;
  WsLayout L[3];
  WsTag tag[3];
  int64_t* off_dev[3];
  int32_t* order[3];
  WsTag* tag_dev[3];
  void* G[3];
  StoreFmt fmt[3];
  bool pairs_fit = true;
  for (int h = 0; h < n_proj; ++h) {
    if (!K[h]) return ISOPO_ERR_INVALID_ARG;
    isopo_status s = check_layer_args(X, dY[h], dtype, T, d_in, d_out[h], seq_offsets_host, B, ISOPO_PATH_MATERIALISE, ws[h]);
    if (s != ISOPO_OK) return s;
    for (int g = 0; g < h; ++g)
      if (ws[g] == ws[h]) return ISOPO_ERR_INVALID_ARG;  // every projection keeps its own gradients
    L[h] = ws_layout(dtype, T, d_in, d_out[h], B, ISOPO_PATH_MATERIALISE);
    if (ws_bytes[h] < L[h].total) return ISOPO_ERR_WORKSPACE;
    char* w = (char*)ws[h];
    tag[h] = make_ws_tag(dtype, T, d_in, d_out[h], B, seq_offsets_host);
    off_dev[h] = (int64_t*)(w + L[h].off_offsets);
    order[h] = (int32_t*)(w + L[h].off_order);
    tag_dev[h] = (WsTag*)(w + L[h].off_tag);
    G[h] = w + L[h].off_G;
    fmt[h] = store_fmt(L[h], B, ws[h]);
    pairs_fit = pairs_fit && (L[h].tiles_m % 2 == 0 || L[h].tiles_m >= 7);
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  isopo_status s = launch_prep_stored_multi(seq_offsets_host, B, n_proj, tag, off_dev, order, tag_dev, K, st);
  if (s != ISOPO_OK) return s;
  for (int h = 0; h < n_proj; ++h)
    if (fmt[h].split) {
      s = launch_seq_scales(X, dY[h], d_in, d_out[h], off_dev[0], B, (float*)fmt[h].scales, fmt[h].kdiag, st);
      if (s != ISOPO_OK) return s;
    }
  if (pairs_fit) {
    s = bf16_seq_grad_pair_shared(X, n_proj, dY, d_out, T, d_in, off_dev[0], order[0], B, L, G, fmt, info, st);
    if (s != ISOPO_OK) return s;
  } else {  // a projection with an odd, small number of 128-row tiles would idle half of its pairs: one launch each
    for (int h = 0; h < n_proj; ++h) {
      s = bf16_seq_grad(X, dY[h], T, d_in, d_out[h], seq_offsets_host, off_dev[h], order[h], B, L[h], G[h], fmt[h], info, st);
      if (s != ISOPO_OK) return s;
    }
  }
  for (int h = 0; h < n_proj; ++h) {
    float* kpart = deterministic_mode() ? (float*)((char*)ws[h] + L[h].off_kpart) : nullptr;
    s = bf16_ntk(G[h], L[h], B, K[h], /*k_is_zero=*/true, kpart, fmt[h], info, st);
    if (s != ISOPO_OK) return s;
  }
  return ISOPO_OK;
}

size_t isopo_sampled_workspace_bytes(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, int n_samples) {
  if (!sizes_ok(dtype, T, d_in, d_out, B) || n_samples < 1 || n_samples > ISOPO_MAX_SAMPLES) return 0;
  return sampled_layout(dtype, T, d_in, d_out, B, n_samples).total;
}

isopo_status isopo_sampled_coefficients(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                                        const int64_t* seq_offsets_host, int B, const int64_t* sample_rows_host,
                                        int n_samples, const float* A, float lambda, float* coeffs, float* F2, void* ws,
                                        size_t ws_bytes, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_sampled_coefficients");
  if (!A || !coeffs || !info || !sample_rows_host) return ISOPO_ERR_INVALID_ARG;
  if (!(lambda >= 0.0f)) return ISOPO_ERR_INVALID_ARG;
  isopo_status s = check_layer_args(X, dY, dtype, T, d_in, d_out, seq_offsets_host, B, ISOPO_PATH_GRAM, ws);
  if (s != ISOPO_OK) return s;
  if (n_samples < 1 || n_samples > ISOPO_MAX_SAMPLES) return ISOPO_ERR_INVALID_ARG;
  for (int j = 0; j < n_samples; ++j)
    if (sample_rows_host[j] < 0 || sample_rows_host[j] >= T) return ISOPO_ERR_INVALID_ARG;
  const SampledLayout S = sampled_layout(dtype, T, d_in, d_out, B, n_samples);
  if (ws_bytes < S.total) return ISOPO_ERR_WORKSPACE;
  const WsLayout L = ws_layout(dtype, T, d_in, d_out, B, ISOPO_PATH_GRAM);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* w = (char*)ws;
  int32_t* tokseq = (int32_t*)(w + L.off_tokseq);
  s = launch_prep(seq_offsets_host, B, T, (int64_t*)(w + L.off_offsets), tokseq, st);
  if (s != ISOPO_OK) return s;
  return sampled_coefficients(X, dY, dtype, T, d_in, d_out, tokseq, B, sample_rows_host, n_samples, w, S, A, lambda, coeffs,
                              F2, info, st);
}

isopo_status isopo_transform_advantages(const float* K, const float* A, int B, isopo_variant variant, float lambda,
                                        const float* opt_pqr_regs, float* coeffs, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_advantages");
  if (!K || !A || !coeffs || !info || B < 1) return ISOPO_ERR_INVALID_ARG;
  if ((int)variant < 0 || (int)variant > (int)ISOPO_VAR_NORMALISED_RAW) return ISOPO_ERR_INVALID_ARG;
  if (!(lambda >= 0.0f)) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_GENERAL && !opt_pqr_regs) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_INTERACTING && B > 256) return ISOPO_ERR_UNSUPPORTED;
  return transform(K, A, B, variant, lambda, opt_pqr_regs, nullptr, coeffs, info, (cudaStream_t)cuda_stream);
}

size_t isopo_transform_large_workspace_bytes(int B) {
  return B >= 1 && B <= ISOPO_MAX_LARGE_SEQS ? transform_large_workspace_bytes(B) : 0;
}

isopo_status isopo_transform_advantages_large(const float* K, const float* A, int B, float lambda, float* coeffs,
                                              void* workspace, size_t workspace_bytes, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_advantages_large");
  if (!K || !A || !coeffs || !info || !workspace || B < 1) return ISOPO_ERR_INVALID_ARG;
  if (!(lambda >= 0.0f) || ((uintptr_t)workspace & 15)) return ISOPO_ERR_INVALID_ARG;
  if (B > ISOPO_MAX_LARGE_SEQS) return ISOPO_ERR_UNSUPPORTED;
  if (workspace_bytes < transform_large_workspace_bytes(B)) return ISOPO_ERR_WORKSPACE;
  return transform_large(K, A, B, lambda, coeffs, (float*)workspace, info, (cudaStream_t)cuda_stream);
}

isopo_status isopo_reg_ema_update(const float* K, int B, float decay, float* state, void* cuda_stream) {
  ApiRange nvtx_range("isopo_reg_ema_update");
  if (!K || !state || B < 1 || !(decay >= 0.0f && decay < 1.0f)) return ISOPO_ERR_INVALID_ARG;
  return reg_ema_update(K, B, decay, state, (cudaStream_t)cuda_stream);
}

isopo_status isopo_transform_advantages_rel(const float* K, const float* A, int B, isopo_variant variant, float factor,
                                            const float* opt_pqr_factors, const float* state, float* coeffs,
                                            int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_advantages_rel");
  if (!K || !A || !coeffs || !info || !state || B < 1) return ISOPO_ERR_INVALID_ARG;
  if ((int)variant < 0 || (int)variant > (int)ISOPO_VAR_NORMALISED_RAW) return ISOPO_ERR_INVALID_ARG;
  if (!(factor >= 0.0f)) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_GENERAL && !opt_pqr_factors) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_INTERACTING && B > 256) return ISOPO_ERR_UNSUPPORTED;
  return transform(K, A, B, variant, factor, opt_pqr_factors, state, coeffs, info, (cudaStream_t)cuda_stream);
}

isopo_status isopo_transform_advantages_batched(int n_layers, const float* const* K, const float* A, int B,
                                                isopo_variant variant, const float* lambda,
                                                const float* opt_pqr_regs, const float* const* states,
                                                float* const* coeffs, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_advantages_batched");
  if (n_layers < 1 || n_layers > ISOPO_MAX_BATCH) return ISOPO_ERR_INVALID_ARG;
  if (!K || !A || !lambda || !coeffs || !info || B < 1) return ISOPO_ERR_INVALID_ARG;
  if ((int)variant < 0 || (int)variant > (int)ISOPO_VAR_NORMALISED_RAW) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_GENERAL && !opt_pqr_regs) return ISOPO_ERR_INVALID_ARG;
  if (variant == ISOPO_VAR_INTERACTING && B > 256) return ISOPO_ERR_UNSUPPORTED;
  for (int l = 0; l < n_layers; ++l) {
    if (!K[l] || !coeffs[l] || !(lambda[l] >= 0.0f) || (states && !states[l])) return ISOPO_ERR_INVALID_ARG;
  }
  return transform_batched(n_layers, K, A, B, variant, lambda, opt_pqr_regs, states, coeffs, info,
                           (cudaStream_t)cuda_stream);
}

isopo_status isopo_selftest_bounded_wait(int64_t limit_clocks, int32_t* info, int32_t* roles_at_teardown, void* cuda_stream) {
  ApiRange nvtx_range("isopo_selftest_bounded_wait");
  if (!info || !roles_at_teardown || limit_clocks < 1 || limit_clocks > ((int64_t)1 << 28)) return ISOPO_ERR_INVALID_ARG;
  return wait_probe((long long)limit_clocks, info, roles_at_teardown, (cudaStream_t)cuda_stream);
}

size_t isopo_spectral_workspace_bytes(void) { return spectral_workspace_bytes(); }

isopo_status isopo_transform_spectral(const float* K, const float* A, int B, float lambda, float rel_cutoff,
                                      float* coeffs, float* eigenvalues, void* ws, size_t ws_bytes, int32_t* info,
                                      void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_spectral");
  if (!K || !A || !coeffs || !ws || !info || B < 1) return ISOPO_ERR_INVALID_ARG;
  if (!(lambda >= 0.0f) || !(rel_cutoff >= 0.0f && rel_cutoff < 1.0f)) return ISOPO_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 15) return ISOPO_ERR_INVALID_ARG;
  if (B > 256) return ISOPO_ERR_UNSUPPORTED;
  if (ws_bytes < spectral_workspace_bytes()) return ISOPO_ERR_WORKSPACE;
  return spectral(K, A, B, lambda, rel_cutoff, coeffs, eigenvalues, ws, info, (cudaStream_t)cuda_stream);
}

isopo_status isopo_transform_spectral_batched(int n_layers, const float* const* K, const float* A, int B,
                                              const float* lambda, float rel_cutoff, float* const* coeffs,
                                              float* const* eigenvalues, void* ws, size_t ws_bytes, int32_t* info,
                                              void* cuda_stream) {
  ApiRange nvtx_range("isopo_transform_spectral_batched");
  if (n_layers < 1 || n_layers > ISOPO_MAX_BATCH) return ISOPO_ERR_INVALID_ARG;
  if (!K || !A || !lambda || !coeffs || !ws || !info || B < 1) return ISOPO_ERR_INVALID_ARG;
  if (!(rel_cutoff >= 0.0f && rel_cutoff < 1.0f) || ((uintptr_t)ws & 15)) return ISOPO_ERR_INVALID_ARG;
  if (B > 256) return ISOPO_ERR_UNSUPPORTED;
  for (int l = 0; l < n_layers; ++l)
    if (!K[l] || !coeffs[l] || !(lambda[l] >= 0.0f)) return ISOPO_ERR_INVALID_ARG;
  if (ws_bytes < (size_t)n_layers * spectral_workspace_bytes()) return ISOPO_ERR_WORKSPACE;
  return spectral_batched(n_layers, K, A, B, lambda, rel_cutoff, coeffs, eigenvalues, ws, info,
                          (cudaStream_t)cuda_stream);
}

isopo_status isopo_weight_grad(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                               const float* coeffs, const int64_t* seq_offsets_host, int B, isopo_path path,
                               float* dW, float beta, void* ws, size_t ws_bytes, int32_t* info, void* cuda_stream) {
  ApiRange nvtx_range("isopo_weight_grad");
  if (!coeffs || !dW || !info) return ISOPO_ERR_INVALID_ARG;
  if (beta != 0.0f && beta != 1.0f) return ISOPO_ERR_INVALID_ARG;
  isopo_status s = check_layer_args(X, dY, dtype, T, d_in, d_out, seq_offsets_host, B, path, ws);
  if (s != ISOPO_OK) return s;
  const isopo_path rp = resolve_path(dtype, T, d_in, d_out, B, path);
  if (dtype == ISOPO_BF16 && rp == ISOPO_PATH_MATERIALISE && B > 256) return ISOPO_ERR_UNSUPPORTED;
  const WsLayout L = ws_layout(dtype, T, d_in, d_out, B, rp);
  if (ws_bytes < L.total) return ISOPO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* w = (char*)ws;
  if (rp == ISOPO_PATH_MATERIALISE) {
    // the kernels compare the tag isopo_layer_gram left with the one of this call and touch nothing on a mismatch
    const WsTag tag = make_ws_tag(dtype, T, d_in, d_out, B, seq_offsets_host);
    const WsTag* tag_dev = (const WsTag*)(w + L.off_tag);
    if (dtype == ISOPO_F32)
      return f32_combine((const float*)(w + L.off_G), L.n_pad, B, coeffs, dW, beta, tag_dev, tag, info, st);
    return bf16_combine(w + L.off_G, L, d_in, d_out, B, coeffs, dW, beta, tag_dev, tag, store_fmt(L, B, ws), info, st);
  }
  // GEMM over all tokens: refresh the token -> sequence map so the call also works on its own.
  int64_t* off_dev = (int64_t*)(w + L.off_offsets);
  int32_t* tokseq = (int32_t*)(w + L.off_tokseq);
  if (dtype == ISOPO_F32) {
    s = launch_prep(seq_offsets_host, B, T, off_dev, tokseq, st);
    if (s != ISOPO_OK) return s;
    return f32_weight_grad((const float*)X, (const float*)dY, T, d_in, d_out, coeffs, tokseq, dW, beta, st);
  }
  if (bf16_weight_grad_fold_applies(T, d_in, d_out, B)) {
    s = store_i64(seq_offsets_host, (int64_t)B + 1, off_dev, st);
    if (s != ISOPO_OK) return s;
    return bf16_weight_grad_fold(X, dY, T, d_in, d_out, off_dev, coeffs, B, dW, beta, info, st);
  }
  // one scale per token, so that the kernel's scaler warps need a single independent load per row
  float* tokscale = (float*)tokseq;
  s = launch_tokscale(seq_offsets_host, B, T, off_dev, coeffs, tokscale, st);
  if (s != ISOPO_OK) return s;
  void* scaled = w + L.off_scaled;
  return bf16_weight_grad(X, dY, T, d_in, d_out, tokscale, scaled, dW, beta, info, st);
}

}  // extern "C"
