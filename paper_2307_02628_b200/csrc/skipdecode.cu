// Host side of the C ABI declared in include/skipdecode.h: argument checks, the
// integer schedule, arena carving, and the launch sequence of one prefill / one
// decode step (replayed from a CUDA graph per step shape when enabled).
#include "../../include/skipdecode.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <tuple>
#include <type_traits>
#include <vector>

#include "kernels.cuh"
#include "gemm_tc.cuh"
#include "gemm_persist.cuh"
#include "sample.cuh"
#include "attn_prefill.cuh"
#include "attn_stream.cuh"

namespace {

using bf16 = __nv_bfloat16;

constexpr size_t kAlign = 256;
constexpr int kPrefillTokens = 4096;   // query rows per prefill pass (whole batch rows)
constexpr int kMinChunk = 32;          // smallest split of the decode attention, in keys

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Arena {            // byte offsets into the caller's arena
  std::vector<size_t> k_off, v_off;
  std::vector<size_t> wp_qkv, wp_o, wp_fc1, wp_fc2;   // tile-packed copies of the weight matrices (bf16 mode)
  size_t wp_head;
  bool packable;
  std::vector<int> cap;
  size_t x, u, qkv, o, y, part_acc, part_ml, counters, row_index, ids, logits, scalars, pad, rows, splitk_ws, splitk_count, total;
  int rows_max;
  size_t part_slots;
};

struct Timed { cudaEvent_t a, b; int cls; };

}  // namespace

struct sd_handle {
  sd_config cfg;
  sd_plan plan;
  int hd, esize;
  std::vector<const void*> ln1_g, ln1_b, w_qkv, b_qkv, w_o, b_o, ln2_g, ln2_b, w_fc1, b_fc1, w_fc2, b_fc2;
  const void *tok_emb, *pos_emb, *lnf_g, *lnf_b, *lm_head;
  char* arena;
  Arena A;
  cudaStream_t stream;
  // schedule / sequence state
  std::vector<int> n_active, top_begin;
  int warmup = 0, gen_len = 0;
  bool have_schedule = false, have_prefill = false;
  int B = 0, P = 0, next_pos = 0;
  // ragged batches: left padding per row (host copy; device copy in the arena) and the rows still generating
  std::vector<int> pad, rows;
  bool have_pad = false, have_rows = false;
  bool prefill_attn_ready = false, sample_ready = false;   // large dynamic shared memory enabled for these kernels
  int n_rows() const { return have_rows ? (int)rows.size() : B; }
  const int* d_pad() const { return have_pad ? at<int>(A.pad) : nullptr; }
  const int* d_rows() const { return have_rows ? at<int>(A.rows) : nullptr; }
  int64_t steps = 0, layer_steps = 0, launches = 0;
  // options
  int opt_graphs = 1, opt_chunk = 0, opt_gemm = 0, opt_timing = 0, opt_pdl = SD_PDL_DEFAULT, opt_prefill = 1;
  int opt_attn_staged = 1;   // decode attention in bf16 storage through the shared-memory ring where that pays; 0: never
  unsigned attn_stream_ready = 0;   // bit per head size whose shared-memory attributes are set
  bool packed = false;       // the arena holds tile-packed copies of the weight matrices
  // graphs: key = (B, n, warmup, chunk, n_chunks, ids ptr, logits ptr)
  struct Graph { cudaGraphExec_t exec; int64_t nodes; };
  std::map<std::tuple<int, int, int, int, int, const void*, const void*>, Graph> graphs;
  // timing
  std::vector<Timed> timed;
  double k_ms[SD_K_COUNT] = {};
  int64_t k_launches[SD_K_COUNT] = {};
  sd::TcContext tc;
  sd::PersistContext persist;

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(arena + off); }
  int* status() const { return at<int>(A.scalars); }
  int* d_pos() const { return at<int>(A.scalars) + 1; }
};

namespace {

bool valid_config(const sd_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->d_ffn < 8 || c->vocab < 1 || c->max_pos < 1) return false;
  if (c->max_batch < 1 || c->max_prompt < 1 || c->max_gen < 1) return false;
  if (c->dtype != SD_DTYPE_FP32 && c->dtype != SD_DTYPE_BF16) return false;
  if (c->d_model % c->n_heads) return false;
  const int hd = c->d_model / c->n_heads;
  if (hd != 32 && hd != 64 && hd != 128) return false;
  if (c->d_model % 8 || c->d_ffn % 8) return false;
  if (!(c->ln_eps > 0.f)) return false;
  if ((int64_t)c->max_prompt + c->max_gen > c->max_pos) return false;
  return true;
}

bool valid_schedule_args(int n_layers, int mx, int mn, int w, int G) {
  return 0 <= w && w < mn && mn <= mx && mx <= n_layers && G >= 1;
}

// Section 2.3: the line (1 - t) max + t min with t = g / (G - 1), rounded to nearest with
// halves up, in integers: min + floor((2 (G-1-g) (max-min) + (G-1)) / (2 (G-1))).
int budget_at(int mx, int mn, int g, int G) {
  if (G == 1) return mx;
  const int64_t den = G - 1, D = mx - mn;
  return mn + (int)((2 * (den - g) * D + den) / (2 * den));
}

// Power-law variant (Section 2.3 names it as another possible decay): min + (max - min) (1 - t)^alpha
// with t = g / (G - 1) and an integer exponent, rounded to nearest with halves up, in integers:
// min + floor((2 D (G-1-g)^alpha + (G-1)^alpha) / (2 (G-1)^alpha)).  alpha = 1 is the linear schedule.
// True when 2 (max - min) (G-1)^alpha + (G-1)^alpha fits the 128-bit arithmetic below with room to spare.
bool power_args_fit(int mx, int mn, int G, int alpha) {
  if (G <= 2) return true;
  const unsigned __int128 limit = (((unsigned __int128)1) << 124) / (unsigned __int128)(2 * (mx - mn) + 2);
  unsigned __int128 den = 1;
  for (int i = 0; i < alpha; ++i) {
    if (den > limit / (unsigned)(G - 1)) return false;
    den *= (unsigned)(G - 1);
  }
  return true;
}

int budget_power_at(int mx, int mn, int g, int G, int alpha) {
  if (G == 1) return mx;
  const unsigned __int128 den1 = G - 1, num1 = G - 1 - g;
  unsigned __int128 den = 1, num = 1;
  for (int i = 0; i < alpha; ++i) { den *= den1; num *= num1; }
  const unsigned __int128 D = mx - mn;
  return mn + (int)((2 * D * num + den) / (2 * den));
}

// number of generated indices at which layer l runs under (mx, mn, w, G)
void layer_counts(int L, int mx, int mn, int w, int G, std::vector<int>& count) {
  count.assign(L, 0);
  for (int g = 0; g < G; ++g) {
    const int n = budget_at(mx, mn, g, G), top = L - (n - w);
    for (int l = 0; l < L; ++l)
      if (l < w || l >= top) ++count[l];
  }
}

bool valid_plan(const sd_config* c, const sd_plan* p) {
  return p && valid_schedule_args(c->n_layers, p->max_layers, p->min_layers, p->warmup, p->gen_len) &&
         p->gen_len <= c->max_gen;
}

void carve(const sd_config& c, const sd_plan& p, Arena& A) {
  const int L = c.n_layers, d = c.d_model, H = c.n_heads, hd = d / H;
  const size_t e = c.dtype == SD_DTYPE_FP32 ? 4 : 2;
  std::vector<int> count;
  layer_counts(L, p.max_layers, p.min_layers, p.warmup, p.gen_len, count);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  A.k_off.resize(L); A.v_off.resize(L); A.cap.resize(L);
  for (int l = 0; l < L; ++l) {
    A.cap[l] = c.max_prompt + (p.full_capacity ? c.max_gen : count[l]);
    const size_t bytes = (size_t)c.max_batch * H * A.cap[l] * hd * e;
    A.k_off[l] = take(bytes);
    A.v_off[l] = take(bytes);
  }
  A.packable = c.dtype == SD_DTYPE_BF16 && d % 64 == 0 && c.d_ffn % 64 == 0;
  A.wp_qkv.assign(L, 0); A.wp_o.assign(L, 0); A.wp_fc1.assign(L, 0); A.wp_fc2.assign(L, 0);
  A.wp_head = 0;
  if (A.packable) {
    auto packed_bytes = [](size_t n, size_t k) { return (n + 255) / 256 * 256 * k * 2; };   // whole 256-row pairs of tiles
    for (int l = 0; l < L; ++l) {
      A.wp_qkv[l] = take(packed_bytes(3 * d, d));
      A.wp_o[l] = take(packed_bytes(d, d));
      A.wp_fc1[l] = take(packed_bytes(c.d_ffn, d));
      A.wp_fc2[l] = take(packed_bytes(d, c.d_ffn));
    }
    A.wp_head = take(packed_bytes(c.vocab, d));
  }
  const int chunk_rows = std::max(1, kPrefillTokens / c.max_prompt) * c.max_prompt;
  A.rows_max = std::max(c.max_batch, chunk_rows);
  const size_t R = A.rows_max;
  A.x = take(R * d * 4);
  A.u = take(R * d * 4);                 // GEMM operands: K floats, or K 16-bit slots, per row
  A.qkv = take(R * 3 * d * 4);
  A.o = take(R * d * 4);
  A.y = take(R * (size_t)c.d_ffn * 4);
  const int maxT = c.max_prompt + c.max_gen;
  A.part_slots = std::max((size_t)c.max_batch * H * ((maxT + kMinChunk - 1) / kMinChunk), R * H);
  A.part_acc = take(A.part_slots * hd * 4);
  A.part_ml = take(A.part_slots * 2 * 4);
  A.counters = take((R * H + 64) * 4);   // split-KV arrival counters, one per (row, head), then the persistent attention
                                         // kernel's work counter; all zero between launches
  A.row_index = take((size_t)c.max_batch * 4);
  A.ids = take((size_t)c.max_batch * 4);
  A.logits = take((size_t)c.max_batch * c.vocab * 4);
  A.scalars = take(256);
  A.pad = take((size_t)c.max_batch * 4);     // left-padding slots per batch row (ragged prompts)
  // batch rows still generating; a GEMM epilogue looks up whole token tiles (up to 127 entries past the
  // row count, results unused), so the array is that much longer than the batch
  A.rows = take(((size_t)c.max_batch + 128) * 4);
  // bf16 storage: parked partial tiles and arrival counters of the GEMMs that split K under a non-linear epilogue
  A.splitk_ws = A.splitk_count = 0;
  if (c.dtype == SD_DTYPE_BF16) {
    A.splitk_ws = take((size_t)sd::kSplitSlots * 128 * 128 * 4);
    A.splitk_count = take((size_t)sd::kSplitSlots * 4);
  }
  A.total = off;
}

__global__ void set_int_kernel(int* p, int v) { *p = v; }
__global__ void last_rows_kernel(int* idx, int n, int P) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) idx[i] = i * P + P - 1;
}

// ---- launch helpers -------------------------------------------------------------------

struct Launcher {
  sd_handle* h;
  bool timing;
  float* part_acc;        // split-KV partial accumulators and (max, sum) pairs of this launch sequence
  float* part_ml;
  int err = 0;
  int64_t count = 0;      // kernels enqueued through this launcher
  void begin(int cls) {
    if (!timing) return;
    Timed t; t.cls = cls;
    cudaEventCreate(&t.a); cudaEventCreate(&t.b);
    cudaEventRecord(t.a, h->stream);
    h->timed.push_back(t);
  }
  void cancel() {          // begin() was called but nothing was launched
    if (!timing) return;
    cudaEventDestroy(h->timed.back().a); cudaEventDestroy(h->timed.back().b);
    h->timed.pop_back();
  }
  void end() {
    ++count;
    if (cudaGetLastError() != cudaSuccess) err = SD_ERR_CUDA;
    if (timing) cudaEventRecord(h->timed.back().b, h->stream);
  }
};

// SD_OPT_PDL is a mask over kernel classes (bit = 1 << class): a kernel of a class whose bit is
// set is launched with the programmatic attribute, i.e. may begin before its predecessor ends.
bool pdl_for(const sd_handle* h, int cls) { return (h->opt_pdl >> cls) & 1; }

template <typename T>
void launch_gemm(Launcher& Lc, int cls, const T* A, const T* W, size_t packed_off, const T* bias, int M, int N, int K,
                 void* out, int ldo, int epi) {
  sd_handle* h = Lc.h;
  const T* Wp = h->packed ? h->at<T>(packed_off) : nullptr;
  h->tc.pdl = pdl_for(h, cls);
  Lc.begin(cls);
  bool done = false;
  if (std::is_same<T, bf16>::value && h->opt_gemm != 1) {
    if (!done) done = sd::persist_gemm(h->persist, h->tc, h->stream, A, W, bias, M, N, K, out, ldo, epi, h->status(), nullptr, Wp);
    if (!done) done = sd::tc_gemm(h->tc, h->stream, A, W, bias, M, N, K, out, ldo, epi, h->status(), nullptr, Wp);
  }
  if (!done) {
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    const int lda = K * sd::Operand<T>::PARTS;
    if (epi == sd::EPI_STORE_F32)
      sd::launch_kernel(pdl_for(h, cls), h->stream, sd::gemm_simt_kernel<T, sd::EPI_STORE_F32>, dim3(grid), dim3(256), 0, A, lda, W, K, bias, M, N, K, out, ldo);
    else if (epi == sd::EPI_RELU_T)
      sd::launch_kernel(pdl_for(h, cls), h->stream, sd::gemm_simt_kernel<T, sd::EPI_RELU_T>, dim3(grid), dim3(256), 0, A, lda, W, K, bias, M, N, K, out, ldo);
    else
      sd::launch_kernel(pdl_for(h, cls), h->stream, sd::gemm_simt_kernel<T, sd::EPI_RESIDUAL_F32>, dim3(grid), dim3(256), 0, A, lda, W, K, bias, M, N, K, out, ldo);
  }
  Lc.end();
}

// QKV projection with the K/V rows written straight into the cache by the GEMM epilogue
// (tensor-core path only).  Returns false when that path does not take the product.
template <typename T>
bool launch_qkv_to_cache(Launcher&, const T*, const T*, size_t, const T*, int, int, float*, T*, T*, int, sd::RowMap) { return false; }
template <>
bool launch_qkv_to_cache<bf16>(Launcher& Lc, const bf16* u, const bf16* W, size_t packed_off, const bf16* bias, int rows, int d, float* qkv,
                               bf16* Kc, bf16* Vc, int cap, sd::RowMap map) {
  sd_handle* h = Lc.h;
  if (h->opt_gemm == 1) return false;
  const sd::tc::QkvOut qo{Kc, Vc, d, h->cfg.n_heads, h->hd, cap, map, 0, nullptr};
  const bf16* Wp = h->packed ? h->at<bf16>(packed_off) : nullptr;
  h->tc.pdl = pdl_for(h, SD_K_GEMM_QKV);
  Lc.begin(SD_K_GEMM_QKV);
  bool done = false;
  if (!done) done = sd::persist_gemm(h->persist, h->tc, h->stream, u, W, bias, rows, 3 * d, d, qkv, 3 * d, sd::EPI_QKV_CACHE, h->status(), &qo, Wp);
  if (!done) done = sd::tc_gemm(h->tc, h->stream, u, W, bias, rows, 3 * d, d, qkv, 3 * d, sd::EPI_QKV_CACHE, h->status(), &qo, Wp);
  if (done) Lc.end(); else Lc.cancel();
  return done;
}

// Decode attention with K and V staged through shared memory (bf16 storage).  Returns false when the
// kernel cannot be prepared; the register-only kernel then takes the launch.
template <int HD>
bool launch_attention_stream(Launcher& Lc, const bf16* Kc, const bf16* Vc, int cap, int rows, sd::RowMap map, int chunk, int n_chunks) {
  sd_handle* h = Lc.h;
  constexpr int smem = sd::as::smem_bytes();
  const unsigned bit = HD == 128 ? 1u : HD == 64 ? 2u : 4u;
  if (!(h->attn_stream_ready & bit)) {       // per handle: the attributes belong to the handle's device
    if (cudaFuncSetAttribute(sd::attn_stream_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaFuncSetAttribute(sd::attn_stream_kernel<HD>, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    h->attn_stream_ready |= bit;
  }
  const int H = h->cfg.n_heads;
  Lc.begin(SD_K_ATTENTION);
  dim3 grid(rows * H, n_chunks);
  sd::launch_kernel(pdl_for(h, SD_K_ATTENTION), h->stream, sd::attn_stream_kernel<HD>, dim3(grid), dim3(sd::as::THREADS), smem,
                    (const float*)h->at<float>(h->A.qkv), 3 * h->cfg.d_model, Kc, Vc, cap, H, map, chunk, n_chunks, Lc.part_acc, Lc.part_ml,
                    h->at<int>(h->A.counters), h->at<bf16>(h->A.o), h->status());
  Lc.end();
  return true;
}

// Which decode-attention kernel takes a launch of rows x H (row, head) pairs in bf16 storage.  The staged kernel
// holds 3 blocks per SM, the register-only one 7, and a staged block needs a few microseconds before its first keys
// arrive.  Measured: it pays where the launch is many times its 3 x SMs slots and the rows are long (config 4: 2048
// pairs, 1025..1536 keys, +1.6 % tokens/s; config 5: 8192 pairs, 257..1280 keys, +0.6 %), is level at 512..1024 keys,
// loses at 60..160 keys (-2.3 %) and loses where the other kernel holds the whole launch in one wave (config 3: 1024
// pairs, -12 %).  The length that counts is the handle's maximum, so that the choice does not change inside a sequence.
bool attn_staged(const sd_handle* h, int rows) {
  if (h->cfg.dtype != SD_DTYPE_BF16 || !h->opt_attn_staged) return false;
  if ((long)rows * h->cfg.n_heads < 4L * sd::as::BLOCKS_PER_SM * h->tc.sm_count) return false;
  return h->opt_attn_staged == 2 || h->cfg.max_prompt + h->cfg.max_gen >= 1024;
}

template <typename T, int HD>
void launch_attention_hd(Launcher& Lc, const T* Kc, const T* Vc, int cap, int rows, sd::RowMap map, int chunk,
                         int n_chunks) {
  sd_handle* h = Lc.h;
  if constexpr (std::is_same<T, bf16>::value) {
    if (attn_staged(h, rows) && launch_attention_stream<HD>(Lc, Kc, Vc, cap, rows, map, chunk, n_chunks)) return;
  }
  const int H = h->cfg.n_heads;
  Lc.begin(SD_K_ATTENTION);
  dim3 grid(rows * H, n_chunks);
  sd::launch_kernel(pdl_for(h, SD_K_ATTENTION), h->stream, sd::attn_partial_kernel<T, HD, 4>, dim3(grid), dim3(128), 0, h->at<float>(h->A.qkv), 3 * h->cfg.d_model, Kc, Vc, cap, H, map, chunk, n_chunks, Lc.part_acc, Lc.part_ml,
      h->at<int>(h->A.counters), h->at<T>(h->A.o));
  Lc.end();
}

template <typename T>
void launch_attention(Launcher& Lc, const T* Kc, const T* Vc, int cap, int rows, sd::RowMap map, int chunk, int n_chunks) {
  switch (Lc.h->hd) {
    case 32: launch_attention_hd<T, 32>(Lc, Kc, Vc, cap, rows, map, chunk, n_chunks); break;
    case 64: launch_attention_hd<T, 64>(Lc, Kc, Vc, cap, rows, map, chunk, n_chunks); break;
    default: launch_attention_hd<T, 128>(Lc, Kc, Vc, cap, rows, map, chunk, n_chunks); break;
  }
}

// Prompt pass, bf16 storage, head size 64 or 128: tensor-core tiles over whole sequences.
template <int HD>
bool launch_attention_prefill_hd(Launcher& Lc, const bf16* Kc, const bf16* Vc, int cap, int n_seq, int P, int b0) {
  sd_handle* h = Lc.h;
  constexpr int smem = 2 * 2 * sd::PF_BN * HD * 2;
  if (!h->prefill_attn_ready) {              // per handle: the attribute belongs to the handle's device
    if (cudaFuncSetAttribute(sd::attn_prefill_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    h->prefill_attn_ready = true;
  }
  Lc.begin(SD_K_ATTENTION);
  dim3 grid((P + sd::PF_BM - 1) / sd::PF_BM, n_seq * h->cfg.n_heads);
  sd::launch_kernel(false, h->stream, sd::attn_prefill_kernel<HD>, grid, dim3(sd::PF_THREADS), smem, (const float*)h->at<float>(h->A.qkv),
                    3 * h->cfg.d_model, Kc, Vc, cap, h->cfg.n_heads, P, b0, h->d_pad(), h->at<bf16>(h->A.o));
  Lc.end();
  return true;
}
template <typename T>
bool launch_attention_prefill(Launcher& Lc, const T* Kc, const T* Vc, int cap, int n_seq, int P, int b0) {
  if constexpr (std::is_same<T, bf16>::value) {
    if (!Lc.h->opt_prefill) return false;
    if (Lc.h->hd == 128) return launch_attention_prefill_hd<128>(Lc, Kc, Vc, cap, n_seq, P, b0);
    if (Lc.h->hd == 64) return launch_attention_prefill_hd<64>(Lc, Kc, Vc, cap, n_seq, P, b0);
  }
  return false;
}

int ln_threads(int d) { return std::max(32, std::min(256, (d / 4 + 31) / 32 * 32)); }

// One decoder layer over `rows` query rows (Sections 2.1, 2.2): LN1 -> QKV -> append K,V at
// the rows' positions -> attention over cache positions 0..pos -> out-proj (+residual) ->
// LN2 -> fc1 + ReLU -> fc2 (+residual).
template <typename T>
void enqueue_layer(Launcher& Lc, int l, int rows, sd::RowMap map, int chunk, int n_chunks, int prompt_len = 0) {
  sd_handle* h = Lc.h;
  const sd_config& c = h->cfg;
  const int d = c.d_model, f = c.d_ffn;
  float* x = h->at<float>(h->A.x);
  T* u = h->at<T>(h->A.u);
  float* qkv = h->at<float>(h->A.qkv);
  T* o = h->at<T>(h->A.o);
  T* y = h->at<T>(h->A.y);
  T* Kc = h->at<T>(h->A.k_off[l]);
  T* Vc = h->at<T>(h->A.v_off[l]);
  const int cap = h->A.cap[l];

  Lc.begin(SD_K_LAYERNORM);
  sd::launch_kernel(pdl_for(h, SD_K_LAYERNORM), h->stream, sd::layernorm_kernel<T>, dim3(rows), dim3(ln_threads(d)), 0, x, (const T*)h->ln1_g[l], (const T*)h->ln1_b[l], u, d, c.ln_eps, nullptr);
  Lc.end();
  if (!launch_qkv_to_cache<T>(Lc, u, (const T*)h->w_qkv[l], h->A.wp_qkv[l], (const T*)h->b_qkv[l], rows, d, qkv, Kc, Vc, cap, map)) {
    launch_gemm<T>(Lc, SD_K_GEMM_QKV, u, (const T*)h->w_qkv[l], h->A.wp_qkv[l], (const T*)h->b_qkv[l], rows, 3 * d, d, qkv, 3 * d, sd::EPI_STORE_F32);
    Lc.begin(SD_K_KV_APPEND);
    sd::launch_kernel(pdl_for(h, SD_K_KV_APPEND), h->stream, sd::kv_append_kernel<T>, dim3(rows), dim3(256), 0, qkv, Kc, Vc, d, c.n_heads, h->hd, cap, map);
    Lc.end();
  }
  // prompt_len > 0: the rows are whole sequences of that length (the prompt pass)
  if (!(prompt_len > 0 && prompt_len <= cap && launch_attention_prefill<T>(Lc, Kc, Vc, cap, rows / prompt_len, prompt_len, map.b0)))
    launch_attention<T>(Lc, Kc, Vc, cap, rows, map, chunk, n_chunks);
  launch_gemm<T>(Lc, SD_K_GEMM_OUT, o, (const T*)h->w_o[l], h->A.wp_o[l], (const T*)h->b_o[l], rows, d, d, x, d, sd::EPI_RESIDUAL_F32);
  Lc.begin(SD_K_LAYERNORM);
  sd::launch_kernel(pdl_for(h, SD_K_LAYERNORM), h->stream, sd::layernorm_kernel<T>, dim3(rows), dim3(ln_threads(d)), 0, x, (const T*)h->ln2_g[l], (const T*)h->ln2_b[l], u, d, c.ln_eps, nullptr);
  Lc.end();
  launch_gemm<T>(Lc, SD_K_GEMM_FC1, u, (const T*)h->w_fc1[l], h->A.wp_fc1[l], (const T*)h->b_fc1[l], rows, f, d, y, f * sd::Operand<T>::PARTS, sd::EPI_RELU_T);
  launch_gemm<T>(Lc, SD_K_GEMM_FC2, y, (const T*)h->w_fc2[l], h->A.wp_fc2[l], (const T*)h->b_fc2[l], rows, d, f, x, d, sd::EPI_RESIDUAL_F32);
}

template <typename T>
void enqueue_embed(Launcher& Lc, const int32_t* ids, int rows, sd::RowMap map) {
  sd_handle* h = Lc.h;
  Lc.begin(SD_K_EMBED);
  sd::launch_kernel(pdl_for(h, SD_K_EMBED), h->stream, sd::embed_pos_kernel<T>, dim3(rows), dim3(256), 0, ids, (const T*)h->tok_emb, (const T*)h->pos_emb, h->at<float>(h->A.x),
                                                      h->cfg.d_model, h->cfg.vocab, h->cfg.max_pos, map, h->status());
  Lc.end();
}

// final LayerNorm of `rows` rows (gathered through row_index when given) and the LM head
template <typename T>
void enqueue_head(Launcher& Lc, int rows, const int* row_index, float* d_logits) {
  sd_handle* h = Lc.h;
  const sd_config& c = h->cfg;
  Lc.begin(SD_K_LAYERNORM);
  sd::launch_kernel(pdl_for(h, SD_K_LAYERNORM), h->stream, sd::layernorm_kernel<T>, dim3(rows), dim3(ln_threads(c.d_model)), 0, h->at<float>(h->A.x), (const T*)h->lnf_g, (const T*)h->lnf_b,
                                                                        h->at<T>(h->A.u), c.d_model, c.ln_eps, row_index);
  Lc.end();
  launch_gemm<T>(Lc, SD_K_LM_HEAD, h->at<T>(h->A.u), (const T*)h->lm_head, h->A.wp_head, (const T*)nullptr, rows, c.vocab, c.d_model,
                 d_logits, c.vocab, sd::EPI_STORE_F32);
}

// Keys per split for a decode step with `rows` x H query-heads and T keys each: the candidate
// that minimises (waves of blocks) x (keys a block walks + a fixed cost in key units).  Many
// (row, head) pairs -> one block walks the whole row (no partials at all); few -> short
// splits so that every SM has blocks.
int pick_chunk(const sd_handle* h, int rows, int T) {
  if (h->opt_chunk > 0) return h->opt_chunk;
  const long rh = (long)rows * h->cfg.n_heads;
  // blocks resident at once: 7 per SM by registers for the register-only kernel, 3 rings per SM for the staged one
  const long slots = (attn_staged(h, rows) ? (long)sd::as::BLOCKS_PER_SM : 7L) * h->tc.sm_count;
  const int whole = (h->cfg.max_prompt + h->cfg.max_gen + kMinChunk - 1) / kMinChunk * kMinChunk;
  int best = whole;
  double best_cost = 1e30;
  for (int chunk : {whole, 1024, 768, 512, 256, 128, 64, kMinChunk}) {
    if (chunk > whole) continue;
    const long n_chunks = (T + chunk - 1) / chunk;
    const long waves = (rh * n_chunks + slots - 1) / slots;
    const double cost = (double)waves * (std::min(chunk, T) + 48);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = chunk; }
  }
  return best;
}

template <typename T>
int enqueue_decode(sd_handle* h, const int32_t* d_ids, int pos, bool pos_from_device, float* d_logits, int n, int chunk,
                   int n_chunks, bool timing, int64_t* launched, float* part_acc = nullptr, float* part_ml = nullptr) {
  Launcher Lc{h, timing, part_acc ? part_acc : h->at<float>(h->A.part_acc), part_ml ? part_ml : h->at<float>(h->A.part_ml)};
  const int L = h->cfg.n_layers, w = h->warmup, top = L - (n - w);
  sd::RowMap map{1, 0, pos, pos_from_device ? h->d_pos() : nullptr, h->d_rows(), h->d_pad()};
  const int rows = h->n_rows();
  enqueue_embed<T>(Lc, d_ids, rows, map);
  for (int l = 0; l < L; ++l) {
    if (!(l < w || l >= top)) continue;             // bypassed layer: identity, no K/V written (Section 2.4)
    enqueue_layer<T>(Lc, l, rows, map, chunk, n_chunks);
  }
  enqueue_head<T>(Lc, rows, nullptr, d_logits);
  *launched = Lc.count;
  return Lc.err;
}

template <typename T>
int run_prefill(sd_handle* h, const int32_t* d_tokens, int B, int P, float* d_logits) {
  Launcher Lc{h, h->opt_timing != 0, h->at<float>(h->A.part_acc), h->at<float>(h->A.part_ml)};
  const int L = h->cfg.n_layers;
  // whole batch rows per pass, from the rows the activation buffers were carved for (P <= max_prompt <= rows_max)
  const int per = std::max(1, h->A.rows_max / P);
  for (int b0 = 0; b0 < B; b0 += per) {
    const int nb = std::min(per, B - b0), rows = nb * P;
    sd::RowMap map{P, b0, 0, nullptr, nullptr, h->d_pad()};
    enqueue_embed<T>(Lc, d_tokens + (size_t)b0 * P, rows, map);
    const int chunk = (P + kMinChunk - 1) / kMinChunk * kMinChunk;   // one split: every row reads keys 0..pos
    for (int l = 0; l < L; ++l) enqueue_layer<T>(Lc, l, rows, map, chunk, 1, P);
    last_rows_kernel<<<(nb + 127) / 128, 128, 0, h->stream>>>(h->at<int>(h->A.row_index), nb, P);
    enqueue_head<T>(Lc, nb, h->at<int>(h->A.row_index), d_logits + (size_t)b0 * h->cfg.vocab);
    Lc.count += 1;
  }
  h->launches += Lc.count;
  return Lc.err;
}

void collect_timing(sd_handle* h) {
  if (h->timed.empty()) return;
  cudaStreamSynchronize(h->stream);
  for (Timed& t : h->timed) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, t.a, t.b) == cudaSuccess) { h->k_ms[t.cls] += ms; h->k_launches[t.cls] += 1; }
    cudaEventDestroy(t.a); cudaEventDestroy(t.b);
  }
  h->timed.clear();
}

void drop_graphs(sd_handle* h) {
  for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second.exec);
  h->graphs.clear();
}

int decode_step_impl(sd_handle* h, const int32_t* d_ids, int position, float* d_logits) {
  if (!h || !d_ids || !d_logits) return SD_ERR_ARG;
  if (!h->have_schedule || !h->have_prefill) return SD_ERR_STATE;
  const int g = position - h->P;
  if (position != h->next_pos || g < 0 || g >= h->gen_len || position >= h->cfg.max_pos) return SD_ERR_POSITION;
  const int n = h->n_active[g];
  const int T = position + 1;
  const int chunk = pick_chunk(h, h->n_rows(), T);
  const int n_chunks = (T + chunk - 1) / chunk;
  const bool bf = h->cfg.dtype == SD_DTYPE_BF16;
  int err = 0;
  int64_t launched = 0;
  const bool graphs = h->opt_graphs && !h->opt_timing && !h->tc.test_expire && h->stream != nullptr;
  if (!graphs) {
    err = bf ? enqueue_decode<bf16>(h, d_ids, position, false, d_logits, n, chunk, n_chunks, h->opt_timing != 0, &launched)
             : enqueue_decode<float>(h, d_ids, position, false, d_logits, n, chunk, n_chunks, h->opt_timing != 0, &launched);
  } else {
    auto key = std::make_tuple(h->n_rows(), n, h->warmup, chunk, n_chunks, (const void*)d_ids, (const void*)d_logits);
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
      if (h->graphs.size() >= 256) drop_graphs(h);
      cudaGraph_t graph = nullptr;
      if (cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
      err = bf ? enqueue_decode<bf16>(h, d_ids, position, true, d_logits, n, chunk, n_chunks, false, &launched)
               : enqueue_decode<float>(h, d_ids, position, true, d_logits, n, chunk, n_chunks, false, &launched);
      const cudaError_t ce = cudaStreamEndCapture(h->stream, &graph);
      if (ce != cudaSuccess || err || !graph) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return SD_ERR_CUDA; }
      cudaGraphExec_t exec = nullptr;
      const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      if (ie != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
      it = h->graphs.emplace(key, sd_handle::Graph{exec, launched}).first;
    }
    set_int_kernel<<<1, 1, 0, h->stream>>>(h->d_pos(), position);
    if (cudaGraphLaunch(it->second.exec, h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
    launched = it->second.nodes + 1;
  }
  if (err) return err;
  h->launches += launched;
  h->next_pos = position + 1;
  h->steps += 1;
  h->layer_steps += n;
  return SD_OK;
}

// ---- static scratch for sd_decode_step_static -------------------------------------------
// Lives in the library image: every GPU that loads the library holds these bytes until the
// process exits.  In host code the symbol below is only a stand-in; the device address comes
// from cudaGetSymbolAddress, looked up once per device with that device current.
constexpr size_t kStaticScratchBytes = SD_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};

int static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return SD_ERR_ARG;
  if (!g_static_scratch_addr[device]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return SD_ERR_CUDA; }
    g_static_scratch_addr[device] = p;
  }
  *out = g_static_scratch_addr[device];
  return SD_OK;
}

}  // namespace

extern "C" {

int sd_arena_bytes(const sd_config* cfg, const sd_plan* plan, size_t* out) {
  if (!valid_config(cfg) || !out || !valid_plan(cfg, plan)) return SD_ERR_ARG;
  Arena A;
  carve(*cfg, *plan, A);
  *out = A.total;
  return SD_OK;
}

int sd_create(const sd_config* cfg, const sd_weights* w, const sd_plan* plan, void* arena, size_t arena_bytes,
              void* stream, sd_handle** out) {
  if (!valid_config(cfg) || !w || !out || !arena || !valid_plan(cfg, plan)) return SD_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(arena) % kAlign) return SD_ERR_ARG;
  const int L = cfg->n_layers;
  const void* const* per_layer[] = {w->ln1_g, w->ln1_b, w->w_qkv, w->b_qkv, w->w_o, w->b_o,
                                    w->ln2_g, w->ln2_b, w->w_fc1, w->b_fc1, w->w_fc2, w->b_fc2};
  for (auto arr : per_layer) {
    if (!arr) return SD_ERR_ARG;
    for (int l = 0; l < L; ++l)
      if (!arr[l]) return SD_ERR_ARG;
  }
  if (!w->tok_emb || !w->pos_emb || !w->lnf_g || !w->lnf_b) return SD_ERR_ARG;
  sd_handle* h = new (std::nothrow) sd_handle();
  if (!h) return SD_ERR_ARG;
  h->cfg = *cfg;
  h->plan = *plan;
  h->hd = cfg->d_model / cfg->n_heads;
  h->esize = cfg->dtype == SD_DTYPE_FP32 ? 4 : 2;
  carve(*cfg, *plan, h->A);
  if (h->A.total > arena_bytes) { delete h; return SD_ERR_CAPACITY; }
  auto copy = [&](std::vector<const void*>& dst, const void* const* src) { dst.assign(src, src + L); };
  copy(h->ln1_g, w->ln1_g); copy(h->ln1_b, w->ln1_b); copy(h->w_qkv, w->w_qkv); copy(h->b_qkv, w->b_qkv);
  copy(h->w_o, w->w_o); copy(h->b_o, w->b_o); copy(h->ln2_g, w->ln2_g); copy(h->ln2_b, w->ln2_b);
  copy(h->w_fc1, w->w_fc1); copy(h->b_fc1, w->b_fc1); copy(h->w_fc2, w->w_fc2); copy(h->b_fc2, w->b_fc2);
  h->tok_emb = w->tok_emb; h->pos_emb = w->pos_emb; h->lnf_g = w->lnf_g; h->lnf_b = w->lnf_b;
  h->lm_head = w->lm_head ? w->lm_head : w->tok_emb;
  h->arena = static_cast<char*>(arena);
  h->stream = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(h->arena + h->A.scalars, 0, 256, h->stream) != cudaSuccess ||
      cudaMemsetAsync(h->arena + h->A.counters, 0, ((size_t)h->A.rows_max * cfg->n_heads + 64) * 4, h->stream) != cudaSuccess) {
    cudaGetLastError(); delete h; return SD_ERR_CUDA;
  }
  if (cfg->dtype == SD_DTYPE_BF16) {
    if (cudaMemsetAsync(h->arena + h->A.splitk_count, 0, (size_t)sd::kSplitSlots * 4, h->stream) != cudaSuccess) {
      cudaGetLastError(); delete h; return SD_ERR_CUDA;
    }
    h->tc.splitk_ws = h->at<float>(h->A.splitk_ws);
    h->tc.splitk_count = h->at<int>(h->A.splitk_count);
  }
  sd::tc_init(h->tc);
  sd::persist_init(h->persist, h->tc);
  if (h->tc.ready && h->A.packable) {            // tile-packed copies of the matrices, made once
    const int d = cfg->d_model, f = cfg->d_ffn;
    auto pack = [&](const void* W, size_t off, int n, int k) {
      const int tiles = (n + 255) / 256 * 2 * (k / 64);
      sd::tc::pack_tiles_kernel<<<tiles, 256, 0, h->stream>>>(static_cast<const bf16*>(W), h->at<bf16>(off), n, k, h->status());
    };
    for (int l = 0; l < L; ++l) {
      pack(h->w_qkv[l], h->A.wp_qkv[l], 3 * d, d);
      pack(h->w_o[l], h->A.wp_o[l], d, d);
      pack(h->w_fc1[l], h->A.wp_fc1[l], f, d);
      pack(h->w_fc2[l], h->A.wp_fc2[l], d, f);
    }
    pack(h->lm_head, h->A.wp_head, cfg->vocab, d);
    if (cudaGetLastError() != cudaSuccess) { delete h; return SD_ERR_CUDA; }
    h->packed = true;
  }
  *out = h;
  return SD_OK;
}

int sd_schedule(sd_handle* h, int mx, int mn, int w, int G, int32_t* n_active, int32_t* top_begin) {
  if (!h || !valid_schedule_args(h->cfg.n_layers, mx, mn, w, G) || G > h->cfg.max_gen) return SD_ERR_ARG;
  const int L = h->cfg.n_layers;
  std::vector<int> count;
  layer_counts(L, mx, mn, w, G, count);
  for (int l = 0; l < L; ++l)
    if (h->cfg.max_prompt + count[l] > h->A.cap[l]) return SD_ERR_CAPACITY;
  h->n_active.resize(G); h->top_begin.resize(G);
  for (int g = 0; g < G; ++g) {
    h->n_active[g] = budget_at(mx, mn, g, G);
    h->top_begin[g] = L - (h->n_active[g] - w);
    if (n_active) n_active[g] = h->n_active[g];
    if (top_begin) top_begin[g] = h->top_begin[g];
  }
  h->warmup = w; h->gen_len = G;
  h->have_schedule = true;
  // the prompt's cache does not depend on the schedule: keep it when the new length still fits
  if (h->have_prefill && (int64_t)h->P + G > h->cfg.max_pos) h->have_prefill = false;
  h->next_pos = h->P;
  return SD_OK;
}

int sd_schedule_power_compute(int n_layers, int mx, int mn, int w, int G, int alpha, int32_t* n_active, int32_t* top_begin) {
  if (!valid_schedule_args(n_layers, mx, mn, w, G) || alpha < 1 || alpha > 8 || !power_args_fit(mx, mn, G, alpha)) return SD_ERR_ARG;
  for (int g = 0; g < G; ++g) {
    const int n = budget_power_at(mx, mn, g, G, alpha);
    if (n_active) n_active[g] = n;
    if (top_begin) top_begin[g] = n_layers - (n - w);
  }
  return SD_OK;
}

int sd_schedule_custom(sd_handle* h, const int32_t* n_active, int w, int G, int32_t* top_begin) {
  if (!h || !n_active || G < 1 || G > h->cfg.max_gen || w < 0) return SD_ERR_ARG;
  const int L = h->cfg.n_layers;
  for (int g = 0; g < G; ++g) {
    if (n_active[g] <= w || n_active[g] > L) return SD_ERR_ARG;
    if (g > 0 && n_active[g] > n_active[g - 1]) return SD_ERR_ARG;      // budgets never grow (Section 2.2)
  }
  std::vector<int> count(L, 0);
  for (int g = 0; g < G; ++g) {
    const int top = L - (n_active[g] - w);
    for (int l = 0; l < L; ++l)
      if (l < w || l >= top) ++count[l];
  }
  for (int l = 0; l < L; ++l)
    if (h->cfg.max_prompt + count[l] > h->A.cap[l]) return SD_ERR_CAPACITY;
  h->n_active.assign(n_active, n_active + G);
  h->top_begin.resize(G);
  for (int g = 0; g < G; ++g) {
    h->top_begin[g] = L - (n_active[g] - w);
    if (top_begin) top_begin[g] = h->top_begin[g];
  }
  h->warmup = w; h->gen_len = G;
  h->have_schedule = true;
  if (h->have_prefill && (int64_t)h->P + G > h->cfg.max_pos) h->have_prefill = false;
  h->next_pos = h->P;
  return SD_OK;
}

int sd_schedule_compute(int n_layers, int mx, int mn, int w, int G, int32_t* n_active, int32_t* top_begin) {
  if (!valid_schedule_args(n_layers, mx, mn, w, G)) return SD_ERR_ARG;
  for (int g = 0; g < G; ++g) {
    const int n = budget_at(mx, mn, g, G);
    if (n_active) n_active[g] = n;
    if (top_begin) top_begin[g] = n_layers - (n - w);
  }
  return SD_OK;
}

int sd_layer_capacity(const sd_config* cfg, const sd_plan* plan, int32_t* capacity) {
  if (!valid_config(cfg) || !valid_plan(cfg, plan) || !capacity) return SD_ERR_ARG;
  Arena A;
  carve(*cfg, *plan, A);
  for (int l = 0; l < cfg->n_layers; ++l) capacity[l] = A.cap[l];
  return SD_OK;
}

int sd_prefill(sd_handle* h, const int32_t* d_tokens, int B, int P, float* d_logits) {
  if (!h || !d_tokens || !d_logits || B < 1 || P < 1) return SD_ERR_ARG;
  if (!h->have_schedule) return SD_ERR_STATE;
  if (B > h->cfg.max_batch || P > h->cfg.max_prompt || (int64_t)P + h->gen_len > h->cfg.max_pos) return SD_ERR_CAPACITY;
  if (h->have_pad) {                        // every row keeps at least one real token
    if ((int)h->pad.size() != B) return SD_ERR_ARG;
    for (int b = 0; b < B; ++b)
      if (h->pad[b] >= P) return SD_ERR_ARG;
  }
  if (h->have_rows) { h->have_rows = false; h->rows.clear(); drop_graphs(h); }   // a new batch: all rows generate
  // a new batch starts with a clean status word (a bit set earlier has been reported through sd_status by now or is lost)
  if (cudaMemsetAsync(h->status(), 0, sizeof(int), h->stream) != cudaSuccess ||
      cudaMemsetAsync(h->arena + h->A.counters, 0, ((size_t)h->A.rows_max * h->cfg.n_heads + 64) * 4, h->stream) != cudaSuccess) {
    cudaGetLastError();
    return SD_ERR_CUDA;
  }
  const int err = h->cfg.dtype == SD_DTYPE_BF16 ? run_prefill<bf16>(h, d_tokens, B, P, d_logits)
                                                : run_prefill<float>(h, d_tokens, B, P, d_logits);
  if (err) return err;
  h->B = B; h->P = P; h->next_pos = P; h->have_prefill = true;
  return SD_OK;
}

int sd_set_padding(sd_handle* h, const int32_t* h_pad, int B) {
  if (!h) return SD_ERR_ARG;
  if (!h_pad) {
    if (h->have_pad) drop_graphs(h);
    h->have_pad = false; h->pad.clear(); h->have_prefill = false;
    return SD_OK;
  }
  if (B < 1 || B > h->cfg.max_batch) return SD_ERR_ARG;
  for (int b = 0; b < B; ++b)
    if (h_pad[b] < 0 || h_pad[b] >= h->cfg.max_prompt) return SD_ERR_ARG;
  if (!h->have_pad) drop_graphs(h);
  h->pad.assign(h_pad, h_pad + B);
  h->have_pad = true;
  h->have_prefill = false;                  // the cache was filled under another alignment
  if (cudaMemcpyAsync(h->arena + h->A.pad, h->pad.data(), (size_t)B * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  return SD_OK;
}

int sd_set_rows(sd_handle* h, const int32_t* h_rows, int n) {
  if (!h) return SD_ERR_ARG;
  if (!h->have_prefill) return SD_ERR_STATE;
  if (!h_rows) {
    if (h->have_rows) drop_graphs(h);
    h->have_rows = false; h->rows.clear();
    return SD_OK;
  }
  if (n < 1 || n > h->B) return SD_ERR_ARG;
  for (int i = 0; i < n; ++i)
    if (h_rows[i] < 0 || h_rows[i] >= h->B || (i && h_rows[i] <= h_rows[i - 1])) return SD_ERR_ARG;
  if (!h->have_rows) drop_graphs(h);
  h->rows.assign(h_rows, h_rows + n);
  h->have_rows = true;
  if (cudaMemcpyAsync(h->arena + h->A.rows, h->rows.data(), (size_t)n * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  return SD_OK;
}

int sd_decode_step(sd_handle* h, const int32_t* d_token_ids, int position, float* d_logits) {
  return decode_step_impl(h, d_token_ids, position, d_logits);
}

int sd_rewind(sd_handle* h) {
  if (!h) return SD_ERR_ARG;
  if (!h->have_schedule || !h->have_prefill) return SD_ERR_STATE;
  h->next_pos = h->P;
  return SD_OK;
}

int sd_launch_count(sd_handle* h, int64_t* launches) {
  if (!h || !launches) return SD_ERR_ARG;
  *launches = h->launches;
  return SD_OK;
}

int sd_decode_step_static(sd_handle* h, const int32_t* d_ids, int position, float* d_logits) {
  if (!h || !d_ids || !d_logits) return SD_ERR_ARG;
  if (!h->have_schedule || !h->have_prefill) return SD_ERR_STATE;
  const int g = position - h->P;
  if (position != h->next_pos || g < 0 || g >= h->gen_len || position >= h->cfg.max_pos) return SD_ERR_POSITION;
  int device = -1;
  cudaPointerAttributes attr;
  if (cudaGetDevice(&device) != cudaSuccess || cudaPointerGetAttributes(&attr, h->arena) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  if (attr.device != device) return SD_ERR_ARG;       // the static array of another GPU would be handed to this handle's kernels
  const int n = h->n_active[g];
  const int T = position + 1;
  const int chunk = pick_chunk(h, h->n_rows(), T);
  const int n_chunks = (T + chunk - 1) / chunk;
  const size_t slots = (size_t)h->n_rows() * h->cfg.n_heads * n_chunks;
  const size_t acc_bytes = align_up(slots * h->hd * sizeof(float)), ml_bytes = slots * 2 * sizeof(float);
  if (acc_bytes + ml_bytes > kStaticScratchBytes) return SD_ERR_CAPACITY;   // split-KV partials beyond the static array
  void* base = nullptr;
  const int rc = static_scratch_address(device, &base);
  if (rc != SD_OK) return rc;
  float* part_acc = static_cast<float*>(base);
  float* part_ml = reinterpret_cast<float*>(static_cast<char*>(base) + acc_bytes);
  int64_t launched = 0;
  // every partial slot the merging block reads was written earlier in the same attention launch,
  // so nothing in the array has to start at zero
  const int err = h->cfg.dtype == SD_DTYPE_BF16
      ? enqueue_decode<bf16>(h, d_ids, position, false, d_logits, n, chunk, n_chunks, false, &launched, part_acc, part_ml)
      : enqueue_decode<float>(h, d_ids, position, false, d_logits, n, chunk, n_chunks, false, &launched, part_acc, part_ml);
  if (err) return err;
  h->launches += launched;
  h->next_pos = position + 1;
  h->steps += 1;
  h->layer_steps += n;
  return SD_OK;
}

int sd_decode_step_host(sd_handle* h, const int32_t* h_ids, int position, float* h_logits) {
  if (!h || !h_ids || !h_logits) return SD_ERR_ARG;
  if (!h->have_schedule || !h->have_prefill) return SD_ERR_STATE;
  int32_t* d_ids = h->at<int32_t>(h->A.ids);
  float* d_logits = h->at<float>(h->A.logits);
  if (cudaMemcpyAsync(d_ids, h_ids, (size_t)h->n_rows() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  const int err = decode_step_impl(h, d_ids, position, d_logits);
  if (err) return err;
  if (cudaMemcpyAsync(h_logits, d_logits, (size_t)h->n_rows() * h->cfg.vocab * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  return SD_OK;
}

int sd_greedy(sd_handle* h, const float* d_logits, int B, int32_t* d_next) {
  if (!h || !d_logits || !d_next || B < 1) return SD_ERR_ARG;
  sd::greedy_kernel<<<B, 1024, 0, h->stream>>>(d_logits, h->cfg.vocab, d_next);
  h->launches += 1;
  return cudaGetLastError() == cudaSuccess ? SD_OK : SD_ERR_CUDA;
}

int sd_sample_top_p(sd_handle* h, const float* d_logits, int B, float temperature, float top_p,
                    const float* d_uniforms, int32_t* d_next) {
  if (!h || !d_logits || !d_uniforms || !d_next || B < 1) return SD_ERR_ARG;
  if (!std::isfinite(temperature) || !(temperature > 0.0f) || !std::isfinite(top_p) || !(top_p > 0.0f) || top_p > 1.0f)
    return SD_ERR_ARG;
  const int vocab = h->cfg.vocab;
  if (vocab <= sd::SAMPLE_MAX_SMEM_VOCAB) {        // the row is staged in shared memory
    if (!h->sample_ready) {                  // per handle: the attribute belongs to the handle's device
      if (cudaFuncSetAttribute(sd::sample_top_p_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               sd::SAMPLE_MAX_SMEM_VOCAB * 4) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
      h->sample_ready = true;
    }
    sd::sample_top_p_kernel<true><<<B, sd::SAMPLE_THREADS, (size_t)vocab * 4, h->stream>>>(d_logits, vocab, d_uniforms,
                                                                                        1.0f / temperature, top_p, d_next);
  } else {
    sd::sample_top_p_kernel<false><<<B, sd::SAMPLE_THREADS, 0, h->stream>>>(d_logits, vocab, d_uniforms,
                                                                           1.0f / temperature, top_p, d_next);
  }
  h->launches += 1;
  return cudaGetLastError() == cudaSuccess ? SD_OK : SD_ERR_CUDA;
}

int sd_status(sd_handle* h, int32_t* device_status) {
  if (!h) return SD_ERR_ARG;
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, h->status(), 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess) { cudaGetLastError(); return SD_ERR_CUDA; }
  if (device_status) *device_status = v;
  return v ? SD_ERR_DEVICE : SD_OK;
}

int sd_stats(sd_handle* h, int64_t* steps, int64_t* layer_steps) {
  if (!h) return SD_ERR_ARG;
  if (steps) *steps = h->steps;
  if (layer_steps) *layer_steps = h->layer_steps;
  return SD_OK;
}

int sd_set_option(sd_handle* h, int option, int value) {
  if (!h) return SD_ERR_ARG;
  switch (option) {
    case SD_OPT_GRAPHS: h->opt_graphs = value ? 1 : 0; return SD_OK;
    case SD_OPT_ATTN_CHUNK:
      if (value != 0 && (value < kMinChunk || value % kMinChunk)) return SD_ERR_ARG;
      h->opt_chunk = value; return SD_OK;
    case SD_OPT_GEMM:
      if (value < 0 || value > 2) return SD_ERR_ARG;
      if (value != h->opt_gemm) drop_graphs(h);
      h->opt_gemm = value; return SD_OK;
    case SD_OPT_GEMM_SPLITK:
      if (value < 0 || value > 8) return SD_ERR_ARG;
      if (value != h->tc.splitk) drop_graphs(h);
      h->tc.splitk = value; return SD_OK;
    case SD_OPT_GEMM_PERSISTENT:
      if (value < 0 || value > 2) return SD_ERR_ARG;
      drop_graphs(h);
      h->persist.enabled = value ? 1 : 0;
      h->persist.allow_96 = value == 1 ? 1 : 0; return SD_OK;
    case SD_OPT_PREFILL_ATTN:
      h->opt_prefill = value ? 1 : 0; return SD_OK;
    case SD_OPT_PDL:
      if (value < 0 || value >= (1 << SD_K_COUNT)) return SD_ERR_ARG;
      if (value != h->opt_pdl) drop_graphs(h);
      h->opt_pdl = value; return SD_OK;
    case SD_OPT_ATTN_STAGED:
      if (value != h->opt_attn_staged) drop_graphs(h);
      if (value < 0 || value > 2) return SD_ERR_ARG;
      h->opt_attn_staged = value; return SD_OK;
    case SD_OPT_DETERMINISTIC:
      if ((value != 0) != (h->tc.deterministic != 0)) drop_graphs(h);
      h->tc.deterministic = value ? 1 : 0; return SD_OK;
    case SD_OPT_TEST_WAIT_EXPIRY:
      drop_graphs(h);                       // the marked launch must not be replayed from a graph
      h->tc.test_expire = value ? 1 : 0; return SD_OK;
    case SD_OPT_TIMING:
      if (h->opt_timing && !value) collect_timing(h);
      h->opt_timing = value ? 1 : 0; return SD_OK;
    default: return SD_ERR_ARG;
  }
}

int sd_kernel_time(sd_handle* h, int cls, double* ms, int64_t* launches) {
  if (!h || cls < 0 || cls >= SD_K_COUNT) return SD_ERR_ARG;
  collect_timing(h);
  if (ms) *ms = h->k_ms[cls];
  if (launches) *launches = h->k_launches[cls];
  return SD_OK;
}

int sd_kernel_time_reset(sd_handle* h) {
  if (!h) return SD_ERR_ARG;
  collect_timing(h);
  for (int i = 0; i < SD_K_COUNT; ++i) { h->k_ms[i] = 0; h->k_launches[i] = 0; }
  return SD_OK;
}

const char* sd_strerror(int code) {
  switch (code) {
    case SD_OK: return "ok";
    case SD_ERR_ARG: return "invalid argument";
    case SD_ERR_STATE: return "schedule or prefill missing";
    case SD_ERR_POSITION: return "position out of order or outside the schedule";
    case SD_ERR_CAPACITY: return "capacity exceeded";
    case SD_ERR_CUDA: return "CUDA call failed";
    case SD_ERR_DEVICE: return "device status word is set";
    default: return "unknown error";
  }
}

void sd_destroy(sd_handle* h) {
  if (!h) return;
  collect_timing(h);
  drop_graphs(h);
  sd::tc_destroy(h->tc);
  delete h;
}

}  // extern "C"
