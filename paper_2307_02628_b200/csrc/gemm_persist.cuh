// Persistent variant of the 128-row tensor-core GEMM for token tiles of 128 (prompt pass, batches
// above 64): one CTA per SM walks over many output tiles, and the accumulator is double-buffered in
// tensor memory (2 x 128 columns), so the epilogue of tile i (TMEM -> registers -> global) runs
// while the MMA warp is already issuing tile i + 1 and the producer keeps the shared-memory ring
// full across tile boundaries.  Same operands, tile shapes, descriptors and epilogues as
// gemm_tc_kernel<128, EPI>; no split-K (there are at least as many tiles as SMs where it is used).
//
// Barriers: full[s] / empty[s] per pipeline stage as in the one-tile kernel, plus per accumulator
// buffer tfull[b] (MMA warp -> epilogue: accumulator complete) and tempty[b] (128 epilogue threads ->
// MMA warp: accumulator read out).  Every wait is bounded and reports through the status word.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

namespace tcp {
using namespace tc;

// Token tile NB = 128, or 96 where that needs fewer rounds of tiles per block (config 5's QKV: 96 x 2 = 192
// tiles of 128 tokens are two rounds for 148 blocks, 96 x 3 = 288 tiles of 96 tokens two rounds of 3/4 the work).
constexpr int A_BYTES = BM * BK * 2;
constexpr int TMEM_COLS = 256;                   // two accumulators, 128 columns apart, of NB columns each
constexpr int ACC_STRIDE = 128;
__host__ __device__ constexpr int stages(int nb) { return nb >= 128 ? 6 : 7; }
__host__ __device__ constexpr int stage_bytes(int nb) { return A_BYTES + nb * BK * 2; }
__host__ __device__ constexpr int smem_bytes(int nb) { return stages(nb) * stage_bytes(nb) + 1024 /*alignment*/ + 256 /*barriers*/ + 1024 /*per-column cache rows*/; }

// Order in which the CTAs walk over the output tiles.  The CTAs that run at the same time hold
// consecutive tile numbers, and what they read at the same time they fetch from DRAM once (the rest are
// L2 hits).  Tiles are therefore numbered in bands of BAND weight tiles, weight tile fastest inside a
// band: one wave of CTAs then covers about BAND weight tiles x (SMs / BAND) token tiles instead of every
// weight tile for a single token tile.  A 128-token tile is as large as a weight tile, so a wave of S CTAs
// fetches about BAND + S / BAND tile units: flat around its minimum at sqrt(S) = 12; 16 divides the tile counts here.
constexpr int BAND = 16;
__device__ __forceinline__ void tile_coords(int tile, int tiles_n, int tiles_m, int& tn, int& tm) {
  const int band_tiles = BAND * tiles_m;
  const int band = tile / band_tiles, r = tile - band * band_tiles;
  const int width = min(BAND, tiles_n - band * BAND);        // the last band may be narrower
  tm = r / width;
  tn = band * BAND + (r - tm * width);
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int NB, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_tc_persist_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                       const __nv_bfloat16* __restrict__ bias, void* __restrict__ out, int ldo, int M, int N, int K,
                       int tiles_n, int tiles_total, int* __restrict__ status, const QkvOut qo) {
  constexpr int STAGES = stages(NB), STAGE_BYTES = stage_bytes(NB);
  constexpr int ACC_COLS = ACC_STRIDE;           // one accumulator: NB columns, one per token of the tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + STAGES * STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES, tfull0 = full0 + 16 * STAGES, tempty0 = tfull0 + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  long long* col_row = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(bars) + 256);   // [NB], QKV epilogue only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb = K / BK;
  const int tiles_m = tiles_total / tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, 128); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
      // the first stages' weight tiles depend on nothing: stream them before waiting for the previous kernel
      const int first_tile = blockIdx.x;
      const int early = nkb < STAGES ? nkb : STAGES;
      {
        int tn, tm;
        tile_coords(first_tile, tiles_n, tiles_m, tn, tm);
        const int n0 = tn * BM;
        for (int i = 0; i < early; ++i) {
          const uint32_t fb = full0 + 8 * i;
          mbar_expect_tx(fb, STAGE_BYTES);
          load_w_tile(tiles + i * STAGE_BYTES, &map_w, qo, i, n0, fb);
        }
      }
      pdl_wait();
      int it = 0;
      bool ok = true;
      for (int tile = first_tile; tile < tiles_total && ok; tile += gridDim.x) {
        int tn, tm;
        tile_coords(tile, tiles_n, tiles_m, tn, tm);
        const int n0 = tn * BM, m0 = tm * NB;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES, round = it / STAGES;
          const uint32_t fb = full0 + 8 * s;
          const uint32_t a_dst = tiles + s * STAGE_BYTES;
          if (it >= early) {
            if (round > 0 && !mbar_wait(empty0 + 8 * s, (round - 1) & 1, abort_flag, status)) { ok = false; break; }
            mbar_expect_tx(fb, STAGE_BYTES);
            load_w_tile(a_dst, &map_w, qo, kb, n0, fb);
          }
          tma_load_2d(a_dst + A_BYTES, &map_x, kb * BK, m0, fb);
        }
      }
      if (*abort_flag) {
        // drain: wait (bounded) until every copy issued has landed before the CTA exits
        const int issued = it > early ? it : early;
        const int first = issued > STAGES ? issued - STAGES : 0;
        for (int i = first; i < issued; ++i) {
          const long long t0 = clock64();
          while (!mbar_try(full0 + 8 * (i % STAGES), (i / STAGES) & 1) && clock64() - t0 < kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(NB);
      int it = 0, i = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < tiles_total && ok; tile += gridDim.x, ++i) {
        const int buf = i & 1, use = i >> 1;
        if (use > 0) ok = mbar_wait(tempty0 + 8 * buf, (use - 1) & 1, abort_flag, status);   // the epilogue has read this accumulator out
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + (uint32_t)(buf * ACC_COLS);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES, round = it / STAGES;
          ok = mbar_wait(full0 + 8 * s, round & 1, abort_flag, status);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = tiles + s * STAGE_BYTES;
          const uint64_t a_desc = smem_desc(a_addr), b_desc = smem_desc(a_addr + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma(acc, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(empty0 + 8 * s);
        }
        if (ok) umma_commit(tfull0 + 8 * buf);
      }
    }
  } else {
    pdl_wait();
    const int quarter = warp & 3;
    const int t_epi = threadIdx.x - 64;           // 0..127 over the four epilogue warps
    int i = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles_total && ok; tile += gridDim.x, ++i) {
      const int buf = i & 1, use = i >> 1;
      int tn, tm;
      tile_coords(tile, tiles_n, tiles_m, tn, tm);
      const int n0 = tn * BM, m0 = tm * NB;
      const int n = n0 + quarter * 32 + lane;
      int kv_head = 0, kv_elem = 0;
      __nv_bfloat16* kv_base = nullptr;
      if (EPI == EPI_QKV_CACHE) {
        if (t_epi < NB) {
          int b, pos;
          qo.map.get(m0 + t_epi, b, pos);
          col_row[t_epi] = (m0 + t_epi < M && pos < qo.cap) ? (long long)b * qo.H * qo.cap + pos : -1;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (n >= qo.d && n < N) {
          const int cc = n < 2 * qo.d ? n - qo.d : n - 2 * qo.d;
          kv_head = cc / qo.hd;
          kv_elem = cc - kv_head * qo.hd;
          kv_base = n < 2 * qo.d ? qo.Kc : qo.Vc;
        }
      }
      const float b = (bias != nullptr && n < N) ? __bfloat162float(bias[n]) : 0.f;   // a weight: fetched before the wait
      ok = mbar_wait(tfull0 + 8 * buf, use & 1, abort_flag, status);
      if (tile + (int)gridDim.x >= tiles_total) pdl_launch_dependents();   // this CTA's last main loop is over
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c = 0; c < NB; c += 32) {
        uint32_t r[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * ACC_COLS + c);
        tmem_ld32(taddr, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (n < N) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int m = m0 + c + j;
            if (m < M) {
              const float v = __uint_as_float(r[j]) + b;
              const size_t idx = (size_t)m * ldo + n;
              if (EPI == EPI_STORE_F32) reinterpret_cast<float*>(out)[idx] = v;
              else if (EPI == EPI_QKV_CACHE) {
                if (kv_base == nullptr) {
                  reinterpret_cast<float*>(out)[idx] = v;
                } else {
                  const long long row = col_row[c + j];
                  if (row >= 0) kv_base[((size_t)row + (size_t)kv_head * qo.cap) * qo.hd + kv_elem] = __float2bfloat16_rn(v);
                }
              }
              else if (EPI == EPI_RELU_T)
                Operand<__nv_bfloat16>::store(reinterpret_cast<__nv_bfloat16*>(out) + (size_t)m * ldo, N, n, fmaxf(v, 0.f));
              else atomicAdd(reinterpret_cast<float*>(out) + idx, v);
            }
          }
        }
      }
      // this thread's reads of the accumulator are complete: hand the buffer back to the MMA warp
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(tempty0 + 8 * buf);
      if (EPI == EPI_QKV_CACHE) asm volatile("bar.sync 1, 128;" ::: "memory");   // col_row is rewritten for the next tile
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tcp

struct PersistContext { int ready = 0; int enabled = 1; int allow_96 = 1; };

template <int EPI>
inline bool persist_prepare() {
  return cudaFuncSetAttribute(tcp::gemm_tc_persist_kernel<128, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tcp::smem_bytes(128)) == cudaSuccess &&
         cudaFuncSetAttribute(tcp::gemm_tc_persist_kernel<96, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tcp::smem_bytes(96)) == cudaSuccess;
}
template <int NB>
inline void persist_launch(bool pdl, cudaStream_t st, int sms, const CUtensorMap* mw, const CUtensorMap* mx, const __nv_bfloat16* bias,
                           void* out, int ldo, int M, int N, int K, int tiles_n, int total, int epi, int* status, const tc::QkvOut& qo) {
  const dim3 grid(sms), block(192);
  constexpr int smem = tcp::smem_bytes(NB);
  if (epi == EPI_STORE_F32)
    launch_kernel(pdl, st, tcp::gemm_tc_persist_kernel<NB, EPI_STORE_F32>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, tiles_n, total, status, qo);
  else if (epi == EPI_RELU_T)
    launch_kernel(pdl, st, tcp::gemm_tc_persist_kernel<NB, EPI_RELU_T>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, tiles_n, total, status, qo);
  else if (epi == EPI_QKV_CACHE)
    launch_kernel(pdl, st, tcp::gemm_tc_persist_kernel<NB, EPI_QKV_CACHE>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, tiles_n, total, status, qo);
  else
    launch_kernel(pdl, st, tcp::gemm_tc_persist_kernel<NB, EPI_RESIDUAL_F32>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, tiles_n, total, status, qo);
}
inline void persist_init(PersistContext& p, const TcContext& c) {
  if (!c.ready) return;
  if (!(persist_prepare<EPI_STORE_F32>() && persist_prepare<EPI_RELU_T>() && persist_prepare<EPI_RESIDUAL_F32>() &&
        persist_prepare<EPI_QKV_CACHE>())) {
    cudaGetLastError();
    return;
  }
  p.ready = 1;
}

// Takes the product when the token tile is 128 and there are more tiles than SMs (so that K is not split);
// false leaves it to tc_gemm.
inline bool persist_gemm(PersistContext& p, TcContext& c, cudaStream_t st, const __nv_bfloat16* X, const __nv_bfloat16* W,
                         const __nv_bfloat16* bias, int M, int N, int K, void* out, int ldo, int epi, int* status,
                         const tc::QkvOut* qkv_out = nullptr, const __nv_bfloat16* Wp = nullptr) {
  if (!p.ready || !p.enabled || !c.ready || !Wp || K % tc::BK || M <= 64 || N < 1) return false;
  if (epi == EPI_QKV_CACHE && (!qkv_out || qkv_out->d % tc::BM || N != 3 * qkv_out->d)) return false;
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 15) return false;
  const int tiles_n = (N + tc::BM - 1) / tc::BM;
  if (tiles_n * ((M + 127) / 128) <= c.sm_count) return false;
  if (K / tc::BK > 128) return false;       // long main loops hide little behind them (measured: fc2 3 % slower here)
  // token tile: the one whose tiles take less time per block, counted as rounds of tiles x tokens per tile
  auto cost = [&](int nb) { return (tiles_n * ((M + nb - 1) / nb) + c.sm_count - 1) / c.sm_count * nb; };
  const int nb = (p.allow_96 && cost(96) < cost(128)) ? 96 : 128;
  const int total = tiles_n * ((M + nb - 1) / nb);
  tc::QkvOut qo = qkv_out ? *qkv_out : tc::QkvOut{};
  qo.packed_kb = Wp ? K / tc::BK : 0;
  qo.w_packed = Wp;
  CUtensorMap mw_v, mx_v;
  const CUtensorMap *mw = &mw_v, *mx = &mx_v;
  if (!tc_map(c, W, N, K, tc::BM, &mw_v) || !tc_map(c, X, M, K, nb, &mx_v)) return false;
  if (nb == 96) persist_launch<96>(c.pdl, st, c.sm_count, mw, mx, bias, out, ldo, M, N, K, tiles_n, total, epi, status, qo);
  else persist_launch<128>(c.pdl, st, c.sm_count, mw, mx, bias, out, ldo, M, N, K, tiles_n, total, epi, status, qo);
  return true;
}
template <typename T>
inline bool persist_gemm(PersistContext&, TcContext&, cudaStream_t, const T*, const T*, const T*, int, int, int, void*, int, int, int*,
                         const tc::QkvOut* = nullptr, const T* = nullptr) {
  return false;
}

}  // namespace sd
