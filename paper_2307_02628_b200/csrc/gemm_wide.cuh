// Wide-tile tensor-core GEMM for the weight-streaming regime (few tokens, bf16 operands):
// out[m, n] (+)= sum_k X[m, k] W[n, k] + bias[n], X carried as hi + lo (see Operand).
//
// A measured alternative to the 128-row kernel, selectable with SD_OPT_GEMM = 3.  A block owns
// 256 weight rows (two 128 x 2NB accumulators in tensor memory) per operand tile, which halves
// the operand bytes per weight byte, and the blocks of a thread-block cluster split K between
// them so that enough blocks exist.  For the store epilogues the cluster finishes with a
// reduce-scatter through distributed shared memory: each block ships the accumulator rows it
// does not own to their owner (32-row groups dealt round-robin), then adds what it received
// to its own rows and runs the epilogue on them.  The residual epilogue needs no exchange
// (fp32 atomics).  On B200 at 64 tokens it is slower than the 128-row kernel: the main loop is
// paced by the number of MMA instructions per SM, which this layout does not reduce, and its
// epilogue is longer.
//
// Warp roles as in gemm_tc.cuh.  All threads of all blocks of a cluster reach both cluster
// barriers on every path, also when a bounded mbarrier wait has expired (the data movement
// is then skipped and STATUS_WAIT_EXPIRED is set), so the cluster barriers always complete.
#pragma once
#include "gemm_tc.cuh"

namespace sd {
namespace tcw {

using namespace tc;

constexpr int ROWS = 256;            // weight rows per block: two MMA tiles of 128
constexpr int MAX_CLUSTER = 4;

__host__ __device__ constexpr int stages_for(int nb) { return nb >= 128 ? 3 : nb >= 64 ? 4 : nb >= 32 ? 5 : 6; }
__host__ __device__ constexpr int stage_bytes(int nb) { return ROWS * BK * 2 + 2 * nb * BK * 2; }
__host__ __device__ constexpr int smem_bytes(int nb) { return stages_for(nb) * stage_bytes(nb) + 1024 + 256 + 1024; }

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Row groups: accumulator a (0, 1) x lane quarter q (0..3) -> g = 4a + q, rows [128a + 32q, +32).
// Group g is finished by block g % S of the cluster; there it is that block's slot g / S.
template <int NB, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                 const __nv_bfloat16* __restrict__ bias, void* __restrict__ out, int ldo, int M, int N, int K,
                 int kb_per_split, int* __restrict__ status, const QkvOut qo) {
  constexpr int STAGES = stages_for(NB);
  constexpr int A_BYTES = ROWS * BK * 2, A_HALF = A_BYTES / 2, B_BYTES = NB * BK * 2, STAGE_BYTES = A_BYTES + 2 * B_BYTES;
  constexpr int TMEM_COLS = 4 * NB;             // per accumulator: W.hi in [0, NB), W.lo in [NB, 2 NB)
  constexpr int CW = NB < 32 ? 16 : 32;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + STAGES * STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES, accum_bar = full0 + 16 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  long long* col_row = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(bars) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = (int)cluster_size(), crank = (int)cluster_rank();
  const int n0 = (blockIdx.x / S) * ROWS, m0 = blockIdx.y * NB;
  const int kb_total = (K + BK - 1) / BK;
  // K range of this split (blockIdx.z), then of this block inside its cluster; the host keeps
  // every block's share non-empty
  const int zb0 = blockIdx.z * kb_per_split, zb1 = min(zb0 + kb_per_split, kb_total);
  const int zlen = zb1 - zb0;
  const int kb0 = zb0 + (int)((long long)zlen * crank / S), kb1 = zb0 + (int)((long long)zlen * (crank + 1) / S);
  const int nkb = kb1 - kb0;
  const bool exchange = (S > 1) && (EPI != EPI_RESIDUAL_F32);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(accum_bar, 1);
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
  pdl_launch_dependents();

  bool accum_ok = false;
  if (warp == 0) {
    if (lane == 0 && nkb > 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
      const int early = nkb < STAGES ? nkb : STAGES;     // weights do not depend on the previous kernel
      for (int i = 0; i < early; ++i) {
        const uint32_t fb = full0 + 8 * i, dst = tiles + i * STAGE_BYTES;
        mbar_expect_tx(fb, STAGE_BYTES);
        load_w_tile(dst, &map_w, qo, kb0 + i, n0, fb);
        load_w_tile(dst + A_HALF, &map_w, qo, kb0 + i, n0 + 128, fb);
      }
      pdl_wait();
      int issued = early;
      for (int i = 0; i < nkb; ++i) {
        const int s = i % STAGES, round = i / STAGES;
        const uint32_t fb = full0 + 8 * s, dst = tiles + s * STAGE_BYTES;
        if (round > 0) {
          if (!mbar_wait(empty0 + 8 * s, (round - 1) & 1, abort_flag, status)) break;
          mbar_expect_tx(fb, STAGE_BYTES);
          load_w_tile(dst, &map_w, qo, kb0 + i, n0, fb);
          load_w_tile(dst + A_HALF, &map_w, qo, kb0 + i, n0 + 128, fb);
        }
        tma_load_2d(dst + A_BYTES, &map_x, (kb0 + i) * BK, m0, fb);
        tma_load_2d(dst + A_BYTES + B_BYTES, &map_x, K + (kb0 + i) * BK, m0, fb);
        if (i + 1 > issued) issued = i + 1;
      }
      if (*abort_flag) {
        const int first = issued > STAGES ? issued - STAGES : 0;
        for (int i = first; i < issued; ++i) {
          const long long t0 = clock64();
          while (!mbar_try(full0 + 8 * (i % STAGES), (i / STAGES) & 1) && clock64() - t0 < kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && nkb > 0) {
      constexpr uint32_t idesc = instr_desc(2 * NB);   // hi and lo tiles back to back = one operand of 2 NB rows
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const int s = i % STAGES, round = i / STAGES;
        ok = mbar_wait(full0 + 8 * s, round & 1, abort_flag, status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = tiles + s * STAGE_BYTES;
        const uint64_t a0 = smem_desc(a_addr), a1 = smem_desc(a_addr + A_HALF), bd = smem_desc(a_addr + A_BYTES);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          const uint32_t acc = (i > 0 || k > 0) ? 1u : 0u;
          umma(tmem_base, a0 + 2 * k, bd + 2 * k, idesc, acc);
          umma(tmem_base + 2 * NB, a1 + 2 * k, bd + 2 * k, idesc, acc);
        }
        umma_commit(empty0 + 8 * s);
      }
      if (ok) umma_commit(accum_bar);
    }
  } else {
    pdl_wait();
    if (EPI == EPI_QKV_CACHE) {
      const int t = threadIdx.x - 64;
      if (t < NB) {
        int b, pos;
        qo.map.get(m0 + t, b, pos);
        col_row[t] = (m0 + t < M && pos < qo.cap) ? (long long)b * qo.H * qo.cap + pos : -1;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    accum_ok = nkb > 0 && mbar_wait(accum_bar, 0, abort_flag, status);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
  __syncwarp();
  accum_ok = __all_sync(0xffffffffu, accum_ok);   // warp-uniform: the TMEM loads below are warp-wide

  const int quarter = warp & 3;
  const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
  // receive area: [slot][source][column][lane] floats at the start of the (now idle) stage buffers
  if (exchange) {
    cluster_sync();                               // every block of the cluster has finished its MMAs
    if (warp >= 2 && accum_ok) {
#pragma unroll 1
      for (int a = 0; a < 2; ++a) {
        const int g = 4 * a + quarter, owner = g % S;
        if (owner == crank) continue;
        const int slot = g / S, src = crank < owner ? crank : crank - 1;
        const uint32_t dst0 = map_to_cta(tiles, (uint32_t)owner) + (uint32_t)(((slot * (S - 1) + src) * NB) * 32 + lane) * 4u;
#pragma unroll 1
        for (int c = 0; c < NB; c += CW) {
          uint32_t r[32], rl[32];
          const uint32_t taddr = tmem_base + lane_base + (uint32_t)(a * 2 * NB + c);
          if (CW == 32) { tmem_ld32(taddr, r); tmem_ld32(taddr + NB, rl); } else { tmem_ld16(taddr, r); tmem_ld16(taddr + NB, rl); }
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < CW; ++j)
            st_cluster_f32(dst0 + (uint32_t)((c + j) * 32) * 4u, __uint_as_float(r[j]) + __uint_as_float(rl[j]));
        }
      }
    }
    cluster_sync();                               // everything sent to this block has arrived
  }

  if (warp >= 2 && accum_ok) {
    const float* recv = reinterpret_cast<const float*>(tiles_ptr);
#pragma unroll 1
    for (int a = 0; a < 2; ++a) {
      const int g = 4 * a + quarter;
      if (exchange && g % S != crank) continue;
      const int slot = g / S;
      const int n = n0 + a * 128 + quarter * 32 + lane;
      const bool add_bias = bias != nullptr && n < N && (EPI != EPI_RESIDUAL_F32 || (blockIdx.z == 0 && crank == 0));
      const float b = add_bias ? __bfloat162float(bias[n]) : 0.f;
      int kv_head = 0, kv_elem = 0;
      __nv_bfloat16* kv_base = nullptr;
      if (EPI == EPI_QKV_CACHE && n >= qo.d && n < N) {
        const int cc = n < 2 * qo.d ? n - qo.d : n - 2 * qo.d;
        kv_head = cc / qo.hd;
        kv_elem = cc - kv_head * qo.hd;
        kv_base = n < 2 * qo.d ? qo.Kc : qo.Vc;
      }
#pragma unroll 1
      for (int c = 0; c < NB; c += CW) {
        uint32_t r[32], rl[32];
        const uint32_t taddr = tmem_base + lane_base + (uint32_t)(a * 2 * NB + c);
        if (CW == 32) { tmem_ld32(taddr, r); tmem_ld32(taddr + NB, rl); } else { tmem_ld16(taddr, r); tmem_ld16(taddr + NB, rl); }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (n < N) {
#pragma unroll
          for (int j = 0; j < CW; ++j) {
            const int m = m0 + c + j;
            if (m < M) {
              float v = (__uint_as_float(r[j]) + __uint_as_float(rl[j])) + b;
              if (exchange) {
                for (int s = 0; s < S - 1; ++s) v += recv[((slot * (S - 1) + s) * NB + (c + j)) * 32 + lane];
              }
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
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tcw

// ---- host side ------------------------------------------------------------------------

template <int NB, int EPI>
inline bool wide_prepare() {
  return cudaFuncSetAttribute(tcw::gemm_wide_kernel<NB, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tcw::smem_bytes(NB)) == cudaSuccess;
}
template <int NB>
inline bool wide_prepare_nb() {
  return wide_prepare<NB, EPI_STORE_F32>() && wide_prepare<NB, EPI_RELU_T>() && wide_prepare<NB, EPI_RESIDUAL_F32>() &&
         wide_prepare<NB, EPI_QKV_CACHE>();
}

struct WideContext {
  int ready = 0;
  int max_clusters[tcw::MAX_CLUSTER + 1] = {};   // co-resident clusters of size S (one block per SM), measured at init
  int force_cluster = 0;                          // 0 = choose; 1..MAX_CLUSTER = use this size where K allows
};

template <int NB, int EPI>
inline cudaError_t wide_launch_one(bool pdl, cudaStream_t st, dim3 grid, int S, const CUtensorMap* mw, const CUtensorMap* mx,
                                   const __nv_bfloat16* bias, void* out, int ldo, int M, int N, int K, int kb_per_split,
                                   int* status, const tc::QkvOut& qo) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = tcw::smem_bytes(NB); cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, tcw::gemm_wide_kernel<NB, EPI>, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
}

template <int NB>
inline cudaError_t wide_launch(bool pdl, cudaStream_t st, dim3 grid, int S, int epi, const CUtensorMap* mw, const CUtensorMap* mx,
                               const __nv_bfloat16* bias, void* out, int ldo, int M, int N, int K, int kb_per_split, int* status,
                               const tc::QkvOut& qo) {
  switch (epi) {
    case EPI_STORE_F32: return wide_launch_one<NB, EPI_STORE_F32>(pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
    case EPI_RELU_T: return wide_launch_one<NB, EPI_RELU_T>(pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
    case EPI_QKV_CACHE: return wide_launch_one<NB, EPI_QKV_CACHE>(pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
    default: return wide_launch_one<NB, EPI_RESIDUAL_F32>(pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
  }
}

inline void wide_init(WideContext& w, const TcContext& c) {
  if (!c.ready) return;
  if (!(wide_prepare_nb<16>() && wide_prepare_nb<32>() && wide_prepare_nb<64>() && wide_prepare_nb<128>())) { cudaGetLastError(); return; }
  // how many clusters of each size fit at once (one block per SM by shared memory)
  for (int S = 1; S <= tcw::MAX_CLUSTER; ++S) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S * 64); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = tcw::smem_bytes(64);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tcw::gemm_wide_kernel<64, EPI_STORE_F32>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    w.max_clusters[S] = n;
  }
  w.ready = w.max_clusters[1] > 0;
}

// Picks the cluster size (store epilogues) or the number of K splits (residual epilogue) that
// minimises waves x (block time), with block time ~ share of K plus a fixed cost.
inline bool wide_gemm(WideContext& w, TcContext& c, cudaStream_t st, const __nv_bfloat16* X, const __nv_bfloat16* W,
                      const __nv_bfloat16* bias, int M, int N, int K, void* out, int ldo, int epi, int* status,
                      const tc::QkvOut* qkv_out = nullptr, const __nv_bfloat16* Wp = nullptr) {
  if (!w.ready || !c.ready || K % tc::BK || M < 1 || N < 1) return false;
  if (epi == EPI_QKV_CACHE && (!qkv_out || qkv_out->d % 128 || N != 3 * qkv_out->d)) return false;
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 15) return false;
  tc::QkvOut qo = qkv_out ? *qkv_out : tc::QkvOut{};
  qo.packed_kb = Wp ? K / tc::BK : 0;
  qo.w_packed = Wp;
  const int nb = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128;
  const CUtensorMap* mw = tc_map(c, W, N, K, tc::BM);
  const CUtensorMap* mx = tc_map(c, X, M, 2 * K, nb);
  if (!mw || !mx) return false;
  const int kb_total = K / tc::BK;
  const int tiles = ((N + tcw::ROWS - 1) / tcw::ROWS) * ((M + nb - 1) / nb);
  int S = 1, splits = 1;
  if (epi == EPI_RESIDUAL_F32) {
    splits = std::max(1, std::min(kb_total / 4, w.max_clusters[1] / tiles));
  } else {
    double best = 1e30;
    for (int s = 1; s <= tcw::MAX_CLUSTER; ++s) {
      if (w.max_clusters[s] < 1 || kb_total < 4 * s) continue;
      if (w.force_cluster && s != w.force_cluster) continue;
      const int waves = (tiles + w.max_clusters[s] - 1) / w.max_clusters[s];
      const double t = waves * (1.0 / s + 0.12);          // 0.12: fixed cost of a block relative to a full-K block
      if (t < best - 1e-9) { best = t; S = s; }
    }
  }
  int kb_per_split = (kb_total + splits - 1) / splits;
  splits = (kb_total + kb_per_split - 1) / kb_per_split;
  dim3 grid(((N + tcw::ROWS - 1) / tcw::ROWS) * S, (M + nb - 1) / nb, splits);
  cudaError_t e;
  switch (nb) {
    case 16: e = wide_launch<16>(c.pdl, st, grid, S, epi, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    case 32: e = wide_launch<32>(c.pdl, st, grid, S, epi, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    case 64: e = wide_launch<64>(c.pdl, st, grid, S, epi, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    default: e = wide_launch<128>(c.pdl, st, grid, S, epi, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
  }
  if (e != cudaSuccess) { cudaGetLastError(); return false; }
  return true;
}

template <typename T>
inline bool wide_gemm(WideContext&, TcContext&, cudaStream_t, const T*, const T*, const T*, int, int, int, void*, int, int, int*,
                      const tc::QkvOut* = nullptr, const T* = nullptr) {
  return false;                                  // fp32 storage runs on the CUDA-core kernel
}

}  // namespace sd
