// Token-stationary tensor-core GEMM for decode steps of up to 64 tokens (bf16 operands):
// out[m, n] (+)= sum_k X[m, k] W[n, k] + bias[n], X carried as hi + lo (see Operand).
//
// Measured on B200: at these sizes a tcgen05.mma of 128 x N x 16 takes about the same time
// for N = 32 ... 256, so the instruction count decides the speed of the main loop.  Here the
// hi and lo rows of the 64 tokens are the MMA's M = 128 and 256 WEIGHT rows are its N: one
// instruction per 16 columns of K covers 256 weight rows, half the instructions per weight
// byte of the weight-stationary kernel (gemm_tc.cuh).  A block owns 256 weight rows; for the
// store epilogues two blocks of a cluster split K and exchange halves of the result through
// distributed shared memory; the residual epilogue splits K over blockIdx.z and adds with
// vector atomics.
//
// Accumulator layout: TMEM lane r < 64 holds token r against Xhi, lane 64 + r the same token
// against Xlo; column c is weight row n0 + c.  The epilogue first copies all 128 lanes to
// shared memory (the pipeline stages are idle by then), so that one thread can add a
// token's hi and lo rows and write 8 consecutive outputs with 16-byte stores.
//
// Warp roles and bounded waits as in gemm_tc.cuh; every thread reaches both cluster barriers
// on every path.
#pragma once
#include "gemm_wide.cuh"

namespace sd {
namespace txs {

using namespace tc;
using tcw::cluster_rank;
using tcw::cluster_size;
using tcw::cluster_sync;
using tcw::map_to_cta;
using tcw::st_cluster_f32;

constexpr int WN = 256;              // weight rows per block = MMA N
constexpr int XM = 128;              // MMA M: 64 tokens x (hi, lo)
constexpr int TOK = 64;
constexpr int STAGES = 4;
constexpr int W_BYTES = WN * BK * 2, X_BYTES = XM * BK * 2, STAGE_BYTES = W_BYTES + X_BYTES;   // 32 KB + 16 KB
constexpr int DUMP_LD = WN + 1;      // floats per accumulator row in shared memory (odd: no bank conflicts)
constexpr int RECV_LD = 129;
constexpr int DUMP_BYTES = XM * DUMP_LD * 4, RECV_BYTES = TOK * RECV_LD * 4;
static_assert(DUMP_BYTES + RECV_BYTES <= STAGES * STAGE_BYTES, "epilogue scratch must fit in the stage buffers");
__host__ __device__ constexpr int smem_bytes() { return STAGES * STAGE_BYTES + 1024 + 256 + 1024; }

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

template <int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_xs_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __nv_bfloat16* __restrict__ bias, void* __restrict__ out, int ldo, int M, int N, int K,
               int kb_per_split, int* __restrict__ status, const QkvOut qo) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + STAGES * STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES, accum_bar = full0 + 16 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  long long* col_row = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(bars) + 256);   // [TOK] cache rows (QKV)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = (int)cluster_size(), crank = (int)cluster_rank();
  const int n0 = (blockIdx.x / S) * WN;
  const int kb_total = K / BK;
  const int zb0 = blockIdx.z * kb_per_split, zb1 = min(zb0 + kb_per_split, kb_total);
  const int zlen = zb1 - zb0;
  const int kb0 = zb0 + (int)((long long)zlen * crank / S), kb1 = zb0 + (int)((long long)zlen * (crank + 1) / S);
  const int nkb = kb1 - kb0;                       // the host keeps every block's share non-empty
  const bool exchange = (S > 1) && (EPI != EPI_RESIDUAL_F32);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(accum_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(WN) : "memory");
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
      const int early = nkb < STAGES ? nkb : STAGES;      // weights do not depend on the previous kernel
      for (int i = 0; i < early; ++i) {
        const uint32_t fb = full0 + 8 * i, dst = tiles + i * STAGE_BYTES;
        mbar_expect_tx(fb, STAGE_BYTES);
        load_w_tile(dst, &map_w, qo, kb0 + i, n0, fb);
        load_w_tile(dst + W_BYTES / 2, &map_w, qo, kb0 + i, n0 + 128, fb);
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
          load_w_tile(dst + W_BYTES / 2, &map_w, qo, kb0 + i, n0 + 128, fb);
        }
        tma_load_2d(dst + W_BYTES, &map_x, (kb0 + i) * BK, 0, fb);                    // hi rows of the tokens
        tma_load_2d(dst + W_BYTES + X_BYTES / 2, &map_x, K + (kb0 + i) * BK, 0, fb);  // lo rows
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
      constexpr uint32_t idesc = instr_desc(WN);           // M = 128 (tokens x hi/lo), N = 256 weight rows
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const int s = i % STAGES, round = i / STAGES;
        ok = mbar_wait(full0 + 8 * s, round & 1, abort_flag, status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t w_addr = tiles + s * STAGE_BYTES;
        const uint64_t x_desc = smem_desc(w_addr + W_BYTES), w_desc = smem_desc(w_addr);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          umma(tmem_base, x_desc + 2 * k, w_desc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
        umma_commit(empty0 + 8 * s);
      }
      if (ok) umma_commit(accum_bar);
    }
  } else {
    pdl_wait();
    if (EPI == EPI_QKV_CACHE) {
      const int t = threadIdx.x - 64;
      if (t < TOK) {
        int b, pos;
        qo.map.get(t, b, pos);
        col_row[t] = (t < M && pos < qo.cap) ? (long long)b * qo.H * qo.cap + pos : -1;
      }
    }
    accum_ok = nkb > 0 && mbar_wait(accum_bar, 0, abort_flag, status);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
  __syncwarp();
  accum_ok = __all_sync(0xffffffffu, accum_ok);

  float* dump = reinterpret_cast<float*>(tiles_ptr);                     // [XM][DUMP_LD]
  float* recv = reinterpret_cast<float*>(tiles_ptr + DUMP_BYTES);        // [TOK][RECV_LD]
  if (warp >= 2 && accum_ok) {                    // all 128 accumulator lanes -> shared memory
    const int quarter = warp & 3;
    float* row = dump + (size_t)(quarter * 32 + lane) * DUMP_LD;
#pragma unroll 1
    for (int c = 0; c < WN; c += 32) {
      uint32_t r[32];
      tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int j = 0; j < 32; ++j) row[c + j] = __uint_as_float(r[j]);
    }
  }
  const int t = threadIdx.x - 64;                 // epilogue thread: token m, column group sub
  const int m = t & 63, sub = t >> 6;
  const int ncols = exchange ? 64 : 128;          // columns this thread finishes
  const int c0 = exchange ? 128 * crank + 64 * sub : 128 * sub;
  if (exchange) {
    cluster_sync();                               // both blocks have their accumulators in shared memory
    if (warp >= 2 && accum_ok) {
      const int peer = crank ^ 1;
      const int s0 = 128 * peer + 64 * sub;       // columns the peer owns
      const uint32_t dst = map_to_cta(tiles + DUMP_BYTES, (uint32_t)peer) + (uint32_t)(m * RECV_LD + 64 * sub) * 4u;
      const float* hi = dump + (size_t)m * DUMP_LD + s0;
      const float* lo = dump + (size_t)(m + TOK) * DUMP_LD + s0;
#pragma unroll 8
      for (int j = 0; j < 64; ++j) st_cluster_f32(dst + 4u * j, hi[j] + lo[j]);
    }
    cluster_sync();                               // the peer's half has arrived
  } else {
    if (warp >= 2) asm volatile("bar.sync 1, 128;" ::: "memory");
  }

  if (warp >= 2 && accum_ok && m < M) {
    const float* hi = dump + (size_t)m * DUMP_LD + c0;
    const float* lo = dump + (size_t)(m + TOK) * DUMP_LD + c0;
    const float* rc = recv + (size_t)m * RECV_LD + 64 * sub;
    const bool add_bias = bias != nullptr && (EPI != EPI_RESIDUAL_F32 || blockIdx.z == 0);
    const long long cache_row = EPI == EPI_QKV_CACHE ? col_row[m] : 0;
#pragma unroll 1
    for (int j = 0; j < ncols; j += 8) {
      const int n = n0 + c0 + j;
      if (n >= N) break;
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        v[e] = hi[j + e] + lo[j + e];
        if (exchange) v[e] += rc[j + e];
        if (add_bias && n + e < N) v[e] += __bfloat162float(bias[n + e]);
      }
      const bool whole = n + 8 <= N;
      if (EPI == EPI_STORE_F32 || (EPI == EPI_QKV_CACHE && n < qo.d)) {
        float* o = reinterpret_cast<float*>(out) + (size_t)m * ldo + n;
        if (whole && (ldo & 3) == 0) {
          reinterpret_cast<float4*>(o)[0] = make_float4(v[0], v[1], v[2], v[3]);
          reinterpret_cast<float4*>(o)[1] = make_float4(v[4], v[5], v[6], v[7]);
        } else {
          for (int e = 0; e < 8 && n + e < N; ++e) o[e] = v[e];
        }
      } else if (EPI == EPI_QKV_CACHE) {          // 8 consecutive elements of one head's K or V row
        if (cache_row >= 0) {
          const int cc = n < 2 * qo.d ? n - qo.d : n - 2 * qo.d;
          const int head = cc / qo.hd, elem = cc - head * qo.hd;
          __nv_bfloat16* dst = (n < 2 * qo.d ? qo.Kc : qo.Vc) + ((size_t)cache_row + (size_t)head * qo.cap) * qo.hd + elem;
          *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
        }
      } else if (EPI == EPI_RELU_T) {             // the next product's operand: hi | lo halves of a row of 2N bf16
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + (size_t)m * ldo + n;
        if (whole) {
          uint32_t ph[4], pl[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float a = fmaxf(v[2 * e], 0.f), b = fmaxf(v[2 * e + 1], 0.f);
            const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
            ph[e] = pack_bf16(__bfloat162float(ah), __bfloat162float(bh));
            pl[e] = pack_bf16(a - __bfloat162float(ah), b - __bfloat162float(bh));
          }
          *reinterpret_cast<uint4*>(o) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
          *reinterpret_cast<uint4*>(o + N) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
        } else {
          for (int e = 0; e < 8 && n + e < N; ++e) Operand<__nv_bfloat16>::store(o - n, N, n + e, fmaxf(v[e], 0.f));
        }
      } else {                                    // residual: partial sums of the K splits add up in x
        float* o = reinterpret_cast<float*>(out) + (size_t)m * ldo + n;
        if (whole && (ldo & 3) == 0) {
          red_add_v4(o, v[0], v[1], v[2], v[3]);
          red_add_v4(o + 4, v[4], v[5], v[6], v[7]);
        } else {
          for (int e = 0; e < 8 && n + e < N; ++e) atomicAdd(o + e, v[e]);
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(WN) : "memory");
  }
}

}  // namespace txs

struct XsContext {
  int ready = 0;
  int max_clusters2 = 0;       // co-resident 2-block clusters
};

template <int EPI>
inline bool xs_prepare() {
  return cudaFuncSetAttribute(txs::gemm_xs_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, txs::smem_bytes()) == cudaSuccess;
}

inline void xs_init(XsContext& x, const TcContext& c) {
  if (!c.ready) return;
  if (!(xs_prepare<EPI_STORE_F32>() && xs_prepare<EPI_RELU_T>() && xs_prepare<EPI_RESIDUAL_F32>() && xs_prepare<EPI_QKV_CACHE>())) {
    cudaGetLastError();
    return;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(128); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = txs::smem_bytes();
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, txs::gemm_xs_kernel<EPI_STORE_F32>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  x.max_clusters2 = n;
  x.ready = 1;
}

template <int EPI>
inline cudaError_t xs_launch(bool pdl, cudaStream_t st, dim3 grid, int S, const CUtensorMap* mw, const CUtensorMap* mx,
                             const __nv_bfloat16* bias, void* out, int ldo, int M, int N, int K, int kb_per_split, int* status,
                             const tc::QkvOut& qo) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = txs::smem_bytes(); cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, txs::gemm_xs_kernel<EPI>, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
}

// Takes products of up to 64 tokens whose output rows are 8-aligned where vectors are stored.
inline bool xs_gemm(XsContext& x, TcContext& c, cudaStream_t st, const __nv_bfloat16* X, const __nv_bfloat16* W,
                    const __nv_bfloat16* bias, int M, int N, int K, void* out, int ldo, int epi, int* status,
                    const tc::QkvOut* qkv_out = nullptr, const __nv_bfloat16* Wp = nullptr, int force_cluster = 0) {
  if (!x.ready || !c.ready || K % tc::BK || M < 1 || M > txs::TOK || N < 1) return false;
  if (epi == EPI_QKV_CACHE && (!qkv_out || qkv_out->d % 128 || qkv_out->hd % 8 || N != 3 * qkv_out->d)) return false;
  if (epi == EPI_RELU_T && (N % 8 || ldo != 2 * N)) return false;
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(out)) & 15) return false;
  tc::QkvOut qo = qkv_out ? *qkv_out : tc::QkvOut{};
  qo.packed_kb = Wp ? K / tc::BK : 0;
  qo.w_packed = Wp;
  const CUtensorMap* mw = tc_map(c, W, N, K, tc::BM);
  const CUtensorMap* mx = tc_map(c, X, M, 2 * K, txs::TOK);
  if (!mw || !mx) return false;
  const int kb_total = K / tc::BK;
  const int tiles = (N + txs::WN - 1) / txs::WN;
  int S = 1, splits = 1;
  if (epi == EPI_RESIDUAL_F32) {
    splits = std::max(1, std::min(kb_total / 4, c.sm_count / tiles));
  } else if (kb_total >= 8 && x.max_clusters2 > 0 && force_cluster != 1) {
    const int w1 = (tiles + c.sm_count - 1) / c.sm_count, w2 = (tiles + x.max_clusters2 - 1) / x.max_clusters2;
    if (force_cluster == 2 || w2 * (0.5 + 0.2) < w1 * (1.0 + 0.2)) S = 2;
  }
  int kb_per_split = (kb_total + splits - 1) / splits;
  splits = (kb_total + kb_per_split - 1) / kb_per_split;
  dim3 grid(tiles * S, 1, splits);
  cudaError_t e;
  switch (epi) {
    case EPI_STORE_F32: e = xs_launch<EPI_STORE_F32>(c.pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    case EPI_RELU_T: e = xs_launch<EPI_RELU_T>(c.pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    case EPI_QKV_CACHE: e = xs_launch<EPI_QKV_CACHE>(c.pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
    default: e = xs_launch<EPI_RESIDUAL_F32>(c.pdl, st, grid, S, mw, mx, bias, out, ldo, M, N, K, kb_per_split, status, qo); break;
  }
  if (e != cudaSuccess) { cudaGetLastError(); return false; }
  return true;
}
template <typename T>
inline bool xs_gemm(XsContext&, TcContext&, cudaStream_t, const T*, const T*, const T*, int, int, int, void*, int, int, int*,
                    const tc::QkvOut* = nullptr, const T* = nullptr, int = 0) {
  return false;
}

}  // namespace sd
