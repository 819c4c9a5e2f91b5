// Tensor-core GEMM for bf16 storage on sm_100a: out[m, n] (+)= sum_k X[m, k] W[n, k] + bias[n].
// X rows are Operand rows (kernels.cuh): the activations rounded to fp16.  W is read from the tile-packed copy that
// sd_create makes of every matrix, in which each bf16 weight is stored as the fp16 bit pattern of the same value,
// so that one fp16 x fp16 MMA pass gives the product of the bf16 weights with 11-bit activations.
//
// The weight's output dimension sits on the MMA M axis (D^T = W X^T): a CTA owns 128 rows
// of W, so tiles are full even when the token count M is 16..256, which becomes the MMA N.
// Operands reach shared memory by TMA (128-byte swizzle, K-major; every CTA loads its own tiles), the
// accumulator lives in tensor memory, and one thread issues tcgen05.mma.  Warp roles:
// warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue (each
// reads its own quarter of the 128 TMEM lanes).  K can be split over blockIdx.z for the
// residual epilogue, whose partial sums are added to the fp32 residual stream atomically.
//
// Every mbarrier wait is bounded: on expiry the CTA raises an abort flag, records
// STATUS_WAIT_EXPIRED in the status word, drains the copies it issued and frees its TMEM.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <map>
#include <tuple>

#include "kernels.cuh"

namespace sd {

namespace tc {

constexpr int BM = 128;              // W rows (output features) per CTA = MMA M
constexpr int BK = 64;               // bf16 elements per k-block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr long long kWaitLimit = 4000000000LL;   // clock cycles (~2 s) before a wait gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
      : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another wait expired).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long limit = kWaitLimit) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      atomicOr(status, STATUS_WAIT_EXPIRED);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// K-major operand tile in shared memory, rows of 128 bytes, 128-byte swizzle, groups of 8
// rows 1024 bytes apart.  Fields: start address >> 4 [0,14), leading byte offset >> 4
// [16,30) (unused for swizzled K-major, set to 1), stride byte offset >> 4 [32,46) = 64,
// descriptor version 1 [46,48), layout type 2 = SWIZZLE_128B [61,64).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// kind::f16 instruction descriptor: D = fp32 [4,6), A and B formats [7,10) [10,13) = 0 (fp16; 1 would be bf16), both
// K-major, N >> 3 at [17,23), M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}

// Where the QKV epilogue puts its rows: features [0, d) are the query (fp32, into the qkv
// buffer), [d, 2d) the key and [2d, 3d) the value, written straight into the layer's cache at
// each token's position.  A 128-row tile never straddles two sections because d % 128 == 0.
struct QkvOut {
  __nv_bfloat16* Kc;
  __nv_bfloat16* Vc;
  int d, H, hd, cap;
  RowMap map;
  int packed_kb;     // every epilogue: 0 = W is row-major [N, K]; else W is tile-packed with K/64 tiles per row tile
  const __nv_bfloat16* w_packed;
  // K split under an epilogue that is not linear (ReLU, rounding into the cache, plain store): every
  // split parks its partial tile in ws[(tile * splits + split)][token column][weight row] and bumps
  // ws_count[tile]; the block that arrives last adds the partials in split order and runs the epilogue.
  float* ws;
  int* ws_count;     // zero between launches (the last block puts it back)
  int fix_residual;  // 1: the residual epilogue takes the same route (partials added in split order, one plain update per
                     //    element) instead of atomic adds in arrival order: bit-identical results from run to run
  int test_expire;   // test hook: the MMA warp never reports the accumulator complete and the epilogue gives up its wait
                     //    after about a millisecond; every copy has landed and every MMA has been issued by then
};

// Tile-packed weights: [ceil(N/128)][K/64] tiles of 128 rows x 64 columns, each tile stored as
// the 16 KB shared-memory image the MMA wants (128-byte rows with the 128-byte swizzle already
// applied: 16-byte chunk c of row r sits at chunk c ^ (r & 7)).  A tile is then one contiguous
// 1-D bulk copy, with no per-row address generation, and the tiles a block streams (fixed row
// tile, consecutive k-blocks) are adjacent in HBM.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void load_w_tile(uint32_t dst, const CUtensorMap* map, const QkvOut& qo, int kb, int n_row0, uint32_t bar) {
  if (qo.packed_kb)
    bulk_load(dst, qo.w_packed + ((size_t)(n_row0 >> 7) * qo.packed_kb + kb) * (BM * BK), BM * BK * 2, bar);
  else
    tma_load_2d(dst, map, kb * BK, n_row0, bar);
}
// `count` consecutive k-blocks of one row tile: adjacent in the packed copy, so one bulk copy brings them all
__device__ __forceinline__ void load_w_tiles(uint32_t dst, const CUtensorMap* map, const QkvOut& qo, int kb, int count, int n_row0, uint32_t bar) {
  if (qo.packed_kb)
    bulk_load(dst, qo.w_packed + ((size_t)(n_row0 >> 7) * qo.packed_kb + kb) * (BM * BK), count * (BM * BK * 2), bar);
  else
    for (int t = 0; t < count; ++t) tma_load_2d(dst + t * (BM * BK * 2), map, (kb + t) * BK, n_row0, bar);
}

// Epilogue warps: a warp can only read the quarter of the tensor-memory lanes that matches its index
// mod 4, so there are four warps per group; with two groups each takes half of the token columns,
// which halves the serial part of the epilogue (loads from tensor memory, then one store per column).
__host__ __device__ constexpr int epi_warps(int nb) { return nb >= 32 ? 8 : 4; }
__host__ __device__ constexpr int block_threads(int nb) { return 64 + 32 * epi_warps(nb); }
// k-blocks per pipeline stage.  The thread that issues the MMAs pays a fixed price per stage (one barrier
// wait, one fence, one commit) beside the four instructions of a k-block, and at 64 tokens or fewer that
// chain, not the tensor pipe, paces the block: two k-blocks per stage halve the fixed part.
__host__ __device__ constexpr int kps_for(int nb) { return nb >= 128 ? 1 : 2; }
__host__ __device__ constexpr int stage_bytes(int nb) { return kps_for(nb) * (BM * BK * 2 + nb * BK * 2); }   // W tiles, then X tiles
// 6 stages of 32 KB at 128 tokens (a 7th fits and measured no faster), else all that fit in 227 KB: 4, 5, 6 at 64, 32, 16 tokens
__host__ __device__ constexpr int stages_for(int nb) { return nb >= 128 ? 6 : (227 * 1024 - 2304) / stage_bytes(nb); }
__host__ __device__ constexpr int smem_bytes(int nb) { return stages_for(nb) * stage_bytes(nb) + 1024 /*alignment*/ + 256 /*barriers*/ + 1024 /*per-column cache rows*/; }

template <int NB, int EPI>
__global__ void __launch_bounds__(block_threads(NB), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __nv_bfloat16* __restrict__ bias, void* __restrict__ out, int ldo, int M, int N, int K,
               int kb_per_split, int* __restrict__ status, const QkvOut qo) {
  constexpr int STAGES = stages_for(NB), KPS = kps_for(NB);
  constexpr int A_BYTES = BM * BK * 2, B_BYTES = NB * BK * 2, STAGE_BYTES = KPS * (A_BYTES + B_BYTES);
  constexpr int X_OFF = KPS * A_BYTES;           // a stage holds KPS weight tiles, then KPS token tiles
  constexpr int TMEM_COLS = NB < 32 ? 32 : NB;   // one accumulator column per token; a power of two >= 32
  constexpr int EW = epi_warps(NB);              // epilogue warps: 4, or 8 = two groups that split the columns
  constexpr int GROUP_COLS = NB / (EW / 4);      // token columns per group of four warps
  constexpr int CW = GROUP_COLS < 32 ? 16 : 32;  // accumulator columns read per tcgen05.ld

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // swizzled tiles need 1024-byte alignment
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + STAGES * STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES, accum_bar = full0 + 16 * STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);   // split K with fix-up: this block arrived last
  long long* col_row = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(bars) + 256);   // [NB], QKV epilogue only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BM, m0 = blockIdx.y * NB;
  const int kb_total = (K + BK - 1) / BK;
  const int kb0 = blockIdx.z * kb_per_split, kb1 = min(kb0 + kb_per_split, kb_total);
  const int nkb = kb1 - kb0;                                     // >= 1 by construction of the grid
  const int nst = (nkb + KPS - 1) / KPS;                         // pipeline stages' worth of k-blocks; the last may be short

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

  if (warp == 0) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
      // The weights do not depend on the previous kernel: start streaming the first stages'
      // W tiles while it is still finishing, and only then wait for it before touching X.
      const int early = nst < STAGES ? nst : STAGES;
      for (int i = 0; i < early; ++i) {
        const uint32_t fb = full0 + 8 * i;
        const int c = min(KPS, nkb - i * KPS);
        mbar_expect_tx(fb, c * (A_BYTES + B_BYTES));
        load_w_tiles(tiles + i * STAGE_BYTES, &map_w, qo, kb0 + i * KPS, c, n0, fb);
      }
      pdl_wait();
      int issued = early;
      for (int i = 0; i < nst; ++i) {
        const int s = i % STAGES, round = i / STAGES;
        const uint32_t fb = full0 + 8 * s;
        const uint32_t a_dst = tiles + s * STAGE_BYTES;
        const int c = min(KPS, nkb - i * KPS);
        if (round > 0) {
          if (!mbar_wait(empty0 + 8 * s, (round - 1) & 1, abort_flag, status)) break;
          mbar_expect_tx(fb, c * (A_BYTES + B_BYTES));
          load_w_tiles(a_dst, &map_w, qo, kb0 + i * KPS, c, n0, fb);
        }
        for (int t = 0; t < c; ++t)
          tma_load_2d(a_dst + X_OFF + t * B_BYTES, &map_x, (kb0 + i * KPS + t) * BK, m0, fb);
        if (i + 1 > issued) issued = i + 1;
      }
      if (*abort_flag) {
        // drain: wait (bounded) until every copy issued has landed before the CTA exits
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
      bool ok = true;
      for (int i = 0; i < nst && ok; ++i) {
        const int s = i % STAGES, round = i / STAGES;
        ok = mbar_wait(full0 + 8 * s, round & 1, abort_flag, status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = tiles + s * STAGE_BYTES;
        const int c = min(KPS, nkb - i * KPS);
#pragma unroll
        for (int t = 0; t < KPS; ++t) {
          if (t < c) {
            const uint64_t a_desc = smem_desc(a_addr + t * A_BYTES), b_desc = smem_desc(a_addr + X_OFF + t * B_BYTES);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)   // 32 bytes further along K inside the swizzle row
              umma(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i > 0 || t > 0 || k > 0) ? 1u : 0u);
          }
        }
        umma_commit(empty0 + 8 * s);              // the stage is free once these MMAs have read it
      }
      if (ok && !qo.test_expire) umma_commit(accum_bar);   // the accumulator is complete
    }
  } else {
    pdl_wait();                                   // bias aside, the epilogue reads and writes buffers earlier kernels own
    const int quarter = warp & 3;                 // TMEM lanes [32 * quarter, +32) belong to this warp
    const int n = n0 + quarter * 32 + lane;
    // QKV epilogue: cache row (b * H * cap + pos) of every token column, worked out once per block;
    // this thread's feature picks the head and the element inside the row
    int kv_head = 0, kv_elem = 0;
    __nv_bfloat16* kv_base = nullptr;
    if (EPI == EPI_QKV_CACHE) {
      const int t = threadIdx.x - 64;             // 0.. over the epilogue warps
      if (t < NB) {
        int b, pos;
        qo.map.get(m0 + t, b, pos);
        col_row[t] = (m0 + t < M && pos < qo.cap) ? (long long)b * qo.H * qo.cap + pos : -1;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(32 * EW) : "memory");
      if (n >= qo.d && n < N) {
        const int cc = n < 2 * qo.d ? n - qo.d : n - 2 * qo.d;
        kv_head = cc / qo.hd;
        kv_elem = cc - kv_head * qo.hd;
        kv_base = n < 2 * qo.d ? qo.Kc : qo.Vc;
      }
    }
    // the bias is a weight: fetched now, so that its latency hides behind the main loop.  It goes in once: with the
    // fix-up by the block that finishes the tile, else by the first split
    const bool fix = (EPI != EPI_RESIDUAL_F32 || qo.fix_residual) && gridDim.z > 1;
    const float b = (bias != nullptr && n < N && (fix || EPI != EPI_RESIDUAL_F32 || blockIdx.z == 0)) ? __bfloat162float(bias[n]) : 0.f;
    const bool accum_ok = mbar_wait(accum_bar, 0, abort_flag, status, qo.test_expire ? 2000000LL : kWaitLimit);
    // The main loop is over: let the next kernel of the stream become resident now, so that its
    // launch and set-up overlap this kernel's epilogue (earlier would only park its blocks on the
    // SMs for the whole main loop).
    pdl_launch_dependents();
    // K split under a non-linear epilogue: park the partial tile, count arrivals, and let
    // the block that arrives last finish the tile from the parked partials
    bool go = accum_ok;
    if (fix) {
      // the fix-up meets at a named barrier: all epilogue threads take it or none (a bounded wait may
      // have expired for some of them only)
      int all;
      asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 q, %1, 0;\n bar.red.and.pred p, 1, %2, q;\n selp.b32 %0, 1, 0, p;\n}\n"
                   : "=r"(all) : "r"((int)accum_ok), "n"(32 * EW) : "memory");
      go = all != 0;
    }
    if (go) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int c_begin = ((warp - 2) >> 2) * GROUP_COLS;
      const int splits = (int)gridDim.z, tile_id = (int)(blockIdx.y * gridDim.x + blockIdx.x);
      float* ws_tile = fix ? qo.ws + (size_t)tile_id * splits * (NB * BM) + quarter * 32 + lane : nullptr;
      bool emit = true;
      if (fix) {
        float* mine = ws_tile + (size_t)blockIdx.z * (NB * BM);
#pragma unroll 1
        for (int c = c_begin; c < c_begin + GROUP_COLS; c += CW) {
          uint32_t r[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c;
          if (CW == 32) tmem_ld32(taddr, r); else tmem_ld16(taddr, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < CW; ++j)             // 32 lanes = 32 consecutive weight rows: one 128-byte store per column
            __stcg(mine + (size_t)(c + j) * BM, __uint_as_float(r[j]));
        }
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(32 * EW) : "memory");
        if (threadIdx.x == 64) {
          const int arrived = atomicAdd(qo.ws_count + tile_id, 1);
          const int last = arrived == splits - 1;
          if (last) qo.ws_count[tile_id] = 0;     // every split has arrived: ready for the next launch
          *last_flag = last;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * EW) : "memory");
        emit = *last_flag != 0;
        if (emit) __threadfence();
      }
#pragma unroll 1
      for (int c = c_begin; emit && c < c_begin + GROUP_COLS; c += CW) {
        uint32_t r[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c;
        if (fix) {
          // partials added in split order, so the result does not depend on which block came last; all
          // loads of one split are in flight together
#pragma unroll
          for (int j = 0; j < CW; ++j) r[j] = 0u;
#pragma unroll 1
          for (int z = 0; z < splits; ++z) {
            const float* src = ws_tile + (size_t)z * (NB * BM) + (size_t)c * BM;
            float t[CW];
#pragma unroll
            for (int j = 0; j < CW; ++j) t[j] = __ldcg(src + (size_t)j * BM);
#pragma unroll
            for (int j = 0; j < CW; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + t[j]);
          }
        } else {
          if (CW == 32) tmem_ld32(taddr, r); else tmem_ld16(taddr, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        }
        if (n < N) {
#pragma unroll
          for (int j = 0; j < CW; ++j) {
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
              else if (EPI == EPI_RELU_T)      // the result is the next product's operand row
                Operand<__nv_bfloat16>::store(reinterpret_cast<__nv_bfloat16*>(out) + (size_t)m * ldo, N, n, fmaxf(v, 0.f));
              else if (fix) reinterpret_cast<float*>(out)[idx] += v;      // the only block that touches this tile's elements now
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

// One block per 128 x 64 tile: tile (tn, kb) holds W[tn * 128 + r][kb * 64 + 8 c .. +8] at 16-byte
// piece r * 8 + (c ^ (r & 7)); rows past N are zero.  Each bf16 weight is written as the fp16 with the same value:
// exact for magnitudes in [2^-14, 65504] (every bf16 has at most 8 significant bits); smaller ones land on the fp16
// subnormal grid (absolute error at most 2^-25), larger ones saturate and raise STATUS_WEIGHT_RANGE.
__global__ void pack_tiles_kernel(const __nv_bfloat16* __restrict__ W, __nv_bfloat16* __restrict__ P, int N, int K, int* __restrict__ status) {
  const int KB = K / BK;
  const int tn = blockIdx.x / KB, kb = blockIdx.x - tn * KB;
  uint4* dst = reinterpret_cast<uint4*>(P + (size_t)blockIdx.x * BM * BK);
  for (int i = threadIdx.x; i < BM * BK / 8; i += blockDim.x) {      // 16-byte pieces: 8 per tile row
    const int r = i >> 3, c8 = i & 7;
    const int n = tn * BM + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (n < N) {
      const uint4 w = *reinterpret_cast<const uint4*>(W + (size_t)n * K + kb * BK + c8 * 8);
      const uint32_t in[4] = {w.x, w.y, w.z, w.w};
      uint32_t out[4];
      bool clipped = false;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = __uint_as_float(in[e] << 16), b = __uint_as_float(in[e] & 0xffff0000u);
        clipped = clipped || fabsf(a) > 65504.f || fabsf(b) > 65504.f;
        const __half2 h = __floats2half2_rn(sat_f16(a), sat_f16(b));
        out[e] = *reinterpret_cast<const uint32_t*>(&h);
      }
      if (clipped) atomicOr(status, STATUS_WEIGHT_RANGE);
      v = make_uint4(out[0], out[1], out[2], out[3]);
    }
    dst[r * 8 + (c8 ^ (r & 7))] = v;
  }
}

}  // namespace tc

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kSplitSlots = 160;   // parked partial tiles: tiles x splits of one launch never exceed this

struct TcContext {
  EncodeTiledFn encode = nullptr;
  int ready = 0;
  int sm_count = 148;
  bool pdl = false;      // launch with the programmatic-dependent-launch attribute
  // split K under a non-linear epilogue: parked partial tiles (kSplitSlots of 128 x 128 floats) and arrival counters
  float* splitk_ws = nullptr;
  int* splitk_count = nullptr;
  int splitk = 8;        // most splits of K under a non-linear epilogue; 0: K is split for the residual products only
  int deterministic = 0; // 1: split-K partial sums of the residual products are added in split order too (no atomics)
  int test_expire = 0;   // test hook: the next product makes its accumulator wait expire (one shot)
  // (pointer, rows, cols, box rows) -> tensor map of a row-major bf16 matrix, 64-column boxes, 128-byte swizzle
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> maps;
};

template <int NB, int EPI>
inline bool tc_prepare() {
  return cudaFuncSetAttribute(tc::gemm_tc_kernel<NB, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::smem_bytes(NB)) == cudaSuccess;
}
template <int NB>
inline bool tc_prepare_nb() {
  return tc_prepare<NB, EPI_STORE_F32>() && tc_prepare<NB, EPI_RELU_T>() && tc_prepare<NB, EPI_RESIDUAL_F32>() &&
         tc_prepare<NB, EPI_QKV_CACHE>();
}

inline void tc_init(TcContext& c) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return;
  }
  c.encode = reinterpret_cast<EncodeTiledFn>(fn);
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return; }
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (major != 10) return;                       // tcgen05 exists on sm_100 only
  if (sms > 0) c.sm_count = sms;
  if (!(tc_prepare_nb<16>() && tc_prepare_nb<32>() && tc_prepare_nb<64>() && tc_prepare_nb<128>())) {
    cudaGetLastError();
    return;
  }
  c.ready = 1;
}
inline void tc_destroy(TcContext& c) { c.maps.clear(); c.ready = 0; }

// Looks the map up (or encodes it) and copies it into *out: the cache may evict entries on a later call, so
// callers keep no pointer into it.
inline bool tc_map(TcContext& c, const void* ptr, int rows, int cols, int box_rows, CUtensorMap* out) {
  auto key = std::make_tuple(ptr, rows, cols, box_rows);
  auto it = c.maps.find(key);
  if (it != c.maps.end()) { *out = it->second; return true; }
  CUtensorMap m;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)tc::BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  if (c.encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (c.maps.size() > 4096) c.maps.clear();
  c.maps.emplace(key, m);
  *out = m;
  return true;
}

template <int NB>
inline bool tc_launch(bool pdl, cudaStream_t st, const CUtensorMap* mw, const CUtensorMap* mx, const __nv_bfloat16* bias, void* out,
                      int ldo, int M, int N, int K, int kb_per_split, int splits, int epi, int* status, const tc::QkvOut& qo) {
  dim3 grid((N + tc::BM - 1) / tc::BM, (M + NB - 1) / NB, splits);
  const dim3 block(tc::block_threads(NB));
  const int smem = tc::smem_bytes(NB);
  if (epi == EPI_STORE_F32)
    launch_kernel(pdl, st, tc::gemm_tc_kernel<NB, EPI_STORE_F32>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
  else if (epi == EPI_RELU_T)
    launch_kernel(pdl, st, tc::gemm_tc_kernel<NB, EPI_RELU_T>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
  else if (epi == EPI_QKV_CACHE)
    launch_kernel(pdl, st, tc::gemm_tc_kernel<NB, EPI_QKV_CACHE>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
  else
    launch_kernel(pdl, st, tc::gemm_tc_kernel<NB, EPI_RESIDUAL_F32>, grid, block, smem, *mw, *mx, bias, out, ldo, M, N, K, kb_per_split, status, qo);
  return true;
}

// Returns true when the product was enqueued on the tensor-core path; false leaves it to the caller.
inline bool tc_gemm(TcContext& c, cudaStream_t st, const __nv_bfloat16* X, const __nv_bfloat16* W, const __nv_bfloat16* bias,
                    int M, int N, int K, void* out, int ldo, int epi, int* status, const tc::QkvOut* qkv_out = nullptr,
                    const __nv_bfloat16* Wp = nullptr) {
  if (!c.ready || K % tc::BK || M < 1 || N < 1) return false;   // whole k-blocks only
  if (epi == EPI_QKV_CACHE && (!qkv_out || qkv_out->d % tc::BM || N != 3 * qkv_out->d)) return false;
  tc::QkvOut qo = qkv_out ? *qkv_out : tc::QkvOut{};
  qo.packed_kb = Wp ? K / tc::BK : 0;
  qo.w_packed = Wp;
  if (!Wp) return false;                       // the MMAs take the weights from the packed fp16 copy only
  if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 15) return false;
  const int nb = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128;
  CUtensorMap mw_v, mx_v;
  const CUtensorMap *mw = &mw_v, *mx = &mx_v;                 // W's map is not used by the kernel (packed copy)
  if (!tc_map(c, W, N, K, tc::BM, &mw_v) || !tc_map(c, X, M, K, nb, &mx_v)) return false;
  const int kb_total = (K + tc::BK - 1) / tc::BK;
  int splits = 1;
  if (epi == EPI_RESIDUAL_F32) {                 // partial sums may be added in any order
    const int tiles = ((N + tc::BM - 1) / tc::BM) * ((M + nb - 1) / nb);
    splits = std::max(1, std::min(kb_total / 4, c.sm_count / tiles));     // one wave: never more blocks than SMs
    if (c.deterministic && c.splitk_ws) {        // ... or in split order, through the parked partial tiles
      splits = std::max(1, std::min(splits, kSplitSlots / tiles));
      qo.ws = c.splitk_ws;
      qo.ws_count = c.splitk_count;
      qo.fix_residual = 1;
    }
  } else if (c.splitk && c.splitk_ws) {
    // The other epilogues are not linear, so the block that arrives last finishes the tile from parked
    // partials.  That costs a second pass over the tile: only where fewer than half of the SMs would hold
    // a block and every split keeps at least 8 k-blocks (the main loop is paced per MMA instruction, so
    // the time saved is the k-blocks a block no longer issues).
    const int tiles = ((N + tc::BM - 1) / tc::BM) * ((M + nb - 1) / nb);
    if (2 * tiles <= c.sm_count)
      splits = std::max(1, std::min(std::min(std::min(kb_total / 8, c.sm_count / tiles), kSplitSlots / tiles), c.splitk));
    qo.ws = c.splitk_ws;
    qo.ws_count = c.splitk_count;
  }
  int kb_per_split = (kb_total + splits - 1) / splits;
  splits = (kb_total + kb_per_split - 1) / kb_per_split;      // no empty split
  if (c.test_expire) { qo.test_expire = 1; c.test_expire = 0; }
  switch (nb) {
    case 16: return tc_launch<16>(c.pdl, st, mw, mx, bias, out, ldo, M, N, K, kb_per_split, splits, epi, status, qo);
    case 32: return tc_launch<32>(c.pdl, st, mw, mx, bias, out, ldo, M, N, K, kb_per_split, splits, epi, status, qo);
    case 64: return tc_launch<64>(c.pdl, st, mw, mx, bias, out, ldo, M, N, K, kb_per_split, splits, epi, status, qo);
    default: return tc_launch<128>(c.pdl, st, mw, mx, bias, out, ldo, M, N, K, kb_per_split, splits, epi, status, qo);
  }
}
template <typename T>
inline bool tc_gemm(TcContext&, cudaStream_t, const T*, const T*, const T*, int, int, int, void*, int, int, int*,
                    const tc::QkvOut* = nullptr, const T* = nullptr) {
  return false;                                  // fp32 storage runs on the CUDA-core kernel
}

}  // namespace sd
