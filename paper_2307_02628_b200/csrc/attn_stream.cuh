// Split-KV decode attention for bf16 storage with the keys and values staged through shared memory.
//
// Same arithmetic, thread-to-key mapping and merge as attn_partial_kernel (one block per (row, head) and
// split; hd/8 lanes per key, each with 8 elements of q; base-2 online softmax per lane group; the last
// split to arrive merges).  What differs is how K and V reach the threads.  A (batch row, head) K stream is
// contiguous in the cache, T * hd * 2 bytes, and so is its V stream: a fifth warp copies them in pieces of
// 8 KB with 1-D bulk copies into a ring of four shared-memory stages (K piece | V piece), and the four
// consumer warps read their 16-byte slices from there and hand a stage back as soon as it is in registers.
// The bytes a block keeps in flight are then its ring at every moment, instead of eight 16-byte loads per
// thread that are all consumed before the next eight are issued.
//
// Barriers: full[s] (producer's expect_tx + the two copies' bytes) and empty[s] (one arrival per consumer
// warp).  Every wait is bounded; on expiry the block sets the wait-expired bit of the status word, the
// producer waits (bounded) for the copies it has issued, and the block's result is garbage.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

namespace as {
using tc::smem_u32;

constexpr int NW = 4;                           // consumer warps (eight measured 1 % slower)
constexpr int THREADS = 32 * (NW + 1);          // the consumer warps and the producer warp
constexpr int TILE = 8192;                      // bytes of K (and of V) per stage: one bulk copy each
constexpr int STAGES = 4;                       // 64 KB of ring per block, three blocks per SM
constexpr int BLOCKS_PER_SM = 3;
__host__ __device__ constexpr int smem_bytes() { return STAGES * 2 * TILE; }

__device__ __forceinline__ void lds16(uint32_t addr, float (&o)[8]) {
  uint32_t w[4];
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
#pragma unroll
  for (int i = 0; i < 4; ++i) {                 // bf16 -> fp32 is a 16-bit shift
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
}  // namespace as

template <int HD>
__global__ void __launch_bounds__(as::THREADS)
attn_stream_kernel(const float* __restrict__ qkv, int ldq, const __nv_bfloat16* __restrict__ Kc,
                   const __nv_bfloat16* __restrict__ Vc, int cap, int H, RowMap map, int chunk, int max_chunks,
                   float* part_acc, float* part_ml, int* __restrict__ counters, __nv_bfloat16* __restrict__ o,
                   int* __restrict__ status) {
  using T = __nv_bfloat16;
  constexpr int VEC = 8;
  constexpr int LPK = HD / VEC;              // lanes per key
  constexpr int KPW = 32 / LPK;              // keys per warp step
  constexpr int NW = as::NW;                 // consumer warps
  constexpr int G = NW * KPW;                // keys per block step
  constexpr int ROW = HD * 2;                // bytes per key
  constexpr int KC = as::TILE / ROW;         // keys per stage
  constexpr int UNROLL = (KC / G) < 4 ? (KC / G) : 4;   // block steps per pass over registers
  constexpr int SUBK = G * UNROLL;           // keys per pass
  constexpr int PASSES = KC / SUBK;          // passes per stage
  static_assert(LPK >= 1 && LPK <= 32 && (LPK & (LPK - 1)) == 0 && KC % SUBK == 0 && PASSES >= 1, "head size");

  extern __shared__ __align__(128) uint8_t ring[];          // [as::STAGES][K tile | V tile]
  __shared__ uint64_t bars[2 * as::STAGES];
  __shared__ int abort_word;
  __shared__ float sm_acc[NW][HD];
  __shared__ float sm_m[NW], sm_l[NW];
  __shared__ int sm_last;

  pdl_begin();
  const int rh = blockIdx.x, r = rh / H, h = rh - r * H;
  int b, pos;
  map.get(r, b, pos);
  const int T_len = min(pos + 1, cap);
  if ((int)blockIdx.y * chunk >= T_len) return;
  const int k1 = min((int)blockIdx.y * chunk + chunk, T_len);
  // left padding: keys before the row's first slot do not exist for it.  A chunk that lies wholly
  // in the padding walks no keys and publishes an empty partial (max -inf, sum 0).
  const int k0 = max((int)blockIdx.y * chunk, map.first_key(b, pos));
  const int n_it = k1 > k0 ? (k1 - k0 + KC - 1) / KC : 0;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t ring0 = as::smem_u32(ring);
  const uint32_t full0 = as::smem_u32(bars), empty0 = full0 + 8 * as::STAGES;
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    for (int s = 0; s < as::STAGES; ++s) { tc::mbar_init(full0 + 8 * s, 1); tc::mbar_init(empty0 + 8 * s, NW); }
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == NW) {
    // producer: one thread streams the (row, head)'s keys k0..k1 and their values, KC keys per stage
    if (lane == 0) {
      const size_t base = ((size_t)b * H + h) * cap * HD;
      const T* Kp = Kc + base;
      const T* Vp = Vc + base;
      int issued = 0;
      for (int it = 0; it < n_it; ++it) {
        const int s = it % as::STAGES, round = it / as::STAGES;
        if (round > 0 && !tc::mbar_wait(empty0 + 8 * s, (round - 1) & 1, abort_flag, status)) break;
        const int key = k0 + it * KC;
        const uint32_t bytes = (uint32_t)min(KC, k1 - key) * ROW;
        const uint32_t fb = full0 + 8 * s, dst = ring0 + s * (2 * as::TILE);
        tc::mbar_expect_tx(fb, 2 * bytes);
        tc::bulk_load(dst, Kp + (size_t)key * HD, bytes, fb);
        tc::bulk_load(dst + as::TILE, Vp + (size_t)key * HD, bytes, fb);
        issued = it + 1;
      }
      if (*abort_flag) {
        // a wait expired somewhere in the block: let every copy issued land before the block can exit
        const int first = issued > as::STAGES ? issued - as::STAGES : 0;
        for (int i = first; i < issued; ++i) {
          const long long t0 = clock64();
          while (!tc::mbar_try(full0 + 8 * (i % as::STAGES), (i / as::STAGES) & 1) && clock64() - t0 < tc::kWaitLimit) {}
        }
      }
    }
    return;
  }

  const int grp = lane / LPK, sub = lane % LPK;
  // q, scaled by hd^-1/2 and by log2(e) so the softmax runs on exp2
  float q[VEC];
  {
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
    const float* qp = qkv + (size_t)r * ldq + h * HD + sub * VEC;
#pragma unroll
    for (int v = 0; v < VEC; ++v) q[v] = qp[v] * sc;
  }
  float m = -INFINITY, l = 0.f, acc[VEC];
#pragma unroll
  for (int v = 0; v < VEC; ++v) acc[v] = 0.f;

  const int in_stage = warp * KPW + grp;       // this lane group's key inside a block step
  for (int it = 0; it < n_it; ++it) {
    const int s = it % as::STAGES, round = it / as::STAGES;
    // the vote keeps the warp together: the shuffles below name all 32 lanes
    if (!__all_sync(0xffffffffu, tc::mbar_wait(full0 + 8 * s, round & 1, abort_flag, status))) break;
    const int nk_stage = min(KC, k1 - (k0 + it * KC));        // keys this stage holds
    const uint32_t kt0 = ring0 + s * (2 * as::TILE) + sub * 16;
#pragma unroll
    for (int ps = 0; ps < PASSES; ++ps) {
      const int nk = nk_stage - ps * SUBK;                    // keys left from this pass on (uniform over the block)
      if (nk > 0) {
        const uint32_t kt = kt0 + ps * SUBK * ROW, vt = kt + as::TILE;
        float kv[UNROLL][VEC], vv[UNROLL][VEC], sc[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const int j = min(in_stage + u * G, nk - 1);        // clamp: bytes past the stage's keys are stale
          as::lds16(kt + j * ROW, kv[u]);
          as::lds16(vt + j * ROW, vv[u]);
        }
        if (ps == PASSES - 1 || nk <= SUBK) {
          // the last keys of the stage are in registers: hand it back to the producer
          __syncwarp();
          if (lane == 0) as::mbar_arrive(empty0 + 8 * s);
        }
        float mx = m;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          float t = 0.f;
#pragma unroll
          for (int v = 0; v < VEC; ++v) t = fmaf(q[v], kv[u][v], t);
#pragma unroll
          for (int o2 = LPK / 2; o2 > 0; o2 >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o2);
          sc[u] = (in_stage + u * G < nk) ? t : -INFINITY;
          mx = fmaxf(mx, sc[u]);
        }
        const float sc_old = exp2_safe(m, mx);
        l *= sc_old;
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] *= sc_old;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const float p = exp2_safe(sc[u], mx);
          l += p;
#pragma unroll
          for (int v = 0; v < VEC; ++v) acc[v] = fmaf(p, vv[u][v], acc[v]);
        }
        m = mx;
      }
    }
  }

  // merge the KPW groups of the warp
#pragma unroll
  for (int o2 = LPK; o2 < 32; o2 <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o2);
    const float l2 = __shfl_xor_sync(0xffffffffu, l, o2);
    const float mn = fmaxf(m, m2);
    const float a = exp2_safe(m, mn), c = exp2_safe(m2, mn);
    l = l * a + l2 * c;
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const float a2 = __shfl_xor_sync(0xffffffffu, acc[v], o2);
      acc[v] = acc[v] * a + a2 * c;
    }
    m = mn;
  }
  // merge the consumer warps (the producer warp has left: barrier 1 counts the 128 consumer threads)
  if (grp == 0) {
#pragma unroll
    for (int v = 0; v < VEC; ++v) sm_acc[warp][sub * VEC + v] = acc[v];
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(32 * as::NW) : "memory");
  float M = sm_m[0];
#pragma unroll
  for (int w = 1; w < NW; ++w) M = fmaxf(M, sm_m[w]);
  float L = 0.f;
#pragma unroll
  for (int w = 0; w < NW; ++w) L += sm_l[w] * exp2_safe(sm_m[w], M);
  const int n_valid = (T_len + chunk - 1) / chunk;          // chunks of this (row, head) that hold keys
  T* orow = o + (size_t)r * H * HD * Operand<T>::PARTS;
  if (n_valid == 1) {                                       // the only chunk: normalise and finish here
    const float inv = 1.f / L;
    for (int c = threadIdx.x; c < HD; c += 32 * NW) {
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) a += sm_acc[w][c] * exp2_safe(sm_m[w], M);
      Operand<T>::store(orow, H * HD, h * HD + c, a * inv);
    }
    return;
  }
  const size_t slot0 = (size_t)rh * max_chunks;
  const size_t slot = slot0 + blockIdx.y;
  for (int c = threadIdx.x; c < HD; c += 32 * NW) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) a += sm_acc[w][c] * exp2_safe(sm_m[w], M);
    part_acc[slot * HD + c] = a;
  }
  if (threadIdx.x == 0) {
    part_ml[slot * 2] = M;
    part_ml[slot * 2 + 1] = L;
  }
  // The block that finishes last for this (row, head) merges all chunks.  Nobody waits: each
  // block publishes its partial, bumps the counter and leaves; only the last one goes on.
  __threadfence();
  asm volatile("bar.sync 1, %0;" ::"n"(32 * as::NW) : "memory");
  if (threadIdx.x == 0) {
    const int done = atomicAdd(&counters[rh], 1);
    sm_last = (done == n_valid - 1);
    if (sm_last) counters[rh] = 0;                          // ready for the next launch
  }
  asm volatile("bar.sync 1, %0;" ::"n"(32 * as::NW) : "memory");
  if (!sm_last) return;
  __threadfence();
  float Mg = -INFINITY;
  for (int s = 0; s < n_valid; ++s) Mg = fmaxf(Mg, __ldcg(part_ml + (slot0 + s) * 2));
  float Lg = 0.f;
  for (int s = 0; s < n_valid; ++s)
    Lg += __ldcg(part_ml + (slot0 + s) * 2 + 1) * exp2_safe(__ldcg(part_ml + (slot0 + s) * 2), Mg);
  const float inv = 1.f / Lg;
  for (int c = threadIdx.x; c < HD; c += 32 * NW) {
    float a = 0.f;
    for (int s = 0; s < n_valid; ++s)
      a += __ldcg(part_acc + (slot0 + s) * HD + c) * exp2_safe(__ldcg(part_ml + (slot0 + s) * 2), Mg);
    Operand<T>::store(orow, H * HD, h * HD + c, a * inv);
  }
}




}  // namespace sd
