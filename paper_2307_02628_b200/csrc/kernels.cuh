// CUDA-core kernels of the skip-decode step: embedding, LayerNorm, KV append,
// split-KV decode attention (with its merge), greedy argmax, and the CUDA-core GEMM
// used by the fp32 configuration (and as the fallback for shapes the tensor-core
// GEMM does not take).  T is the storage type: float or __nv_bfloat16.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sd {

enum : int { STATUS_BAD_TOKEN = 1, STATUS_WAIT_EXPIRED = 2, STATUS_BAD_SHAPE = 4, STATUS_WEIGHT_RANGE = 8 };

// Programmatic dependent launch.  Every kernel of the step calls pdl_begin() before it touches
// anything an earlier kernel wrote: it lets the next kernel in the stream start its own
// prologue early and then blocks until the previous kernel has completed and its writes are
// visible.  Both instructions do nothing when the launch carries no programmatic attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_begin() { pdl_launch_dependents(); pdl_wait(); }

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte vector of T, widened to fp32.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void load(const float* p, float (&o)[4]) {
    float4 v = __ldg(reinterpret_cast<const float4*>(p));
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&o)[8]) {
    uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {       // bf16 -> fp32 is a 16-bit shift
      o[2 * i] = __uint_as_float(w[i] << 16);
      o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

// GEMM input operands (activations).  In fp32 storage an operand row is K floats.  In bf16 storage it is K
// 16-bit slots that hold the value rounded to fp16 (11 significant bits, against the 8 of a bf16), saturated at
// the largest finite fp16: the tensor-core kernels multiply them with the weights' values held as fp16 as well (a
// bf16 weight is an fp16 value exactly unless its magnitude is below 2^-14 or above 65504, see pack_tiles_kernel),
// one MMA pass per product.  Weights as the caller stores them and the KV cache stay bf16.  The operand buffers are
// typed as the storage type; only the two functions below know what the 16 bits mean.
template <typename T> struct Operand;
template <> struct Operand<float> {
  static constexpr int PARTS = 1;
  __device__ static __forceinline__ void store(float* row, int K, int c, float v) { row[c] = v; }
  __device__ static __forceinline__ float load(const float* row, int K, int c) { return row[c]; }
};
__device__ __forceinline__ float sat_f16(float v) { return fminf(fmaxf(v, -65504.f), 65504.f); }
template <> struct Operand<__nv_bfloat16> {
  static constexpr int PARTS = 1;
  __device__ static __forceinline__ void store(__nv_bfloat16* row, int K, int c, float v) {
    reinterpret_cast<__half*>(row)[c] = __float2half_rn(sat_f16(v));
  }
  __device__ static __forceinline__ float load(const __nv_bfloat16* row, int K, int c) {
    return __half2float(reinterpret_cast<const __half*>(row)[c]);
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block; every thread gets the result.  scratch: >= 33 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = lane < nw ? scratch[lane] : 0.f;
    t = warp_sum(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

// Row r of a launch covers batch row b = b0 + r / q_per_b at position (cache slot)
// pos0 + r % q_per_b.  d_pos, when not null, supplies pos0 from device memory (graph replay).
// rows, when not null (decode steps, q_per_b = 1), lists the batch rows still generating:
// b = rows[r].  pad, when not null, holds each batch row's number of left-padding slots: the
// row's sequence starts at slot pad[b], so its learned position is pos - pad[b] and it
// attends to slots pad[b]..pos only (a padding slot attends to itself alone).
struct RowMap {
  int q_per_b, b0, pos0;
  const int* d_pos;
  const int* rows;
  const int* pad;
  __device__ __forceinline__ void get(int r, int& b, int& pos) const {
    const int p0 = d_pos ? *d_pos : pos0;
    b = rows ? rows[r] : b0 + r / q_per_b;
    pos = p0 + r % q_per_b;
  }
  __device__ __forceinline__ int first_key(int b, int pos) const { return pad ? min(pad[b], pos) : 0; }
  __device__ __forceinline__ int seq_pos(int b, int pos) const { return pad ? max(pos - pad[b], 0) : pos; }
};

// x[r, :] = tok_emb[ids[r], :] + pos_emb[pos(r), :]      (fp32 residual stream)
template <typename T>
__global__ void embed_pos_kernel(const int32_t* __restrict__ ids, const T* __restrict__ tok_emb,
                                 const T* __restrict__ pos_emb, float* __restrict__ x, int d, int vocab,
                                 int max_pos, RowMap map, int* __restrict__ status) {
  pdl_begin();
  const int r = blockIdx.x;
  int b, pos;
  map.get(r, b, pos);
  pos = map.seq_pos(b, pos);
  int id = ids[r];
  if (id < 0 || id >= vocab || pos < 0 || pos >= max_pos) {   // record and clamp: never read out of range
    if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_TOKEN);
    id = min(max(id, 0), vocab - 1);
    pos = min(max(pos, 0), max_pos - 1);
  }
  const T* te = tok_emb + (size_t)id * d;
  const T* pe = pos_emb + (size_t)pos * d;
  float* xr = x + (size_t)r * d;
  if (sizeof(T) == 2 && (d & 3) == 0 && ((reinterpret_cast<uintptr_t>(tok_emb) | reinterpret_cast<uintptr_t>(pos_emb)) & 7) == 0) {
    // bf16 tables: four elements per 8-byte load (a bf16 is the upper half of the float with the same value)
    const uint2* te2 = reinterpret_cast<const uint2*>(te);
    const uint2* pe2 = reinterpret_cast<const uint2*>(pe);
    for (int k = threadIdx.x; k < (d >> 2); k += blockDim.x) {
      const uint2 a = te2[k], p = pe2[k];
      reinterpret_cast<float4*>(xr)[k] =
          make_float4(__uint_as_float(a.x << 16) + __uint_as_float(p.x << 16),
                      __uint_as_float(a.x & 0xffff0000u) + __uint_as_float(p.x & 0xffff0000u),
                      __uint_as_float(a.y << 16) + __uint_as_float(p.y << 16),
                      __uint_as_float(a.y & 0xffff0000u) + __uint_as_float(p.y & 0xffff0000u));
    }
    return;
  }
  for (int c = threadIdx.x; c < d; c += blockDim.x) xr[c] = to_f32(te[c]) + to_f32(pe[c]);
}

// u[r, :] = (x[r, :] - mean) / sqrt(var + eps) * gamma + beta, biased variance, fp32 statistics.
// Two passes over the row (mean, then centred second moment) for accuracy.  u is a GEMM
// operand (see Operand).
template <typename T>
__global__ void __launch_bounds__(256)
layernorm_kernel(const float* __restrict__ x, const T* __restrict__ gamma, const T* __restrict__ beta,
                 T* __restrict__ u, int d, float eps, const int* __restrict__ row_index) {
  constexpr int MAXV = 4;                       // float4 vectors a thread keeps in registers
  __shared__ float red[33];
  pdl_begin();
  const int r = blockIdx.x;
  const float* xr = x + (size_t)(row_index ? row_index[r] : r) * d;
  T* ur = u + (size_t)r * d * Operand<T>::PARTS;
  const int nvec = d >> 2;                      // d is a multiple of 8
  if (nvec <= MAXV * (int)blockDim.x) {         // the row fits in registers: one read of x
    float4 v[MAXV];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int k = i * blockDim.x + threadIdx.x;
      v[i] = k < nvec ? reinterpret_cast<const float4*>(xr)[k] : make_float4(0.f, 0.f, 0.f, 0.f);
      s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
    // bf16 storage: gain and offset as 8-byte vectors, fetched before the reductions so that their latency
    // hides behind them, and the operand row written as 8-byte vectors (4 fp16)
    constexpr bool kVec = sizeof(T) == 2;
    const bool vec = kVec && ((reinterpret_cast<uintptr_t>(gamma) | reinterpret_cast<uintptr_t>(beta)) & 7) == 0;
    uint2 gv[MAXV], bv[MAXV];
    if (vec) {
#pragma unroll
      for (int i = 0; i < MAXV; ++i) {
        const int k = i * blockDim.x + threadIdx.x;
        gv[i] = k < nvec ? reinterpret_cast<const uint2*>(gamma)[k] : make_uint2(0u, 0u);
        bv[i] = k < nvec ? reinterpret_cast<const uint2*>(beta)[k] : make_uint2(0u, 0u);
      }
    }
    const float mean = block_sum(s, red) / d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int k = i * blockDim.x + threadIdx.x;
      if (k < nvec) {
        const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
        q += (a * a + b * b) + (c * c + e * e);
      }
    }
    const float rstd = rsqrtf(block_sum(q, red) / d + eps);
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int k = i * blockDim.x + threadIdx.x;
      if (k < nvec) {
        const float vals[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        if (vec) {
          // a bf16 is the upper half of the float with the same value
          const float g[4] = {__uint_as_float(gv[i].x << 16), __uint_as_float(gv[i].x & 0xffff0000u),
                              __uint_as_float(gv[i].y << 16), __uint_as_float(gv[i].y & 0xffff0000u)};
          const float o[4] = {__uint_as_float(bv[i].x << 16), __uint_as_float(bv[i].x & 0xffff0000u),
                              __uint_as_float(bv[i].y << 16), __uint_as_float(bv[i].y & 0xffff0000u)};
          float y[4];
#pragma unroll
          for (int t = 0; t < 4; ++t) y[t] = sat_f16((vals[t] - mean) * rstd * g[t] + o[t]);
          const __half2 h01 = __floats2half2_rn(y[0], y[1]), h23 = __floats2half2_rn(y[2], y[3]);
          reinterpret_cast<uint2*>(ur)[k] = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
        } else {
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const int c = 4 * k + t;
            Operand<T>::store(ur, d, c, (vals[t] - mean) * rstd * to_f32(gamma[c]) + to_f32(beta[c]));
          }
        }
      }
    }
    return;
  }
  float s = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) s += xr[c];
  const float mean = block_sum(s, red) / d;
  float q = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) { const float t = xr[c] - mean; q += t * t; }
  const float rstd = rsqrtf(block_sum(q, red) / d + eps);
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    Operand<T>::store(ur, d, c, (xr[c] - mean) * rstd * to_f32(gamma[c]) + to_f32(beta[c]));
}

// Writes this launch's keys and values into the layer's cache, in place:
// K[b, h, pos, :] = qkv[r, d + h*hd : ...], V likewise from 2d.  Cache layout
// [max_batch, H, cap, hd]; positions already present are not touched.
template <typename T>
__global__ void kv_append_kernel(const float* __restrict__ qkv, T* __restrict__ Kc, T* __restrict__ Vc,
                                 int d, int H, int hd, int cap, RowMap map) {
  pdl_begin();
  const int r = blockIdx.x;
  int b, pos;
  map.get(r, b, pos);
  if (pos >= cap) return;
  const float* src = qkv + (size_t)r * 3 * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const int h = c / hd, e = c - h * hd;
    const size_t off = (((size_t)b * H + h) * cap + pos) * hd + e;
    Kc[off] = from_f32<T>(src[d + c]);
    Vc[off] = from_f32<T>(src[2 * d + c]);
  }
}

// ---- split-KV decode attention --------------------------------------------------------
// One block per (query row x head, key chunk) = (blockIdx.x, blockIdx.y).  A group of
// LPK = HD / VEC lanes owns one key at a time: each lane holds VEC consecutive dims (one
// 16-byte load of K and of V), the dot product is finished with xor-shuffles inside the
// group, and every group runs its own online softmax in base 2.  Groups are merged by
// shuffles inside a warp and through shared memory across warps.  With one chunk the block
// writes the attention output o[r, h*HD + c] (a GEMM operand) itself; with several, every
// block stores (unnormalised accumulator[HD], running max m as a base-2 exponent, sum l) and
// the block that arrives last at a per-(row, head) counter merges them:
// o = sum_s acc_s 2^(m_s - M) / sum_s l_s 2^(m_s - M).  Partials written by other SMs are read
// with L2 loads (the buffers are reused every layer, so L1 could hold stale lines).
__device__ __forceinline__ float exp2_safe(float a, float m) {   // 2^(a - m), 0 when a = -inf
  return a == -INFINITY ? 0.f : exp2f(a - m);
}

template <typename T, int HD, int UNROLL>
__global__ void __launch_bounds__(128, 7)
attn_partial_kernel(const float* __restrict__ qkv, int ldq, const T* __restrict__ Kc, const T* __restrict__ Vc,
                    int cap, int H, RowMap map, int chunk, int max_chunks,
                    float* part_acc, float* part_ml, int* __restrict__ counters, T* __restrict__ o) {
  constexpr int VEC = Vec16<T>::N;
  constexpr int LPK = HD / VEC;              // lanes per key
  constexpr int KPW = 32 / LPK;              // keys per warp step
  constexpr int NW = 4;
  constexpr int G = NW * KPW;                // key groups per block
  static_assert(LPK >= 1 && LPK <= 32 && (LPK & (LPK - 1)) == 0, "head_dim / vector width must be a power of two <= 32");

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

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane / LPK, sub = lane % LPK;

  // q, scaled by hd^-1/2 and by log2(e) so the softmax runs on exp2
  float q[VEC];
  {
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
    const float* qp = qkv + (size_t)r * ldq + h * HD + sub * VEC;
#pragma unroll
    for (int v = 0; v < VEC; ++v) q[v] = qp[v] * sc;
  }
  const size_t base = ((size_t)b * H + h) * cap * HD + sub * VEC;
  const T* Kp = Kc + base;
  const T* Vp = Vc + base;

  float m = -INFINITY, l = 0.f, acc[VEC];
#pragma unroll
  for (int v = 0; v < VEC; ++v) acc[v] = 0.f;

  // the loop bound is uniform over the warp (the shuffles below use the full mask); a group
  // whose key falls past the chunk end loads a clamped address and masks the score
  for (int jb = k0 + warp * KPW; jb < k1; jb += G * UNROLL) {
    const int j0 = jb + grp;
    float kv[UNROLL][VEC], vv[UNROLL][VEC], s[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int j = min(j0 + u * G, k1 - 1);          // clamp: the load stays inside the cache
      Vec16<T>::load(Kp + (size_t)j * HD, kv[u]);
      Vec16<T>::load(Vp + (size_t)j * HD, vv[u]);
    }
    float mx = m;
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      float t = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) t = fmaf(q[v], kv[u][v], t);
#pragma unroll
      for (int o = LPK / 2; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      s[u] = (j0 + u * G < k1) ? t : -INFINITY;
      mx = fmaxf(mx, s[u]);
    }
    const float sc_old = exp2_safe(m, mx);
    l *= sc_old;
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] *= sc_old;
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const float p = exp2_safe(s[u], mx);
      l += p;
#pragma unroll
      for (int v = 0; v < VEC; ++v) acc[v] = fmaf(p, vv[u][v], acc[v]);
    }
    m = mx;
  }

  // merge the KPW groups of the warp
#pragma unroll
  for (int o = LPK; o < 32; o <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float l2 = __shfl_xor_sync(0xffffffffu, l, o);
    const float mn = fmaxf(m, m2);
    const float a = exp2_safe(m, mn), c = exp2_safe(m2, mn);
    l = l * a + l2 * c;
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const float a2 = __shfl_xor_sync(0xffffffffu, acc[v], o);
      acc[v] = acc[v] * a + a2 * c;
    }
    m = mn;
  }
  // merge the warps
  __shared__ float sm_acc[NW][HD];
  __shared__ float sm_m[NW], sm_l[NW];
  __shared__ int sm_last;
  if (grp == 0) {
#pragma unroll
    for (int v = 0; v < VEC; ++v) sm_acc[warp][sub * VEC + v] = acc[v];
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
  }
  __syncthreads();
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
    for (int c = threadIdx.x; c < HD; c += blockDim.x) {
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) a += sm_acc[w][c] * exp2_safe(sm_m[w], M);
      Operand<T>::store(orow, H * HD, h * HD + c, a * inv);
    }
    return;
  }
  const size_t slot0 = (size_t)rh * max_chunks;
  const size_t slot = slot0 + blockIdx.y;
  for (int c = threadIdx.x; c < HD; c += blockDim.x) {
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
  __syncthreads();
  if (threadIdx.x == 0) {
    const int done = atomicAdd(&counters[rh], 1);
    sm_last = (done == n_valid - 1);
    if (sm_last) counters[rh] = 0;                          // ready for the next launch
  }
  __syncthreads();
  if (!sm_last) return;
  __threadfence();
  float Mg = -INFINITY;
  for (int s = 0; s < n_valid; ++s) Mg = fmaxf(Mg, __ldcg(part_ml + (slot0 + s) * 2));
  float Lg = 0.f;
  for (int s = 0; s < n_valid; ++s)
    Lg += __ldcg(part_ml + (slot0 + s) * 2 + 1) * exp2_safe(__ldcg(part_ml + (slot0 + s) * 2), Mg);
  const float inv = 1.f / Lg;
  for (int c = threadIdx.x; c < HD; c += blockDim.x) {
    float a = 0.f;
    for (int s = 0; s < n_valid; ++s)
      a += __ldcg(part_acc + (slot0 + s) * HD + c) * exp2_safe(__ldcg(part_ml + (slot0 + s) * 2), Mg);
    Operand<T>::store(orow, H * HD, h * HD + c, a * inv);
  }
}

// Host side: launch with the programmatic-dependent-launch attribute when `pdl` is set.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool pdl, cudaStream_t stream, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// next[b] = lowest index of the maximum of logits[b, :]
__global__ void greedy_kernel(const float* __restrict__ logits, int vocab, int32_t* __restrict__ next) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const float* row = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  if ((vocab & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0) {
    // 16-byte loads, four in flight per thread: the row is read once and the kernel is latency-bound
    const float4* row4 = reinterpret_cast<const float4*>(row);
    const int n4 = vocab >> 2;
#pragma unroll 4
    for (int c4 = threadIdx.x; c4 < n4; c4 += blockDim.x) {
      const float4 v = row4[c4];
      const int c = c4 << 2;                    // a thread's columns increase, so ">" keeps the lowest index of a tie
      if (v.x > best) { best = v.x; bi = c; }
      if (v.y > best) { best = v.y; bi = c + 1; }
      if (v.z > best) { best = v.z; bi = c + 2; }
      if (v.w > best) { best = v.w; bi = c + 3; }
    }
  } else {
    for (int c = threadIdx.x; c < vocab; c += blockDim.x) {
      const float v = row[c];
      if (v > best || (v == best && c < bi)) { best = v; bi = c; }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float v2 = __shfl_xor_sync(0xffffffffu, best, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
    if (v2 > best || (v2 == best && i2 < bi)) { best = v2; bi = i2; }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sv[warp] = best; si[warp] = bi; }
  __syncthreads();
  if (warp == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    best = lane < nw ? sv[lane] : -INFINITY;
    bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float v2 = __shfl_xor_sync(0xffffffffu, best, o);
      const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
      if (v2 > best || (v2 == best && i2 < bi)) { best = v2; bi = i2; }
    }
    if (lane == 0) next[blockIdx.x] = bi == 0x7fffffff ? 0 : bi;
  }
}

// ---- CUDA-core GEMM -------------------------------------------------------------------
// out[m, n] (+)= sum_k A[m, k] W[n, k] + bias[n], fp32 accumulation, 64x64 tile, 16-wide
// k-steps, 256 threads with a 4x4 register tile each.  A is an Operand row; the ReLU
// epilogue writes an Operand row.
enum : int { EPI_STORE_F32 = 0, EPI_RELU_T = 1, EPI_RESIDUAL_F32 = 2, EPI_QKV_CACHE = 3 /* tensor-core kernel only */ };

template <typename T, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, int lda, const T* __restrict__ W, int ldw,
                 const T* __restrict__ bias, int M, int N, int K, void* __restrict__ out, int ldo) {
  constexpr int BM = 64, BN = 64, BK = 16;
  pdl_begin();
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[4][4] = {};
  const int lr = threadIdx.x >> 2;            // 0..63: tile row this thread loads
  const int lc = (threadIdx.x & 3) * 4;       // 0,4,8,12: first of its 4 k-columns
  const int am = m0 + lr, wn = n0 + lr;
  const T* arow = am < M ? A + (size_t)am * lda : nullptr;       // lda = K * Operand<T>::PARTS
  const T* wrow = wn < N ? W + (size_t)wn * ldw : nullptr;
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int k = k0 + lc + i;
      As[lc + i][lr] = (arow && k < K) ? Operand<T>::load(arow, K, k) : 0.f;
      Ws[lc + i][lr] = (wrow && k < K) ? to_f32(wrow[k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      const float v = acc[i][j] + (bias ? to_f32(bias[n]) : 0.f);
      if (EPI == EPI_STORE_F32) reinterpret_cast<float*>(out)[(size_t)m * ldo + n] = v;
      else if (EPI == EPI_RELU_T) Operand<T>::store(reinterpret_cast<T*>(out) + (size_t)m * ldo, N, n, fmaxf(v, 0.f));   // ldo = N * PARTS
      else reinterpret_cast<float*>(out)[(size_t)m * ldo + n] += v;
    }
  }
}

}  // namespace sd
