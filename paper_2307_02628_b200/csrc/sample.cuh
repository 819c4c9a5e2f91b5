// Token selection on the device: temperature softmax, top-p nucleus, inverse-CDF draw
// (the generation settings of Section 3.2: beam 1, top-p 0.7, temperature 0.3).
//
// One block per batch row, no sort.  The row is copied to shared memory once.  Every logit gets a
// fixed-point mass floor(2^40 * 2^((x - max) / T * log2 e)) (64-bit integers: sums and comparisons are
// exact and do not depend on the order in which threads add).  The rank, in order of decreasing
// probability, at which the running mass passes a target is found in two stages:
//   1. a histogram of mass over 1024 equal-width slices of the logit range that can hold mass at all
//      ([max - 41 T ln 2, max]; anything lower has mass 0).  The slice index is a monotone function
//      of the logit, so the slices cut the sorted order into consecutive pieces, and a scan over the
//      slices gives the total Z and the slice in which the target is passed;
//   2. inside that slice, a radix descent over the logits' order-preserving bit patterns (four 8-bit
//      digits, most significant first), which only the slice's few elements take part in.
// The histogram is built once and serves both targets: top_p * Z (the nucleus boundary) and u * M (the
// draw, M = nucleus mass).  Equal logits are taken in order of increasing token id.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace sd {

constexpr int SAMPLE_THREADS = 1024;
constexpr int SAMPLE_SLICES = 1024;
constexpr float SAMPLE_FIX = 1099511627776.0f;   // 2^40
constexpr int SAMPLE_MAX_SMEM_VOCAB = 52224;     // a row of this many floats fits beside the histograms

// Bit pattern that orders like the value: larger float <=> larger key.  NaN counts as -inf.
__device__ __forceinline__ uint32_t sample_key(float x) {
  if (!(x == x)) return 0u;
  const uint32_t b = __float_as_uint(x + 0.0f);   // -0 becomes +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float sample_unkey(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// Fixed-point mass of a logit: floor(2^40 * 2^((x - m) * s)), s = log2(e) / temperature.
__device__ __forceinline__ unsigned long long sample_mass(float x, float m, float s) {
  if (!(x == x)) return 0ull;
  return __float2ull_rd(exp2f((x - m) * s) * SAMPLE_FIX);
}
// Slice of a logit: 0 holds the maximum, higher slices lower logits; monotone in x.
__device__ __forceinline__ int sample_slice(float x, float m, float slice_scale) {
  const float d = (m - x) * slice_scale;
  return d >= (float)(SAMPLE_SLICES - 1) ? SAMPLE_SLICES - 1 : (int)d;
}

struct SampleShared {
  unsigned long long slices[SAMPLE_SLICES];
  unsigned long long hist[256];
  unsigned long long red[32];
  float redf[32];
  int redi[32];
  uint32_t prefix;
  int slice;
  unsigned long long above, tie, total;
};

// Warp 0: the slice in which the running mass (slice 0 first) first EXCEEDS target, and the mass of
// the slices before it.  Results in sh.slice / sh.above; the caller synchronises.
__device__ __forceinline__ void sample_find_slice(SampleShared& sh, unsigned long long target, int lane) {
  constexpr int PER = SAMPLE_SLICES / 32;
  unsigned long long mine = 0ull;
#pragma unroll 1
  for (int j = 0; j < PER; ++j) mine += sh.slices[lane * PER + j];
  unsigned long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  const unsigned ballot = __ballot_sync(0xffffffffu, incl > target);
  const int owner = ballot ? __ffs(ballot) - 1 : 31;          // target < total mass makes ballot non-zero
  if (lane == owner) {
    unsigned long long run = incl - mine;
    int b = lane * PER + PER - 1;
#pragma unroll 1
    for (int j = 0; j < PER; ++j) {
      const unsigned long long t = sh.slices[lane * PER + j];
      if (run + t > target) { b = lane * PER + j; break; }
      if (j < PER - 1) run += t;
    }
    sh.slice = b;
    sh.above = run;
  }
  if (lane == 31) sh.total = incl;
}

// Inside slice sh.slice (mass sh.above before it): the key at which the running mass, keys in
// decreasing order, first EXCEEDS target.  On return, for every thread: key; above = mass of
// everything that precedes the elements equal to key; tie = mass of the elements equal to key.
__device__ void sample_select(const float* __restrict__ src, int vocab, float m, float s, float slice_scale,
                              unsigned long long target, SampleShared& sh,
                              uint32_t& key, unsigned long long& above, unsigned long long& tie) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int slice = sh.slice;
  if (tid == 0) { sh.prefix = 0u; sh.tie = 0ull; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) sh.hist[tid] = 0ull;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    for (int c = tid; c < vocab; c += SAMPLE_THREADS) {
      const float x = src[c];
      if (sample_slice(x, m, slice_scale) != slice) continue;     // cheap test first: few elements pass it
      const unsigned long long w = sample_mass(x, m, s);
      if (w == 0ull) continue;
      const uint32_t k = sample_key(x);
      if (pass == 0 || (k >> (shift + 8)) == prefix) atomicAdd(&sh.hist[(k >> shift) & 255u], w);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 255-8l ... 248-8l: a descending scan over lanes, then over the lane's digits
      const int top = 255 - 8 * lane;
      unsigned long long mine = 0ull;
#pragma unroll 1
      for (int j = 0; j < 8; ++j) mine += sh.hist[top - j];
      unsigned long long incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const unsigned long long base = sh.above;
      const unsigned ballot = __ballot_sync(0xffffffffu, base + incl > target);
      const int owner = ballot ? __ffs(ballot) - 1 : 31;
      if (lane == owner) {
        unsigned long long run = base + incl - mine;
        int d = top - 7;
        unsigned long long t_d = sh.hist[d];
#pragma unroll 1
        for (int j = 0; j < 8; ++j) {
          const unsigned long long t = sh.hist[top - j];
          if (run + t > target) { d = top - j; t_d = t; break; }
          if (j < 7) run += t;
        }
        sh.prefix = (prefix << 8) | (uint32_t)d;
        sh.above = run;
        sh.tie = t_d;
      }
    }
    __syncthreads();
  }
  key = sh.prefix;
  above = sh.above;
  tie = sh.tie;
  __syncthreads();
}

// next[b] ~ nucleus(top_p) of softmax(logits[b, :] / temperature), drawn with uniforms[b] in [0, 1).
// ROW_IN_SMEM: the row is staged in dynamic shared memory (vocab floats); otherwise every pass reads it
// from global memory (L2), for vocabularies that do not fit.
template <bool ROW_IN_SMEM>
__global__ void __launch_bounds__(SAMPLE_THREADS)
sample_top_p_kernel(const float* __restrict__ logits, int vocab, const float* __restrict__ uniforms,
                    float inv_temperature, float top_p, int32_t* __restrict__ next) {
  extern __shared__ float sample_row[];
  __shared__ SampleShared sh;
  const float* row = logits + (size_t)blockIdx.x * vocab;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // stage the row, find its maximum, clear the slice histogram
  float m = -INFINITY;
  for (int c = tid; c < vocab; c += SAMPLE_THREADS) {
    const float x = row[c];
    if (ROW_IN_SMEM) sample_row[c] = x;
    if (x > m) m = x;
  }
  for (int i = tid; i < SAMPLE_SLICES; i += SAMPLE_THREADS) sh.slices[i] = 0ull;
  const float* src = ROW_IN_SMEM ? sample_row : row;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) sh.redf[warp] = m;
  __syncthreads();
  m = sh.redf[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (!(m > -INFINITY) || m == INFINITY) {   // no finite maximum: nothing to weigh, answer the first maximum
    if (tid == 0) {
      int best = 0;
      for (int c = 0; c < vocab; ++c) if (row[c] == m) { best = c; break; }
      next[blockIdx.x] = best;
    }
    return;
  }
  const float s = 1.44269504088896340736f * inv_temperature;
  const float slice_scale = (float)SAMPLE_SLICES * s / 41.0f;       // mass is 0 below max - 41 / s

  // mass per slice (the maximum contributes exactly 2^40, so the total is positive)
  for (int c = tid; c < vocab; c += SAMPLE_THREADS) {
    const float x = src[c];
    const unsigned long long w = sample_mass(x, m, s);
    if (w) atomicAdd(&sh.slices[sample_slice(x, m, slice_scale)], w);
  }
  __syncthreads();

  // nucleus: the smallest leading set with mass >= top_p * Z, i.e. whose mass exceeds target1 - 1
  if (warp == 0) sample_find_slice(sh, ~0ull, lane);                 // only the total is wanted here
  __syncthreads();
  const unsigned long long z = sh.total;
  unsigned long long target1 = __double2ull_ru((double)top_p * (double)z);
  target1 = target1 < 1ull ? 1ull : (target1 > z ? z : target1);
  __syncthreads();
  if (warp == 0) sample_find_slice(sh, target1 - 1ull, lane);
  __syncthreads();
  uint32_t key1, key2;
  unsigned long long above1, tie1, above2, tie2;
  sample_select(src, vocab, m, s, slice_scale, target1 - 1ull, sh, key1, above1, tie1);
  const unsigned long long w1 = sample_mass(sample_unkey(key1), m, s);
  unsigned long long c1 = w1 ? (target1 - above1 + w1 - 1ull) / w1 : 1ull;   // equal logits taken from the boundary value
  const unsigned long long n1 = w1 ? tie1 / w1 : 1ull;
  c1 = c1 < 1ull ? 1ull : (c1 > n1 ? n1 : c1);
  const unsigned long long mass = above1 + c1 * w1;

  // draw: first element whose running mass exceeds u * M
  float u = uniforms[blockIdx.x];
  u = (u >= 0.0f) ? u : 0.0f;
  unsigned long long target2 = __double2ull_rd((double)u * (double)mass);
  if (target2 >= mass) target2 = mass - 1ull;
  if (warp == 0) sample_find_slice(sh, target2, lane);
  __syncthreads();
  sample_select(src, vocab, m, s, slice_scale, target2, sh, key2, above2, tie2);
  const unsigned long long w2 = sample_mass(sample_unkey(key2), m, s);
  unsigned long long j = w2 ? (target2 - above2) / w2 : 0ull;     // which of the equal logits, by token id
  const unsigned long long n2 = w2 ? tie2 / w2 : 1ull;
  if (j >= n2) j = n2 - 1ull;
  if (key2 < key1 || (key2 == key1 && j >= c1)) { key2 = key1; j = c1 - 1ull; }   // never outside the nucleus

  // the j-th element equal to key2 in token order.  Thread t holds tokens t, t + 1024, ...: token order is
  // round by round, and inside a round by thread.
  const int want = (int)j;
  if (tid == 0) next[blockIdx.x] = 0;   // overwritten below; only a row without any match keeps it
  int before = 0;
  for (int c0 = 0; c0 < vocab; c0 += SAMPLE_THREADS) {
    const int c = c0 + tid;
    const bool match = c < vocab && sample_key(src[c]) == key2 && sample_mass(src[c], m, s) != 0ull;
    const int cnt = __syncthreads_count(match);
    if (want < before + cnt) {                                  // uniform over the block: the answer is in this round
      const unsigned ballot = __ballot_sync(0xffffffffu, match);
      if (lane == 0) sh.redi[warp] = __popc(ballot);
      __syncthreads();
      int rank = before + __popc(ballot & ((1u << lane) - 1u));
      for (int wI = 0; wI < warp; ++wI) rank += sh.redi[wI];
      if (match && rank == want) next[blockIdx.x] = c;
      break;
    }
    before += cnt;
  }
}

}  // namespace sd
