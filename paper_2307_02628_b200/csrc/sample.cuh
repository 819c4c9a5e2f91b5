// Token selection on the device: temperature softmax, top-p nucleus, inverse-CDF draw
// (the generation settings of Section 3.2: beam 1, top-p 0.7, temperature 0.3).
//
// One block per batch row.  No sort: the position in the order of decreasing probability at
// which the running probability mass passes a target is found by a radix descent over the
// logits' bit patterns (four 8-bit digits, most significant first), each pass summing the mass
// of the candidates per digit value.  Masses are 2^-40 fixed-point integers, so every sum and
// comparison is exact and independent of the order in which threads add; the same descent runs
// twice, first for the nucleus boundary (target top_p * Z), then for the draw (target u * M with
// M the nucleus mass).  Equal logits are taken in order of increasing token id.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace sd {

constexpr int SAMPLE_THREADS = 1024;
constexpr int SAMPLE_HISTS = 16;        // one histogram per pair of warps
constexpr float SAMPLE_FIX = 1099511627776.0f;   // 2^40

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

struct SampleShared {
  unsigned long long hist[SAMPLE_HISTS][256];
  unsigned long long tot[256];
  unsigned long long red[32];
  float redf[32];
  int redi[32];
  uint32_t prefix;
  unsigned long long above, tie;
};

// Finds the key at which the mass accumulated over keys in decreasing order first EXCEEDS
// `target` (target < total mass).  On return, for every thread: key; above = mass of the keys
// strictly greater; tie = mass of the elements equal to key (count * mass of one).
__device__ void sample_select(const float* __restrict__ row, int vocab, float m, float s,
                              unsigned long long target, SampleShared& sh,
                              uint32_t& key, unsigned long long& above, unsigned long long& tie) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { sh.prefix = 0u; sh.above = 0ull; sh.tie = 0ull; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < SAMPLE_HISTS * 256; i += SAMPLE_THREADS) (&sh.hist[0][0])[i] = 0ull;
    __syncthreads();
    const uint32_t prefix = sh.prefix;
    unsigned long long* hist = sh.hist[warp >> 1];
    for (int c = tid; c < vocab; c += SAMPLE_THREADS) {
      const float x = row[c];
      const uint32_t k = sample_key(x);
      if (pass == 0 || (k >> (shift + 8)) == prefix) {
        const unsigned long long w = sample_mass(x, m, s);
        if (w) atomicAdd(&hist[(k >> shift) & 255u], w);
      }
    }
    __syncthreads();
    if (tid < 256) {
      unsigned long long t = 0ull;
#pragma unroll
      for (int hI = 0; hI < SAMPLE_HISTS; ++hI) t += sh.hist[hI][tid];
      sh.tot[tid] = t;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 255-8l ... 248-8l: a descending scan over lanes, then over the lane's digits
      const int top = 255 - 8 * lane;
      unsigned long long mine = 0ull;
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += sh.tot[top - j];
      unsigned long long incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const unsigned long long base = sh.above;
      const unsigned ballot = __ballot_sync(0xffffffffu, base + incl > target);
      // ballot is non-zero whenever target < total mass; otherwise fall to the lowest digit that has mass
      const int owner = ballot ? __ffs(ballot) - 1 : 31;
      if (lane == owner) {
        unsigned long long run = base + incl - mine;
        int d = top - 7;
        unsigned long long t_d = sh.tot[d];
        for (int j = 0; j < 8; ++j) {
          const unsigned long long t = sh.tot[top - j];
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
__global__ void __launch_bounds__(SAMPLE_THREADS)
sample_top_p_kernel(const float* __restrict__ logits, int vocab, const float* __restrict__ uniforms,
                    float inv_temperature, float top_p, int32_t* __restrict__ next) {
  __shared__ SampleShared sh;
  const float* row = logits + (size_t)blockIdx.x * vocab;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // row maximum
  float m = -INFINITY;
  for (int c = tid; c < vocab; c += SAMPLE_THREADS) { const float x = row[c]; if (x > m) m = x; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) sh.redf[warp] = m;
  __syncthreads();
  m = sh.redf[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __syncthreads();
  if (!(m > -INFINITY) || m == INFINITY) {   // no finite maximum: nothing to weigh, answer the first maximum
    if (tid == 0) {
      int best = 0;
      for (int c = 0; c < vocab; ++c) if (row[c] == m) { best = c; break; }
      next[blockIdx.x] = best;
    }
    return;
  }
  const float s = 1.44269504088896340736f * inv_temperature;

  // total mass Z (the maximum contributes exactly 2^40, so Z > 0)
  unsigned long long z = 0ull;
  for (int c = tid; c < vocab; c += SAMPLE_THREADS) z += sample_mass(row[c], m, s);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if (lane == 0) sh.red[warp] = z;
  __syncthreads();
  z = sh.red[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  __syncthreads();

  // nucleus: the smallest leading set with mass >= top_p * Z, i.e. whose mass exceeds target1 - 1
  unsigned long long target1 = __double2ull_ru((double)top_p * (double)z);
  target1 = target1 < 1ull ? 1ull : (target1 > z ? z : target1);
  uint32_t key1, key2;
  unsigned long long above1, tie1, above2, tie2;
  sample_select(row, vocab, m, s, target1 - 1ull, sh, key1, above1, tie1);
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
  sample_select(row, vocab, m, s, target2, sh, key2, above2, tie2);
  const unsigned long long w2 = sample_mass(sample_unkey(key2), m, s);
  unsigned long long j = w2 ? (target2 - above2) / w2 : 0ull;     // which of the equal logits, by token id
  const unsigned long long n2 = w2 ? tie2 / w2 : 1ull;
  if (j >= n2) j = n2 - 1ull;
  if (key2 < key1 || (key2 == key1 && j >= c1)) { key2 = key1; j = c1 - 1ull; }   // never outside the nucleus

  // the j-th element equal to key2 in token order: contiguous ranges per thread, then a block scan
  const int per = (vocab + SAMPLE_THREADS - 1) / SAMPLE_THREADS;
  const int c0 = tid * per, c_end = min(vocab, c0 + per);
  int cnt = 0;
  for (int c = c0; c < c_end; ++c) cnt += sample_key(row[c]) == key2;
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) sh.redi[warp] = incl;
  __syncthreads();
  int wbase = 0;
  for (int wI = 0; wI < warp; ++wI) wbase += sh.redi[wI];
  const int excl = wbase + incl - cnt;
  const int want = (int)j;
  if (tid == 0) next[blockIdx.x] = 0;   // overwritten below; only a row without any match keeps it
  __syncthreads();
  if (cnt > 0 && want >= excl && want < excl + cnt) {
    int seen = excl;
    for (int c = c0; c < c_end; ++c)
      if (sample_key(row[c]) == key2) {
        if (seen == want) { next[blockIdx.x] = c; break; }
        ++seen;
      }
  }
}

}  // namespace sd
