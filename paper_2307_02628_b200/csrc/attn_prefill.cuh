// Causal attention over the prompt (the full-depth prompt pass that precedes generation,
// Section 2.3): every prompt position attends to positions 0..pos of its own sequence, all
// layers.  Unlike a decode step this is a dense contraction (P queries against P keys per
// sequence and head), so it runs on the tensor cores: 64 queries x 64 keys per tile, four warps
// of 16 query rows each, register-level bf16 MMAs with fp32 accumulation and a base-2 online
// softmax.  q arrives in fp32 and the softmax weights are fp32, so both are fed as a (hi, lo)
// pair of bf16 values, two MMAs each, which keeps the error at fp32-accumulation level; K and V
// are the bf16 cache rows that the QKV epilogue has just written.  K/V tiles are staged in
// shared memory with 16-byte asynchronous copies, two tiles in flight, 16-byte chunks XOR-swizzled
// by the key index so that the 8x8 matrix loads are free of bank conflicts.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace sd {

constexpr int PF_BM = 64, PF_BN = 64, PF_THREADS = 128;

__device__ __forceinline__ void pf_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void pf_ldmatrix(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void pf_ldmatrix_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// 16-byte asynchronous copy; bytes = 0 fills the destination with zeros and reads nothing
__device__ __forceinline__ void pf_cp16(uint32_t dst, const void* src, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" :: "r"(dst), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void pf_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void pf_wait() { asm volatile("cp.async.wait_group %0;\n" :: "n"(N)); }

// two floats -> packed bf16 pair of the values (hi) and of what the rounding left (lo)
__device__ __forceinline__ void pf_split(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
  const __nv_bfloat16 lx = __float2bfloat16_rn(x - __bfloat162float(hx));
  const __nv_bfloat16 ly = __float2bfloat16_rn(y - __bfloat162float(hy));
  hi = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
}

// grid (query tiles of a sequence, sequences of this pass x heads); block 128 threads.
// qkv: fp32 [n_seq * P, ldq], q of head h at columns h*HD..; row = seq * P + pos.
// Kc, Vc: bf16 [B, H, cap, HD] of this layer; sequences b0.. of the batch.
// o: operand rows [n_seq * P, H * HD] for the out-projection (fp16 values in 16-bit slots, see Operand).
// pad (may be null): left-padding slots per batch row; a row's keys start at slot pad[b], and a
// padding slot attends to itself alone (its output is never used).
template <int HD>
__global__ void __launch_bounds__(PF_THREADS)
attn_prefill_kernel(const float* __restrict__ qkv, int ldq, const __nv_bfloat16* __restrict__ Kc,
                    const __nv_bfloat16* __restrict__ Vc, int cap, int H, int P, int b0,
                    const int* __restrict__ pad, __nv_bfloat16* __restrict__ o) {
  constexpr int ROW_BYTES = HD * 2, CHUNKS = HD / 8;            // 16-byte chunks per key row
  constexpr int TILE_BYTES = PF_BN * ROW_BYTES;
  constexpr int KS = HD / 16;                                  // k-steps of Q K^T
  constexpr int NT_S = PF_BN / 8, NT_O = HD / 8;               // 8-wide accumulator tiles of S and of O
  extern __shared__ __align__(128) unsigned char pf_smem[];    // [stage][K | V][key][chunk]

  const int n_qt = (P + PF_BM - 1) / PF_BM;
  const int qt = n_qt - 1 - (int)blockIdx.x;                   // the longest rows first
  const int seq = blockIdx.y / H, h = blockIdx.y - seq * H;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int q0 = qt * PF_BM + warp * 16;                        // first query position of this warp
  const int n_kt = qt + 1;                                     // key tiles ..qt (the last one is masked)
  const int first = pad ? pad[b0 + seq] : 0;                   // first slot of this row's own sequence
  const int kt0 = min(first, qt * PF_BM) / PF_BN;              // tiles wholly inside the padding are skipped

  const size_t head_base = ((size_t)(b0 + seq) * H + h) * (size_t)cap * HD;
  const __nv_bfloat16* Kh = Kc + head_base;
  const __nv_bfloat16* Vh = Vc + head_base;
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(pf_smem);

  auto load_tile = [&](int kt, int stage) {
    const uint32_t kdst = smem0 + stage * 2 * TILE_BYTES, vdst = kdst + TILE_BYTES;
    for (int i = tid; i < PF_BN * CHUNKS; i += PF_THREADS) {
      const int key = i / CHUNKS, ch = i - key * CHUNKS;
      const int j = kt * PF_BN + key;
      const bool ok = j < P;                                    // rows past the prompt: zeros, never read from memory
      const size_t src = (size_t)(ok ? j : 0) * HD + ch * 8;
      const uint32_t off = key * ROW_BYTES + ((ch ^ (key & 7)) << 4);
      pf_cp16(kdst + off, Kh + src, ok ? 16 : 0);
      pf_cp16(vdst + off, Vh + src, ok ? 16 : 0);
    }
  };

  load_tile(kt0, kt0 & 1);
  pf_commit();

  // q of this warp's 16 rows as MMA A fragments, scaled by hd^-1/2 log2(e), split into hi and lo
  uint32_t qh[KS][4], ql[KS][4];
  {
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
    const int p_lo = min(q0 + g, P - 1), p_hi = min(q0 + g + 8, P - 1);   // rows past the prompt repeat the last one; never stored
    const float* r_lo = qkv + ((size_t)seq * P + p_lo) * ldq + h * HD;
    const float* r_hi = qkv + ((size_t)seq * P + p_hi) * ldq + h * HD;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int c = ks * 16 + 2 * t;
      const float2 a = *reinterpret_cast<const float2*>(r_lo + c), b = *reinterpret_cast<const float2*>(r_hi + c);
      const float2 a8 = *reinterpret_cast<const float2*>(r_lo + c + 8), b8 = *reinterpret_cast<const float2*>(r_hi + c + 8);
      pf_split(a.x * sc, a.y * sc, qh[ks][0], ql[ks][0]);
      pf_split(b.x * sc, b.y * sc, qh[ks][1], ql[ks][1]);
      pf_split(a8.x * sc, a8.y * sc, qh[ks][2], ql[ks][2]);
      pf_split(b8.x * sc, b8.y * sc, qh[ks][3], ql[ks][3]);
    }
  }

  float acc[NT_O][4];
#pragma unroll
  for (int n = 0; n < NT_O; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  const int mi = lane >> 3, mr = lane & 7;                     // matrix and row this lane addresses in an x4 load

  for (int kt = kt0; kt < n_kt; ++kt) {
    const int stage = kt & 1;
    if (kt + 1 < n_kt) { load_tile(kt + 1, stage ^ 1); pf_commit(); pf_wait<1>(); }
    else pf_wait<0>();
    __syncthreads();
    const uint32_t ks_base = smem0 + stage * 2 * TILE_BYTES, vs_base = ks_base + TILE_BYTES;

    // S = Q K^T for 16 queries x 64 keys
    float s[NT_S][4];
#pragma unroll
    for (int n = 0; n < NT_S; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
#pragma unroll
    for (int np = 0; np < NT_S / 2; ++np) {
      const int key = np * 16 + ((mi >> 1) << 3) + mr;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int ch = 2 * ks + (mi & 1);
        uint32_t b[4];
        pf_ldmatrix(b, ks_base + key * ROW_BYTES + ((ch ^ (key & 7)) << 4));
        pf_mma(s[2 * np], qh[ks], b[0], b[1]);
        pf_mma(s[2 * np], ql[ks], b[0], b[1]);
        pf_mma(s[2 * np + 1], qh[ks], b[2], b[3]);
        pf_mma(s[2 * np + 1], ql[ks], b[2], b[3]);
      }
    }
    // causal mask: only the last tile holds keys beyond a query's own position; padding mask: only
    // tiles that begin before the row's first slot hold keys it must not see
    if (kt == n_kt - 1 || kt * PF_BN < first) {
      const int p_lo = q0 + g, p_hi = p_lo + 8;
      const int f_lo = min(first, p_lo), f_hi = min(first, p_hi);
#pragma unroll
      for (int n = 0; n < NT_S; ++n) {
        const int j = kt * PF_BN + n * 8 + 2 * t;
        if (j > p_lo || j < f_lo) s[n][0] = -INFINITY;
        if (j + 1 > p_lo || j + 1 < f_lo) s[n][1] = -INFINITY;
        if (j > p_hi || j < f_hi) s[n][2] = -INFINITY;
        if (j + 1 > p_hi || j + 1 < f_hi) s[n][3] = -INFINITY;
      }
    }
    // online softmax (base 2); a row's values sit in the four lanes of a quad
    float mx_lo = m_lo, mx_hi = m_hi;
#pragma unroll
    for (int n = 0; n < NT_S; ++n) {
      mx_lo = fmaxf(mx_lo, fmaxf(s[n][0], s[n][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[n][2], s[n][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    // a row may have seen no key yet (tiles before its first slot): its maximum is still -inf, every
    // weight of the tile is 0, and the reference point of the exponentials is set to 0 to keep them finite
    const float sc_lo = m_lo == -INFINITY ? 0.f : exp2f(m_lo - mx_lo);
    const float sc_hi = m_hi == -INFINITY ? 0.f : exp2f(m_hi - mx_hi);
    m_lo = mx_lo; m_hi = mx_hi;
    if (mx_lo == -INFINITY) mx_lo = 0.f;
    if (mx_hi == -INFINITY) mx_hi = 0.f;
    l_lo *= sc_lo; l_hi *= sc_hi;
#pragma unroll
    for (int n = 0; n < NT_O; ++n) { acc[n][0] *= sc_lo; acc[n][1] *= sc_lo; acc[n][2] *= sc_hi; acc[n][3] *= sc_hi; }
    uint32_t ph[NT_S / 2][4], pl[NT_S / 2][4];                 // P as A fragments: k-step = 16 keys
#pragma unroll
    for (int n = 0; n < NT_S; ++n) {
      const float p0 = exp2f(s[n][0] - mx_lo), p1 = exp2f(s[n][1] - mx_lo);
      const float p2 = exp2f(s[n][2] - mx_hi), p3 = exp2f(s[n][3] - mx_hi);
      l_lo += p0 + p1; l_hi += p2 + p3;
      pf_split(p0, p1, ph[n >> 1][(n & 1) * 2], pl[n >> 1][(n & 1) * 2]);
      pf_split(p2, p3, ph[n >> 1][(n & 1) * 2 + 1], pl[n >> 1][(n & 1) * 2 + 1]);
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < NT_S / 2; ++kk) {
      const int key = kk * 16 + ((mi & 1) << 3) + mr;
#pragma unroll
      for (int np = 0; np < NT_O / 2; ++np) {
        const int ch = 2 * np + (mi >> 1);
        uint32_t b[4];
        pf_ldmatrix_t(b, vs_base + key * ROW_BYTES + ((ch ^ (key & 7)) << 4));
        pf_mma(acc[2 * np], ph[kk], b[0], b[1]);
        pf_mma(acc[2 * np], pl[kk], b[0], b[1]);
        pf_mma(acc[2 * np + 1], ph[kk], b[2], b[3]);
        pf_mma(acc[2 * np + 1], pl[kk], b[2], b[3]);
      }
    }
    __syncthreads();                                           // the other stage is refilled at the top of the next round
  }

  // row sums across the quad, normalise, write the operand rows (fp16 values)
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
  const int d = H * HD;
  const int p_lo = q0 + g, p_hi = p_lo + 8;
#pragma unroll
  for (int n = 0; n < NT_O; ++n) {
    const int c = h * HD + n * 8 + 2 * t;
    if (p_lo < P) {
      const __half2 v = __floats2half2_rn(fminf(fmaxf(acc[n][0] * inv_lo, -65504.f), 65504.f), fminf(fmaxf(acc[n][1] * inv_lo, -65504.f), 65504.f));
      *reinterpret_cast<__half2*>(o + ((size_t)seq * P + p_lo) * d + c) = v;
    }
    if (p_hi < P) {
      const __half2 v = __floats2half2_rn(fminf(fmaxf(acc[n][2] * inv_hi, -65504.f), 65504.f), fminf(fmaxf(acc[n][3] * inv_hi, -65504.f), 65504.f));
      *reinterpret_cast<__half2*>(o + ((size_t)seq * P + p_hi) * d + c) = v;
    }
  }
}

}  // namespace sd
