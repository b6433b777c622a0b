// Warp-level block-vs-cache attention on the legacy tensor path (mma.sync m16n8k16, bf16 in, fp32
// accumulate), shared by the streaming chain kernel and the row-batched attention kernel: each warp
// holds the 16 query rows of an m-tile as A fragments and walks 16-key slices of K / V tiles that
// sit in shared memory as 128-byte rows with the 16-byte chunks XOR-swizzled by (row & 7) -- the
// layout a 128B-swizzle TMA box produces -- keeping the running maximum, normaliser and output in
// registers (online softmax).  Attention here is bound by the K/V stream and by latency, not by
// tensor throughput (9-32 query rows per sequence), which is why it does not use tcgen05.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>

#include <cstdint>

namespace vvs {
namespace attmma {

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int HD>
struct AttState {
  float m[2], l[2];
  float o[HD / 8][4];
};

// 16 keys (rows row0 .. row0 + 15 of a K tile / V tile pair in shared memory) against the 16 query
// rows of this warp's m-tile.  vis[i]: bit k set = key k of the slice is visible to row g + 8 i;
// vmem: bit k set = row k of the V tile holds data (others are zeroed before they are multiplied).
template <int HD>
__device__ __forceinline__ void att_slice(AttState<HD>& st, const uint32_t (&qa)[HD / 16][4], uint32_t k_base,
                                          uint32_t v_base, uint32_t tile_stride, int row0, int lane, float sl2,
                                          const uint32_t (&vis)[2], uint32_t vmem) {
  const int c = lane & 3, mi = lane >> 3, ri = lane & 7;
  float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
  {
    const int key = row0 + ((mi >> 1) << 3) + ri;
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk) {
      const int cc = 2 * kk + (mi & 1);
      uint32_t r0, r1, r2, r3;
      ldsm4(k_base + (cc >> 3) * tile_stride + key * 128 + (((cc & 7) ^ ri) << 4), r0, r1, r2, r3);
      mma16816(s0, qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], r0, r1);
      mma16816(s1, qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], r2, r3);
    }
  }
  // online softmax for rows g (i = 0) and g + 8 (i = 1); this lane holds keys 2c, 2c+1, 2c+8, 2c+9
  uint32_t pa[4];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const uint32_t vb = vis[i] >> (2 * c);
    float v[4];
    v[0] = (vb & 1u) ? s0[2 * i] * sl2 : -CUDART_INF_F;
    v[1] = (vb & 2u) ? s0[2 * i + 1] * sl2 : -CUDART_INF_F;
    v[2] = (vb & 0x100u) ? s1[2 * i] * sl2 : -CUDART_INF_F;
    v[3] = (vb & 0x200u) ? s1[2 * i + 1] * sl2 : -CUDART_INF_F;
    float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(st.m[i], mx);
    const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
    const float alpha = ex2(st.m[i] - m_safe);
    st.m[i] = m_new;
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = ex2(v[e] - m_safe);
    st.l[i] = st.l[i] * alpha + (v[0] + v[1]) + (v[2] + v[3]);
#pragma unroll
    for (int j = 0; j < HD / 8; ++j) {
      st.o[j][2 * i] *= alpha;
      st.o[j][2 * i + 1] *= alpha;
    }
    pa[i] = pack2(v[0], v[1]);
    pa[2 + i] = pack2(v[2], v[3]);
  }
  // O += P V
  const uint32_t vlo = ((vmem >> (2 * c)) & 1u ? 0x0000ffffu : 0u) | ((vmem >> (2 * c + 1)) & 1u ? 0xffff0000u : 0u);
  const uint32_t vhi = ((vmem >> (2 * c + 8)) & 1u ? 0x0000ffffu : 0u) | ((vmem >> (2 * c + 9)) & 1u ? 0xffff0000u : 0u);
  {
    const int key = row0 + ((mi & 1) << 3) + ri;
#pragma unroll
    for (int jj = 0; jj < HD / 16; ++jj) {
      const int cc = 2 * jj + (mi >> 1);
      uint32_t r0, r1, r2, r3;
      ldsm4t(v_base + (cc >> 3) * tile_stride + key * 128 + (((cc & 7) ^ ri) << 4), r0, r1, r2, r3);
      mma16816(st.o[2 * jj], pa[0], pa[1], pa[2], pa[3], r0 & vlo, r1 & vhi);
      mma16816(st.o[2 * jj + 1], pa[0], pa[1], pa[2], pa[3], r2 & vlo, r3 & vhi);
    }
  }
}

}  // namespace attmma
}  // namespace vvs
