// Rotary position embedding and split of a packed QKV projection, the step between a decoder
// layer's QKV GEMM and the cache (Section 2: attention itself is unchanged by the method, so the
// position encoding is the model's own; the paper's models use rotary embeddings with the half-split
// pairing: coordinate j of a head is paired with coordinate j + D/2 and the pair is turned by the
// angle pos * theta^(-2j/D)).
//
// One thread block per batch row.  The row's D/2 angles are the same for all of its heads: the first
// D/2 threads compute them once, in double precision (pos * theta^(-2j/D) reaches 10^4..10^5 radians
// at the positions of long reasoning traces; single precision would lose the angle's low bits before
// the range reduction), and leave cos and sin rounded to fp32 in shared memory.  Then every thread
// takes 16-byte pieces: for a q or k head one piece of the lower half and the piece D/2 further on,
// rotates the eight pairs in fp32 and stores both rounded to bf16; for a v head a plain copy.
// The three outputs are contiguous [n, heads, D] arrays, the layout the cache calls take.
// The work is a few KB per row: the launch is bound by latency, not by bandwidth.
#include "bc_common.cuh"

namespace {

constexpr int kRopeThreads = 256;

__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&p);
}

// lo, hi: eight coordinates j0..j0+7 and j0+D/2..j0+D/2+7; cs: cos and sin of angles j0..j0+7
__device__ __forceinline__ void rotate8(uint4& lo, uint4& hi, const float* c, const float* s) {
  uint32_t* a = reinterpret_cast<uint32_t*>(&lo);
  uint32_t* b = reinterpret_cast<uint32_t*>(&hi);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float x0 = bf_lo(a[i]), x1 = bf_hi(a[i]), y0 = bf_lo(b[i]), y1 = bf_hi(b[i]);
    const float c0 = c[2 * i], c1 = c[2 * i + 1], s0 = s[2 * i], s1 = s[2 * i + 1];
    a[i] = pack_bf16(fmaf(x0, c0, -y0 * s0), fmaf(x1, c1, -y1 * s1));
    b[i] = pack_bf16(fmaf(y0, c0, x0 * s0), fmaf(y1, c1, x1 * s1));
  }
}

__global__ void __launch_bounds__(kRopeThreads) k_rope_split(const uint4* __restrict__ qkv, const int32_t* __restrict__ positions,
                                                            int q_heads, int kv_heads, int head_dim, double log2_theta,
                                                            uint4* __restrict__ q_out, uint4* __restrict__ k_out,
                                                            uint4* __restrict__ v_out) {
  __shared__ float s_cos[128], s_sin[128];     // head_dim <= 256
  const int row = blockIdx.x, half = head_dim >> 1;
  if ((int)threadIdx.x < half) {
    const int j = threadIdx.x;
    const double inv_freq = exp2(-2.0 * (double)j / (double)head_dim * log2_theta);
    double sn, cs;
    sincos((double)positions[row] * inv_freq, &sn, &cs);
    s_cos[j] = (float)cs;
    s_sin[j] = (float)sn;
  }
  __syncthreads();
  const int hv = head_dim >> 3;                 // 16-byte pieces per head
  const int hp = hv >> 1;                       // pieces per half head
  const int rot_heads = q_heads + kv_heads;
  const int rot_units = rot_heads * hp, units = rot_units + kv_heads * hv;
  const uint4* in = qkv + (size_t)row * (q_heads + 2 * kv_heads) * hv;
  for (int u = threadIdx.x; u < units; u += kRopeThreads) {
    if (u < rot_units) {
      const int h = u / hp, piece = u - h * hp;
      uint4 lo = in[h * hv + piece], hi = in[h * hv + hp + piece];
      rotate8(lo, hi, s_cos + piece * 8, s_sin + piece * 8);
      uint4* dst = h < q_heads ? q_out + ((size_t)row * q_heads + h) * hv : k_out + ((size_t)row * kv_heads + (h - q_heads)) * hv;
      dst[piece] = lo;
      dst[hp + piece] = hi;
    } else {
      const int w = u - rot_units;
      v_out[(size_t)row * kv_heads * hv + w] = in[rot_heads * hv + w];
    }
  }
}

}  // namespace

cudaError_t bc_launch_rope_split(const void* qkv, const int32_t* positions, int n, int q_heads, int kv_heads, int head_dim,
                                 double theta, void* q_out, void* k_out, void* v_out, cudaStream_t s) {
  k_rope_split<<<n, kRopeThreads, 0, s>>>((const uint4*)qkv, positions, q_heads, kv_heads, head_dim, log2(theta), (uint4*)q_out,
                                          (uint4*)k_out, (uint4*)v_out);
  return cudaGetLastError();
}
