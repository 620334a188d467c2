// Row-wise and element-wise operators of a decoder layer around the cache calls: what a decode step runs
// between its GEMMs.  The paper's models (Experimental Setup: Qwen2.5-1.5B-Instruct, Phi-4-mini-instruct) are
// pre-norm decoders with a residual stream, RMSNorm in front of the attention and the MLP block, a gated MLP
// with the SiLU activation, and the latency protocol decodes greedily (Algorithm 1 samples the next token).
//
//   k_add_rmsnorm  h' = h + delta (rounded to bf16, the residual stream's type), y = h' / sqrt(mean(h'^2) + eps) * w
//   k_swiglu       out = silu(gate) * up, gate and up the two halves of the packed projection's rows
//   k_argmax_rows  the lowest index of every row's maximum
//
// All three are bound by memory latency at decode sizes (a few hundred KB per call; the logits of a step are
// 19 MB); each replaces a chain of framework kernels (seven for the norm, three for the gate, and the residual
// add) by one launch.  Arithmetic in fp32, 16-byte accesses, one block per row for the two row-wise ones.
#include <cooperative_groups.h>

#include "bc_common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kRowThreads = 256;
constexpr int kMaxChunksPerThread = 4;   // hidden <= 256 * 4 * 8 = 8192

__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&p);
}

__device__ __forceinline__ float block_sum(float x) {
  __shared__ float warp_part[kRowThreads / 32];
  __shared__ float total;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = x;
  __syncthreads();
  if (threadIdx.x < 32) {
    float y = threadIdx.x < kRowThreads / 32 ? warp_part[threadIdx.x] : 0.f;
#pragma unroll
    for (int d = 4; d > 0; d >>= 1) y += __shfl_xor_sync(0xffffffffu, y, d);
    if (threadIdx.x == 0) total = y;
  }
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(kRowThreads) k_add_rmsnorm(const uint4* h, const uint4* delta,
                                                            const uint4* __restrict__ weight, int chunks, float inv_hidden, float eps,
                                                            uint4* h_out, uint4* __restrict__ normed) {
  const int64_t row = (int64_t)blockIdx.x * chunks;
  uint4 s[kMaxChunksPerThread];
  float sq = 0.f;
#pragma unroll
  for (int k = 0; k < kMaxChunksPerThread; ++k) {
    const int ch = threadIdx.x + k * kRowThreads;
    if (ch < chunks) {
      uint4 a = h[row + ch];
      if (delta != nullptr) {
        const uint4 b = delta[row + ch];
        a.x = pack_bf16(bf_lo(a.x) + bf_lo(b.x), bf_hi(a.x) + bf_hi(b.x));
        a.y = pack_bf16(bf_lo(a.y) + bf_lo(b.y), bf_hi(a.y) + bf_hi(b.y));
        a.z = pack_bf16(bf_lo(a.z) + bf_lo(b.z), bf_hi(a.z) + bf_hi(b.z));
        a.w = pack_bf16(bf_lo(a.w) + bf_lo(b.w), bf_hi(a.w) + bf_hi(b.w));
      }
      s[k] = a;
      if (h_out != nullptr) h_out[row + ch] = a;
      // the norm sees the residual stream as it is stored (bf16)
      sq += bf_lo(a.x) * bf_lo(a.x) + bf_hi(a.x) * bf_hi(a.x) + bf_lo(a.y) * bf_lo(a.y) + bf_hi(a.y) * bf_hi(a.y) +
            bf_lo(a.z) * bf_lo(a.z) + bf_hi(a.z) * bf_hi(a.z) + bf_lo(a.w) * bf_lo(a.w) + bf_hi(a.w) * bf_hi(a.w);
    }
  }
  const float r = rsqrtf(block_sum(sq) * inv_hidden + eps);
#pragma unroll
  for (int k = 0; k < kMaxChunksPerThread; ++k) {
    const int ch = threadIdx.x + k * kRowThreads;
    if (ch < chunks) {
      const uint4 a = s[k];
      float w[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
      if (weight != nullptr) {
        const uint4 ww = weight[ch];
        w[0] = bf_lo(ww.x); w[1] = bf_hi(ww.x); w[2] = bf_lo(ww.y); w[3] = bf_hi(ww.y);
        w[4] = bf_lo(ww.z); w[5] = bf_hi(ww.z); w[6] = bf_lo(ww.w); w[7] = bf_hi(ww.w);
      }
      uint4 y;
      y.x = pack_bf16(bf_lo(a.x) * r * w[0], bf_hi(a.x) * r * w[1]);
      y.y = pack_bf16(bf_lo(a.y) * r * w[2], bf_hi(a.y) * r * w[3]);
      y.z = pack_bf16(bf_lo(a.z) * r * w[4], bf_hi(a.z) * r * w[5]);
      y.w = pack_bf16(bf_lo(a.w) * r * w[6], bf_hi(a.w) * r * w[7]);
      normed[row + ch] = y;
    }
  }
}

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.f + __expf(-g)) * u; }

// gate_up rows are [gate (m) | up (m)]; one thread per 16-byte piece of the output
__global__ void __launch_bounds__(256) k_swiglu(const uint4* __restrict__ gate_up, int64_t pieces, int chunks_m, uint4* __restrict__ out) {
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < pieces; idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = idx / chunks_m;
    const int ch = (int)(idx - row * chunks_m);
    const uint4 g = gate_up[row * 2 * chunks_m + ch], u = gate_up[row * 2 * chunks_m + chunks_m + ch];
    uint4 y;
    y.x = pack_bf16(silu_mul(bf_lo(g.x), bf_lo(u.x)), silu_mul(bf_hi(g.x), bf_hi(u.x)));
    y.y = pack_bf16(silu_mul(bf_lo(g.y), bf_lo(u.y)), silu_mul(bf_hi(g.y), bf_hi(u.y)));
    y.z = pack_bf16(silu_mul(bf_lo(g.z), bf_lo(u.z)), silu_mul(bf_hi(g.z), bf_hi(u.z)));
    y.w = pack_bf16(silu_mul(bf_lo(g.w), bf_lo(u.w)), silu_mul(bf_hi(g.w), bf_hi(u.w)));
    out[idx] = y;
  }
}

constexpr int kArgThreads = 512;
constexpr int kArgCluster = 8;   // thread blocks per row: a cluster, reduced through distributed shared memory
__device__ __forceinline__ void take(float& best, int& at, float v, int i) {
  if (v > best || (v == best && i < at)) { best = v; at = i; }
}
// One CLUSTER of kArgCluster blocks per row (19 MB of logits per decode step of the 1.5B model: 64 rows are too few
// blocks to draw the memory bandwidth with one block each).  Every block scans its slice of the row with 16-byte
// loads, reduces it to (maximum, lowest index), and leaves the pair in its shared memory; after a cluster barrier
// the first block of the cluster folds the pairs of all blocks, read through distributed shared memory.
__global__ void __launch_bounds__(kArgThreads) k_argmax_rows(const __nv_bfloat16* __restrict__ z, int vocab, long long* __restrict__ out) {
  cg::cluster_group cluster = cg::this_cluster();
  const int part = (int)cluster.block_rank(), parts = (int)cluster.num_blocks();
  const int64_t r = blockIdx.x / parts;
  const __nv_bfloat16* row = z + r * vocab;
  float best = -INFINITY;
  int at = 0x7fffffff;
  const int chunks = vocab >> 3;   // the row starts on a 16-byte boundary when vocab is a multiple of 8 (checked by the host)
  const int per = (chunks + parts - 1) / parts, c0 = part * per, c1 = min(chunks, c0 + per);
  const uint4* r4 = reinterpret_cast<const uint4*>(row);
  for (int ch = c0 + threadIdx.x; ch < c1; ch += kArgThreads) {
    const uint4 a = __ldcs(r4 + ch);
    const int i = ch << 3;
    take(best, at, bf_lo(a.x), i); take(best, at, bf_hi(a.x), i + 1); take(best, at, bf_lo(a.y), i + 2); take(best, at, bf_hi(a.y), i + 3);
    take(best, at, bf_lo(a.z), i + 4); take(best, at, bf_hi(a.z), i + 5); take(best, at, bf_lo(a.w), i + 6); take(best, at, bf_hi(a.w), i + 7);
  }
  __shared__ float sh_v[kArgThreads / 32];
  __shared__ int sh_i[kArgThreads / 32];
  __shared__ float blk_v;
  __shared__ int blk_i;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const float v = __shfl_xor_sync(0xffffffffu, best, d);
    const int i = __shfl_xor_sync(0xffffffffu, at, d);
    take(best, at, v, i);
  }
  if ((threadIdx.x & 31) == 0) { sh_v[threadIdx.x >> 5] = best; sh_i[threadIdx.x >> 5] = at; }
  __syncthreads();
  if (threadIdx.x < 32) {
    best = threadIdx.x < kArgThreads / 32 ? sh_v[threadIdx.x] : -INFINITY;
    at = threadIdx.x < kArgThreads / 32 ? sh_i[threadIdx.x] : 0x7fffffff;
#pragma unroll
    for (int d = 8; d > 0; d >>= 1) {
      const float v = __shfl_xor_sync(0xffffffffu, best, d);
      const int i = __shfl_xor_sync(0xffffffffu, at, d);
      take(best, at, v, i);
    }
    if (threadIdx.x == 0) { blk_v = best; blk_i = at; }
  }
  cluster.sync();   // every block's pair is in its shared memory
  if (part == 0 && threadIdx.x == 0) {
    for (int b = 1; b < parts; ++b) take(best, at, *cluster.map_shared_rank(&blk_v, b), *cluster.map_shared_rank(&blk_i, b));
    out[r] = at == 0x7fffffff ? 0 : at;   // a row of -inf / NaN: index 0
  }
  cluster.sync();   // no block leaves while its shared memory may still be read
}

}  // namespace

cudaError_t bc_launch_add_rmsnorm(const void* h, const void* delta, const void* weight, int n, int hidden, float eps, void* h_out,
                                  void* normed, cudaStream_t s) {
  k_add_rmsnorm<<<n, kRowThreads, 0, s>>>((const uint4*)h, (const uint4*)delta, (const uint4*)weight, hidden >> 3, 1.f / (float)hidden, eps,
                                          (uint4*)h_out, (uint4*)normed);
  return cudaGetLastError();
}
cudaError_t bc_launch_swiglu(const void* gate_up, int n, int m, void* out, cudaStream_t s) {
  const int64_t pieces = (int64_t)n * (m >> 3);
  const int blocks = (int)((pieces + 255) / 256 < 148 * 8 ? (pieces + 255) / 256 : 148 * 8);
  k_swiglu<<<blocks, 256, 0, s>>>((const uint4*)gate_up, pieces, m >> 3, (uint4*)out);
  return cudaGetLastError();
}
cudaError_t bc_launch_argmax(const void* logits, int n, int vocab, long long* out, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n * kArgCluster); cfg.blockDim = dim3(kArgThreads); cfg.dynamicSmemBytes = 0; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kArgCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_argmax_rows, (const __nv_bfloat16*)logits, vocab, out);
}
int bc_rmsnorm_max_hidden() { return kRowThreads * kMaxChunksPerThread * 8; }
