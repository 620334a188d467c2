// Distillation loss of Section 3.2 (Eq. 1): mean over trajectories of the mean over positions of
// KL(teacher || student), with the teacher stored as its top-K log-probabilities per position
// (Implementation Details: the top 100 per time step) and the student given by its logits over the
// whole vocabulary.  Optionally the gradient with respect to the student logits.
//
// The work is one streaming read of the student logits (rows x vocab bf16, hundreds of KB per
// row): HBM-bound.  One thread block per position keeps an online log-sum-exp per thread over
// 16-byte loads, reduces it across the block, gathers the K stored entries and writes the row's
// loss.  With a gradient buffer the block reads its row a second time (it is still in L2) and
// writes w * (q * sum_k p_k - p [stored]) in bf16.  The batch mean is a second, single-block kernel
// that adds in a fixed order (deterministic).
#include "bc_common.cuh"

namespace {

constexpr int kRowThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// Online log-sum-exp state in the log2 domain: sum_j 2^(x_j * log2e - m).
struct Lse {
  float m, s;
  __device__ __forceinline__ void add8(const uint4& v) {
    float x[8] = {bf_lo(v.x), bf_hi(v.x), bf_lo(v.y), bf_hi(v.y), bf_lo(v.z), bf_hi(v.z), bf_lo(v.w), bf_hi(v.w)};
    float vm = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
    const float mn = fmaxf(m, vm * kLog2e);
    const float ms = mn == -INFINITY ? 0.f : mn;   // a row of -inf logits must not produce inf - inf
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += ex2(fmaf(x[i], kLog2e, -ms));
    s = s * ex2(m - ms) + acc;
    m = mn;
  }
  __device__ __forceinline__ void add1(float x) {
    const float mn = fmaxf(m, x * kLog2e);
    const float ms = mn == -INFINITY ? 0.f : mn;
    s = s * ex2(m - ms) + ex2(fmaf(x, kLog2e, -ms));
    m = mn;
  }
  __device__ __forceinline__ void merge(float m2, float s2) {
    const float mn = fmaxf(m, m2);
    const float ms = mn == -INFINITY ? 0.f : mn;
    s = s * ex2(m - ms) + s2 * ex2(m2 - ms);
    m = mn;
  }
};

__global__ void __launch_bounds__(kRowThreads) k_kl_rows(const __nv_bfloat16* __restrict__ logits, const int32_t* __restrict__ tidx,
                                                        const float* __restrict__ tlogp, const int32_t* __restrict__ cu_rows,
                                                        int n_traj, int vocab, int top_k, float* __restrict__ row_loss,
                                                        __nv_bfloat16* __restrict__ grad) {
  const int64_t r = blockIdx.x;
  const __nv_bfloat16* z = logits + r * vocab;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ float sh_m[kRowThreads / 32], sh_s[kRowThreads / 32], sh_acc[kRowThreads / 32], sh_p[kRowThreads / 32];
  __shared__ float sh_lse, sh_psum;

  // ---- log-sum-exp of the row: scalar head up to a 16-byte boundary, 16-byte body, scalar tail -------
  const int head = min(vocab, (int)(((16 - (reinterpret_cast<uintptr_t>(z) & 15)) & 15) >> 1));
  const int nvec = (vocab - head) >> 3;
  const int tail0 = head + (nvec << 3);
  Lse st = {-INFINITY, 0.f};
  if (tid < head) st.add1(__bfloat162float(z[tid]));
  const uint4* zv = reinterpret_cast<const uint4*>(z + head);
  // read once -> streaming loads; with a gradient the row is read again, so it should stay in L2
  const bool reread = grad != nullptr;
  auto ld = [&](const uint4* p) { return reread ? *p : __ldcs(p); };
  int i = tid;
  for (; i + 3 * kRowThreads < nvec; i += 4 * kRowThreads) {   // four loads in flight per thread
    const uint4 a = ld(zv + i), b = ld(zv + i + kRowThreads), c = ld(zv + i + 2 * kRowThreads), d = ld(zv + i + 3 * kRowThreads);
    st.add8(a); st.add8(b); st.add8(c); st.add8(d);
  }
  for (; i < nvec; i += kRowThreads) st.add8(ld(zv + i));
  if (tail0 + tid < vocab) st.add1(__bfloat162float(z[tail0 + tid]));
  // block reduction, fixed order
#pragma unroll
  for (int d = 16; d; d >>= 1) st.merge(__shfl_xor_sync(0xffffffffu, st.m, d), __shfl_xor_sync(0xffffffffu, st.s, d));
  if (lane == 0) { sh_m[warp] = st.m; sh_s[warp] = st.s; }
  __syncthreads();
  if (warp == 0) {
    Lse t = {lane < kRowThreads / 32 ? sh_m[lane] : -INFINITY, lane < kRowThreads / 32 ? sh_s[lane] : 0.f};
#pragma unroll
    for (int d = 16; d; d >>= 1) t.merge(__shfl_xor_sync(0xffffffffu, t.m, d), __shfl_xor_sync(0xffffffffu, t.s, d));
    if (lane == 0) sh_lse = (t.m + log2f(t.s)) * kLn2;   // natural-log normaliser of the student
  }
  __syncthreads();
  const float lse = sh_lse;

  // ---- the K stored teacher entries --------------------------------------------------------------------
  float acc = 0.f, psum = 0.f;
  for (int k = tid; k < top_k; k += kRowThreads) {
    const float lp = tlogp[r * top_k + k];
    const int j = tidx[r * top_k + k];
    if (lp > -INFINITY && j >= 0 && j < vocab) {   // entries without mass or with an index outside the vocabulary are ignored
      const float p = __expf(lp);
      const float lq = __bfloat162float(z[j]) - lse;
      acc += p * (lp - lq);
      psum += p;
    }
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) { acc += __shfl_xor_sync(0xffffffffu, acc, d); psum += __shfl_xor_sync(0xffffffffu, psum, d); }
  if (lane == 0) { sh_acc[warp] = acc; sh_p[warp] = psum; }
  __syncthreads();
  if (tid == 0) {
    float a = 0.f, p = 0.f;
    for (int w = 0; w < kRowThreads / 32; ++w) { a += sh_acc[w]; p += sh_p[w]; }
    row_loss[r] = a;
    sh_psum = p;
  }
  if (grad == nullptr) return;
  __syncthreads();

  // ---- gradient row: w * (q * sum_k p_k - p [stored]) ------------------------------------------------
  int lo = 0, hi = n_traj;   // trajectory of this row: largest b with cu_rows[b] <= r
  while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cu_rows[mid] <= r) lo = mid; else hi = mid; }
  const float w = 1.f / ((float)n_traj * (float)(cu_rows[lo + 1] - cu_rows[lo]));
  const float coef = w * sh_psum, lse2 = lse * kLog2e;
  __nv_bfloat16* g = grad + r * vocab;   // same alignment as z: rows have the same stride
  if (tid < head) g[tid] = __float2bfloat16_rn(coef * ex2(fmaf(__bfloat162float(z[tid]), kLog2e, -lse2)));
  uint4* gv = reinterpret_cast<uint4*>(g + head);
  auto grad8 = [&](const uint4& v) {
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const __nv_bfloat162 t = __floats2bfloat162_rn(coef * ex2(fmaf(bf_lo(in[q]), kLog2e, -lse2)),
                                                     coef * ex2(fmaf(bf_hi(in[q]), kLog2e, -lse2)));
      o[q] = *reinterpret_cast<const uint32_t*>(&t);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
  };
  int j = tid;
  for (; j + 3 * kRowThreads < nvec; j += 4 * kRowThreads) {   // four loads in flight per thread
    const uint4 a = zv[j], b = zv[j + kRowThreads], c = zv[j + 2 * kRowThreads], d = zv[j + 3 * kRowThreads];
    __stcs(gv + j, grad8(a)); __stcs(gv + j + kRowThreads, grad8(b));
    __stcs(gv + j + 2 * kRowThreads, grad8(c)); __stcs(gv + j + 3 * kRowThreads, grad8(d));
  }
  for (; j < nvec; j += kRowThreads) __stcs(gv + j, grad8(zv[j]));
  if (tail0 + tid < vocab) g[tail0 + tid] = __float2bfloat16_rn(coef * ex2(fmaf(__bfloat162float(z[tail0 + tid]), kLog2e, -lse2)));
  __syncthreads();   // the dense row is written; the stored entries overwrite their elements
  for (int k = tid; k < top_k; k += kRowThreads) {
    const float lp = tlogp[r * top_k + k];
    const int j = tidx[r * top_k + k];
    if (lp > -INFINITY && j >= 0 && j < vocab) {
      g[j] = __float2bfloat16_rn(coef * ex2(fmaf(__bfloat162float(z[j]), kLog2e, -lse2)) - w * __expf(lp));
    }
  }
}

// loss = (1 / n_traj) * sum_b mean(row_loss[cu[b] .. cu[b+1])): one block, one warp per trajectory in
// turn, additions in a fixed order.
__global__ void k_kl_mean(const float* __restrict__ row_loss, const int32_t* __restrict__ cu_rows, int n_traj, float* __restrict__ loss) {
  __shared__ float sh[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  float mine = 0.f;
  for (int b = warp; b < n_traj; b += nw) {
    const int a = cu_rows[b], e = cu_rows[b + 1];
    float s = 0.f;
    for (int i = a + lane; i < e; i += 32) s += row_loss[i];
#pragma unroll
    for (int d = 16; d; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
    if (e > a) mine += s / (float)(e - a);
  }
  if (lane == 0) sh[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += sh[w];
    *loss = t / (float)n_traj;
  }
}

}  // namespace

extern "C" bc_status bc_distill_loss(int32_t n_traj, const int32_t* cu_rows, int64_t rows, int32_t vocab, int32_t top_k,
                                     const void* student_logits, const int32_t* teacher_idx, const float* teacher_logprob,
                                     float* row_loss, float* loss, void* grad, void* stream) {
  if (n_traj < 1 || !cu_rows || rows < 0 || vocab < 1 || top_k < 1 || !row_loss || !loss) return BC_ERR_INVALID_ARG;
  if (rows > 0 && (!student_logits || !teacher_idx || !teacher_logprob)) return BC_ERR_INVALID_ARG;
  if (rows > 0x7fffffff) return BC_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(student_logits) | reinterpret_cast<uintptr_t>(grad)) & 1) return BC_ERR_INVALID_ARG;
  // the gradient rows must be aligned like the logit rows (same 16-byte phase)
  if (grad && ((reinterpret_cast<uintptr_t>(student_logits) ^ reinterpret_cast<uintptr_t>(grad)) & 15)) return BC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (rows > 0)
    k_kl_rows<<<(unsigned)rows, kRowThreads, 0, s>>>((const __nv_bfloat16*)student_logits, teacher_idx, teacher_logprob, cu_rows,
                                                     n_traj, vocab, top_k, row_loss, (__nv_bfloat16*)grad);
  k_kl_mean<<<1, 1024, 0, s>>>(row_loss, cu_rows, n_traj, loss);
  return cudaGetLastError() == cudaSuccess ? BC_OK : BC_ERR_CUDA;
}
