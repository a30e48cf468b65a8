// Speculative-sampling acceptance at temperature T > 0 (Appendix B.2 names speculative sampling as the acceptance
// strategy).  The drafts come from retrieval or the schema, so the draft distribution is a point mass on the drafted
// token x and the rule reads: accept x with probability p(x), p = softmax(logits / T) of the row that predicts it;
// on the first rejection emit one sample of p with x removed (renormalised) and stop; if every draft is accepted
// emit one sample of the last row's p.  Over a draft tree the children of a node are tried in node order against
// the residual of the refused ones.  The uniforms are inputs: uni[node c] decides node c, the root's draws the sample
// (the host renames a chain's uniforms accordingly).  A sample is the smallest index whose running sum of weights, in index order, exceeds
// u times the total.
#include "kernels.h"

namespace ts {

static constexpr int kStatThreads = 256;
static constexpr int kStatSlices = 16;        // CTAs per row in the statistics kernel
static constexpr int kSampleThreads = 1024;   // 32 warps: one contiguous stretch of the vocabulary each

// the row maximum, from the packed (ordered value bits, ~id) word the LM-head epilogue reduced
__device__ __forceinline__ float row_max_of(unsigned long long word) {
  const uint32_t u = (uint32_t)(word >> 32);
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// grid = (rows, slices): sum of exp((l - max) / T) over one slice of one row
__global__ void __launch_bounds__(kStatThreads)
row_expsum_kernel(const float *logits, const unsigned long long *amax, int V, float inv_t, float *part) {
  __shared__ float red[kStatThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x, sl = blockIdx.y;
  const float *row = logits + (size_t)r * V;
  const float mx = row_max_of(amax[r]);
  const int per = (V + kStatSlices - 1) / kStatSlices;
  const int i0 = sl * per, i1 = min(V, i0 + per);
  float sum = 0.f;
  for (int i = i0 + threadIdx.x; i < i1; i += blockDim.x) sum += __expf((row[i] - mx) * inv_t);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < kStatThreads / 32; ++w) t += red[w];
    part[(size_t)r * kStatSlices + sl] = t;
  }
}

// grid = sequences.  The chunk is a draft tree (a chain is the tree with parents j - 1).  Thread c < k computes the
// weight of node c's token under its parent's row; thread 0 then walks from the root: the children of a node are
// tried in node order against the residual (the parent's weights with the tokens of refused children removed),
// child c accepted iff uni[c] * residual total < its weight.  Where the walk ends the block draws the step's one
// sample from the residual with uni[root]: the refused tokens' logits are set to -inf for the draw and put back
// afterwards; warp w owns ids [w * S, (w + 1) * S), read 32 at a time; the running sum goes warp by warp, then group
// of 32 by group, then lane by lane, so it is non-decreasing in the id and the first id above the target is found.
__global__ void __launch_bounds__(kSampleThreads)
sample_accept_kernel(SampleArgs a) {
  __shared__ float seg_total[kSampleThreads / 32];
  __shared__ float w_node[64], tot_node[64];
  __shared__ int refused[64];
  __shared__ float refused_logit[64];
  __shared__ int sh_l, sh_last, sh_nref, sh_tok;
  pdl_launch_dependents();
  pdl_wait();
  const int seq = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r0 = a.in.cu_rows[seq], k = a.in.cu_rows[seq + 1] - r0;
  int32_t *path = a.path + (size_t)seq * a.k_max;
  for (int r = r0 + threadIdx.x; r < r0 + k; r += blockDim.x)
    a.argmax[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)(a.amax[r] & 0xFFFFFFFFull));
  if ((int)threadIdx.x < k) {
    const int c = threadIdx.x;
    float tot = 0.f;
    for (int s = 0; s < kStatSlices; ++s) tot += a.part[(size_t)(r0 + c) * kStatSlices + s];
    tot_node[c] = tot;                                   // total weight of node c's own row
    const int par = a.in.parent[r0 + c];
    w_node[c] = par < 0 ? 0.f
                        : __expf((a.logits[(size_t)(r0 + par) * a.V + a.in.tokens[r0 + c]] - row_max_of(a.amax[r0 + par])) * a.inv_t);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int v = 0, l = 0, nref = 0;
    path[0] = 0;
    for (;;) {
      float R = tot_node[v];
      nref = 0;
      int nxt = -1;
      for (int c = v + 1; c < k; ++c) {
        if (a.in.parent[r0 + c] != v) continue;
        if (a.uni[r0 + c] * R < w_node[c]) { nxt = c; break; }
        R -= w_node[c];
        refused[nref++] = a.in.tokens[r0 + c];
      }
      if (nxt < 0) break;
      v = nxt;
      path[++l] = v;
    }
    sh_l = l; sh_last = v; sh_nref = nref; sh_tok = -1;
    // the refused tokens leave the row for the draw
    float *row_w = a.logits + (size_t)(r0 + v) * a.V;
    for (int i = 0; i < nref; ++i) { refused_logit[i] = row_w[refused[i]]; row_w[refused[i]] = -INFINITY; }
    __threadfence_block();
  }
  __syncthreads();
  const int l = sh_l, last = sh_last;
  const float *row = a.logits + (size_t)(r0 + last) * a.V;
  const float mx = row_max_of(a.amax[r0 + last]);
  const int S = ((a.V + kSampleThreads - 1) / kSampleThreads) * 32;   // ids per warp, a multiple of 32
  const int i0 = warp * S, i1 = min(a.V, i0 + S);
  auto weight = [&](int i) { return i < i1 ? __expf((__ldcg(row + i) - mx) * a.inv_t) : 0.f; };
  float part = 0.f;
  for (int i = i0 + lane; i < i1; i += 32) part += weight(i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0) seg_total[warp] = part;
  __syncthreads();
  float before = 0.f, total = 0.f;
  for (int w = 0; w < kSampleThreads / 32; ++w) {
    if (w < warp) before += seg_total[w];
    total += seg_total[w];
  }
  const float target = a.uni[r0] * total;
  if (before + seg_total[warp] > target && !(before > target)) {   // the running sum passes the target in this stretch
    float run = before;
    int tok = -1, lastw = -1;                          // lastw: the last id of the stretch that carries weight
    for (int g0 = i0; g0 < i1 && tok < 0; g0 += 32) {
      const float w = weight(g0 + lane);
      float inc = w;                                   // inclusive prefix over the group's 32 lanes
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, run + inc > target && w > 0.f);
      const unsigned any = __ballot_sync(0xffffffffu, w > 0.f);
      if (any) lastw = g0 + 31 - __clz(any);
      if (hit) tok = g0 + __ffs(hit) - 1;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) sh_tok = tok >= 0 ? tok : lastw;    // (the two summation orders may round apart by an ulp)
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int tok = sh_tok;
    if (tok < 0) {   // rounding kept every partial sum at or below the target: the last id that carries weight
      for (tok = a.V - 1; tok > 0 && !(__expf((row[tok] - mx) * a.inv_t) > 0.f); --tok) {}
    }
    float *row_w = a.logits + (size_t)(r0 + last) * a.V;
    for (int i = 0; i < sh_nref; ++i) row_w[refused[i]] = refused_logit[i];   // the logits are an output: put them back
    int32_t *em = a.emitted + (size_t)seq * a.k_max;
    for (int j = 1; j <= l; ++j) em[j - 1] = a.in.tokens[r0 + path[j]];
    em[l] = tok;
    a.accept_len[seq] = l;
    a.new_len[seq] = a.in.seq_len[seq] + l + 1;
    a.new_pending[seq] = tok;
  }
}

template <typename K, typename... Args>
static cudaError_t launch_pdl1(K kernel, dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_sample_accept(const SampleArgs &a, cudaStream_t st) {
  cudaError_t e = launch_pdl1(row_expsum_kernel, dim3(a.in.M, kStatSlices), dim3(kStatThreads), st, a.logits, a.amax,
                              a.V, a.inv_t, a.part);
  if (e != cudaSuccess) return e;
  return launch_pdl1(sample_accept_kernel, dim3(a.in.B), dim3(kSampleThreads), st, a);
}

}  // namespace ts
