// K5 and the small index kernels of the step prologue.
//
//  * scatter_kv:   cache write-back of the active rows' fresh K, V (Algorithm 1 line 11).
//  * scatter_rows: fp32 row scatter (hidden_out rows of the active tokens; sampled rows
//                  into the stack input).
//  * gather_table_rows, fill_mask_rows: assembly of the decoder's input (Eq. 2).
//  * step_flags:   per-step bookkeeping of the token sets of Algorithm 1 lines 1-4:
//                  which active rows are generating tokens, which tokens may be picked
//                  for refresh.
//  * build_active: A = G u N u R by concatenation.
//  * validate:     optional device-side check of the index sets.
// All are pure copies / integer work, bound by HBM (rows) or launch latency (indices).
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

// One warp per (row, K|V) pair; 16-byte vectors, row_vecs = D*sizeof(T)/16 per row.
__global__ void __launch_bounds__(256)
scatter_kv_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, long ld_vecs,
                  const int32_t* __restrict__ idx, int n, int S, int row_vecs, long total_rows,
                  long kv_stride_vecs, uint4* __restrict__ cache) {
  const long w = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= 2 * total_rows) return;
  pdl_sync();
  const int which = (int)(w & 1);
  const long r = w >> 1;
  const int b = (int)(r / n), j = (int)(r - (long)b * n);
  const int t = idx ? idx[r] : j;
  const uint4* src = (which ? v : k) + r * ld_vecs;
  uint4* dst = cache + which * kv_stride_vecs + ((long)b * S + t) * row_vecs;
  for (int c = lane; c < row_vecs; c += 32) dst[c] = __ldg(src + c);
}

__global__ void __launch_bounds__(256)
scatter_rows_kernel(const float4* __restrict__ rows, const int32_t* __restrict__ idx, int n, int S,
                    int row_vecs, long total_rows, float4* __restrict__ dst) {
  const long r = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= total_rows) return;
  pdl_sync();
  const int b = (int)(r / n), j = (int)(r - (long)b * n);
  const int t = idx ? idx[r] : j;
  const float4* src = rows + r * row_vecs;
  float4* d = dst + ((long)b * S + t) * row_vecs;
  for (int c = lane; c < row_vecs; c += 32) d[c] = __ldg(src + c);
}

__global__ void __launch_bounds__(256)
gather_rows_kernel(const float4* __restrict__ src, const int32_t* __restrict__ idx, int n, int S, int row_vecs,
                   long total_rows, float4* __restrict__ out) {
  const long r = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= total_rows) return;
  pdl_sync();
  const int b = (int)(r / n);
  const float4* s = src + ((long)b * S + idx[r]) * row_vecs;
  float4* d = out + r * row_vecs;
  for (int c = lane; c < row_vecs; c += 32) d[c] = __ldg(s + c);
}

// out[r] = table[idx[r]]: rows of a table shared by all samples (positional embedding), one warp per row.
__global__ void __launch_bounds__(256)
gather_table_rows_kernel(const float4* __restrict__ table, const int32_t* __restrict__ idx, int row_vecs,
                         long total_rows, float4* __restrict__ out) {
  const long r = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= total_rows) return;
  pdl_sync();
  const float4* s = table + (long)idx[r] * row_vecs;
  float4* d = out + r * row_vecs;
  for (int c = lane; c < row_vecs; c += 32) d[c] = __ldg(s + c);
}

// out[b][s] = mask_token + pos[s] for every token of every sample (Eq. 2: the decoder's input at a
// masked position); the rows of known tokens are overwritten afterwards.
__global__ void __launch_bounds__(256)
fill_mask_rows_kernel(const float4* __restrict__ mask_token, const float4* __restrict__ pos, int S, int row_vecs,
                      long total_rows, float4* __restrict__ out) {
  const long r = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= total_rows) return;
  pdl_sync();
  const float4* p = pos + (r % S) * row_vecs;
  float4* d = out + r * row_vecs;
  for (int c = lane; c < row_vecs; c += 32) {
    const float4 m = __ldg(mask_token + c), q = __ldg(p + c);
    d[c] = make_float4(m.x + q.x, m.y + q.y, m.z + q.z, m.w + q.w);
  }
}

// One CTA per sample.  mark bit0 = generating token, bit1 = excluded token.
__global__ void __launch_bounds__(256)
step_flags_kernel(const int32_t* __restrict__ active_idx, int n_active, const int32_t* __restrict__ new_idx,
                  int n_new, const int32_t* __restrict__ excl_idx, int n_excl, int S,
                  uint8_t* __restrict__ is_new, uint8_t* __restrict__ cand) {
  extern __shared__ uint8_t mark[];
  const int b = blockIdx.x;
  pdl_sync();
  for (int t = threadIdx.x; t < S; t += blockDim.x) mark[t] = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < n_new; i += blockDim.x) mark[new_idx[(long)b * n_new + i]] = 1;
  __syncthreads();
  for (int i = threadIdx.x; i < n_excl; i += blockDim.x) mark[excl_idx[(long)b * n_excl + i]] |= 2;
  __syncthreads();
  if (is_new)
    for (int j = threadIdx.x; j < n_active; j += blockDim.x)
      is_new[(long)b * n_active + j] = active_idx ? (mark[active_idx[(long)b * n_active + j]] & 1) : (mark[j] & 1);
  if (cand)
    for (int t = threadIdx.x; t < S; t += blockDim.x) cand[(long)b * S + t] = mark[t] ? 0 : 1;
}

__global__ void build_active_kernel(const int32_t* __restrict__ a, int na, const int32_t* __restrict__ b, int nb,
                                    const int32_t* __restrict__ c, int nc, int B, int32_t* __restrict__ out) {
  const int n = na + nb + nc;
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)B * n) return;
  pdl_sync();
  const int s = (int)(i / n), j = (int)(i - (long)s * n);
  int32_t v;
  if (j < na) v = a[(long)s * na + j];
  else if (j < na + nb) v = b[(long)s * nb + (j - na)];
  else v = c[(long)s * nc + (j - na - nb)];
  out[i] = v;
}

// One CTA per sample; count[t] bit layout: low nibble = times in active, bit4 = new, bit5 = excl.
__global__ void __launch_bounds__(256)
validate_kernel(const int32_t* __restrict__ active_idx, int n_active, const int32_t* __restrict__ new_idx,
                int n_new, const int32_t* __restrict__ excl_idx, int n_excl, int S, int* status) {
  extern __shared__ int cnt[];
  __shared__ int bad;
  const int b = blockIdx.x;
  pdl_sync();
  if (threadIdx.x == 0) bad = 0;
  for (int t = threadIdx.x; t < 3 * S; t += blockDim.x) cnt[t] = 0;
  __syncthreads();
  int* ca = cnt; int* cn = cnt + S; int* cx = cnt + 2 * S;
  for (int i = threadIdx.x; i < n_active; i += blockDim.x) {
    const int t = active_idx[(long)b * n_active + i];
    if (t < 0 || t >= S) bad = 1; else atomicAdd(&ca[t], 1);
  }
  for (int i = threadIdx.x; i < n_new; i += blockDim.x) {
    const int t = new_idx[(long)b * n_new + i];
    if (t < 0 || t >= S) bad = 1; else atomicAdd(&cn[t], 1);
  }
  for (int i = threadIdx.x; i < n_excl; i += blockDim.x) {
    const int t = excl_idx[(long)b * n_excl + i];
    if (t < 0 || t >= S) bad = 1; else atomicAdd(&cx[t], 1);
  }
  __syncthreads();
  for (int t = threadIdx.x; t < S; t += blockDim.x) {
    if (ca[t] > 1 || cn[t] > 1 || cx[t] > 1) bad = 1;          // duplicates
    if (active_idx && cn[t] && !ca[t]) bad = 1;                 // new not in active
    if (cn[t] && cx[t]) bad = 1;                                // exclude overlaps new
  }
  __syncthreads();
  if (threadIdx.x == 0 && bad) *status = 1;
}

cudaError_t launch_scatter_kv(bool bf16_t, const void* k, const void* v, int ld_kv, const int32_t* idx,
                              int B, int n, int S, int D, void* cache_layer, cudaStream_t st) {
  const int eb = bf16_t ? 2 : 4;
  if ((D * eb) % 16 || (ld_kv * eb) % 16) return cudaErrorInvalidValue;
  const long rows = (long)B * n;
  if (rows == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((2 * rows + 7) / 8);
  return launch_pdl(scatter_kv_kernel, dim3(grid), dim3(256), 0, st, (const uint4*)k, (const uint4*)v,
                    (long)ld_kv * eb / 16, idx, n, S, D * eb / 16, rows, (long)B * S * D * eb / 16, (uint4*)cache_layer);
}

cudaError_t launch_scatter_rows(const float* rows, const int32_t* idx, int B, int n, int S, int D,
                                float* dst, cudaStream_t st) {
  if (D % 4) return cudaErrorInvalidValue;
  const long total = (long)B * n;
  if (total == 0) return cudaSuccess;
  return launch_pdl(scatter_rows_kernel, dim3((unsigned)((total + 7) / 8)), dim3(256), 0, st, (const float4*)rows, idx,
                    n, S, D / 4, total, (float4*)dst);
}

cudaError_t launch_gather_rows(const float* src, const int32_t* idx, int B, int n, int S, int D, float* out,
                               cudaStream_t st) {
  if (D % 4) return cudaErrorInvalidValue;
  const long total = (long)B * n;
  if (total == 0) return cudaSuccess;
  return launch_pdl(gather_rows_kernel, dim3((unsigned)((total + 7) / 8)), dim3(256), 0, st, (const float4*)src, idx, n,
                    S, D / 4, total, (float4*)out);
}

cudaError_t launch_gather_table_rows(const float* table, const int32_t* idx, long total_rows, int D, float* out,
                                     cudaStream_t st) {
  if (D % 4) return cudaErrorInvalidValue;
  if (total_rows == 0) return cudaSuccess;
  return launch_pdl(gather_table_rows_kernel, dim3((unsigned)((total_rows + 7) / 8)), dim3(256), 0, st,
                    (const float4*)table, idx, D / 4, total_rows, (float4*)out);
}

cudaError_t launch_fill_mask_rows(const float* mask_token, const float* pos, int B, int S, int D, float* out,
                                  cudaStream_t st) {
  if (D % 4) return cudaErrorInvalidValue;
  const long total = (long)B * S;
  return launch_pdl(fill_mask_rows_kernel, dim3((unsigned)((total + 7) / 8)), dim3(256), 0, st,
                    (const float4*)mask_token, (const float4*)pos, S, D / 4, total, (float4*)out);
}

cudaError_t launch_step_flags(const int32_t* active_idx, int n_active, const int32_t* new_idx, int n_new,
                              const int32_t* excl_idx, int n_excl, int B, int S, uint8_t* is_new,
                              uint8_t* cand, cudaStream_t st) {
  return launch_pdl(step_flags_kernel, dim3(B), dim3(256), (size_t)S, st, active_idx, n_active, new_idx, n_new, excl_idx,
                    n_excl, S, is_new, cand);
}

cudaError_t launch_build_active(const int32_t* a, int na, const int32_t* b, int nb, const int32_t* c, int nc,
                                int B, int32_t* out, cudaStream_t st) {
  const long total = (long)B * (na + nb + nc);
  if (total == 0) return cudaSuccess;
  return launch_pdl(build_active_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, a, na, b, nb, c, nc,
                    B, out);
}

cudaError_t launch_validate(const int32_t* active_idx, int n_active, const int32_t* new_idx, int n_new,
                            const int32_t* excl_idx, int n_excl, int B, int S, int* status, cudaStream_t st) {
  return launch_pdl(validate_kernel, dim3(B), dim3(256), 3 * S * sizeof(int), st, active_idx, n_active, new_idx, n_new,
                    excl_idx, n_excl, S, status);
}

}  // namespace marche
