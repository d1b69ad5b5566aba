// Memory-bound glue kernels: RMSNorm (RoPE, the KV-cache write and SwiGLU live in the GEMM
// epilogues) and the seeded synthetic fill used by the measurement harness.
#include "pd_common.cuh"
#include "pd_ptx.cuh"

namespace pd {
namespace {

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = ptx::bf16_lo(v.x); f[1] = ptx::bf16_hi(v.x);
  f[2] = ptx::bf16_lo(v.y); f[3] = ptx::bf16_hi(v.y);
  f[4] = ptx::bf16_lo(v.z); f[5] = ptx::bf16_hi(v.z);
  f[6] = ptx::bf16_lo(v.w); f[7] = ptx::bf16_hi(v.w);
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 o;
  o.x = ptx::pack_bf16(f[0], f[1]);
  o.y = ptx::pack_bf16(f[2], f[3]);
  o.z = ptx::pack_bf16(f[4], f[5]);
  o.w = ptx::pack_bf16(f[6], f[7]);
  return o;
}

// ------------------------------------------------------- FP8 row quantisation
// One block per row: pass 1 finds max|x|, pass 2 (the row is still in L1/L2) divides by
// scale = max / 448 in fp32 (IEEE division, the precision in which the codes are defined) and
// converts with round-to-nearest-even, saturating.  An all-zero row gets scale 1.
constexpr int QNT_THREADS = 256;

__global__ void __launch_bounds__(QNT_THREADS) quantize_rows_fp8_kernel(const bf16* __restrict__ x, int ldx, int k,
                                                                         uint8_t* __restrict__ codes, int ldq,
                                                                         float* __restrict__ scale_out) {
  const int row = blockIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const uint4* xr = reinterpret_cast<const uint4*>(x + static_cast<size_t>(row) * ldx);
  const int chunks = k / 8;
  float amax = 0.f;
  for (int c = threadIdx.x; c < chunks; c += QNT_THREADS) {
    float f[8];
    unpack8(xr[c], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
  }
  __shared__ float red[QNT_THREADS / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < QNT_THREADS / 32; ++w) tot = fmaxf(tot, red[w]);
  const float scale = tot > 0.f ? __fdiv_rn(tot, 448.f) : 1.f;
  if (threadIdx.x == 0) scale_out[row] = scale;
  uint2* qr = reinterpret_cast<uint2*>(codes + static_cast<size_t>(row) * ldq);
  for (int c = threadIdx.x; c < chunks; c += QNT_THREADS) {
    float f[8];
    unpack8(xr[c], f);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = __fdiv_rn(f[e], scale);
    uint2 o;
    o.x = ptx::cvt_e4m3x2(f[0], f[1]) | (ptx::cvt_e4m3x2(f[2], f[3]) << 16);
    o.y = ptx::cvt_e4m3x2(f[4], f[5]) | (ptx::cvt_e4m3x2(f[6], f[7]) << 16);
    qr[c] = o;
  }
}

// ------------------------------------------------------------------- RMSNorm
// y = x * rsqrt(mean(x^2) + eps) * g; one block per row, row kept in registers.
constexpr int RMS_THREADS = 256;
constexpr int RMS_MAX_CHUNKS = 8;  // 8 chunks * 8 elements * 256 threads = d up to 16384 (largest instantiation)

// With q_out != NULL the row is also quantised to E4M3 exactly as quantize_rows_fp8_kernel would quantise the
// stored bf16 row (the maximum and the quotients are taken on the bf16-rounded values).
// Rows are taken grid-stride (gridDim.x blocks, `rows` rows): while a row is being reduced and written, the loads of
// the block's next row are already in flight.
template <int NCH>  // 16-byte chunks per thread: d <= NCH * 8 * RMS_THREADS
__global__ void __launch_bounds__(RMS_THREADS) rmsnorm_kernel(const bf16* __restrict__ x,
                                                               const bf16* __restrict__ gain, bf16* __restrict__ y,
                                                               int rows, int d, float eps, float* zero_ptr,
                                                               int zero_cols, uint8_t* __restrict__ q_out,
                                                               float* __restrict__ s_out) {
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const uint4* gr = reinterpret_cast<const uint4*>(gain);
  const int chunks = d / 8;
  __shared__ float red[2][RMS_THREADS / 32];
  uint4 v[NCH], nxt[NCH];
  auto load_row = [&](int r, uint4 (&dst)[NCH]) {
    const uint4* xr = reinterpret_cast<const uint4*>(x + static_cast<size_t>(r) * d);
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int c = threadIdx.x + i * RMS_THREADS;
      if (c < chunks) dst[i] = xr[c];
    }
  };
  int row = blockIdx.x;
  if (row < rows) load_row(row, nxt);
  for (; row < rows; row += gridDim.x) {
#pragma unroll
    for (int i = 0; i < NCH; ++i) v[i] = nxt[i];
    if (row + static_cast<int>(gridDim.x) < rows) load_row(row + gridDim.x, nxt);
    if (zero_ptr) {  // fp32 sums of a later decode projection, idle while this kernel runs
      float4* q = reinterpret_cast<float4*>(zero_ptr + static_cast<size_t>(row) * zero_cols);
      for (int i = threadIdx.x; i < zero_cols / 4; i += RMS_THREADS) q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint4* yr = reinterpret_cast<uint4*>(y + static_cast<size_t>(row) * d);
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int c = threadIdx.x + i * RMS_THREADS;
      if (c < chunks) {
        float f[8];
        unpack8(v[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < RMS_THREADS / 32; ++w) tot += red[0][w];
    const float scale = rsqrtf(tot / static_cast<float>(d) + eps);
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int c = threadIdx.x + i * RMS_THREADS;
      if (c < chunks) {
        float f[8], g[8];
        unpack8(v[i], f);
        unpack8(gr[c], g);
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = f[e] * scale * g[e];
        v[i] = pack8(f);
        yr[c] = v[i];
        if (q_out) {
          unpack8(v[i], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(f[e]));
        }
      }
    }
    if (q_out) {  // block-uniform
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if ((threadIdx.x & 31) == 0) red[1][threadIdx.x >> 5] = amax;
      __syncthreads();
      float mx = 0.f;
#pragma unroll
      for (int w = 0; w < RMS_THREADS / 32; ++w) mx = fmaxf(mx, red[1][w]);
      const float qs = mx > 0.f ? __fdiv_rn(mx, 448.f) : 1.f;
      if (threadIdx.x == 0) s_out[row] = qs;
      uint2* qr = reinterpret_cast<uint2*>(q_out + static_cast<size_t>(row) * d);
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        const int c = threadIdx.x + i * RMS_THREADS;
        if (c < chunks) {
          float f[8];
          unpack8(v[i], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = __fdiv_rn(f[e], qs);
          uint2 o;
          o.x = ptx::cvt_e4m3x2(f[0], f[1]) | (ptx::cvt_e4m3x2(f[2], f[3]) << 16);
          o.y = ptx::cvt_e4m3x2(f[4], f[5]) | (ptx::cvt_e4m3x2(f[6], f[7]) << 16);
          qr[c] = o;
        }
      }
    }
    __syncthreads();  // red[] is reused by the block's next row
  }
}

// ------------------------------------------------------------- seeded fill
__device__ __forceinline__ uint64_t splitmix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(256) fill_normal_kernel(bf16* dst, size_t n, uint64_t key, float mean, float std) {
  // One hash per pair of outputs, Box-Muller on its two 32-bit halves.
  const size_t pairs = (n + 1) / 2;
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < pairs;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const uint64_t h = splitmix64(key ^ splitmix64(i));
    const float u1 = (static_cast<float>(static_cast<uint32_t>(h >> 32) >> 8) + 0.5f) * (1.0f / 16777216.0f);
    const float u2 = (static_cast<float>(static_cast<uint32_t>(h) >> 8) + 0.5f) * (1.0f / 16777216.0f);
    const float rad = sqrtf(-2.0f * __logf(u1));
    float s, c;
    __sincosf(6.283185307179586f * u2, &s, &c);
    dst[2 * i] = __float2bfloat16(mean + std * rad * c);
    if (2 * i + 1 < n) dst[2 * i + 1] = __float2bfloat16(mean + std * rad * s);
  }
}

}  // namespace

// Picks the instantiation for the row length; all blocks are resident (148 SMs x 4) and take further rows grid-stride.
static cudaError_t launch_rmsnorm_any(const bf16* x, const bf16* gain, bf16* y, int rows, int d, float eps, float* zero_ptr,
                                      int zero_cols, uint8_t* q_out, float* s_out, cudaStream_t s) {
  const int grid = rows < 148 * 4 ? rows : 148 * 4;
  const int per_thread = (d / 8 + RMS_THREADS - 1) / RMS_THREADS;
  const dim3 g(grid), b(RMS_THREADS);
  if (per_thread <= 1) return launch_pdl(rmsnorm_kernel<1>, g, b, 0, s, x, gain, y, rows, d, eps, zero_ptr, zero_cols, q_out, s_out);
  if (per_thread <= 2) return launch_pdl(rmsnorm_kernel<2>, g, b, 0, s, x, gain, y, rows, d, eps, zero_ptr, zero_cols, q_out, s_out);
  if (per_thread <= 4) return launch_pdl(rmsnorm_kernel<4>, g, b, 0, s, x, gain, y, rows, d, eps, zero_ptr, zero_cols, q_out, s_out);
  return launch_pdl(rmsnorm_kernel<8>, g, b, 0, s, x, gain, y, rows, d, eps, zero_ptr, zero_cols, q_out, s_out);
}

pd_status launch_rmsnorm(const bf16* x, const bf16* gain, bf16* y, int rows, int d, float eps, cudaStream_t s,
                         uint8_t* q_out, float* s_out) {
  if (rows == 0) return PD_OK;
  if (d % 8 != 0 || d > RMS_THREADS * RMS_MAX_CHUNKS * 8 || (q_out && !s_out)) return PD_ERR_UNSUPPORTED_SHAPE;
  float* no_zero = nullptr;
  PD_CUDA_TRY(launch_rmsnorm_any(x, gain, y, rows, d, eps, no_zero, 0, q_out, s_out, s));
  count_launch();
  return PD_OK;
}

pd_status launch_rmsnorm_decode(const bf16* x, const bf16* gain, bf16* y, int rows, int d, float eps, float* zero_ptr,
                                int zero_cols, cudaStream_t s, uint8_t* q_out, float* s_out) {
  if (rows == 0) return PD_OK;
  if (d % 8 != 0 || d > RMS_THREADS * RMS_MAX_CHUNKS * 8 || (zero_ptr && zero_cols % 4 != 0) || (q_out && !s_out))
    return PD_ERR_UNSUPPORTED_SHAPE;
  PD_CUDA_TRY(launch_rmsnorm_any(x, gain, y, rows, d, eps, zero_ptr, zero_cols, q_out, s_out, s));
  count_launch();
  return PD_OK;
}

pd_status launch_quantize_rows_fp8(const bf16* x, int ldx, int rows, int k, uint8_t* codes, int ldq, float* scale,
                                   cudaStream_t s) {
  if (rows == 0) return PD_OK;
  if (!x || !codes || !scale || rows < 0 || k <= 0) return PD_ERR_INVALID_ARG;
  if (k % 16 != 0 || ldx % 8 != 0 || ldq % 16 != 0 || ldx < k || ldq < k) return PD_ERR_UNSUPPORTED_SHAPE;
  PD_CUDA_TRY(launch_pdl(quantize_rows_fp8_kernel, dim3(rows), dim3(QNT_THREADS), 0, s, x, ldx, k, codes, ldq, scale));
  count_launch();
  return PD_OK;
}

pd_status launch_fill_normal(bf16* dst, size_t n, uint64_t seed, uint64_t stream_id, float mean, float std,
                             cudaStream_t s) {
  if (n == 0) return PD_OK;
  const uint64_t key = seed * 0xD1342543DE82EF95ull + stream_id * 0x2545F4914F6CDD1Dull + 0x632BE59BD9B4E019ull;
  fill_normal_kernel<<<148 * 8, 256, 0, s>>>(dst, n, key, mean, std);
  PD_CUDA_TRY(cudaGetLastError());
  return PD_OK;
}

}  // namespace pd

extern "C" pd_status pd_quantize_fp8_rows(const void* x, int32_t ldx, int32_t rows, int32_t k, void* codes,
                                          float* scales, void* stream) {
  return pd::launch_quantize_rows_fp8(static_cast<const pd::bf16*>(x), ldx, rows, k, static_cast<uint8_t*>(codes), k,
                                      scales, static_cast<cudaStream_t>(stream));
}
