// Device side of the seeded input generators: the same counter-based hash and the same fp32 operations as
// gen.py, so a tensor filled here is bit-identical to the numpy one.  Inputs only: no method arithmetic.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr uint64_t kM1 = 0xBF58476D1CE4E5B9ull, kM2 = 0x94D049BB133111EBull, kGold = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kStreamKBase = 1ull << 20, kStreamKNoise = 2ull << 20, kStreamKRedraw = 3ull << 20;
constexpr uint64_t kRedrawThreshold = 5033165ull;

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x ^= x >> 30; x *= kM1;
  x ^= x >> 27; x *= kM2;
  x ^= x >> 31;
  return x;
}
__device__ __forceinline__ uint64_t stream_key(uint64_t seed, uint64_t stream) { return mix64(seed * kGold + stream); }
__device__ __forceinline__ uint64_t hash_at(uint64_t key, uint64_t idx) { return mix64(key + idx * kGold); }

__device__ __forceinline__ float normal_at(uint64_t key, uint64_t idx) {
  const uint64_t h0 = hash_at(key, 2 * idx), h1 = hash_at(key, 2 * idx + 1);
  uint32_t s = 0;
#pragma unroll
  for (int sh = 0; sh < 64; sh += 16) s += static_cast<uint32_t>((h0 >> sh) & 0xFFFF) + static_cast<uint32_t>((h1 >> sh) & 0xFFFF);
  const float x = static_cast<float>(s);
  return __fmul_rn(__fsub_rn(x, 262140.0f), static_cast<float>(1.0 / 53509.98));
}
__device__ __forceinline__ uint16_t bf16_rne(float f) {
  const uint32_t u = __float_as_uint(f);
  return static_cast<uint16_t>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

__global__ void fill_normal(uint16_t* out, uint64_t seed, uint64_t stream, uint64_t idx0, uint64_t n) {
  const uint64_t key = stream_key(seed, stream);
  for (uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<uint64_t>(gridDim.x) * blockDim.x)
    out[i] = bf16_rne(normal_at(key, idx0 + i));
}

// One warp-sized group of threads per (frame, position) row would also work; a flat element loop is enough here.
__global__ void fill_keys(uint16_t* out, uint64_t seed, uint64_t layer, uint64_t g0, uint64_t n_frames, uint64_t T,
                          uint64_t D, float sigma) {
  const uint64_t kb = stream_key(seed, kStreamKBase + layer), kn = stream_key(seed, kStreamKNoise + layer),
                 kr = stream_key(seed, kStreamKRedraw + layer);
  const uint64_t n = n_frames * T * D;
  for (uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<uint64_t>(gridDim.x) * blockDim.x) {
    const uint64_t c = i % D, fp = i / D, p = fp % T, g = g0 + fp / T;
    uint64_t src = g;   // latest frame <= g at which position p was redrawn (frame 0 always is)
    while (src > 0 && (hash_at(kr, src * T + p) >> 40) >= kRedrawThreshold) --src;
    const float base = normal_at(kb, (src * T + p) * D + c);
    const float eps = normal_at(kn, (g * T + p) * D + c);
    out[i] = bf16_rne(__fadd_rn(base, __fmul_rn(sigma, eps)));
  }
}

}  // namespace

extern "C" {

int wkin_fill_normal_bf16(void* out_dev, uint64_t seed, uint64_t stream_id, uint64_t idx0, uint64_t n, void* cuda_stream) {
  if (n == 0) return 0;
  const int threads = 256;
  const uint64_t want = (n + threads - 1) / threads;
  const int blocks = static_cast<int>(want < 148 * 32 ? want : 148 * 32);
  fill_normal<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<uint16_t*>(out_dev), seed, stream_id,
                                                                             idx0, n);
  return static_cast<int>(cudaGetLastError());
}

int wkin_fill_keys_bf16(void* out_dev, uint64_t seed, uint64_t layer, uint64_t g0, uint64_t n_frames, uint64_t T, uint64_t D,
                        float sigma, void* cuda_stream) {
  const uint64_t n = n_frames * T * D;
  if (n == 0) return 0;
  const int threads = 256;
  const uint64_t want = (n + threads - 1) / threads;
  const int blocks = static_cast<int>(want < 148 * 32 ? want : 148 * 32);
  fill_keys<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<uint16_t*>(out_dev), seed, layer, g0,
                                                                           n_frames, T, D, sigma);
  return static_cast<int>(cudaGetLastError());
}

}  // extern "C"
