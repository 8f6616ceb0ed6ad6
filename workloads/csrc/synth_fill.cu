// Native twins of the synthetic input generator (the Python module beside this folder): a
// device kernel that fills KV pools and transfer buffers far too large to generate on the host,
// and a plain host loop for tests that regenerate such content chunk by chunk.  Input
// generation only - none of the library's own operations is implemented here, and libaibx does
// not link this file.
//
// Logical content: 64-bit word w of the block-major byte stream [block][layer][tile] equals
// splitmix64's output function of (w + 1) * GOLD + seed * SEEDMUL, stored little-endian.  A
// layer-major pool holds the same logical content at its own physical place.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__host__ __device__ __forceinline__ unsigned long long mix64(unsigned long long seed,
                                                    unsigned long long counter) {
  unsigned long long z = (counter + 1ULL) * 0x9E3779B97F4A7C15ULL + seed * 0xD1B54A32D192ED03ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

// layout 0: physical word == logical word (offset by first_word).
// layout 1: physical [layer][block][tile] -> logical [block][layer][tile].
// layout 2: physical [layer][K/V][block][half tile] -> logical [block][layer][K/V][half tile].
__global__ void fill_kernel(unsigned long long* dst, unsigned long long n_words,
                            unsigned long long seed, unsigned long long first_word, int layout,
                            unsigned long long num_layers, unsigned long long num_blocks,
                            unsigned long long tile_words) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long pw = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
       pw < n_words; pw += stride) {
    unsigned long long lw = first_word + pw;
    if (layout == 1) {
      const unsigned long long per_layer = num_blocks * tile_words;
      const unsigned long long l = pw / per_layer;
      const unsigned long long rem = pw - l * per_layer;
      const unsigned long long b = rem / tile_words;
      const unsigned long long j = rem - b * tile_words;
      lw = (b * num_layers + l) * tile_words + j;
    } else if (layout == 2) {
      const unsigned long long half_words = tile_words / 2;
      const unsigned long long per_plane = num_blocks * half_words;
      const unsigned long long plane = pw / per_plane;            // 2 * layer + kv
      const unsigned long long rem = pw - plane * per_plane;
      const unsigned long long b = rem / half_words;
      const unsigned long long j = rem - b * half_words;
      lw = (b * 2 * num_layers + plane) * half_words + j;
    }
    dst[pw] = mix64(seed, lw);
  }
}

}  // namespace

extern "C" {

// d_dst: device pointer, 8-byte aligned; n_bytes and first_byte multiples of 8.
int32_t aibx_synth_fill_linear(void* d_dst, uint64_t n_bytes, uint64_t seed, uint64_t first_byte,
                               void* stream) {
  if (!d_dst || (n_bytes & 7) || (first_byte & 7)) return -1;
  if (n_bytes == 0) return 0;
  fill_kernel<<<148 * 16, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<unsigned long long*>(d_dst), n_bytes / 8, seed, first_byte / 8, 0, 1, 1, 1);
  return cudaPeekAtLastError() == cudaSuccess ? 0 : -4;
}

// The same stream written by the calling host thread: h_dst (host memory, 8-byte aligned) <-
// bytes [first_byte, first_byte + n_bytes) of stream `seed`.  No CUDA call is made.
int32_t aibx_synth_fill_host(void* h_dst, uint64_t n_bytes, uint64_t seed, uint64_t first_byte) {
  if (!h_dst || (n_bytes & 7) || (first_byte & 7) || (reinterpret_cast<uintptr_t>(h_dst) & 7))
    return -1;
  unsigned long long* dst = static_cast<unsigned long long*>(h_dst);
  const unsigned long long first_word = first_byte / 8;
  const unsigned long long n_words = n_bytes / 8;
  for (unsigned long long w = 0; w < n_words; ++w) dst[w] = mix64(seed, first_word + w);
  return 0;
}

// Whole pool in its physical layout (0 block-major, 1 layer-major, 2 layer-major with the K and
// V halves of the tiles in separate planes); tile_bytes multiple of 8 (16 for layout 2).
int32_t aibx_synth_fill_pool(void* d_pool, uint64_t seed, int32_t layout, uint64_t num_layers,
                             uint64_t num_blocks, uint64_t tile_bytes, void* stream) {
  if (!d_pool || (tile_bytes & 7) || layout < 0 || layout > 2) return -1;
  if (layout == 2 && (tile_bytes & 15)) return -1;
  const unsigned long long n_words = num_layers * num_blocks * (tile_bytes / 8);
  if (n_words == 0) return 0;
  fill_kernel<<<148 * 16, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<unsigned long long*>(d_pool), n_words, seed, 0, layout, num_layers, num_blocks,
      tile_bytes / 8);
  return cudaPeekAtLastError() == cudaSuccess ? 0 : -4;
}

}  // extern "C"
