// Microbenchmark of the two L2 streams that bound the key-block-major tile kernels:
//   gather : 1 KB pieces (the G*d*2 bytes of one token's query rows, G = 4, d = 128) fetched from random
//            tokens of a 16384-token window into shared memory with 16-byte cp.async (what the producer
//            warps of lse_ws / pv_ws do), 4 or 8 issuing warps per SM, several tiles in flight;
//   reduce : 2 KB of fp32 per (token, block) pair added into an L2-resident accumulator window with
//            red.global.add.v4.f32 (what the reducer warps of pv_ws do);
//   mix    : both at once in the kernels' 1 : 2 byte ratio;
//   half   : the reduce and the gather stream from half of the SMs (is the limit on the SM's path or in L2?);
//   bulk   : the reduction stream through the copy engine (cp.reduce.async.bulk from shared memory, 2 KB per
//            token), alone, from half of the SMs, and side by side with the vector reductions.
// One CTA per SM.  Prints one line per case: name, milliseconds, TB/s, bytes per clock and SM at the SM
// clock the run saw.  Build: nvcc -gencode arch=compute_100a,code=sm_100a -O3 l2_streams.cu -o l2_streams
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <cuda_runtime.h>

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda error %s at line %d\n", cudaGetErrorString(e_), __LINE__); return 1; } } while (0)

constexpr int kTileBytes = 32768;     // 32 tokens x 1 KB
constexpr int kDepth = 4;             // tiles in flight per SM

// warps [0, gw): gather; warps [gw, gw + rw): reduce.  tok: [ctas][tiles][32] token ids.
__global__ void streams_kernel(const uint8_t* __restrict__ q, long long tok_stride, const int* __restrict__ tok,
                               int tiles, int gw, int rw, float* acc, long long acc_tok_stride) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int* my = tok + (long long)blockIdx.x * tiles * 32;
  if (warp < gw) {
    // 16-byte chunk ck of rows rb, rb + rpp, ... of a 128-row tile (row = token * 4 + head, 256 bytes each)
    const int p = warp * 32 + lane, ck = p % 16, rb = p / 16, rpp = gw * 2;
    for (int t = 0; t < tiles; ++t) {
      uint8_t* dst = smem + (t % kDepth) * kTileBytes;
      for (int row = rb; row < 128; row += rpp) {
        const uint8_t* src = q + (long long)my[t * 32 + (row >> 2)] * tok_stride + (row & 3) * 256 + ck * 16;
        const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + row * 256 + ((ck ^ (row & 7)) * 16));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else if (warp < gw + rw) {
    // lane = output column d of a [token][d = 128][4 heads] accumulator; a warp adds 512 contiguous bytes per
    // instruction, one instruction per token of the tile; rw warps cover the 128 columns in 128 / (32 * rw) passes
    const int w = warp - gw;
    for (int t = 0; t < tiles; ++t)
      for (int col0 = w * 32; col0 < 128; col0 += rw * 32)
        for (int i = 0; i < 32; ++i) {
          float* dst = acc + (long long)my[t * 32 + i] * acc_tok_stride + (col0 + lane) * 4;
          asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %1, %1, %1};" ::"l"(dst), "f"(1.0f) : "memory");
        }
  }
}

// The reduction stream through the copy engine instead of the SM's load/store path: one warp, every lane adds one
// token's 2 KB (shared memory -> accumulator row) with a bulk reduction, two tiles in flight.
template <int DEPTH>
__global__ void bulk_reduce_kernel(const int* __restrict__ tok, int tiles, float* acc, long long acc_tok_stride) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int lane = threadIdx.x & 31;
  const int* my = tok + (long long)blockIdx.x * tiles * 32;
  for (int i = threadIdx.x; i < 2 * 65536 / 4; i += blockDim.x) reinterpret_cast<float*>(smem)[i] = 1.0f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < 32) {
    for (int t = 0; t < tiles; ++t) {
      float* dst = acc + (long long)my[t * 32 + lane] * acc_tok_stride;
      const uint32_t src = (uint32_t)__cvta_generic_to_shared(smem + (t & 1) * 65536 + lane * 2048);
      asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(2048)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(DEPTH - 1) : "memory");
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
}

// Both paths at once: warps 0-3 add the first 16 tokens of a tile with vector reductions, warp 4 the other 16 with
// bulk reductions.
__global__ void split_reduce_kernel(const int* __restrict__ tok, int tiles, float* acc, long long acc_tok_stride) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int* my = tok + (long long)blockIdx.x * tiles * 32;
  for (int i = threadIdx.x; i < 65536 / 4; i += blockDim.x) reinterpret_cast<float*>(smem)[i] = 1.0f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (warp < 4) {
    for (int t = 0; t < tiles; ++t)
      for (int i = 0; i < 16; ++i) {
        float* dst = acc + (long long)my[t * 32 + i] * acc_tok_stride + (warp * 32 + lane) * 4;
        asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %1, %1, %1};" ::"l"(dst), "f"(1.0f) : "memory");
      }
  } else if (lane < 16) {
    for (int t = 0; t < tiles; ++t) {
      float* dst = acc + (long long)my[t * 32 + 16 + lane] * acc_tok_stride;
      const uint32_t src = (uint32_t)__cvta_generic_to_shared(smem + (t & 1) * 32768 + lane * 2048);
      asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(2048)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
}

// Both paths from the same four warps, no barrier between them: every warp adds its 512-byte column share of 24 of a
// tile's tokens with vector reductions and of the other 8 with one bulk reduction each (lanes 0-7 issue them).
__global__ void warp_split_kernel(const int* __restrict__ tok, int tiles, float* acc, long long acc_tok_stride) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int* my = tok + (long long)blockIdx.x * tiles * 32;
  for (int i = threadIdx.x; i < 32768 / 4; i += blockDim.x) reinterpret_cast<float*>(smem)[i] = 1.0f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  for (int t = 0; t < tiles; ++t) {
    for (int i = 0; i < 24; ++i) {
      float* dst = acc + (long long)my[t * 32 + i] * acc_tok_stride + (warp * 32 + lane) * 4;
      asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %1, %1, %1};" ::"l"(dst), "f"(1.0f) : "memory");
    }
    if (lane < 8) {
      float* dst = acc + (long long)my[t * 32 + 24 + lane] * acc_tok_stride + warp * 128;
      const uint32_t src = (uint32_t)__cvta_generic_to_shared(smem + (t & 1) * 16384 + warp * 4096 + lane * 512);
      asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(512)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
    }
    __syncwarp();
  }
  if (lane < 8) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

static int run_warp_split(const char* name, const int* tok, int tiles, float* acc, int sms, double clk_hz) {
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
  CK(cudaFuncSetAttribute(warp_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768));
  warp_split_kernel<<<sms, 128, 32768>>>(tok, tiles, acc, 512);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(a));
  warp_split_kernel<<<sms, 128, 32768>>>(tok, tiles, acc, 512);
  CK(cudaEventRecord(b));
  CK(cudaDeviceSynchronize());
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, a, b));
  const double bytes = (double)sms * tiles * 65536.0;
  printf("%-44s %8.3f ms %6.2f TB/s %6.1f B/clk/SM\n", name, ms, bytes / ms * 1e-9, bytes / sms / (ms * 1e-3 * clk_hz));
  return 0;
}

static int run_split(const char* name, const int* tok, int tiles, float* acc, int sms, double clk_hz) {
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
  CK(cudaFuncSetAttribute(split_reduce_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536));
  split_reduce_kernel<<<sms, 160, 65536>>>(tok, tiles, acc, 512);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(a));
  split_reduce_kernel<<<sms, 160, 65536>>>(tok, tiles, acc, 512);
  CK(cudaEventRecord(b));
  CK(cudaDeviceSynchronize());
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, a, b));
  const double bytes = (double)sms * tiles * 65536.0;
  printf("%-44s %8.3f ms %6.2f TB/s %6.1f B/clk/SM\n", name, ms, bytes / ms * 1e-9, bytes / sms / (ms * 1e-3 * clk_hz));
  return 0;
}

template <int DEPTH>
static int run_bulk(const char* name, const int* tok, int tiles, float* acc, int sms, double clk_hz) {
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
  CK(cudaFuncSetAttribute(bulk_reduce_kernel<DEPTH>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 65536));
  bulk_reduce_kernel<DEPTH><<<sms, 128, 2 * 65536>>>(tok, tiles, acc, 512);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(a));
  bulk_reduce_kernel<DEPTH><<<sms, 128, 2 * 65536>>>(tok, tiles, acc, 512);
  CK(cudaEventRecord(b));
  CK(cudaDeviceSynchronize());
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, a, b));
  const double bytes = (double)sms * tiles * 65536.0;
  printf("%-44s %8.3f ms %6.2f TB/s %6.1f B/clk/SM\n", name, ms, bytes / ms * 1e-9, bytes / sms / (ms * 1e-3 * clk_hz));
  return 0;
}

static int run(const char* name, const uint8_t* q, const int* tok, int tiles, int gw, int rw, float* acc, int sms,
               double clk_hz) {
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
  const int threads = (gw + rw) * 32;
  CK(cudaFuncSetAttribute(streams_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDepth * kTileBytes));
  streams_kernel<<<sms, threads, kDepth * kTileBytes>>>(q, 8192, tok, tiles, gw, rw, acc, 512);
  CK(cudaDeviceSynchronize());
  CK(cudaEventRecord(a));
  streams_kernel<<<sms, threads, kDepth * kTileBytes>>>(q, 8192, tok, tiles, gw, rw, acc, 512);
  CK(cudaEventRecord(b));
  CK(cudaDeviceSynchronize());
  float ms = 0.f;
  CK(cudaEventElapsedTime(&ms, a, b));
  const double bytes = (double)sms * tiles * ((gw ? 32768.0 : 0.0) + (rw ? 65536.0 : 0.0));
  printf("%-44s %8.3f ms %6.2f TB/s %6.1f B/clk/SM\n", name, ms, bytes / ms * 1e-9, bytes / sms / (ms * 1e-3 * clk_hz));
  return 0;
}

int main() {
  int dev = 0, sms = 0, khz = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  CK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
  const double clk = khz * 1e3;
  const int tiles = 512, window = 16384;
  const long long ntok = 131072;
  uint8_t* q;
  CK(cudaMalloc(&q, ntok * 8192));                    // q of 32 heads x 128 x bf16 per token: 1.07 GB
  CK(cudaMemset(q, 1, ntok * 8192));
  float* acc;
  CK(cudaMalloc(&acc, ntok * 512 * sizeof(float)));   // one KV head's accumulator [token][128][4]: 268 MB
  CK(cudaMemset(acc, 0, ntok * 512 * sizeof(float)));
  // all CTAs work in the same window at the same time; the window advances with the tile index
  std::vector<int> h((size_t)sms * tiles * 32);
  srand(1);
  for (int c = 0; c < sms; ++c)
    for (int t = 0; t < tiles; ++t)
      for (int i = 0; i < 32; ++i) h[((size_t)c * tiles + t) * 32 + i] = (t * 8 / tiles) * window + rand() % window;
  int* tok;
  CK(cudaMalloc(&tok, h.size() * sizeof(int)));
  CK(cudaMemcpy(tok, h.data(), h.size() * sizeof(int), cudaMemcpyHostToDevice));
  printf("SMs %d, SM clock %.0f MHz (bytes per clock use this clock)\n", sms, clk * 1e-6);
  if (run("gather 1 KB pieces, 4 warps", q, tok, tiles, 4, 0, acc, sms, clk)) return 1;
  if (run("gather 1 KB pieces, 8 warps", q, tok, tiles, 8, 0, acc, sms, clk)) return 1;
  if (run("reduce fp32 v4, 4 warps", q, tok, tiles, 0, 4, acc, sms, clk)) return 1;
  if (run("reduce fp32 v4, 8 warps", q, tok, tiles, 0, 8, acc, sms, clk)) return 1;
  if (run("mix: gather 4 warps + reduce 4 warps", q, tok, tiles, 4, 4, acc, sms, clk)) return 1;
  if (run("mix: gather 8 warps + reduce 4 warps", q, tok, tiles, 8, 4, acc, sms, clk)) return 1;
  if (run("mix: gather 8 warps + reduce 8 warps", q, tok, tiles, 8, 8, acc, sms, clk)) return 1;
  // the same streams from half of the SMs: a limit that sits in L2 leaves the total where it was (twice the rate per
  // active SM), a limit on the SM's own path halves the total
  if (run("reduce fp32 v4, 4 warps, half of the SMs", q, tok, tiles, 0, 4, acc, sms / 2, clk)) return 1;
  if (run("gather 1 KB pieces, 4 warps, half of the SMs", q, tok, tiles, 4, 0, acc, sms / 2, clk)) return 1;
  if (run_bulk<2>("bulk reductions of 2 KB, 2 tiles in flight", tok, tiles, acc, sms, clk)) return 1;
  if (run_bulk<2>("bulk reductions of 2 KB, half of the SMs", tok, tiles, acc, sms / 2, clk)) return 1;
  if (run_split("half vector reductions, half bulk reductions", tok, tiles, acc, sms, clk)) return 1;
  if (run_warp_split("3/4 vector, 1/4 bulk (512 B), per warp", tok, tiles, acc, sms, clk)) return 1;
  return 0;
}
