// Diagnostic kernels behind the pivot_debug_* entry points.  Not part of the method.
//
// wait_expiry_probe: every tensor-core kernel of the library waits on mbarriers through
// ptx::mbar_wait / mbar_wait_poll, which give up after a wall-clock limit, raise the CTA's abort
// flag and let the kernel end with DEV_WAIT_EXPIRED in the status word instead of hanging the GPU.
// In a correct run that path never executes.  This kernel runs it: 128 threads wait -- through the
// same two functions, with a short limit passed in -- for a barrier phase that nothing will ever
// complete, fall through when the limit runs out, and report the status exactly as the real
// kernels do at their teardown.  Nothing traps and nothing spins without bound.
#include <cuda.h>

#include "kernels.h"
#include "ptx.cuh"

namespace pivot {
namespace {

__global__ void __launch_bounds__(128, 1) wait_expiry_probe_kernel(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  __shared__ int returned_false;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);         // one arrival expected; nobody arrives
    abort_flag = 0;
    returned_false = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  bool ok;
  if (warp == 0) ok = ptx::mbar_wait(&bar, 0, &abort_flag, 64, limit_ns);          // sleeping poll (single-thread roles)
  else if (warp == 1) ok = ptx::mbar_wait_poll(&bar, 0, &abort_flag, limit_ns);     // the MMA issuer's poll
  else ok = ptx::mbar_wait(&bar, 0, &abort_flag, 0, limit_ns);                      // epilogue warps
  if (!ok) atomicAdd(&returned_false, 1);
  __syncthreads();
  // same report as the scan / re-score / decode kernels make at their teardown; the wait must have
  // failed in every thread (whoever saw the limit first raised the flag for the others)
  if (threadIdx.x == 0 && abort_flag && returned_false == (int)blockDim.x) set_status(status, DEV_WAIT_EXPIRED);
}

}  // namespace

cudaError_t launch_wait_expiry_probe(int* status, unsigned long long limit_ns, cudaStream_t st) {
  wait_expiry_probe_kernel<<<1, 128, 0, st>>>(status, limit_ns);
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace pivot

// ------------------------------------------------------------------------------------------------
// mma_model_probe: what the tensor pipe, the tensor-memory port and the warp-to-warp hand-overs of
// one SM cost for the instruction shapes the scan and the re-score are built from -- the numbers
// the per-tile time model of those kernels rests on.  One CTA; thread 0 issues tcgen05.mma streams
// over zero operands (timing only), optionally while other warps keep the tensor-memory port busy
// the way the kernels' ReLU / score passes do.  Every wait is bounded.
namespace pivot {
namespace {

constexpr int PROBE_TILES = 64;

__device__ __forceinline__ void mma_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t acc, int kind) {
  if (kind == 0)
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
  else if (kind == 1)
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
  else
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

// issuer variants (per "tile"; buffers alternate between TMEM columns 0 and 256)
enum {
  V_M1_256 = 0,        // first MMA: fp8, N = 256, four K steps
  V_M1_192,            // N = 192 (three rows)
  V_M1_128x2,          // two N = 128 halves
  V_M2_BF16_16,        // second MMA: bf16 A in tensor memory, N = 16, sixteen K steps
  V_M2_BF16_8,         // ... eight K steps (two rows' worth)
  V_M2_F8_8,           // fp8 A in tensor memory, eight K steps of 32
  V_M2_I8_8,           // 8-bit integer A in tensor memory, eight K steps of 32
  V_M1_M2_BF16_16,     // alternating, as the scan issues them
  V_M1_M2_BF16_8,
  V_M1_M2_I8_8,
  V_M1_192_M2_I8_6,
  V_LIN_16,            // one fp8 MMA from shared memory, N = 16, four K steps (a linear-term column block)
  V_M1_LIN,            // first MMA + that
  V_COUNT
};

struct ProbeCtrl {
  uint64_t done[2 * V_COUNT + 8];
  uint64_t ping, pong;
  uint32_t tbase;
  int abort;
  volatile int traffic_on;
  volatile int traffic_kind;
  unsigned long long traffic_clk[8];
  unsigned int traffic_passes[8];
};

__global__ void __launch_bounds__(416, 1) mma_model_probe_kernel(long long* out) {
  extern __shared__ uint8_t raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  ProbeCtrl& ct = *reinterpret_cast<ProbeCtrl*>(smem + 16384 + 32768 + 8192);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < (16384 + 32768 + 8192) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0u;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2 * V_COUNT + 8; ++i) ptx::mbar_init(&ct.done[i], 1);
    ptx::mbar_init(&ct.ping, 1);
    ptx::mbar_init(&ct.pong, 1);
    ct.abort = 0; ct.traffic_on = 0; ct.traffic_kind = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 0) { ptx::tmem_alloc(&ct.tbase, 512); ptx::tmem_relinquish(); }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before(); __syncthreads(); ptx::tc_fence_after();
  const uint32_t tb = ct.tbase;
  volatile int* abort_flag = &ct.abort;

  // ---- phases: for traffic kind 0 (none), 1 (ReLU pass: load 32 columns, pack, store 16), 2 (loads only, as an
  //      fp32 head sum would) with 4 warps, 3 = kind 2 with 8 warps (two per lane quarter)
  for (int phase = 0; phase < 4; ++phase) {
    __syncthreads();
    if (threadIdx.x == 0) { ct.traffic_kind = phase; ct.traffic_on = phase ? 1 : 0; }
    __syncthreads();
    if (threadIdx.x == 0) {
      const uint32_t k_addr = ptx::smem_u32(smem), q_addr = k_addr + 16384, w_addr = q_addr + 32768;
      const uint32_t id256 = ptx::make_idesc(0u, 128, 256), id192 = ptx::make_idesc(0u, 128, 192);
      const uint32_t id128 = ptx::make_idesc(0u, 128, 128), id16f8 = ptx::make_idesc(0u, 128, 16);
      const uint32_t id2 = ptx::make_idesc(1u, 128, 16);
      const uint32_t idi8 = (2u << 4) | (0u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);   // s32 += u8 x s8
      auto m1 = [&](uint32_t d, uint32_t idesc, uint32_t qoff) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          ptx::tc_mma<true>(d, ptx::smem_desc_sw128(k_addr + ks * 32), ptx::smem_desc_sw128(q_addr + qoff + ks * 32), idesc,
                            ks ? 1u : 0u);
      };
      auto m2 = [&](uint32_t d, uint32_t a, int n, uint32_t idesc, int kind) {
        for (int j = 0; j < n; ++j)
          mma_a_tmem(d, a + j * 8, ptx::smem_desc_sw128(w_addr + (j >> 2) * 2048 + (j & 3) * 32), idesc, j ? 1u : 0u, kind);
      };
      for (int v = 0; v < V_COUNT; ++v) {
        const long long t0 = clock64();
        for (int r = 0; r < PROBE_TILES; ++r) {
          const uint32_t buf = tb + (r & 1) * 256, other = buf ^ 256;
          switch (v) {
            case V_M1_256: m1(buf, id256, 0); break;
            case V_M1_192: m1(buf, id192, 0); break;
            case V_M1_128x2: m1(buf, id128, 0); m1(buf + 128, id128, 16384); break;
            case V_M2_BF16_16: m2(buf + 128, buf, 16, id2, 0); break;
            case V_M2_BF16_8: m2(buf + 128, buf, 8, id2, 0); break;
            case V_M2_F8_8: m2(buf + 128, buf, 8, id16f8, 1); break;
            case V_M2_I8_8: m2(buf + 128, buf, 8, idi8, 2); break;
            case V_M1_M2_BF16_16: m1(buf, id256, 0); m2(other + 128, other, 16, id2, 0); break;
            case V_M1_M2_BF16_8: m1(buf, id256, 0); m2(other + 128, other, 8, id2, 0); break;
            case V_M1_M2_I8_8: m1(buf, id256, 0); m2(other + 128, other, 8, idi8, 2); break;
            case V_M1_192_M2_I8_6: m1(buf, id192, 0); m2(other + 192, other, 6, idi8, 2); break;
            case V_LIN_16: m1(buf + 240, id16f8, 0); break;
            case V_M1_LIN: m1(buf, id256, 0); m1(other + 240, id16f8, 0); break;
          }
        }
        uint64_t* bar = &ct.done[(phase & 1) * V_COUNT + v];
        const uint32_t parity = (phase >> 1) & 1;
        ptx::tc_commit(bar);
        (void)ptx::mbar_wait(bar, parity, abort_flag);
        out[phase * 32 + v] = (clock64() - t0) / PROBE_TILES;
      }
      ct.traffic_on = 0;
    } else if (warp >= 4 && warp < 12) {
      // ---- tensor-memory traffic on this warp's lane quarter while the issuer runs
      const int tw = warp - 4;
      const uint32_t lq = (uint32_t)(warp & 3);
      const uint32_t xb0 = tb + ((lq * 32u) << 16);
      unsigned int passes = 0;
      const int kind = ct.traffic_kind;
      const bool active = kind == 1 ? tw < 4 : kind == 2 ? tw < 4 : kind == 3;
      const long long t0 = clock64();
      uint32_t sink = 0;
      while (active && ct.traffic_on && !*abort_flag) {
        const uint32_t xb = xb0 + (passes & 1) * 256;
        uint32_t va[32];
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          ptx::tmem_ld_32x32(xb + c * 32, va);
          ptx::tmem_wait_ld();
          if (kind == 1) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = ptx::relu_pack_bf16x2(__uint_as_float(va[2 * i]), __uint_as_float(va[2 * i + 1]));
            ptx::tmem_st_32x16(xb + c * 16, pk);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) sink ^= va[i];
          }
        }
        if (kind == 1) ptx::tmem_wait_st();
        ++passes;
        if (passes > 2000000u) break;
      }
      if (lane == 0 && active) {
        ct.traffic_clk[tw] = (unsigned long long)(clock64() - t0);
        ct.traffic_passes[tw] = passes;
      }
      if (sink == 0x12345678u) out[255] = sink;
    }
    __syncthreads();
    if (threadIdx.x < 8 && phase) {
      const unsigned int n = ct.traffic_passes[threadIdx.x];
      out[phase * 32 + 16 + threadIdx.x] = n ? (long long)(ct.traffic_clk[threadIdx.x] / n) : 0;
      ct.traffic_passes[threadIdx.x] = 0;
    }
  }
  __syncthreads();

  // ---- hand-over latency: warp 1 (lane 0) and warp 2 (lane 0) bounce an mbarrier pair
  {
    constexpr int ROUNDS = 256;
    for (int mode = 0; mode < 2; ++mode) {          // 0: try_wait polls, 1: test_wait polls
      __syncthreads();
      if (threadIdx.x == 32) {
        const long long t0 = clock64();
        for (int r = 0; r < ROUNDS; ++r) {
          const uint32_t ph = (uint32_t)((mode * ROUNDS + r) & 1);
          ptx::mbar_arrive(&ct.ping);
          if (mode == 0) (void)ptx::mbar_wait(&ct.pong, ph, abort_flag);
          else (void)ptx::mbar_wait_poll(&ct.pong, ph, abort_flag);
        }
        out[128 + mode] = (clock64() - t0) / (2 * ROUNDS);      // one way
      } else if (threadIdx.x == 64) {
        for (int r = 0; r < ROUNDS; ++r) {
          const uint32_t ph = (uint32_t)((mode * ROUNDS + r) & 1);
          if (mode == 0) (void)ptx::mbar_wait(&ct.ping, ph, abort_flag);
          else (void)ptx::mbar_wait_poll(&ct.ping, ph, abort_flag);
          ptx::mbar_arrive(&ct.pong);
        }
      }
    }
    __syncthreads();
    // tcgen05.commit -> waiting thread: an empty commit (nothing outstanding) bounced back by a plain arrive
    if (threadIdx.x == 0) {
      const long long t0 = clock64();
      for (int r = 0; r < ROUNDS; ++r) {
        const uint32_t ph = (uint32_t)(r & 1);      // ping / pong have each completed 2 * ROUNDS phases
        ptx::tc_commit(&ct.ping);
        (void)ptx::mbar_wait_poll(&ct.pong, ph, abort_flag);
      }
      out[130] = (clock64() - t0) / ROUNDS;           // commit -> other thread -> back
    } else if (threadIdx.x == 64) {
      for (int r = 0; r < ROUNDS; ++r) {
        const uint32_t ph = (uint32_t)(r & 1);
        (void)ptx::mbar_wait_poll(&ct.ping, ph, abort_flag);
        ptx::mbar_arrive(&ct.pong);
      }
    }
  }
  ptx::tc_fence_before(); __syncthreads(); ptx::tc_fence_after();
  if (warp == 0) ptx::tmem_dealloc(tb, 512);
  if (threadIdx.x == 0) out[254] = ct.abort;
}

}  // namespace

// Key-tile streaming alone: every CTA pulls 16 KB key tiles (128 keys x 128 B, the scan's TMA box) of
// one L2-resident key tensor through a ring of `stages` shared-memory stages and does nothing with
// them -- the rate at which L2 can feed all SMs the scan's key stream.  Each CTA starts at its own
// offset and walks `tiles` consecutive tiles (wrapping), as the scan's CTAs do.
__global__ void __launch_bounds__(160, 1) key_stream_probe_kernel(const __grid_constant__ CUtensorMap tm_k, const uint8_t* keys,
                                                                  int n_tiles_total, int tiles, int stages, int mode,
                                                                  long long* out) {
  // mode 0: one TMA ring (warp 0).  mode 1: a second, independent TMA ring on warp 1.  mode 2: warp 0's
  // TMA ring plus warps 1-4 streaming other tiles with 16-byte cp.async (the load/store unit's path).
  extern __shared__ uint8_t raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full[2][12];
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 24; ++i) ptx::mbar_init(&full[0][0] + i, 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int start = (int)(((long long)blockIdx.x * 977) % n_tiles_total);
  if (mode < 3 && (warp == 0 || (warp == 1 && mode == 1)) && lane == 0) {
    ptx::prefetch_tensormap(&tm_k);
    uint8_t* ring = smem + warp * stages * 16384;
    const int first = start + warp * (n_tiles_total / 2);
    auto issue = [&](int t) {
      const int s = t % stages;
      ptx::mbar_arrive_expect_tx(&full[warp][s], 16384);
      ptx::tma_load_2d(ring + s * 16384, &tm_k, 0, ((first + t) % n_tiles_total) * 128, &full[warp][s]);
    };
    for (int t = 0; t < stages && t < tiles; ++t) issue(t);
    const long long t0 = clock64();
    for (int t = 0; t < tiles; ++t) {
      const int s = t % stages;
      if (!ptx::mbar_wait_poll(&full[warp][s], (uint32_t)((t / stages) & 1), &abort_flag)) break;
      if (t + stages < tiles) issue(t + stages);
    }
    out[blockIdx.x * 2 + warp] = (clock64() - t0) / tiles;
    if (abort_flag) out[blockIdx.x * 2 + warp] = -1;
  } else if (mode >= 3 && warp == 0 && (lane == 0 || (mode == 4 && lane < 4))) {
    // mode 3: one thread issues the tile as four boxes of 32 keys; mode 4: four lanes issue one box each
    ptx::prefetch_tensormap(&tm_k);
    auto issue = [&](int t) {
      const int s = t % stages;
      if (lane == 0) ptx::mbar_arrive_expect_tx(&full[0][s], 16384);
      __syncwarp(mode == 4 ? 0xfu : 0x1u);
      for (int i = (mode == 4 ? lane : 0); i < 4; i += (mode == 4 ? 4 : 1))
        ptx::tma_load_2d(smem + s * 16384 + i * 4096, &tm_k, 0, ((start + t) % n_tiles_total) * 128 + i * 32, &full[0][s]);
    };
    for (int t = 0; t < stages && t < tiles; ++t) issue(t);
    const long long t0 = clock64();
    for (int t = 0; t < tiles; ++t) {
      const int s = t % stages;
      if (!ptx::mbar_wait_poll(&full[0][s], (uint32_t)((t / stages) & 1), &abort_flag)) break;
      if (t + stages < tiles) issue(t + stages);
    }
    if (lane == 0) out[blockIdx.x * 2] = (clock64() - t0) / tiles;
  } else if (mode == 2 && warp >= 1) {
    // four warps share the second stream: warp w copies quarter w of every tile
    uint8_t* ring = smem + stages * 16384;
    const int first = start + n_tiles_total / 2;
    const int wq = warp - 1;
    const long long t0 = clock64();
    for (int t = 0; t < tiles; ++t) {
      const uint8_t* src = keys + (size_t)((first + t) % n_tiles_total) * 16384 + wq * 4096;
      const uint32_t dst = ptx::smem_u32(ring + (t % stages) * 16384 + wq * 4096);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (i * 32 + lane) * 16), "l"(src + (i * 32 + lane) * 16)
                     : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 3;" ::: "memory");
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (lane == 0 && wq == 0) out[blockIdx.x * 2 + 1] = (clock64() - t0) / tiles;
  }
}

// out: 256 long longs (device).  [phase * 32 + variant] = tensor-pipe clocks per tile for the issuer variants
// (phase 0 alone, 1 with ReLU-pass traffic, 2 with load-only traffic from 4 warps, 3 from 8 warps);
// [phase * 32 + 16 + w] = clocks per 256-column pass of traffic warp w; [128], [129] one-way mbarrier
// hand-over with try_wait / test_wait polls; [130] commit round trip; [254] abort flag.
cudaError_t launch_mma_model_probe(long long* out, cudaStream_t st) {
  const size_t smem = 1024 + 16384 + 32768 + 8192 + sizeof(ProbeCtrl);
  static bool attr[kMaxDevices] = {};
  if (cudaError_t e = opt_in_dynamic_smem(mma_model_probe_kernel, smem, attr); e != cudaSuccess) return e;
  mma_model_probe_kernel<<<1, 416, smem, st>>>(out);
  ++launch_counter();
  return cudaGetLastError();
}

bool make_operand_map(CUtensorMap* m, const void* base, long long rows, int dtype, int box_rows, int row_stride);

// keys: an FP8 key tensor [n_keys, 128] (device), n_keys a multiple of 128; out: one slot per CTA
// (clocks per tile seen by that CTA's first and, with mode 1 / 2, second stream: out[2 cta], out[2 cta + 1]).
cudaError_t launch_key_stream_probe(const void* keys, int n_keys, int ctas, int tiles, int stages, int mode, long long* out,
                                    cudaStream_t st) {
  if (mode < 0 || mode > 4 || ((mode == 1 || mode == 2) && stages > 6)) return cudaErrorInvalidValue;
  if (stages < 1 || stages > 12 || n_keys < 128 || (n_keys & 127) || ctas < 1 || tiles < 1) return cudaErrorInvalidValue;
  CUtensorMap mk;
  if (!make_operand_map(&mk, keys, n_keys, DT_FP8, mode >= 3 ? 32 : 128, 0)) return cudaErrorInvalidValue;
  const size_t smem = 1024 + (size_t)stages * 16384 * ((mode == 1 || mode == 2) ? 2 : 1);
  if (cudaError_t e = cudaFuncSetAttribute(key_stream_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e != cudaSuccess)
    return e;
  key_stream_probe_kernel<<<ctas, 160, smem, st>>>(mk, (const uint8_t*)keys, n_keys / 128, tiles, stages, mode, out);
  ++launch_counter();
  return cudaGetLastError();
}

}  // namespace pivot
