// Chunk-scan carry of the prefill for bf16 I/O and d = 128 on the tensor cores, at fp32 accuracy:
//   S += phi(K')^T V',  z += sum phi(K')      over the chunk's delayed tokens (k'_i = k_{i-w}).
// V' is bf16 already.  phi(K') is fp32 in the chunk scratch; every value is split into three bf16 terms
// (x = hi + mid + lo, each the bf16 rounding of what the previous ones left: an error-free split of the 24-bit
// significand), so the three products phi_term^T V' are exact in fp32 and only the fp32 accumulation of the tensor
// core rounds.  The carry therefore stays an fp32 quantity, as the method's chunk scan requires, while the
// 2 C d^2 multiply-adds per KV head leave the CUDA cores (a bf16 or tf32 product of phi(K') itself would miss the
// 1e-5 state tolerance).  z is summed in fp32 on the CUDA cores from the same staged values.
//
// One CTA of 4 warps per (unit, 64 state rows); warp w owns rows 16 w .. 16 w + 15 and all 128 columns
// (16 n-tiles of m16n8k16, 64 accumulators per thread).  Tokens are staged 32 at a time through two shared-memory
// buffers filled by cp.async; row strides are padded (272 bytes) so that the scalar reads of the A fragments and
// the ldmatrix reads of V' are free of bank conflicts.
#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kThreads = 128;
constexpr int kRowsPerCta = 64;
constexpr int kTok = 32;                      // tokens per stage
constexpr int kPhiStride = 68;                // floats per staged phi row (64 + 4: conflict-free fragment reads)
constexpr int kVStride = 272;                 // bytes per staged V' row (256 + 16: conflict-free ldmatrix)
constexpr int kPhiBytes = kTok * kPhiStride * 4;
constexpr int kVBytes = kTok * kVStride;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp16(uint32_t dst, const void *src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0: writes zeros, reads nothing
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// x0, x1 -> three packed bf16 pairs (x0 in the low half) whose sums give x0, x1 back to fp32 accuracy
__device__ __forceinline__ void split3(float x0, float x1, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  const float r0 = x0 - __low2float(h), r1 = x1 - __high2float(h);
  const __nv_bfloat162 m = __floats2bfloat162_rn(r0, r1);
  const float s0 = r0 - __low2float(m), s1 = r1 - __high2float(m);
  const __nv_bfloat162 l = __floats2bfloat162_rn(s0, s1);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  mid = *reinterpret_cast<const uint32_t *>(&m);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

__global__ void __launch_bounds__(kThreads) prefill_state_mma_kernel(const PrefillParams p) {
  using bf16 = __nv_bfloat16;
  __shared__ __align__(16) unsigned char stage[2][kPhiBytes + kVBytes];
  const int blocks_per_unit = p.dp / kRowsPerCta;   // rows of S: d, or 2 d with the learned feature map
  const int64_t u = blockIdx.x / blocks_per_unit;
  const int rb = blockIdx.x % blocks_per_unit;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const int64_t first = p.n0 + p.c0 - ld.wlin;    // delayed token of chunk index 0
  const int i_lo = first < 0 ? int(first < -int64_t(p.C) ? p.C : -first) : 0;
  if (i_lo >= p.C) return;
  const int ub = (b + p.b0) * p.Hkv + g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  // V' rows: the ring for tokens older than the call, the call's own rows otherwise
  const int64_t cap = ld.cap > 0 ? ld.cap : 1;
  const bf16 *ringV = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + size_t(ub) * size_t(ld.cap) * kD;
  const bf16 *callV = reinterpret_cast<const bf16 *>(p.v) + ((size_t(lrel) * p.B + b) * size_t(p.T) * p.Hkv + g) * kD;
  const int64_t call_stride = int64_t(p.Hkv) * kD;
  const float *pk = p.phik + size_t(u) * p.Cmax * p.dp + rb * kRowsPerCta;

  float acc[kD / 8][4];
#pragma unroll
  for (int n = 0; n < kD / 8; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  float zacc = 0.f;   // threads 0..63: z of row rb*64 + tid

  // tokens past the chunk's end are filled with zeros
  auto issue = [&](int buf, int i0) {
    const int nt = min(kTok, p.C - i0);
    const uint32_t sphi = smem_addr(stage[buf]), sv = sphi + kPhiBytes;
    for (int e = tid; e < kTok * (kRowsPerCta / 4); e += kThreads) {
      const int i = e / (kRowsPerCta / 4), c4 = e % (kRowsPerCta / 4);
      cp16(sphi + uint32_t(i * kPhiStride + c4 * 4) * 4u, pk + size_t(i0 + (i < nt ? i : 0)) * p.dp + c4 * 4, i < nt);
    }
    for (int e = tid; e < kTok * 16; e += kThreads) {
      const int i = e >> 4, c = e & 15;
      const int64_t j = first + i0 + (i < nt ? i : 0);
      const bf16 *row = j >= p.n0 ? callV + (j - p.n0) * call_stride : ringV + (j % cap) * kD;
      cp16(sv + uint32_t(i * kVStride + c * 16), row + c * 8, i < nt);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  issue(0, i_lo);
  int buf = 0;
  for (int i0 = i_lo; i0 < p.C; i0 += kTok, buf ^= 1) {
    if (i0 + kTok < p.C) {
      issue(buf ^ 1, i0 + kTok);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const float *sphi = reinterpret_cast<const float *>(stage[buf]);
    const uint32_t sv = smem_addr(stage[buf]) + kPhiBytes;
#pragma unroll
    for (int kk = 0; kk < kTok / 16; ++kk) {
      // A = phi(K')^T: element (row r, k i) = phi(k'_i)[r]; fragment registers a0: (gid, 2 tig + {0,1}),
      // a1: (gid + 8, ..), a2: (gid, 2 tig + 8 + {0,1}), a3: (gid + 8, ..)
      const float *base = sphi + (kk * 16 + 2 * tig) * kPhiStride + warp * 16 + gid;
      uint32_t ah[4], am[4], al[4];
      split3(base[0], base[kPhiStride], ah[0], am[0], al[0]);
      split3(base[8], base[kPhiStride + 8], ah[1], am[1], al[1]);
      split3(base[8 * kPhiStride], base[9 * kPhiStride], ah[2], am[2], al[2]);
      split3(base[8 * kPhiStride + 8], base[9 * kPhiStride + 8], ah[3], am[3], al[3]);
      const int krow = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int dp = 0; dp < kD / 16; ++dp) {
        uint32_t bfr[4];
        ldsm_x4_trans(bfr, sv + uint32_t(krow * kVStride + (2 * dp + (lane >> 4)) * 16));
        // smallest terms first
        mma16816(acc[2 * dp], al, bfr[0], bfr[1]);
        mma16816(acc[2 * dp + 1], al, bfr[2], bfr[3]);
        mma16816(acc[2 * dp], am, bfr[0], bfr[1]);
        mma16816(acc[2 * dp + 1], am, bfr[2], bfr[3]);
        mma16816(acc[2 * dp], ah, bfr[0], bfr[1]);
        mma16816(acc[2 * dp + 1], ah, bfr[2], bfr[3]);
      }
    }
    if (tid < kRowsPerCta) {
#pragma unroll 8
      for (int i = 0; i < kTok; ++i) zacc += sphi[i * kPhiStride + tid];
    }
    __syncthreads();   // the stage is refilled by the next iteration's issue
  }
  // accumulator fragment: c0, c1 -> (row gid, cols 2 tig + {0,1}); c2, c3 -> row gid + 8
  float *Sb = reinterpret_cast<float *>(p.ws + ld.S) + size_t(ub) * p.dp * kD + size_t(rb * kRowsPerCta + warp * 16) * kD;
#pragma unroll
  for (int n = 0; n < kD / 8; ++n) {
    float2 *d0 = reinterpret_cast<float2 *>(Sb + size_t(gid) * kD + n * 8 + 2 * tig);
    float2 *d1 = reinterpret_cast<float2 *>(Sb + size_t(gid + 8) * kD + n * 8 + 2 * tig);
    float2 c0 = *d0, c1 = *d1;
    c0.x += acc[n][0];
    c0.y += acc[n][1];
    c1.x += acc[n][2];
    c1.y += acc[n][3];
    *d0 = c0;
    *d1 = c1;
  }
  if (tid < kRowsPerCta) {
    float *zb = reinterpret_cast<float *>(p.ws + ld.z) + size_t(ub) * p.dp + rb * kRowsPerCta;
    zb[tid] += zacc;
  }
}

}  // namespace

bool prefill_state_mma_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD;
}

int launch_prefill_state_mma(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream) {
  (void)ctx;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  prefill_state_mma_kernel<<<unsigned(units * (p.dp / kRowsPerCta)), kThreads, 0, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? GLIDE_OK : GLIDE_ERR_CUDA;
}

}  // namespace glide
