// Query preparation: RoPE on the elite chunks of q and absorption of B^k into the query
// (score equation of Section 3.1; Section 5 on folding B^k into the neighbouring product).
//
//   q_rope[b,h,2j:2j+2] = q[b,h,chunk idx[h][j]] . R(q_pos[b] * theta_idx[h][j])
//   q_abs [b,h,k]       = sum_i q_nope[b,h,i] * W_uk[k][h*dn + i]
//
// Grid (n_h, ceil(d_c/128) + 1).  A block of the first rows owns one head and 128 latent
// coordinates: per chunk of 16 sequences it computes the [16 x dn] . [dn x 128] product with
// mma.sync (m16n8k16, bf16 in, fp32 accumulate; both operands are bf16 already, so the products
// are exact), one warp per 16 coordinates.  The weights come regrouped as [n_h][dn][d_c]
// (d_c contiguous); the block's [dn x 128] slab is brought into shared memory by one bulk copy
// per weight row, all issued at once by one warp, so the slab costs one trip to memory and
// overlaps the gather of the queries.  The kernel is bound by latency, not by its 11 MB of
// traffic or its 0.2 GFLOP.  The blocks of the last grid row do the query RoPE (three dependent
// loads per element), off the path of the others.  d_c below is the width of the latent the
// scores read: the whole latent row, or the key latent d_ck when keys and values have latents of
// their own (S-LRD, Section 3.2).
#include "tc_ptx.cuh"

namespace {

constexpr int kAbsorbBatch = 16;       // sequences per MMA row tile
constexpr int kAbsorbThreads = 256;    // 8 warps x 16 coordinates
constexpr int kAbsorbCoords = 128;
constexpr int kAbsorbPitch = kAbsorbCoords + 8;   // slab row pitch: 16 bytes of padding spread the fragment loads over the banks

__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kAbsorbThreads)
absorb_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int B,
              const bf16* __restrict__ WukT, const int32_t* __restrict__ qdims,
              const int32_t* __restrict__ idx, const float2* __restrict__ cs, bf16* __restrict__ q_rope,
              bf16* __restrict__ q_abs, int n_h, int d_h, int r, int d_c, int max_pos,
              int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_b[];
  ekv_pdl_trigger();      // nothing later in the stream is held up by this kernel's start
  const int h = blockIdx.x;
  const int dn = d_h - 2 * r;
  const int kpad = (dn + 15) & ~15;                  // K of the product, zero-padded to 16
  const int qpitch = kpad + 8;                       // row pitch of the query tile (bank spread)
  bf16* s_w = (bf16*)smem_b;                         // [kpad][128 + 8] weight slab
  bf16* s_q = s_w + (size_t)kpad * kAbsorbPitch;    // [16][qpitch] un-rotated query dims
  bf16* s_raw = s_q + (size_t)kAbsorbBatch * qpitch;    // [16][d_h] whole query rows as they come (16-byte aligned: both sizes before it are multiples of 8 elements)
  int* s_dims = (int*)(s_raw + (size_t)kAbsorbBatch * d_h);   // [dn] query dim of every K index
  __shared__ __align__(8) uint64_t w_bar;
  __shared__ int s_abort;
  const bool rope_block = blockIdx.y == gridDim.y - 1;      // last grid row: query RoPE only
  const int32_t* dims = qdims + (size_t)h * d_h;

  if (rope_block) {
    for (int e = threadIdx.x; e < B * r; e += blockDim.x) {
      const int b = e / r, j = e % r;
      int p = q_pos[b];
      if (p < 0 || p >= max_pos) {
        ekv_record(status, ELITEKV_ERR_BAD_POSITION, b, p);
        p = 0;
      }
      const float2 w = cs[(size_t)p * (d_h / 2) + idx[h * r + j]];
      const bf16* qq = q + ((size_t)b * n_h + h) * d_h;
      const float x0 = __bfloat162float(qq[dims[2 * j]]), x1 = __bfloat162float(qq[dims[2 * j + 1]]);
      const float y0 = __fsub_rn(__fmul_rn(x0, w.x), __fmul_rn(x1, w.y));
      const float y1 = __fadd_rn(__fmul_rn(x0, w.y), __fmul_rn(x1, w.x));
      bf162* dst = (bf162*)(q_rope + ((size_t)b * n_h + h) * 2 * r + 2 * j);
      *dst = __floats2bfloat162_rn(y0, y1);
    }
    return;
  }

  const int k0 = blockIdx.y * kAbsorbCoords;
  const int kw = min(kAbsorbCoords, d_c - k0);       // coordinates of this slab (a multiple of 8)
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&w_bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();
  if (threadIdx.x < 32 && dn > 0) {
    if (threadIdx.x == 0) mbar_expect_tx(smem_u32(&w_bar), (uint32_t)(dn * kw * 2));
    __syncwarp();
    const bf16* src = WukT + (size_t)h * dn * d_c + k0;
    for (int i = threadIdx.x; i < dn; i += 32)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(s_w + (size_t)i * kAbsorbPitch)), "l"(src + (size_t)i * d_c), "r"(kw * 2),
                     "r"(smem_u32(&w_bar)) : "memory");
  }
  // rows of the slab past dn (K padding) are zeros
  for (int e = threadIdx.x; e < (kpad - dn) * (kAbsorbCoords / 8); e += blockDim.x)
    *(uint4*)(s_w + (size_t)(dn + e / (kAbsorbCoords / 8)) * kAbsorbPitch + (e % (kAbsorbCoords / 8)) * 8) =
        make_uint4(0, 0, 0, 0);
  bool w_ready = dn == 0;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;             // MMA fragment coordinates of this lane
  const int n0 = warp * 16;                          // first coordinate (inside the slab) of this warp
  for (int b0 = 0; b0 < B; b0 += kAbsorbBatch) {
    const int nb = min(kAbsorbBatch, B - b0);
    __syncthreads();
    // un-rotated query dims of 16 sequences, bf16 as they come; K padding and missing rows are
    // zeros.  The dim table and the query rows are fetched side by side (whole rows, 16-byte
    // loads) and the gather runs out of shared memory: one trip to memory instead of two
    // dependent ones.
    if (b0 == 0)
      for (int i = threadIdx.x; i < dn; i += blockDim.x) s_dims[i] = __ldg(dims + 2 * r + i);
    if ((d_h & 7) == 0) {
      for (int e = threadIdx.x; e < kAbsorbBatch * (d_h / 8); e += blockDim.x) {
        const int bb = e / (d_h / 8), v = e % (d_h / 8);
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (bb < nb) raw = __ldg((const uint4*)(q + ((size_t)(b0 + bb) * n_h + h) * d_h) + v);
        *(uint4*)(s_raw + (size_t)bb * d_h + v * 8) = raw;
      }
    } else {      // head dims that are not whole 16-byte units: element by element
      for (int e = threadIdx.x; e < kAbsorbBatch * d_h; e += blockDim.x) {
        const int bb = e / d_h, v = e % d_h;
        s_raw[e] = bb < nb ? q[((size_t)(b0 + bb) * n_h + h) * d_h + v] : __float2bfloat16_rn(0.f);
      }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kAbsorbBatch * kpad; e += blockDim.x) {
      const int bb = e / kpad, i = e % kpad;
      s_q[bb * qpitch + i] = i < dn ? s_raw[(size_t)bb * d_h + s_dims[i]] : __float2bfloat16_rn(0.f);
    }
    __syncthreads();
    if (!w_ready) {
      // the weight slab has landed (bounded wait; a timeout is recorded and the block leaves)
      volatile int* abort_flag = &s_abort;
      w_ready = mbar_wait(smem_u32(&w_bar), 0, abort_flag, 1);
      if (!w_ready) {
        if (threadIdx.x == 0) ekv_record(status, ELITEKV_ERR_TIMEOUT, h, blockIdx.y);
        return;
      }
    }
    if (n0 < kw) {
      float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      for (int kk = 0; kk < kpad; kk += 16) {
        // A fragment (16 sequences x 16 dims): rows g and g+8, dim pairs 2t and 2t+8
        uint32_t a[4];
        a[0] = *(const uint32_t*)(s_q + g * qpitch + kk + 2 * t);
        a[1] = *(const uint32_t*)(s_q + (g + 8) * qpitch + kk + 2 * t);
        a[2] = *(const uint32_t*)(s_q + g * qpitch + kk + 2 * t + 8);
        a[3] = *(const uint32_t*)(s_q + (g + 8) * qpitch + kk + 2 * t + 8);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          // B fragment (16 dims x 8 coordinates): coordinate g, dim pairs 2t and 2t+8
          const unsigned short* wp = (const unsigned short*)(s_w + (size_t)(kk + 2 * t) * kAbsorbPitch + n0 + nt * 8 + g);
          const uint32_t b0r = (uint32_t)wp[0] | ((uint32_t)wp[kAbsorbPitch] << 16);
          const uint32_t b1r = (uint32_t)wp[8 * kAbsorbPitch] | ((uint32_t)wp[9 * kAbsorbPitch] << 16);
          mma_bf16_16816(acc[nt], a, b0r, b1r);
        }
      }
      // C fragment: rows g and g+8, coordinates 2t and 2t+1 of each 8-wide tile
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int k = k0 + n0 + nt * 8 + 2 * t;
        if (k < d_c) {
          if (g < nb)
            *(bf162*)(q_abs + ((size_t)(b0 + g) * n_h + h) * d_c + k) = __floats2bfloat162_rn(acc[nt][0], acc[nt][1]);
          if (g + 8 < nb)
            *(bf162*)(q_abs + ((size_t)(b0 + g + 8) * n_h + h) * d_c + k) = __floats2bfloat162_rn(acc[nt][2], acc[nt][3]);
        }
      }
    }
  }
}

}  // namespace

int ekv_launch_absorb(const elitekv_layer* L, const void* q, const int32_t* q_pos, int B,
                      void* q_rope, void* q_abs, cudaStream_t st) {
  if (B == 0) return ELITEKV_OK;
  // the absorbed query spans the latent columns the scores read (all of them, or the key latent)
  dim3 grid(L->n_h, (L->kw + kAbsorbCoords - 1) / kAbsorbCoords + 1);   // + one row of rope blocks
  const int kpad = (L->dn + 15) & ~15;
  const size_t smem = sizeof(bf16) * ((size_t)kpad * kAbsorbPitch + (size_t)kAbsorbBatch * (kpad + 8) +
                                      (size_t)kAbsorbBatch * L->d_h) + sizeof(int) * (size_t)L->dn + 16;
  if ((int)smem > L->smem_optin || L->kw % 8 != 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  EKV_CUDA_OK(cudaFuncSetAttribute(absorb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  absorb_kernel<<<grid, kAbsorbThreads, smem, st>>>(
      (const bf16*)q, q_pos, B, L->d_WukT, L->d_qdims, L->d_idx, L->d_cs, (bf16*)q_rope,
      (bf16*)q_abs, L->n_h, L->d_h, L->r, L->kw, L->max_pos, L->d_status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
