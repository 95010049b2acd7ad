// Time-batched feed-forward part of the backward pass on the 5th-generation tensor cores (tcgen05, TMEM).
//
//   out[(ts, b)][i] = sum_k W[i][k] * delta_{t0+1+ts}[b][k]        W = W_ff of the layer above, [N][K]
//
// for the (step, sample) pairs of a run of steps: a dense product with M = N rows of W, up to 128 pairs as
// columns and the whole of K contracted, i.e. a real GEMM (the one place on this path where the tensor pipe
// and not HBM sets the pace).  fp32 accuracy comes from three tf32 products per k-block, small terms first:
// x = hi + lo with hi = x cut to 10 mantissa bits and lo = (x - hi) cut likewise (hi + lo differs from x by
// less than 2^-20 |x|), D += W_lo d_hi + W_hi d_lo + W_hi d_hi with fp32 accumulators in tensor memory.
// The cutting is the tensor cores' own: a kind::tf32 operand is read as its 19 high bits (checked on the device:
// results are bit for bit the same with the operands cut beforehand), so the staged fp32 tile itself serves as hi and
// only lo = x - cut(x) is computed and written, to a second tile.
// The tensor cores do not round an accumulation to nearest, and the error of a long chain of accumulations into
// one accumulator grows with its length; so the work is spread over three accumulators, summed in fp32 at the
// end: one for the two small terms of every k-step (they are 2^-11 of the large one: their own rounding no longer
// matters) and two for the large term (even and odd k-steps), 512 accumulations each at K = 8192 instead of 3072.
//
// One CTA = 128 rows of W x one tile of <= 128 pairs.  Warp roles:
//   warp 0      one thread issues the tiled bulk copies (TMA, 128-byte swizzle) of a k-block of 32: the W tile
//               [128 rows][32 k] and the delta tile [pairs][32 k] (a 3-D box: k, sample, step)
//   warp 1      allocates tensor memory; one thread issues the tcgen05.mma instructions (12 per k-block) and
//               commits them to the mbarrier that frees the stage
//   warps 2-9   write lo = x - cut(x) of every staged value to a second tile; warps 2-5 later read the
//               accumulator back (tcgen05.ld: a warp reads the 32 lanes 32 (warp % 4) ..) and store it
// Per stage three mbarriers: bytes landed -> split done -> products done.  All waits are bounded; a wait that
// runs out raises STATUS_SYNC_TIMEOUT, every role leaves its loop, and tensor memory is still released.
#pragma once
#include "kernels.cuh"

namespace snnk {

constexpr int TCG_M = 128;        // rows of W per CTA (lanes of tensor memory)
constexpr int TCG_NMAX = 128;     // pairs per CTA at most (columns of an accumulator)
constexpr int TCG_TMEM_COLS = 512;   // three accumulators of 128 columns; allocations are powers of two
constexpr int TCG_KB = 32;        // contraction values per k-block: one 128-byte swizzle row of fp32
constexpr int TCG_STAGES = 3;
constexpr int TCG_MAX_KSPLIT = 4; // slices of the contraction range at most (layers with few row tiles)
constexpr int TCG_CONV_WARPS = 8;
constexpr int TCG_THREADS = 32 * (2 + TCG_CONV_WARPS);
constexpr uint32_t TCG_A_BYTES = TCG_M * TCG_KB * 4;       // 16 KB
constexpr uint32_t TCG_B_BYTES = TCG_NMAX * TCG_KB * 4;    // 16 KB
constexpr uint32_t TCG_STAGE_BYTES = 2 * TCG_A_BYTES + 2 * TCG_B_BYTES;
constexpr size_t TCG_SMEM_BYTES = 1024 + (size_t)TCG_STAGES * TCG_STAGE_BYTES + 256;   // alignment slack, stages, barriers

struct TcGemmParams {
  CUtensorMap map_w;       // W [N][K] fp32, box 32 k x 128 rows, 128-byte swizzle
  CUtensorMap map_d;       // delta of the run as [n_steps][B][K], box 32 k x B samples x steps_per_tile steps
  float* out;              // [k_split][n_steps * B][N]: one partial product per slice of the contraction range
  size_t out_stride;       // floats between the partial products
  int k_split;             // slices of the contraction range (whole k-blocks each); blockIdx.z selects one
  uint32_t* status;
  int N, K, B, n_steps;
  int steps_per_tile;      // steps whose pairs form one tile: steps_per_tile * B <= 128
  int n_cols;              // steps_per_tile * B rounded up to a multiple of 16: columns of the products
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t n_cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(n_cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled, groups of 8
// rows 1024 bytes apart: start address and offsets in units of 16 bytes, descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);   // start address
  d |= (uint64_t)1 << 16;                          // leading-dimension byte offset: not used by swizzled K-major tiles
  d |= (uint64_t)(1024 >> 4) << 32;                // stride between groups of 8 rows
  d |= (uint64_t)1 << 46;                          // descriptor version
  d |= (uint64_t)2 << 61;                          // 128-byte swizzle
  return d;
}
// Instruction descriptor of kind::tf32: fp32 accumulator, both operands tf32 and K-major, M x N.
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u), "r"(0u) : "memory");
}
// The mbarrier receives one arrival when all tensor-core operations issued so far by this thread are complete.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 columns of 32 bits: thread = lane of tensor memory, registers = consecutive columns.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- the kernel -----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TCG_THREADS, 1) ff_gemm_tc_kernel(const __grid_constant__ TcGemmParams p) {
  pdl_launch_dependents();
  extern __shared__ unsigned char s_tc_raw[];
  // 1024-byte aligned stages (the swizzle pattern repeats every 1024 bytes and descriptors assume that base)
  unsigned char* const s_base = s_tc_raw + ((1024u - (smem_u32(s_tc_raw) & 1023u)) & 1023u);
  uint64_t* const bars = reinterpret_cast<uint64_t*>(s_base + (size_t)TCG_STAGES * TCG_STAGE_BYTES);
  uint64_t* const bar_landed = bars;                      // [TCG_STAGES] bytes of a k-block have landed
  uint64_t* const bar_split = bars + TCG_STAGES;          // [TCG_STAGES] hi / lo tiles are ready
  uint64_t* const bar_free = bars + 2 * TCG_STAGES;       // [TCG_STAGES] the products that read the stage are complete
  uint64_t* const bar_acc = bars + 3 * TCG_STAGES;        // the accumulator is complete
  uint32_t* const s_tmem = reinterpret_cast<uint32_t*>(bars + 3 * TCG_STAGES + 1);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row0 = blockIdx.y * TCG_M, ts0 = blockIdx.x * p.steps_per_tile;
  // this CTA's slice of the contraction range, in k-blocks [kb0, kb0 + n_kb)
  const int n_kb_all = (p.K + TCG_KB - 1) / TCG_KB;
  const int kb0 = (int)((long long)n_kb_all * blockIdx.z / p.k_split);
  const int n_kb = (int)((long long)n_kb_all * (blockIdx.z + 1) / p.k_split) - kb0;
  auto stage_a_hi = [&](int s) { return s_base + (size_t)s * TCG_STAGE_BYTES; };
  auto stage_a_lo = [&](int s) { return s_base + (size_t)s * TCG_STAGE_BYTES + TCG_A_BYTES; };
  auto stage_b_hi = [&](int s) { return s_base + (size_t)s * TCG_STAGE_BYTES + 2 * TCG_A_BYTES; };
  auto stage_b_lo = [&](int s) { return s_base + (size_t)s * TCG_STAGE_BYTES + 2 * TCG_A_BYTES + TCG_B_BYTES; };

  if (tid == 0) {
    for (int s = 0; s < TCG_STAGES; ++s) {
      mbar_init(bar_landed + s, 1);
      mbar_init(bar_split + s, TCG_CONV_WARPS);
      mbar_init(bar_free + s, 1);
    }
    mbar_init(bar_acc, 1);
    mbar_fence_init();
  }
  if (warp == 1) {   // tensor memory: three 128 x n_cols fp32 accumulators, 128 columns apart
    tmem_alloc(s_tmem, TCG_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_acc = *s_tmem;
  pdl_wait();

  // bytes a k-block brings: the boxes are always transferred whole (parts outside the tensors arrive as zeros)
  const uint32_t tx_bytes = TCG_A_BYTES + (uint32_t)(p.steps_per_tile * p.B) * TCG_KB * 4;
  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < n_kb; ++kb) {
        const int s = kb % TCG_STAGES;
        if (kb >= TCG_STAGES && !mbar_wait(bar_free + s, (uint32_t)(kb / TCG_STAGES - 1) & 1u)) {
          atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          break;
        }
        mbar_arrive_expect_tx(bar_landed + s, tx_bytes);
        tma_load_2d(stage_a_hi(s), &p.map_w, (kb0 + kb) * TCG_KB, row0, bar_landed + s);
        tma_load_3d(stage_b_hi(s), &p.map_d, (kb0 + kb) * TCG_KB, 0, ts0, bar_landed + s);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_tf32(TCG_M, p.n_cols);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % TCG_STAGES;
        ok = mbar_wait(bar_split + s, (uint32_t)(kb / TCG_STAGES) & 1u);
        if (!ok) { atomicOr(p.status, STATUS_SYNC_TIMEOUT); break; }
        tc_fence_after_sync();
        const uint32_t a_hi = smem_u32(stage_a_hi(s)), a_lo = smem_u32(stage_a_lo(s));
        const uint32_t b_hi = smem_u32(stage_b_hi(s)), b_lo = smem_u32(stage_b_lo(s));
#pragma unroll
        for (int j = 0; j < TCG_KB / 8; ++j) {   // k-steps of 8: 32 bytes further along the swizzled rows
          const uint32_t o = (uint32_t)j * 32u;
          const uint32_t acc_small = tmem_acc, acc_large = tmem_acc + (uint32_t)(1 + (j & 1)) * TCG_NMAX;
          umma_tf32(acc_small, umma_desc_sw128(a_lo + o), umma_desc_sw128(b_hi + o), idesc, kb > 0 || j > 0);
          umma_tf32(acc_small, umma_desc_sw128(a_hi + o), umma_desc_sw128(b_lo + o), idesc, true);
          umma_tf32(acc_large, umma_desc_sw128(a_hi + o), umma_desc_sw128(b_hi + o), idesc, kb > 0 || j > 1);
        }
        umma_commit(bar_free + s);            // the stage may be refilled once these products are complete
      }
      umma_commit(bar_acc);                   // ... and the accumulator read once all of them are
    }
  } else {
    // ---- split: every 16-byte piece of the landed tiles -> its lo piece in the second tile (same position: the
    // swizzle is a permutation of positions, the split is elementwise); the landed tile itself is read as hi
    const int ctid = tid - 64;   // 0 .. 255
    const int b_pieces = p.n_cols * (TCG_KB / 4);
    bool ok = true;
    for (int kb = 0; kb < n_kb && ok; ++kb) {
      const int s = kb % TCG_STAGES;
      ok = mbar_wait(bar_landed + s, (uint32_t)(kb / TCG_STAGES) & 1u);
      if (!ok) { if (lane == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT); break; }
      float4* const ah = reinterpret_cast<float4*>(stage_a_hi(s));
      float4* const al = reinterpret_cast<float4*>(stage_a_lo(s));
      float4* const bh = reinterpret_cast<float4*>(stage_b_hi(s));
      float4* const bl = reinterpret_cast<float4*>(stage_b_lo(s));
      auto cut = [](float v) { return __uint_as_float(__float_as_uint(v) & 0xffffe000u); };
      auto lo4 = [&](float4 x) {
        return make_float4(x.x - cut(x.x), x.y - cut(x.y), x.z - cut(x.z), x.w - cut(x.w));
      };
#pragma unroll
      for (int q = 0; q < (int)(TCG_A_BYTES / 16) / (32 * TCG_CONV_WARPS); ++q) {
        const int i = ctid + q * 32 * TCG_CONV_WARPS;
        al[i] = lo4(ah[i]);
      }
      for (int i = ctid; i < b_pieces; i += 32 * TCG_CONV_WARPS) {
        bl[i] = lo4(bh[i]);
      }
      fence_proxy_async_smem();   // these writes are read by the tensor cores (asynchronous proxy)
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_split + s);
    }
    // ---- epilogue (warps 2-5: lanes 32 (warp % 4) .. of tensor memory = rows of the tile)
    if (warp < 6) {
      if (ok && mbar_wait(bar_acc, 0u)) {
        tc_fence_after_sync();
        const int q = warp & 3;
        const int i = row0 + 32 * q + lane;
        const int pairs_here = min(p.steps_per_tile, p.n_steps - ts0) * p.B;   // valid columns of this tile
        float* const dst = p.out + (size_t)blockIdx.z * p.out_stride + (size_t)ts0 * p.B * p.N + i;
        for (int c0 = 0; c0 < p.n_cols; c0 += 32) {
          uint32_t small[32], even[32], odd[32];
          const uint32_t at = tmem_acc + ((uint32_t)(32 * q) << 16) + (uint32_t)c0;
          tmem_ld_32x32(at, small);
          tmem_ld_32x32(at + TCG_NMAX, even);
          tmem_ld_32x32(at + 2 * TCG_NMAX, odd);
          tmem_ld_wait();
          if (i < p.N) {
#pragma unroll
            for (int c = 0; c < 32; ++c)   // lanes: consecutive i; the three accumulators in a fixed order
              if (c0 + c < pairs_here)
                dst[(size_t)(c0 + c) * p.N] = (__uint_as_float(even[c]) + __uint_as_float(odd[c])) + __uint_as_float(small[c]);
          }
        }
      } else if (lane == 0) {
        atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, TCG_TMEM_COLS);
}

// Host side: the 3-D tensor map of the deltas of a run, [n_steps][B][K] with the steps slot_stride floats apart.
inline bool make_tensor_map_delta(CUtensorMap* out, const float* base, uint64_t K, uint64_t B, uint64_t n_steps,
                                  uint64_t slot_stride_floats, uint32_t box_steps) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_fn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
      cudaGetLastError();
      return false;
    }
    encode = reinterpret_cast<encode_fn>(fn);
  }
  const cuuint64_t dims[3] = {K, B, n_steps};
  const cuuint64_t strides[2] = {K * sizeof(float), slot_stride_floats * sizeof(float)};
  const cuuint32_t box[3] = {(cuuint32_t)TCG_KB, (cuuint32_t)B, box_steps};
  const cuuint32_t elem[3] = {1, 1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace snnk
