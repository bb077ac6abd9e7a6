// Causal softmax attention inside the sequences of a packed batch, head size 128, on the
// tcgen05 tensor cores (forward only; the gradients use the CUDA-core kernels of attention.cuh).
//
// One CTA = one tile of 128 query rows of one head.  It walks the key rows from the first row of
// the tile's first sequence to the tile's last row in blocks of 128:
//   warp 0 (one lane)  TMA producer: Q once; K and V blocks through a ring of two stages
//   warp 1 (one lane)  MMA issuer:   S = Q K^T into tensor memory (columns 0..127), then, once the
//                                    softmax warps have left P in shared memory, O_blk = P V into
//                                    columns 128..255
//   warps 2..5         softmax:      thread = query row.  Reads S twice from tensor memory (row
//                                    maximum, then exponentials), masks (same sequence, key <= query),
//                                    writes P as bf16 in the K-major swizzled operand layout, then
//                                    adds O_blk into its 128 fp32 output registers, rescaled by
//                                    exp2(m_old - m_new) (online softmax; nothing is rescaled in
//                                    tensor memory).
// Scores are kept in the log2 domain (scale * log2 e folded into one factor).  A row's sequence is
// given per row (seq_start), so a tile may span several sequences: keys before the row's own
// sequence are masked like keys after the row.  Every mbarrier wait is bounded; a wait that runs
// out sets the CTA's abort flag and a device status word, and the CTA leaves through the common
// exit that frees its tensor memory.
#pragma once

#include "gemm_tcgen05.cuh"
#include "ptx.cuh"

namespace mlora {
namespace attn_tc {

constexpr int BM = 128, BN = 128, DH = 128;
constexpr int THREADS = 192;
constexpr int STAGES = 2;
constexpr uint32_t Q_BYTES = BM * DH * 2;     // two 64-wide K-blocks of [128 rows][128 B]
constexpr uint32_t K_BYTES = BN * DH * 2;     // the same for 128 keys
constexpr uint32_t V_BYTES = BN * DH * 2;     // two blocks of 64 keys, each 2 x [64 keys][64 columns] (MN-major operand)
constexpr uint32_t P_BYTES = BM * BN * 2;     // two 64-key K-blocks of [128 rows][128 B]
constexpr uint32_t SMEM_BYTES = 1024 + Q_BYTES + STAGES * (K_BYTES + V_BYTES) + P_BYTES + 256;
constexpr uint32_t TMEM_COLS = 256;

__device__ int32_t g_status;                  // MLORA_ERR_DEVICE_TIMEOUT once a bounded wait ran out

struct Args {
  __nv_bfloat16* o;
  int64_t ldo;
  float* lse;                    // [n_rows, n_heads]
  const int32_t* seq_start;      // [n_rows]
  int32_t n_rows, n_heads, n_kv;
  float scale_log2;              // log2(e) / sqrt(d_head)
};

__global__ void __launch_bounds__(THREADS, 1)
forward_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const Args a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  const uint32_t sQ = base;
  auto sK = [&](int s) { return base + Q_BYTES + (uint32_t)s * (K_BYTES + V_BYTES); };
  auto sV = [&](int s) { return sK(s) + K_BYTES; };
  const uint32_t sP = base + Q_BYTES + STAGES * (K_BYTES + V_BYTES);
  const uint32_t sBar = sP + P_BYTES;
  const uint32_t bar_q = sBar, bar_s = sBar + 8, bar_p = sBar + 16, bar_o = sBar + 24;
  auto bar_kv_full = [&](int s) { return sBar + 32u + 8u * s; };
  auto bar_kv_empty = [&](int s) { return sBar + 48u + 8u * s; };
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(gen + (sBar - base) + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (sBar - base) + 72);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * BM, h = blockIdx.y;
  const int hk = h / (a.n_heads / a.n_kv);
  const int row_last = min(m0 + BM, a.n_rows) - 1;
  const int kmin = a.seq_start[m0];                       // rows and sequences ascend together
  const int nblk = (row_last - kmin) / BN + 1;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_q, 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_p, BM);
    ptx::mbar_init(bar_o, 1);
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(bar_kv_full(s), 1); ptx::mbar_init(bar_kv_empty(s), 1); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ);
    ptx::prefetch_tmap(&tmK);
    ptx::prefetch_tmap(&tmV);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    // ============================ TMA producer ============================
    if (lane == 0) {
      ptx::mbar_arrive_expect_tx(bar_q, Q_BYTES);
      ptx::tma_load_2d(sQ, &tmQ, h * DH, m0, bar_q);
      ptx::tma_load_2d(sQ + 16384, &tmQ, h * DH + 64, m0, bar_q);
      for (int j = 0; j < nblk; ++j) {
        const int s = j % STAGES;
        if (!gemm_wait(bar_kv_empty(s), ((j / STAGES) & 1) ^ 1, abort_flag, &g_status)) break;
        const int key0 = kmin + j * BN;
        ptx::mbar_arrive_expect_tx(bar_kv_full(s), K_BYTES + V_BYTES);
        ptx::tma_load_2d(sK(s), &tmK, hk * DH, key0, bar_kv_full(s));
        ptx::tma_load_2d(sK(s) + 16384, &tmK, hk * DH + 64, key0, bar_kv_full(s));
        ptx::tma_load_3d(sV(s), &tmV, 0, key0, (hk * DH) >> 6, bar_kv_full(s));
        ptx::tma_load_3d(sV(s) + 16384, &tmV, 0, key0 + 64, (hk * DH) >> 6, bar_kv_full(s));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ============================ MMA issuer ============================
    if (lane == 0) {
      constexpr uint32_t idesc_s = ptx::make_idesc_bf16(BM, BN, false, false);   // Q and K both K-major
      constexpr uint32_t idesc_o = ptx::make_idesc_bf16(BM, DH, false, true);    // V: keys are its K-rows
      const uint32_t tS = tmem_base, tO = tmem_base + BN;
      bool ok = gemm_wait(bar_q, 0, abort_flag, &g_status);
      for (int j = 0; j < nblk && ok; ++j) {
        const int s = j % STAGES;
        if (!(ok = gemm_wait(bar_kv_full(s), (j / STAGES) & 1, abort_flag, &g_status))) break;
        ptx::tc_fence_after();
        uint32_t acc = 0;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t ad = ptx::make_smem_desc(sQ + kb * 16384, 16, 1024);
          const uint64_t bd = ptx::make_smem_desc(sK(s) + kb * 16384, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            ptx::umma_f16(tS, ad + (uint64_t)(ks * 2), bd + (uint64_t)(ks * 2), idesc_s, acc);
            acc = 1;
          }
        }
        ptx::umma_commit(bar_s);
        if (!(ok = gemm_wait(bar_p, j & 1, abort_flag, &g_status))) break;     // P in shared memory, S and O_blk read
        ptx::tc_fence_after();
        acc = 0;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t ad = ptx::make_smem_desc(sP + kb * 16384, 16, 1024);
          const uint64_t bd = ptx::make_smem_desc(sV(s) + kb * 16384, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            ptx::umma_f16(tO, ad + (uint64_t)(ks * 2), bd + (uint64_t)(ks * 128), idesc_o, acc);
            acc = 1;
          }
        }
        ptx::umma_commit(bar_o);
        ptx::umma_commit(bar_kv_empty(s));
      }
    }
    __syncwarp();
  } else {
    // ============================ softmax, one query row per thread ============================
    const int e = warp & 3;                         // the quarter of tensor memory this warp may read
    const int row = e * 32 + lane;
    const int i_abs = m0 + row;
    const bool row_ok = i_abs < a.n_rows;
    const int my_start = row_ok ? a.seq_start[i_abs] : 0x7fffffff;
    const uint32_t tS = tmem_base + ((uint32_t)(e * 32) << 16), tO = tS + BN;
    const uint32_t prow = sP + (uint32_t)row * 128u;
    float O[DH];
#pragma unroll
    for (int k = 0; k < DH; ++k) O[k] = 0.f;
    float m = -1e30f, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nblk; ++j) {
      const int key0 = kmin + j * BN;
      ok = __all_sync(0xffffffffu, gemm_wait(bar_s, j & 1, abort_flag, &g_status));   // one decision per warp:
      if (!ok) break;                                                                  // the loads below are warp-wide
      ptx::tc_fence_after();
      float mx = m;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tS + cc * 32, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          const int col = key0 + cc * 32 + k;
          const float sc = (col >= my_start && col <= i_abs) ? __uint_as_float(v[k]) * a.scale_log2 : -1e30f;
          mx = fmaxf(mx, sc);
        }
      }
      const float alpha = exp2f(m - mx);
      float rowsum = 0.f;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tS + cc * 32, v);
        ptx::tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int k = 0; k < 32; k += 2) {
          const int col = key0 + cc * 32 + k;
          const float p0 = (col >= my_start && col <= i_abs) ? exp2f(__uint_as_float(v[k]) * a.scale_log2 - mx) : 0.f;
          const float p1 = (col + 1 >= my_start && col + 1 <= i_abs) ? exp2f(__uint_as_float(v[k + 1]) * a.scale_log2 - mx) : 0.f;
          rowsum += p0 + p1;
          pk[k >> 1] = ptx::pack_bf16(p0, p1);
        }
        // columns 32 cc .. 32 cc + 31 of P: K-block cc / 2, 16-byte pieces 4 (cc % 2) .. + 3 of the row,
        // piece i stored at i ^ (row & 7) (the operand's 128-byte swizzle)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t pc = (uint32_t)((cc & 1) * 4 + q);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(prow + (uint32_t)(cc >> 1) * 16384u + ((pc ^ (uint32_t)(row & 7)) << 4)),
                       "r"(pk[4 * q]), "r"(pk[4 * q + 1]), "r"(pk[4 * q + 2]), "r"(pk[4 * q + 3]) : "memory");
        }
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_p);
      ok = __all_sync(0xffffffffu, gemm_wait(bar_o, j & 1, abort_flag, &g_status));
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tO + cc * 32, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 32; ++k) O[cc * 32 + k] = fmaf(O[cc * 32 + k], alpha, __uint_as_float(v[k]));
      }
      l = fmaf(l, alpha, rowsum);
      m = mx;
    }
    if (ok && row_ok) {
      const float inv = 1.0f / l;
      __nv_bfloat16* dst = a.o + (size_t)i_abs * a.ldo + (size_t)h * DH;
#pragma unroll
      for (int k = 0; k < DH; k += 8) {
        uint4 w;
        w.x = ptx::pack_bf16(O[k] * inv, O[k + 1] * inv);
        w.y = ptx::pack_bf16(O[k + 2] * inv, O[k + 3] * inv);
        w.z = ptx::pack_bf16(O[k + 4] * inv, O[k + 5] * inv);
        w.w = ptx::pack_bf16(O[k + 6] * inv, O[k + 7] * inv);
        *reinterpret_cast<uint4*>(dst + k) = w;
      }
      a.lse[(size_t)i_abs * a.n_heads + h] = (m + log2f(l)) * 0.6931471805599453f;
    }
  }

  // ============================ common exit ============================
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace attn_tc
}  // namespace mlora
