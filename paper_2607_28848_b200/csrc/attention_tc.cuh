// Causal softmax attention inside the sequences of a packed batch, head size 128, on the
// tcgen05 tensor cores: the forward kernel first, the two gradient kernels after it (head size 64
// uses the CUDA-core kernels of attention.cuh).
//
// Forward: one CTA = one tile of 128 query rows of one head.  It walks the key rows from the first row of
// the tile's first sequence to the tile's last row in blocks of 128:
//   warp 0 (one lane)  TMA producer: Q once; K and V blocks through a ring of two stages
//   warp 1 (one lane)  MMA issuer:   S_j = Q K_j^T into one of two score buffers in tensor memory
//                                    (columns 0..127 / 128..255), issued one block ahead: S_{j+1} is
//                                    on the tensor pipe before P_j is waited for; then O_blk = P_j V_j
//                                    into columns 256..383
//   warps 2..9         softmax:      two threads per query row (warps w and w + 4 own the same 32 lanes of
//                                    tensor memory), each with 64 of the block's 128 keys and 64 of the 128
//                                    output columns.  A thread reads its half of S_j twice from tensor memory
//                                    (row maximum - exchanged with its partner through shared memory behind an
//                                    mbarrier of the warp pair - then exponentials), masks (same sequence,
//                                    key <= query) and keeps P_j as packed bf16 in 32 registers; only then it
//                                    takes the previous block's O_blk into its 64 fp32 output registers,
//                                    rescaled by exp2(m_old - m_new) (online softmax; nothing is rescaled in
//                                    tensor memory), and writes P_j in the K-major swizzled operand layout -
//                                    so the product P_{j-1} V_{j-1} and the scores S_{j+1} run on the tensor
//                                    pipe while the threads work on block j.
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
constexpr int FWD_THREADS = 64 + 256;         // forward: producer warp, MMA warp, eight softmax warps
constexpr uint32_t X_BYTES = 3 * 1024;        // forward: row maxima of the two halves (two blocks in flight) and the final row sums
constexpr uint32_t SMEM_BYTES = 1024 + Q_BYTES + STAGES * (K_BYTES + V_BYTES) + P_BYTES + 256 + X_BYTES;
constexpr uint32_t TMEM_COLS = 512;           // forward: S (two buffers of 128 columns), O_blk (128), 128 unused

// 2^x by the special-function unit (the arguments here are differences from a row maximum or a
// log-sum-exp, so nothing overflows; large negative arguments give 0)
__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ int32_t g_status;                  // MLORA_ERR_DEVICE_TIMEOUT once a bounded wait ran out

struct Args {
  __nv_bfloat16* o;
  int64_t ldo;
  float* lse;                    // [n_rows, n_heads]
  const int32_t* seq_start;      // [n_rows]
  int32_t n_rows, n_heads, n_kv;
  float scale_log2;              // log2(e) / sqrt(d_head)
};

__global__ void __launch_bounds__(FWD_THREADS, 1)
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
  const uint32_t bar_q = sBar, bar_p = sBar + 8, bar_o = sBar + 16;
  auto bar_s = [&](int j) { return sBar + 24u + 8u * (j & 1); };
  auto bar_kv_full = [&](int s) { return sBar + 40u + 8u * s; };
  auto bar_kv_empty = [&](int s) { return sBar + 56u + 8u * s; };
  auto bar_x = [&](int e) { return sBar + 72u + 8u * e; };      // one per pair of softmax warps (same 32 rows)
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(gen + (sBar - base) + 104);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (sBar - base) + 112);
  float* xch = reinterpret_cast<float*>(gen + (sBar - base) + 256);   // [3][2 halves][128 rows]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * BM, h = blockIdx.y;
  const int hk = h / (a.n_heads / a.n_kv);
  const int row_last = min(m0 + BM, a.n_rows) - 1;
  const int kmin = a.seq_start[m0];                       // rows and sequences ascend together
  const int nblk = (row_last - kmin) / BN + 1;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_q, 1);
    ptx::mbar_init(bar_s(0), 1);
    ptx::mbar_init(bar_s(1), 1);
    ptx::mbar_init(bar_p, 2 * BM);
    ptx::mbar_init(bar_o, 1);
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(bar_kv_full(s), 1); ptx::mbar_init(bar_kv_empty(s), 1); }
    for (int e = 0; e < 4; ++e) ptx::mbar_init(bar_x(e), 64);
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
      const uint32_t tO = tmem_base + 2 * BN;
      bool ok = gemm_wait(bar_q, 0, abort_flag, &g_status);
      // S_j = Q K_j^T into score buffer j & 1 (its previous reader, the softmax of block j - 2, was done
      // before P_{j-2} arrived, which this thread has waited for)
      auto issue_s = [&](int j) -> bool {
        const int s = j % STAGES;
        if (!gemm_wait(bar_kv_full(s), (j / STAGES) & 1, abort_flag, &g_status)) return false;
        ptx::tc_fence_after();
        const uint32_t tS = tmem_base + (uint32_t)(j & 1) * BN;
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
        ptx::umma_commit(bar_s(j));
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int j = 0; j < nblk && ok; ++j) {
        const int s = j % STAGES;
        if (j + 1 < nblk && !(ok = issue_s(j + 1))) break;                     // one block ahead of the softmax
        if (!(ok = gemm_wait(bar_p, j & 1, abort_flag, &g_status))) break;     // P_j in shared memory, S_j and O_blk of block j - 1 read
        ptx::tc_fence_after();
        uint32_t acc = 0;
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
    // ============================ softmax, two threads per query row ============================
    const int e = warp & 3;                         // the quarter of tensor memory this warp may read
    const int half = (warp - 2) >> 2;               // which 64 keys of a block and which 64 output columns
    const int row = e * 32 + lane;
    const int i_abs = m0 + row;
    const bool row_ok = i_abs < a.n_rows;
    const int my_start = row_ok ? a.seq_start[i_abs] : 0x7fffffff;
    const uint32_t tS0 = tmem_base + ((uint32_t)(e * 32) << 16) + (uint32_t)half * 64u;
    const uint32_t tO = tmem_base + ((uint32_t)(e * 32) << 16) + 2 * BN + (uint32_t)half * 64u;
    const uint32_t prow = sP + (uint32_t)half * 16384u + (uint32_t)row * 128u;       // K-block `half` of P
    float* x_mine = xch + half * BM + row;          // + 256 per slot
    const float* x_peer = xch + (half ^ 1) * BM + row;
    float O[DH / 2];
#pragma unroll
    for (int k = 0; k < DH / 2; ++k) O[k] = 0.f;
    float m = -1e30f, l = 0.f, alpha_prev = 1.f;    // l: the sum over this thread's keys only
    bool ok = true;
    // O += O_blk of one block, the sum so far rescaled to that block's running maximum
    auto take_o = [&](float alpha) {
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tO + cc * 32, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 32; ++k) O[cc * 32 + k] = fmaf(O[cc * 32 + k], alpha, __uint_as_float(v[k]));
      }
    };
    // value exchange between the two threads of a row: slot picks one of three buffers, phase counts the
    // uses of the pair's barrier
    auto exchange = [&](float mine, int slot, int phase, float& peer) -> bool {
      x_mine[slot * 2 * BM] = mine;
      ptx::mbar_arrive(bar_x(e));
      const bool got = __all_sync(0xffffffffu, gemm_wait(bar_x(e), phase & 1, abort_flag, &g_status));
      if (got) peer = x_peer[slot * 2 * BM];
      return got;
    };
    for (int j = 0; j < nblk; ++j) {
      const int key0 = kmin + j * BN + half * 64;
      const uint32_t tS = tS0 + (uint32_t)(j & 1) * BN;
      ok = __all_sync(0xffffffffu, gemm_wait(bar_s(j), (j >> 1) & 1, abort_flag, &g_status));   // one decision per warp:
      if (!ok) break;                                                                            // the loads below are warp-wide
      ptx::tc_fence_after();
      float mx = m;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
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
      float peer_mx;
      if (!(ok = exchange(mx, j & 1, j, peer_mx))) break;
      mx = fmaxf(mx, peer_mx);
      const float alpha = fast_ex2(m - mx);
      float rowsum = 0.f;
      uint32_t pk[32];
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tS + cc * 32, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 32; k += 2) {
          const int col = key0 + cc * 32 + k;
          const float p0 = (col >= my_start && col <= i_abs) ? fast_ex2(__uint_as_float(v[k]) * a.scale_log2 - mx) : 0.f;
          const float p1 = (col + 1 >= my_start && col + 1 <= i_abs) ? fast_ex2(__uint_as_float(v[k + 1]) * a.scale_log2 - mx) : 0.f;
          rowsum += p0 + p1;
          pk[cc * 16 + (k >> 1)] = ptx::pack_bf16(p0, p1);
        }
      }
      if (j > 0) {      // the previous block's P V ran while this block's scores were worked on
        ok = __all_sync(0xffffffffu, gemm_wait(bar_o, (j - 1) & 1, abort_flag, &g_status));
        if (!ok) break;
        ptx::tc_fence_after();
        take_o(alpha_prev);
      }
      // this thread's 64 keys are K-block `half` of P: eight 16-byte pieces of the row, piece i stored at
      // i ^ (row & 7) (the operand's 128-byte swizzle); the previous product has finished reading the buffer
#pragma unroll
      for (int pc = 0; pc < 8; ++pc)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(prow + (((uint32_t)pc ^ (uint32_t)(row & 7)) << 4)),
                     "r"(pk[4 * pc]), "r"(pk[4 * pc + 1]), "r"(pk[4 * pc + 2]), "r"(pk[4 * pc + 3]) : "memory");
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_p);          // P_j is in place, S_j and the previous O_blk have been read
      l = fmaf(l, alpha, rowsum);
      m = mx;
      alpha_prev = alpha;
    }
    float peer_l = 0.f;
    if (ok) {
      ok = __all_sync(0xffffffffu, gemm_wait(bar_o, (nblk - 1) & 1, abort_flag, &g_status));
      if (ok) {
        ptx::tc_fence_after();
        take_o(alpha_prev);
        ok = exchange(l, 2, nblk, peer_l);
      }
    }
    if (ok && row_ok) {
      l += peer_l;
      const float inv = 1.0f / l;
      __nv_bfloat16* dst = a.o + (size_t)i_abs * a.ldo + (size_t)h * DH + half * (DH / 2);
#pragma unroll
      for (int k = 0; k < DH / 2; k += 8) {
        uint4 w;
        w.x = ptx::pack_bf16(O[k] * inv, O[k + 1] * inv);
        w.y = ptx::pack_bf16(O[k + 2] * inv, O[k + 3] * inv);
        w.z = ptx::pack_bf16(O[k + 4] * inv, O[k + 5] * inv);
        w.w = ptx::pack_bf16(O[k + 6] * inv, O[k + 7] * inv);
        *reinterpret_cast<uint4*>(dst + k) = w;
      }
      if (half == 0) a.lse[(size_t)i_abs * a.n_heads + h] = (m + log2f(l)) * 0.6931471805599453f;
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


// =============================================================================================
// Gradients, head size 128.  P is recomputed from the saved log-sum-exp (no running maximum is
// needed), D[i] = sum_d dO[i, d] O[i, d], dS = P o (dP - D):
//   dq kernel : CTA = (128 query rows, head).   Per key block: S = Q K^T and dP = dO V^T into tensor
//               memory, the softmax threads (one query row each) write dS as a bf16 operand, and
//               dQ += dS K accumulates in tensor memory over all key blocks.
//   dkv kernel: CTA = (128 key rows, key-value head).  Per (query head of the group, query block):
//               S^T = K Q^T and dP^T = V dO^T, the threads (one key row each) write P^T and dS^T,
//               dV += P^T dO and dK += dS^T Q accumulate in tensor memory over all heads and blocks,
//               so every element of dk and dv is written once.
// A [rows][64] K-major tile (rows of 128 bytes, 128-byte swizzle) is byte for byte also the
// MN-major operand whose K index is the row, so K, Q and dO are loaded once and used in both roles
// (as an MN-major operand: descriptor start + 8 KiB per 64 rows, 16 KiB between the two 64-column
// blocks).
// =============================================================================================
struct BwdArgs {
  const __nv_bfloat16* o;  int64_t ldo;
  const __nv_bfloat16* dO; int64_t lddo;
  const float* lse;                         // [n_rows, n_heads]
  const int32_t* seq_start;
  const int32_t* seq_end;
  __nv_bfloat16* dq; int64_t lddq;
  __nv_bfloat16* dk; int64_t lddk;
  __nv_bfloat16* dv; int64_t lddv;
  int32_t n_rows, n_heads, n_kv;
  float scale, scale_log2;
};

constexpr uint32_t DQ_SMEM_BYTES = 1024 + 2 * Q_BYTES + P_BYTES + STAGES * (K_BYTES + V_BYTES) + 256;
constexpr uint32_t DKV_SMEM_BYTES = 1024 + 6 * Q_BYTES + 3 * 512 + 256;
constexpr uint32_t BWD_TMEM_COLS = 512;

// 32 columns of a row of a bf16 operand tile: pieces 4 (cc % 2) .. + 3 of K-block cc / 2
__device__ __forceinline__ void store_row_chunk(uint32_t tile, int row, int cc, const uint32_t (&pk)[16]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t pc = (uint32_t)((cc & 1) * 4 + q);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(tile + (uint32_t)row * 128u + (uint32_t)(cc >> 1) * 16384u + ((pc ^ (uint32_t)(row & 7)) << 4)),
                 "r"(pk[4 * q]), "r"(pk[4 * q + 1]), "r"(pk[4 * q + 2]), "r"(pk[4 * q + 3]) : "memory");
  }
}

// 128 x 128 x 128 product of two K-major tiles (two 64-wide K-blocks each) into d_tmem.
__device__ __forceinline__ void mma_kk(uint32_t d_tmem, uint32_t a_tile, uint32_t b_tile, uint32_t first_acc) {
  constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, BN, false, false);
  uint32_t acc = first_acc;
#pragma unroll
  for (int kb = 0; kb < 2; ++kb) {
    const uint64_t ad = ptx::make_smem_desc(a_tile + kb * 16384, 16, 1024);
    const uint64_t bd = ptx::make_smem_desc(b_tile + kb * 16384, 16, 1024);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      ptx::umma_f16(d_tmem, ad + (uint64_t)(ks * 2), bd + (uint64_t)(ks * 2), idesc, acc);
      acc = 1;
    }
  }
}
// d_tmem (+)= A B with A a K-major tile [128][128] (K = its 128 columns) and B a [128 rows][128
// columns] tile read as the MN-major operand whose K index is the row.
__device__ __forceinline__ void mma_kn(uint32_t d_tmem, uint32_t a_tile, uint32_t b_tile, uint32_t first_acc) {
  constexpr uint32_t idesc = ptx::make_idesc_bf16(BM, DH, false, true);
  uint32_t acc = first_acc;
#pragma unroll
  for (int kb = 0; kb < 2; ++kb) {
    const uint64_t ad = ptx::make_smem_desc(a_tile + kb * 16384, 16, 1024);
    const uint64_t bd = ptx::make_smem_desc(b_tile + kb * 8192, 16384, 1024);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      ptx::umma_f16(d_tmem, ad + (uint64_t)(ks * 2), bd + (uint64_t)(ks * 128), idesc, acc);
      acc = 1;
    }
  }
}

__global__ void __launch_bounds__(THREADS, 1)
backward_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmdO,
                   const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const BwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  const uint32_t sQ = base, sdO = base + Q_BYTES, sDS = base + 2 * Q_BYTES;
  auto sK = [&](int s) { return base + 2 * Q_BYTES + P_BYTES + (uint32_t)s * (K_BYTES + V_BYTES); };
  auto sV = [&](int s) { return sK(s) + K_BYTES; };
  const uint32_t sBar = base + 2 * Q_BYTES + P_BYTES + STAGES * (K_BYTES + V_BYTES);
  const uint32_t bar_q = sBar, bar_s = sBar + 8, bar_ds = sBar + 16, bar_done = sBar + 24;
  auto bar_kv_full = [&](int s) { return sBar + 32u + 8u * s; };
  auto bar_kv_empty = [&](int s) { return sBar + 48u + 8u * s; };
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(gen + (sBar - base) + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (sBar - base) + 72);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * BM, h = blockIdx.y;
  const int hk = h / (a.n_heads / a.n_kv);
  const int row_last = min(m0 + BM, a.n_rows) - 1;
  const int kmin = a.seq_start[m0];
  const int nblk = (row_last - kmin) / BN + 1;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_q, 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_ds, BM);
    ptx::mbar_init(bar_done, 1);
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(bar_kv_full(s), 1); ptx::mbar_init(bar_kv_empty(s), 1); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmdO); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), BWD_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    if (lane == 0) {
      ptx::mbar_arrive_expect_tx(bar_q, 2 * Q_BYTES);
      ptx::tma_load_2d(sQ, &tmQ, h * DH, m0, bar_q);
      ptx::tma_load_2d(sQ + 16384, &tmQ, h * DH + 64, m0, bar_q);
      ptx::tma_load_2d(sdO, &tmdO, h * DH, m0, bar_q);
      ptx::tma_load_2d(sdO + 16384, &tmdO, h * DH + 64, m0, bar_q);
      for (int j = 0; j < nblk; ++j) {
        const int s = j % STAGES;
        if (!gemm_wait(bar_kv_empty(s), ((j / STAGES) & 1) ^ 1, abort_flag, &g_status)) break;
        const int key0 = kmin + j * BN;
        ptx::mbar_arrive_expect_tx(bar_kv_full(s), K_BYTES + V_BYTES);
        ptx::tma_load_2d(sK(s), &tmK, hk * DH, key0, bar_kv_full(s));
        ptx::tma_load_2d(sK(s) + 16384, &tmK, hk * DH + 64, key0, bar_kv_full(s));
        ptx::tma_load_2d(sV(s), &tmV, hk * DH, key0, bar_kv_full(s));
        ptx::tma_load_2d(sV(s) + 16384, &tmV, hk * DH + 64, key0, bar_kv_full(s));
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t tS = tmem_base, tP = tmem_base + 128, tDQ = tmem_base + 256;
      bool ok = gemm_wait(bar_q, 0, abort_flag, &g_status);
      for (int j = 0; j < nblk && ok; ++j) {
        const int s = j % STAGES;
        if (!(ok = gemm_wait(bar_kv_full(s), (j / STAGES) & 1, abort_flag, &g_status))) break;
        ptx::tc_fence_after();
        mma_kk(tS, sQ, sK(s), 0);             // S = Q K^T
        mma_kk(tP, sdO, sV(s), 0);            // dP = dO V^T
        ptx::umma_commit(bar_s);
        if (!(ok = gemm_wait(bar_ds, j & 1, abort_flag, &g_status))) break;
        ptx::tc_fence_after();
        mma_kn(tDQ, sDS, sK(s), j > 0 ? 1u : 0u);    // dQ += dS K
        ptx::umma_commit(bar_kv_empty(s));
        if (j == nblk - 1) ptx::umma_commit(bar_done);
      }
    }
    __syncwarp();
  } else {
    const int e = warp & 3;
    const int row = e * 32 + lane;
    const int i_abs = m0 + row;
    const bool row_ok = i_abs < a.n_rows;
    const int my_start = row_ok ? a.seq_start[i_abs] : 0x7fffffff;
    const uint32_t tS = tmem_base + ((uint32_t)(e * 32) << 16), tP = tS + 128, tDQ = tS + 256;
    float lse2 = 0.f, D = 0.f;
    if (row_ok) {
      lse2 = a.lse[(size_t)i_abs * a.n_heads + h] * 1.4426950408889634f;
      const uint4* po = reinterpret_cast<const uint4*>(a.o + (size_t)i_abs * a.ldo + (size_t)h * DH);
      const uint4* pd = reinterpret_cast<const uint4*>(a.dO + (size_t)i_abs * a.lddo + (size_t)h * DH);
#pragma unroll 4
      for (int k = 0; k < DH / 8; ++k) {
        const uint4 x = po[k], y = pd[k];
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          D = fmaf(__uint_as_float(xs[t] << 16), __uint_as_float(ys[t] << 16), D);
          D = fmaf(__uint_as_float(xs[t] & 0xFFFF0000u), __uint_as_float(ys[t] & 0xFFFF0000u), D);
        }
      }
    }
    bool ok = true;
    for (int j = 0; j < nblk; ++j) {
      const int key0 = kmin + j * BN;
      ok = __all_sync(0xffffffffu, gemm_wait(bar_s, j & 1, abort_flag, &g_status));
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t vs[32], vp[32];
        ptx::tmem_ld_32x32b_x32(tS + cc * 32, vs);
        ptx::tmem_ld_32x32b_x32(tP + cc * 32, vp);
        ptx::tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int k = 0; k < 32; k += 2) {
          const int col = key0 + cc * 32 + k;
          const float p0 = (col >= my_start && col <= i_abs) ? fast_ex2(__uint_as_float(vs[k]) * a.scale_log2 - lse2) : 0.f;
          const float p1 = (col + 1 >= my_start && col + 1 <= i_abs) ? fast_ex2(__uint_as_float(vs[k + 1]) * a.scale_log2 - lse2) : 0.f;
          pk[k >> 1] = ptx::pack_bf16(p0 * (__uint_as_float(vp[k]) - D), p1 * (__uint_as_float(vp[k + 1]) - D));
        }
        store_row_chunk(sDS, row, cc, pk);
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_ds);
    }
    if (ok) ok = __all_sync(0xffffffffu, gemm_wait(bar_done, 0, abort_flag, &g_status));
    if (ok) {
      ptx::tc_fence_after();
      __nv_bfloat16* dst = a.dq + (size_t)i_abs * a.lddq + (size_t)h * DH;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(tDQ + cc * 32, v);
        ptx::tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int k = 0; k < 32; k += 8) {
            uint4 w;
            w.x = ptx::pack_bf16(__uint_as_float(v[k]) * a.scale, __uint_as_float(v[k + 1]) * a.scale);
            w.y = ptx::pack_bf16(__uint_as_float(v[k + 2]) * a.scale, __uint_as_float(v[k + 3]) * a.scale);
            w.z = ptx::pack_bf16(__uint_as_float(v[k + 4]) * a.scale, __uint_as_float(v[k + 5]) * a.scale);
            w.w = ptx::pack_bf16(__uint_as_float(v[k + 6]) * a.scale, __uint_as_float(v[k + 7]) * a.scale);
            *reinterpret_cast<uint4*>(dst + cc * 32 + k) = w;
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, BWD_TMEM_COLS);
  }
}

__global__ void __launch_bounds__(THREADS, 1)
backward_dkv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmdO,
                    const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const BwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - ptx::smem_u32(smem_raw));
  const uint32_t sKt = base, sVt = base + Q_BYTES, sQ = base + 2 * Q_BYTES, sdO = base + 3 * Q_BYTES;
  const uint32_t sOP = base + 4 * Q_BYTES;      // the O block, then P^T
  const uint32_t sDS = base + 5 * Q_BYTES;
  float* sL = reinterpret_cast<float*>(gen + 6 * Q_BYTES);            // per query of the block: lse * log2 e
  float* sD = sL + 128;                                               // D
  int* sQS = reinterpret_cast<int*>(sD + 128);                        // first row of the query's sequence
  const uint32_t sBar = base + 6 * Q_BYTES + 3 * 512;
  const uint32_t bar_kv = sBar, bar_s = sBar + 8, bar_p = sBar + 16, bar_done = sBar + 24;
  const uint32_t bar_ld_full = sBar + 32, bar_ld_empty = sBar + 40, bar_tab = sBar + 48;
  uint32_t* tmem_ptr_smem = reinterpret_cast<uint32_t*>(gen + (sBar - base) + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + (sBar - base) + 72);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k0 = blockIdx.x * BM, hk = blockIdx.y;
  const int rep = a.n_heads / a.n_kv;
  const int key_last = min(k0 + BM, a.n_rows) - 1;
  const int qend = a.seq_end[key_last];                    // queries past the last key's sequence see none of these keys
  const int nqb = (qend - k0 + BM - 1) / BM;               // query blocks start at the key tile's first row (causality)
  const int n_it = rep * nqb;

  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_kv, 1);
    ptx::mbar_init(bar_s, 1);
    ptx::mbar_init(bar_p, BM);
    ptx::mbar_init(bar_done, 1);
    ptx::mbar_init(bar_ld_full, 1);
    ptx::mbar_init(bar_ld_empty, 1);
    ptx::mbar_init(bar_tab, BM);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmdO); ptx::prefetch_tmap(&tmO); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), BWD_TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    if (lane == 0) {
      ptx::mbar_arrive_expect_tx(bar_kv, 2 * Q_BYTES);
      ptx::tma_load_2d(sKt, &tmK, hk * DH, k0, bar_kv);
      ptx::tma_load_2d(sKt + 16384, &tmK, hk * DH + 64, k0, bar_kv);
      ptx::tma_load_2d(sVt, &tmV, hk * DH, k0, bar_kv);
      ptx::tma_load_2d(sVt + 16384, &tmV, hk * DH + 64, k0, bar_kv);
      for (int it = 0; it < n_it; ++it) {
        const int h = hk * rep + it / nqb, q0 = k0 + (it % nqb) * BM;
        if (!gemm_wait(bar_ld_empty, (it & 1) ^ 1, abort_flag, &g_status)) break;
        ptx::mbar_arrive_expect_tx(bar_ld_full, 3 * Q_BYTES);
        ptx::tma_load_2d(sQ, &tmQ, h * DH, q0, bar_ld_full);
        ptx::tma_load_2d(sQ + 16384, &tmQ, h * DH + 64, q0, bar_ld_full);
        ptx::tma_load_2d(sdO, &tmdO, h * DH, q0, bar_ld_full);
        ptx::tma_load_2d(sdO + 16384, &tmdO, h * DH + 64, q0, bar_ld_full);
        ptx::tma_load_2d(sOP, &tmO, h * DH, q0, bar_ld_full);
        ptx::tma_load_2d(sOP + 16384, &tmO, h * DH + 64, q0, bar_ld_full);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t tS = tmem_base, tP = tmem_base + 128, tDV = tmem_base + 256, tDK = tmem_base + 384;
      bool ok = gemm_wait(bar_kv, 0, abort_flag, &g_status);
      for (int it = 0; it < n_it && ok; ++it) {
        if (!(ok = gemm_wait(bar_ld_full, it & 1, abort_flag, &g_status))) break;
        ptx::tc_fence_after();
        mma_kk(tS, sKt, sQ, 0);               // S^T = K Q^T
        mma_kk(tP, sVt, sdO, 0);              // dP^T = V dO^T
        ptx::umma_commit(bar_s);
        if (!(ok = gemm_wait(bar_p, it & 1, abort_flag, &g_status))) break;
        ptx::tc_fence_after();
        mma_kn(tDV, sOP, sdO, it > 0 ? 1u : 0u);     // dV += P^T dO
        mma_kn(tDK, sDS, sQ, it > 0 ? 1u : 0u);      // dK += dS^T Q
        ptx::umma_commit(bar_ld_empty);
        if (it == n_it - 1) ptx::umma_commit(bar_done);
      }
    }
    __syncwarp();
  } else {
    const int e = warp & 3;
    const int row = e * 32 + lane;                      // key row of the tile, and the query this thread prepares
    const int j_abs = k0 + row;
    const uint32_t tS = tmem_base + ((uint32_t)(e * 32) << 16), tP = tS + 128, tDV = tS + 256, tDK = tS + 384;
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
      const int h = hk * rep + it / nqb, q0 = k0 + (it % nqb) * BM;
      ok = __all_sync(0xffffffffu, gemm_wait(bar_ld_full, it & 1, abort_flag, &g_status));
      if (!ok) break;
      {   // query q0 + row: D from the staged dO and O rows (same swizzle, so piece by piece), lse, sequence start
        const int i = q0 + row;
        float D = 0.f;
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int pz = 0; pz < 8; ++pz) {
            const uint32_t off = (uint32_t)kb * 16384u + (uint32_t)row * 128u + (uint32_t)pz * 16u;
            uint4 x, y;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "r"(sOP + off));
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(y.x), "=r"(y.y), "=r"(y.z), "=r"(y.w) : "r"(sdO + off));
            const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              D = fmaf(__uint_as_float(xs[t] << 16), __uint_as_float(ys[t] << 16), D);
              D = fmaf(__uint_as_float(xs[t] & 0xFFFF0000u), __uint_as_float(ys[t] & 0xFFFF0000u), D);
            }
          }
        const bool q_ok = i < a.n_rows;
        sD[row] = D;
        sL[row] = q_ok ? a.lse[(size_t)i * a.n_heads + h] * 1.4426950408889634f : 0.f;
        sQS[row] = q_ok ? a.seq_start[i] : 0x7fffffff;
      }
      // the block's tables are complete and every O row has been read once all 128 threads have
      // arrived (an mbarrier with a bounded wait rather than bar.sync: a warp that gave up never arrives)
      ptx::mbar_arrive(bar_tab);
      ok = __all_sync(0xffffffffu, gemm_wait(bar_tab, it & 1, abort_flag, &g_status));
      if (!ok) break;
      ok = __all_sync(0xffffffffu, gemm_wait(bar_s, it & 1, abort_flag, &g_status));
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t vs[32], vp[32];
        ptx::tmem_ld_32x32b_x32(tS + cc * 32, vs);
        ptx::tmem_ld_32x32b_x32(tP + cc * 32, vp);
        ptx::tmem_ld_wait();
        uint32_t pp[16], pd[16];
#pragma unroll
        for (int k4 = 0; k4 < 32; k4 += 4) {       // the per-query tables come in as vectors, four columns at a time
          const int c0 = cc * 32 + k4;
          const float4 l4 = *reinterpret_cast<const float4*>(sL + c0);
          const float4 d4 = *reinterpret_cast<const float4*>(sD + c0);
          const int4 s4 = *reinterpret_cast<const int4*>(sQS + c0);
          const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dv4[4] = {d4.x, d4.y, d4.z, d4.w};
          const int sv[4] = {s4.x, s4.y, s4.z, s4.w};
          float p[4];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const int i = q0 + c0 + t;
            p[t] = (j_abs <= i && j_abs >= sv[t]) ? fast_ex2(__uint_as_float(vs[k4 + t]) * a.scale_log2 - lv[t]) : 0.f;
          }
          pp[k4 >> 1] = ptx::pack_bf16(p[0], p[1]);
          pp[(k4 >> 1) + 1] = ptx::pack_bf16(p[2], p[3]);
          pd[k4 >> 1] = ptx::pack_bf16(p[0] * (__uint_as_float(vp[k4]) - dv4[0]), p[1] * (__uint_as_float(vp[k4 + 1]) - dv4[1]));
          pd[(k4 >> 1) + 1] = ptx::pack_bf16(p[2] * (__uint_as_float(vp[k4 + 2]) - dv4[2]), p[3] * (__uint_as_float(vp[k4 + 3]) - dv4[3]));
        }
        store_row_chunk(sOP, row, cc, pp);
        store_row_chunk(sDS, row, cc, pd);
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      ptx::mbar_arrive(bar_p);
    }
    if (ok) ok = __all_sync(0xffffffffu, gemm_wait(bar_done, 0, abort_flag, &g_status));
    if (ok) {
      ptx::tc_fence_after();
      const bool key_ok = j_abs < a.n_rows;
      __nv_bfloat16* dvp = a.dv + (size_t)j_abs * a.lddv + (size_t)hk * DH;
      __nv_bfloat16* dkp = a.dk + (size_t)j_abs * a.lddk + (size_t)hk * DH;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32], w[32];
        ptx::tmem_ld_32x32b_x32(tDV + cc * 32, v);
        ptx::tmem_ld_32x32b_x32(tDK + cc * 32, w);
        ptx::tmem_ld_wait();
        if (key_ok) {
#pragma unroll
          for (int k = 0; k < 32; k += 8) {
            uint4 x, y;
            x.x = ptx::pack_bf16(__uint_as_float(v[k]), __uint_as_float(v[k + 1]));
            x.y = ptx::pack_bf16(__uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
            x.z = ptx::pack_bf16(__uint_as_float(v[k + 4]), __uint_as_float(v[k + 5]));
            x.w = ptx::pack_bf16(__uint_as_float(v[k + 6]), __uint_as_float(v[k + 7]));
            y.x = ptx::pack_bf16(__uint_as_float(w[k]) * a.scale, __uint_as_float(w[k + 1]) * a.scale);
            y.y = ptx::pack_bf16(__uint_as_float(w[k + 2]) * a.scale, __uint_as_float(w[k + 3]) * a.scale);
            y.z = ptx::pack_bf16(__uint_as_float(w[k + 4]) * a.scale, __uint_as_float(w[k + 5]) * a.scale);
            y.w = ptx::pack_bf16(__uint_as_float(w[k + 6]) * a.scale, __uint_as_float(w[k + 7]) * a.scale);
            *reinterpret_cast<uint4*>(dvp + cc * 32 + k) = x;
            *reinterpret_cast<uint4*>(dkp + cc * 32 + k) = y;
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, BWD_TMEM_COLS);
  }
}

}  // namespace attn_tc
}  // namespace mlora
