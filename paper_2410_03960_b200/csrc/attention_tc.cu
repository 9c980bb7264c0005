// Causal varlen grouped-query flash attention for prefill on tcgen05 tensor cores (head_dim 128, bf16).
//
// One CTA works on one (prompt, 128-query tile, PAIR of query heads that share a KV head): the two heads see
// exactly the same keys, values and causal mask, so they ping-pong on the tensor pipe while sharing every K/V
// tile that TMA brings in.  320 threads:
//   warp 0      : TMA producer (Q of both heads once; K and V tiles of 128 keys through 2-deep rings)
//   warp 1      : MMA issuer: S_w = Q_w K^T into tensor memory, then O_w += P_w V with P_w read straight from
//                 tensor memory (the softmax warps overwrite S_w with bf16 P_w in place)
//   warps 2..5  : softmax of head 0 -- one query row per thread (a TMEM lane), so row max / sum need no shuffles;
//   warps 6..9  : softmax of head 1.
// Online softmax keeps a per-row reference max that only moves when the running max grows by more than 2^8
// (then O_w is rescaled in tensor memory); the final O_w / l_w is exact for any such reference.
// Tensor memory: S0 | S1 | O0 | O1, 128 fp32 columns each (all 512).  Every wait is bounded.
// Two kernels share this design: one CTA per work item (used when only the device knows the lengths), and a persistent
// one that walks a host-balanced list of items and overlaps an item's set-up with the previous item's epilogue.
#include <algorithm>
#include <cstdlib>
#include <functional>
#include <queue>
#include <utility>
#include <vector>

#include <type_traits>

#include "common.cuh"
#include "tc_common.cuh"

namespace skv {
namespace {

constexpr int HD = 128;                 // head dim
constexpr int BQ = 128, BKV = 128;      // query rows / keys per tile
constexpr int ATT_THREADS = 320;
constexpr int TILE_BYTES = 128 * HD * 2;          // 32 KB: one [128 x 128] bf16 tile = two 64-column swizzled chunks
constexpr int CHUNK_BYTES = TILE_BYTES / 2;       // 16 KB
constexpr int KV_STAGES = 2;
constexpr int SM_Q = 0, SM_K = 2 * TILE_BYTES, SM_V = SM_K + KV_STAGES * TILE_BYTES;
constexpr int SM_BAR = SM_V + KV_STAGES * TILE_BYTES;
constexpr int ATT_SMEM = SM_BAR + 256 + 1024;
constexpr float RESCALE_THRESHOLD = 8.0f;          // in log2 units

struct AttnParams {
  const int32_t *cu;        // [n_seqs+1] offsets of each sequence's NEW tokens (the queries) in q / out
  const int32_t *k_row0;    // [n_seqs] first K / V row of each sequence (null: same as cu, i.e. a plain prefill)
  const int32_t *kv_len;    // [n_seqs] keys of each sequence = tokens already cached + new tokens (null: new tokens only)
  const int32_t *blk;       // optional block tables of a paged cache: key tile j of sequence b starts at row
  int blk_stride;           //   blk[b * blk_stride + j] * 128 (a key tile is exactly one page)
  bf16 *out;
  int n_seqs, n_q, n_kv, max_tiles;
  float scale_log2;     // softmax scale * log2(e)
  unsigned int *status;
  int store32;          // out is 32-byte aligned: 32-byte stores in the epilogue
};

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag, unsigned int *status) {
  if (tc::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  // try_wait itself suspends the thread for a while, so the loop is not a busy spin; the abort flag and the clock
  // are looked at only every 32nd round to keep the time from "barrier completed" to "waiter runs" short
  for (unsigned spins = 1;; ++spins) {
    if (tc::mbar_try_wait(bar, parity)) return true;
    if ((spins & 31u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > tc::WAIT_LIMIT_CLOCKS) {
        *abort_flag = 1;
        atomicOr(status, STATUS_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 32 fp32 accumulators of one output row -> * inv -> 16 bits -> 64 contiguous bytes of the row
template <bool ACT_F16>
__device__ __forceinline__ void store_out_chunk(bf16 *dst, const uint32_t (&r)[32], float inv, bool store32) {
  uint32_t v[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = tc::pack_act(__uint_as_float(r[2 * i]) * inv, __uint_as_float(r[2 * i + 1]) * inv, ACT_F16);
  if (store32) {
    tc::st_global_v8(dst, v);
    tc::st_global_v8(dst + 16, v + 8);
  } else {
    uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
    for (int i = 0; i < 4; ++i) d4[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  }
}

// ACT_F16: q, K, V, P and the output are all IEEE halves (else all bfloat16)
template <bool ACT_F16, bool SPLIT_P>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  // ---- which work item: heavy (late) query tiles first
  const int n_pairs = p.n_q >> 1;
  const int per_tile = p.n_seqs * n_pairs;
  const int qt = p.max_tiles - 1 - (int)(blockIdx.x / per_tile);
  const int rem = blockIdx.x % per_tile;
  const int b = rem / n_pairs, pair = rem % n_pairs;
  const int tok0 = p.cu[b], n = p.cu[b + 1] - tok0;
  if (qt * BQ >= n) return;
  const int k0 = p.k_row0 ? p.k_row0[b] : tok0;
  const int past = p.kv_len ? p.kv_len[b] - n : 0;       // query i of this sequence sits at position past + i
  const int h0 = pair * 2;
  const int kvh = h0 / (p.n_q / p.n_kv);
  const int n_kv_tiles = (past + min(n, (qt + 1) * BQ) - 1) / BKV + 1;   // keys 0 .. position of the tile's last query
  const int q_row0 = tok0 + qt * BQ;

  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM_BAR);
  uint64_t *q_full = bars;            // [1]
  uint64_t *k_full = bars + 1;        // [2]
  uint64_t *k_empty = bars + 3;       // [2]
  uint64_t *v_full = bars + 5;        // [2]
  uint64_t *v_empty = bars + 7;       // [2]
  uint64_t *s_full = bars + 9;        // [2]  S_w ready in tensor memory
  uint64_t *p_ready = bars + 11;      // [2]  first 64 keys of P_w written (and O_w rescaled) by the softmax warps
  uint64_t *p_ready2 = bars + 13;     // [2]  last 64 keys of P_w written
  uint64_t *o_full = bars + 15;       // [1]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 16);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(q_full), 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(tc::smem_u32(&k_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&k_empty[s]), 1);
      tc::mbar_init(tc::smem_u32(&v_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&v_empty[s]), 1);
      tc::mbar_init(tc::smem_u32(&s_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&p_ready[s]), 4);   // one arrival per softmax warp
      tc::mbar_init(tc::smem_u32(&p_ready2[s]), 4);
    }
    tc::mbar_init(tc::smem_u32(o_full), 1);
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmQ);
    tc::tma_prefetch_desc(&tmK);
    tc::tma_prefetch_desc(&tmV);
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // tensor-memory columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_w aliases the first 64 of S_w

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------ TMA producer
      const uint32_t qb = tc::smem_u32(q_full);
      tc::mbar_expect_tx(qb, 2 * TILE_BYTES);
      for (int w = 0; w < 2; ++w)
        for (int c = 0; c < 2; ++c)
          tc::tma_load_2d(tc::smem_u32(smem + SM_Q + w * TILE_BYTES + c * CHUNK_BYTES), &tmQ, qb, (h0 + w) * HD + c * 64, q_row0);
      for (int j = 0; j < n_kv_tiles; ++j) {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        const int krow = p.blk ? p.blk[(size_t)b * p.blk_stride + j] * BKV : k0 + j * BKV;
        if (!wait_or_abort(tc::smem_u32(&k_empty[s]), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t kb = tc::smem_u32(&k_full[s]);
        tc::mbar_expect_tx(kb, TILE_BYTES);
        for (int c = 0; c < 2; ++c)
          tc::tma_load_2d(tc::smem_u32(smem + SM_K + s * TILE_BYTES + c * CHUNK_BYTES), &tmK, kb, kvh * HD + c * 64, krow);
        if (!wait_or_abort(tc::smem_u32(&v_empty[s]), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t vb = tc::smem_u32(&v_full[s]);
        tc::mbar_expect_tx(vb, TILE_BYTES);
        for (int c = 0; c < 2; ++c)
          tc::tma_load_2d(tc::smem_u32(smem + SM_V + s * TILE_BYTES + c * CHUNK_BYTES), &tmV, vb, kvh * HD + c * 64, krow);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    // The whole warp walks this code and one elected lane issues every tcgen05.mma and commit: the lane's instruction
    // stream is on the critical path of every key tile (an MMA must leave every 64 clocks), and inside a one-lane
    // branch each descriptor would be per-thread arithmetic.  The key-tile loop is unrolled by the two ring stages so
    // that stage offsets and barrier parities are constants.
    const bool leader = tc::elect_one();
    constexpr uint32_t idesc_qk = tc::umma_idesc(BQ, BKV, 0, 0, ACT_F16, ACT_F16);   // Q, K both K-major (head dim contiguous)
    constexpr uint32_t idesc_pv = tc::umma_idesc(BQ, HD, 0, 1, ACT_F16, ACT_F16);    // V is MN-major (head dim contiguous, keys = K)
    // shared-memory descriptors differ only in their address field (bytes >> 4): one per buffer, plus step offsets
    const uint64_t q_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_Q), 16, 1024);
    const uint64_t k_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_K), 16, 1024);
    const uint64_t v_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_V), CHUNK_BYTES, 1024);
    auto issue_qk = [&](int w, int s) {   // S_w = Q_w K^T : 8 steps of 16 along the head dim
      const uint64_t qd = q_desc0 + (uint64_t)(w * (TILE_BYTES >> 4)), kd = k_desc0 + (uint64_t)(s * (TILE_BYTES >> 4));
      const uint32_t d = tmem_base + w * 128;
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const uint32_t off = ((kk >> 2) * CHUNK_BYTES + (kk & 3) * 32) >> 4;
        tc::umma_ss(d, qd + off, kd + off, idesc_qk, kk != 0);
      }
    };
    // O_w (+)= P_w V : 8 steps of 16 keys, issued in two halves so that the first 64 keys can run on the tensor
    // pipe while the softmax warps still exponentiate the last 64
    auto issue_pv = [&](int w, int s, bool accumulate, int half) {
      const uint64_t vd = v_desc0 + (uint64_t)(s * (TILE_BYTES >> 4));
      const uint32_t d = tmem_base + 256 + w * 128, a_t = tmem_base + w * 128;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const int kk = half * 4 + k4;
        tc::umma_ts(d, a_t + kk * 8, vd + (uint64_t)((kk * 16 * 128) >> 4), idesc_pv, (accumulate || kk != 0) ? 1u : 0u);
      }
    };
    const uint32_t b_kf = tc::smem_u32(&k_full[0]), b_ke = tc::smem_u32(&k_empty[0]), b_vf = tc::smem_u32(&v_full[0]),
                   b_ve = tc::smem_u32(&v_empty[0]), b_sf = tc::smem_u32(&s_full[0]), b_p1 = tc::smem_u32(&p_ready[0]),
                   b_p2 = tc::smem_u32(&p_ready2[0]);
    auto wait = [&](uint32_t bar, uint32_t parity) {
      const bool ok = wait_or_abort(bar, parity, abort_flag, p.status);
      tc::tc_fence_after_sync();
      return ok;
    };
    // key tile j in ring stage s = j & 1 (a compile-time constant here)
    auto tile = [&](auto stage, int j) -> bool {
      constexpr int s = decltype(stage)::value, s1 = s ^ 1;
      const uint32_t ph = (j >> 1) & 1, ph1 = ph ^ s;     // fill parity of stage s for tile j, of stage s1 for tile j + 1
      const bool more = j + 1 < n_kv_tiles, acc = j > 0;
      if (!wait(b_vf + 8 * s, ph) || !wait(b_p1, s)) return false;
      if (leader) issue_pv(0, s, acc, 0);
      if (SPLIT_P && !wait(b_p2, s)) return false;
      if (leader) issue_pv(0, s, acc, 1);
      if (more) {
        if (!wait(b_kf + 8 * s1, ph1)) return false;
        if (leader) {
          issue_qk(0, s1);
          tc::umma_commit(b_sf);
        }
      }
      if (!wait(b_p1 + 8, s)) return false;
      if (leader) issue_pv(1, s, acc, 0);
      if (SPLIT_P && !wait(b_p2 + 8, s)) return false;
      if (leader) {
        issue_pv(1, s, acc, 1);
        tc::umma_commit(b_ve + 8 * s);
        if (more) {
          issue_qk(1, s1);
          tc::umma_commit(b_sf + 8);
          tc::umma_commit(b_ke + 8 * s1);
        }
      }
      return true;
    };
    bool ok = wait(tc::smem_u32(q_full), 0) && wait(b_kf, 0);
    if (ok && leader) {
      issue_qk(0, 0);
      tc::umma_commit(b_sf);
      issue_qk(1, 0);
      tc::umma_commit(b_sf + 8);
      tc::umma_commit(b_ke);
    }
    for (int j = 0; j < n_kv_tiles && ok; j += 2) {
      ok = tile(std::integral_constant<int, 0>{}, j);
      if (ok && j + 1 < n_kv_tiles) ok = tile(std::integral_constant<int, 1>{}, j + 1);
    }
    if (ok && leader) tc::umma_commit(tc::smem_u32(o_full));
    __syncwarp();
  } else {
    // -------------------------------------------------------------- softmax warps: head w, one row per thread
    const int w = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                // query row inside the tile = TMEM lane
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_s = tmem_base + lane_base + w * 128;
    const uint32_t t_o = tmem_base + lane_base + 256 + w * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv_tiles; ++j) {
      if (!wait_or_abort(tc::smem_u32(&s_full[w]), j & 1, abort_flag, p.status)) { ok = false; break; }
      tc::tc_fence_after_sync();
      // causal mask: key column i of this tile is visible to query row r iff i <= r + shift; only the tiles that
      // straddle the diagonal (at most two when the cached prefix is not a multiple of the tile) need it
      const int shift = past + qt * BQ - j * BKV;
      const bool diag = shift < BKV - 1;
      const int lim = row + shift;
      // the whole score row (128 fp32) in registers: one pass over tensor memory, the second half of the loads in
      // flight while the first half is reduced
      uint32_t s[128];
      tc::tmem_ld_32x32b_x32p(t_s, s);
      tc::tmem_ld_32x32b_x32p(t_s + 32, s + 32);
      tc::tmem_ld_wait();
      tc::tmem_ld_32x32b_x32p(t_s + 64, s + 64);
      tc::tmem_ld_32x32b_x32p(t_s + 96, s + 96);
      if (diag) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i > lim) s[i] = 0xff800000u;   // -inf
      }
      float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 8) {
        m0 = tc::max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        m1 = tc::max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        m2 = tc::max3(m2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        m3 = tc::max3(m3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
      }
      tc::tmem_ld_wait();
      if (diag) {
#pragma unroll
        for (int i = 64; i < 128; ++i)
          if (i > lim) s[i] = 0xff800000u;
      }
#pragma unroll
      for (int i = 64; i < 128; i += 8) {
        m0 = tc::max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        m1 = tc::max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        m2 = tc::max3(m2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        m3 = tc::max3(m3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
      }
      const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      // move the reference max only when the running max outgrew it by more than the threshold
      const bool need = (j == 0) || ((mx - m_ref) * c > RESCALE_THRESHOLD);
      const float m_new = need ? mx : m_ref;
      if (j > 0 && __any_sync(0xffffffffu, need)) {
        // S_w of this tile is complete, so every earlier P_w V has retired: O_w is stable and may be rescaled
        const float f = need ? fast_exp2((m_ref - m_new) * c) : 1.f;
        l *= f;
#pragma unroll 1
        for (int ch = 0; ch < 8; ++ch) {
          uint32_t r[16];
          tc::tmem_ld_32x32b_x16(t_o + ch * 16, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
          tc::tmem_st_32x32b_x16(t_o + ch * 16, r);
        }
      }
      m_ref = m_new;
      // p = 2^(s*c - m_ref*c) (masked entries: 2^-inf = 0), row sum, 16-bit P written over S (64 packed columns) in
      // two halves of 64 keys, each announced to the MMA warp as soon as it is in tensor memory
      const float neg_mc = -m_ref * c;
      float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int i = hf * 32; i < hf * 32 + 32; i += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(s[2 * i]), c, neg_mc));
          const float p1 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 1]), c, neg_mc));
          const float p2 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 2]), c, neg_mc));
          const float p3 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 3]), c, neg_mc));
          l0 += p0; l1 += p1; l2 += p2; l3 += p3;
          s[i] = ACT_F16 ? tc::pack_f16x2(p0, p1) : tc::pack_bf16x2(p0, p1);
          s[i + 1] = ACT_F16 ? tc::pack_f16x2(p2, p3) : tc::pack_bf16x2(p2, p3);
        }
        tc::tmem_st_32x32b_x32(t_s + hf * 32, s + hf * 32);
        if (SPLIT_P || hf == 1) {
          tc::tmem_st_wait();
          tc::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(tc::smem_u32((SPLIT_P && hf == 1) ? &p_ready2[w] : &p_ready[w]));
        }
      }
      l += (l0 + l1) + (l2 + l3);
    }
    // ---- epilogue: O_w / l -> bf16 -> out[token, head, :]
    if (ok && wait_or_abort(tc::smem_u32(o_full), 0, abort_flag, p.status)) {
      tc::tc_fence_after_sync();
      const float inv = 1.f / l;
      const bool valid = qt * BQ + row < n;
      bf16 *dst = p.out + ((size_t)(q_row0 + row) * p.n_q + (h0 + w)) * HD;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tc::tmem_ld_32x32b_x32(t_o + ch * 32, r);
        tc::tmem_ld_wait();
        if (valid) store_out_chunk<ACT_F16>(dst + ch * 32, r, inv, p.store32 != 0);
      }
    }
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
}


// ---------------------------------------------------------------------------------------------------------
// Persistent form: one CTA per SM walks a list of work items that the host balanced (longest first, each to the least
// loaded CTA), so that a CTA's fixed cost -- tensor-memory allocation, barrier set-up, Q and first K loads, the first
// Q K^T -- is paid once or hides behind the previous item's last softmax and epilogue: the producer fetches the next
// item's Q as soon as the current item's last Q K^T has retired, and the MMA warp issues the next item's first Q K^T
// while the softmax warps still normalise and store the current output.  Barriers, tensor memory and the K / V rings
// live across items; every role keeps running counts of items (`it`) and key tiles (`gk`) for the barrier parities.
//   sched_off[c] .. sched_off[c + 1] : this CTA's items in sched_items, as indices in the heavy-first item order
// ---------------------------------------------------------------------------------------------------------
struct AttnItem {
  int b, qt, h0, kvh, n, past, k0, n_kv_tiles, q_row0;
};
__device__ __forceinline__ void decode_item(const AttnParams &p, int w, AttnItem &it) {
  const int n_pairs = p.n_q >> 1;
  const int per_tile = p.n_seqs * n_pairs;
  it.qt = p.max_tiles - 1 - w / per_tile;
  const int rem = w % per_tile;
  it.b = rem / n_pairs;
  const int tok0 = p.cu[it.b];
  it.n = p.cu[it.b + 1] - tok0;
  it.k0 = p.k_row0 ? p.k_row0[it.b] : tok0;
  it.past = p.kv_len ? p.kv_len[it.b] - it.n : 0;
  it.h0 = (rem % n_pairs) * 2;
  it.kvh = it.h0 / (p.n_q / p.n_kv);
  it.n_kv_tiles = (it.past + min(it.n, (it.qt + 1) * BQ) - 1) / BKV + 1;
  it.q_row0 = tok0 + it.qt * BQ;
}

template <bool ACT_F16>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_persistent_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                               const __grid_constant__ CUtensorMap tmV, AttnParams p, const int32_t *__restrict__ sched_off,
                               const int32_t *__restrict__ sched_items) {
  const int i_begin = sched_off[blockIdx.x], i_end = sched_off[blockIdx.x + 1];
  if (i_begin >= i_end) return;

  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM_BAR);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 3, *v_full = bars + 5, *v_empty = bars + 7, *s_full = bars + 9,
           *p_ready = bars + 11, *p_ready2 = bars + 13, *o_full = bars + 15;
  uint64_t *q_empty = bars + 16;      // every Q K^T of the item has retired: Q may be overwritten
  uint64_t *o_empty = bars + 17;      // the softmax warps have read the item's O out of tensor memory (8 arrivals)
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 18);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(q_full), 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(tc::smem_u32(&k_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&k_empty[s]), 1);
      tc::mbar_init(tc::smem_u32(&v_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&v_empty[s]), 1);
      tc::mbar_init(tc::smem_u32(&s_full[s]), 1);
      tc::mbar_init(tc::smem_u32(&p_ready[s]), 4);
      tc::mbar_init(tc::smem_u32(&p_ready2[s]), 4);
    }
    tc::mbar_init(tc::smem_u32(o_full), 1);
    tc::mbar_init(tc::smem_u32(q_empty), 1);
    tc::mbar_init(tc::smem_u32(o_empty), 8);
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmQ);
    tc::tma_prefetch_desc(&tmK);
    tc::tma_prefetch_desc(&tmV);
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------ TMA producer
      int gk = 0;
      bool ok = true;
      AttnItem im, nx;
      decode_item(p, sched_items[i_begin], nx);
      for (int i = i_begin; i < i_end && ok; ++i) {
        const int it = i - i_begin;
        im = nx;
        if (i + 1 < i_end) decode_item(p, sched_items[i + 1], nx);     // the next item's description: loads in flight meanwhile
        if (!wait_or_abort(tc::smem_u32(q_empty), (it & 1) ^ 1, abort_flag, p.status)) break;
        const uint32_t qb = tc::smem_u32(q_full);
        tc::mbar_expect_tx(qb, 2 * TILE_BYTES);
        for (int w = 0; w < 2; ++w)
          for (int c = 0; c < 2; ++c)
            tc::tma_load_2d(tc::smem_u32(smem + SM_Q + w * TILE_BYTES + c * CHUNK_BYTES), &tmQ, qb, (im.h0 + w) * HD + c * 64, im.q_row0);
        for (int j = 0; j < im.n_kv_tiles; ++j, ++gk) {
          const int s = gk & 1;
          const uint32_t ph = (gk >> 1) & 1;
          const int krow = p.blk ? p.blk[(size_t)im.b * p.blk_stride + j] * BKV : im.k0 + j * BKV;
          if (!wait_or_abort(tc::smem_u32(&k_empty[s]), ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t kb = tc::smem_u32(&k_full[s]);
          tc::mbar_expect_tx(kb, TILE_BYTES);
          for (int c = 0; c < 2; ++c)
            tc::tma_load_2d(tc::smem_u32(smem + SM_K + s * TILE_BYTES + c * CHUNK_BYTES), &tmK, kb, im.kvh * HD + c * 64, krow);
          if (!wait_or_abort(tc::smem_u32(&v_empty[s]), ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t vb = tc::smem_u32(&v_full[s]);
          tc::mbar_expect_tx(vb, TILE_BYTES);
          for (int c = 0; c < 2; ++c)
            tc::tma_load_2d(tc::smem_u32(smem + SM_V + s * TILE_BYTES + c * CHUNK_BYTES), &tmV, vb, im.kvh * HD + c * 64, krow);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (warp-uniform, one elected lane)
    const bool leader = tc::elect_one();
    constexpr uint32_t idesc_qk = tc::umma_idesc(BQ, BKV, 0, 0, ACT_F16, ACT_F16);
    constexpr uint32_t idesc_pv = tc::umma_idesc(BQ, HD, 0, 1, ACT_F16, ACT_F16);
    const uint64_t q_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_Q), 16, 1024);
    const uint64_t k_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_K), 16, 1024);
    const uint64_t v_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SM_V), CHUNK_BYTES, 1024);
    auto issue_qk = [&](int w, int s) {
      const uint64_t qd = q_desc0 + (uint64_t)(w * (TILE_BYTES >> 4)), kd = k_desc0 + (uint64_t)(s * (TILE_BYTES >> 4));
      const uint32_t d = tmem_base + w * 128;
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const uint32_t off = ((kk >> 2) * CHUNK_BYTES + (kk & 3) * 32) >> 4;
        tc::umma_ss(d, qd + off, kd + off, idesc_qk, kk != 0);
      }
    };
    auto issue_pv = [&](int w, int s, bool accumulate, int half) {
      const uint64_t vd = v_desc0 + (uint64_t)(s * (TILE_BYTES >> 4));
      const uint32_t d = tmem_base + 256 + w * 128, a_t = tmem_base + w * 128;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const int kk = half * 4 + k4;
        tc::umma_ts(d, a_t + kk * 8, vd + (uint64_t)((kk * 16 * 128) >> 4), idesc_pv, (accumulate || kk != 0) ? 1u : 0u);
      }
    };
    const uint32_t b_kf = tc::smem_u32(&k_full[0]), b_ke = tc::smem_u32(&k_empty[0]), b_vf = tc::smem_u32(&v_full[0]),
                   b_ve = tc::smem_u32(&v_empty[0]), b_sf = tc::smem_u32(&s_full[0]), b_p1 = tc::smem_u32(&p_ready[0]),
                   b_p2 = tc::smem_u32(&p_ready2[0]), b_qe = tc::smem_u32(q_empty);
    auto wait = [&](uint32_t bar, uint32_t parity) {
      const bool ok = wait_or_abort(bar, parity, abort_flag, p.status);
      tc::tc_fence_after_sync();
      return ok;
    };
    int gk = 0;
    bool ok = true;
    AttnItem im, nx;
    decode_item(p, sched_items[i_begin], nx);
    for (int i = i_begin; i < i_end && ok; ++i) {
      const int it = i - i_begin;
      im = nx;
      if (i + 1 < i_end) decode_item(p, sched_items[i + 1], nx);
      const int n_kv_tiles = im.n_kv_tiles;
      // the item's first Q K^T: S_w is free as soon as the previous item's last P_w V was issued (the tensor pipe runs in
      // order); it runs while the softmax warps still store the previous item's output
      ok = wait(tc::smem_u32(q_full), it & 1) && wait(b_kf + 8 * (gk & 1), (gk >> 1) & 1);
      if (!ok) break;
      if (leader) {
        issue_qk(0, gk & 1);
        tc::umma_commit(b_sf);
        issue_qk(1, gk & 1);
        tc::umma_commit(b_sf + 8);
        tc::umma_commit(b_ke + 8 * (gk & 1));
        if (n_kv_tiles == 1) tc::umma_commit(b_qe);
      }
      // O_w is overwritten by this item's first P V: the previous item's output must have been read out
      if (!wait(tc::smem_u32(o_empty), (it & 1) ^ 1)) { ok = false; break; }
      for (int j = 0; j < n_kv_tiles; ++j, ++gk) {
        const int s = gk & 1, s1 = s ^ 1;
        const uint32_t ph = (gk >> 1) & 1, ph1 = ph ^ s, pp = gk & 1;
        const bool more = j + 1 < n_kv_tiles, acc = j > 0;
        if (!wait(b_vf + 8 * s, ph) || !wait(b_p1, pp)) { ok = false; break; }
        if (leader) issue_pv(0, s, acc, 0);
        if (!wait(b_p2, pp)) { ok = false; break; }
        if (leader) issue_pv(0, s, acc, 1);
        if (more) {
          if (!wait(b_kf + 8 * s1, ph1)) { ok = false; break; }
          if (leader) {
            issue_qk(0, s1);
            tc::umma_commit(b_sf);
          }
        }
        if (!wait(b_p1 + 8, pp)) { ok = false; break; }
        if (leader) issue_pv(1, s, acc, 0);
        if (!wait(b_p2 + 8, pp)) { ok = false; break; }
        if (leader) {
          issue_pv(1, s, acc, 1);
          tc::umma_commit(b_ve + 8 * s);
          if (more) {
            issue_qk(1, s1);
            tc::umma_commit(b_sf + 8);
            tc::umma_commit(b_ke + 8 * s1);
            if (j + 2 == n_kv_tiles) tc::umma_commit(b_qe);     // the item's last Q K^T is in the pipe
          }
        }
      }
      if (ok && leader) tc::umma_commit(tc::smem_u32(o_full));
    }
    __syncwarp();
  } else {
    // -------------------------------------------------------------- softmax warps: head w, one row per thread
    const int w = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_s = tmem_base + lane_base + w * 128;
    const uint32_t t_o = tmem_base + lane_base + 256 + w * 128;
    const float c = p.scale_log2;
    int gk = 0;
    bool ok = true;
    int w_next = sched_items[i_begin];     // (only the index is fetched ahead here: these warps have no registers to spare)
    for (int i = i_begin; i < i_end && ok; ++i) {
      const int it = i - i_begin;
      AttnItem im;
      decode_item(p, w_next, im);
      if (i + 1 < i_end) w_next = sched_items[i + 1];
      const int n_kv_tiles = im.n_kv_tiles, past = im.past, qt = im.qt;
      float m_ref = -INFINITY, l = 0.f;
      for (int j = 0; j < n_kv_tiles; ++j, ++gk) {
        if (!wait_or_abort(tc::smem_u32(&s_full[w]), gk & 1, abort_flag, p.status)) { ok = false; break; }
        tc::tc_fence_after_sync();
        const int shift = past + qt * BQ - j * BKV;
        const bool diag = shift < BKV - 1;
        const int lim = row + shift;
        uint32_t s[128];
        tc::tmem_ld_32x32b_x32p(t_s, s);
        tc::tmem_ld_32x32b_x32p(t_s + 32, s + 32);
        tc::tmem_ld_wait();
        tc::tmem_ld_32x32b_x32p(t_s + 64, s + 64);
        tc::tmem_ld_32x32b_x32p(t_s + 96, s + 96);
        if (diag) {
#pragma unroll
          for (int e = 0; e < 64; ++e)
            if (e > lim) s[e] = 0xff800000u;   // -inf
        }
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
        for (int e = 0; e < 64; e += 8) {
          m0 = tc::max3(m0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
          m1 = tc::max3(m1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
          m2 = tc::max3(m2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
          m3 = tc::max3(m3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
        }
        tc::tmem_ld_wait();
        if (diag) {
#pragma unroll
          for (int e = 64; e < 128; ++e)
            if (e > lim) s[e] = 0xff800000u;
        }
#pragma unroll
        for (int e = 64; e < 128; e += 8) {
          m0 = tc::max3(m0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
          m1 = tc::max3(m1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
          m2 = tc::max3(m2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
          m3 = tc::max3(m3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
        }
        const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        const bool need = (j == 0) || ((mx - m_ref) * c > RESCALE_THRESHOLD);
        const float m_new = need ? mx : m_ref;
        if (j > 0 && __any_sync(0xffffffffu, need)) {
          const float f = need ? fast_exp2((m_ref - m_new) * c) : 1.f;
          l *= f;
#pragma unroll 1
          for (int ch = 0; ch < 8; ++ch) {
            uint32_t r[16];
            tc::tmem_ld_32x32b_x16(t_o + ch * 16, r);
            tc::tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
            tc::tmem_st_32x32b_x16(t_o + ch * 16, r);
          }
        }
        m_ref = m_new;
        const float neg_mc = -m_ref * c;
        float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
          for (int e = hf * 32; e < hf * 32 + 32; e += 2) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(s[2 * e]), c, neg_mc));
            const float p1 = fast_exp2(fmaf(__uint_as_float(s[2 * e + 1]), c, neg_mc));
            const float p2 = fast_exp2(fmaf(__uint_as_float(s[2 * e + 2]), c, neg_mc));
            const float p3 = fast_exp2(fmaf(__uint_as_float(s[2 * e + 3]), c, neg_mc));
            l0 += p0; l1 += p1; l2 += p2; l3 += p3;
            s[e] = ACT_F16 ? tc::pack_f16x2(p0, p1) : tc::pack_bf16x2(p0, p1);
            s[e + 1] = ACT_F16 ? tc::pack_f16x2(p2, p3) : tc::pack_bf16x2(p2, p3);
          }
          tc::tmem_st_32x32b_x32(t_s + hf * 32, s + hf * 32);
          tc::tmem_st_wait();
          tc::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(tc::smem_u32(hf == 1 ? &p_ready2[w] : &p_ready[w]));
        }
        l += (l0 + l1) + (l2 + l3);
      }
      if (!ok) break;
      // ---- epilogue of the item: O_w / l -> 16 bits -> out[token, head, :], then hand O_w back to the MMA warp
      if (!wait_or_abort(tc::smem_u32(o_full), it & 1, abort_flag, p.status)) { ok = false; break; }
      tc::tc_fence_after_sync();
      const float inv = 1.f / l;
      const bool valid = qt * BQ + row < im.n;
      bf16 *dst = p.out + ((size_t)(im.q_row0 + row) * p.n_q + (im.h0 + w)) * HD;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tc::tmem_ld_32x32b_x32(t_o + ch * 32, r);
        tc::tmem_ld_wait();
        if (ch == 3) {               // the last read of O_w is done: the next item's first P V may overwrite it
          tc::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(tc::smem_u32(o_empty));
        }
        if (valid) store_out_chunk<ACT_F16>(dst + ch * 32, r, inv, p.store32 != 0);
      }
    }
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
}



// ---------------------------------------------------------------------------------------------------------
// Extended-precision scores (activation format "half pairs"): q and K each arrive as a pair of half tensors, value =
// hi + lo, and S = Q K^T is accumulated from three tensor-core passes  Q_hi K_hi^T + Q_lo K_hi^T + Q_hi K_lo^T  (the
// lo-lo term is below fp32 rounding), so the scores carry ~22 significant bits of q and K instead of 11.  This is for
// models whose softmax is so sharp that the 2^-12 rounding of q and K dominates the end-to-end error (the 80-layer
// 70B shape with random weights).  Everything else is attention_tc_kernel: same roles, same softmax, P and V as single
// halves.  Shared memory: Q 4 tiles (hi, lo of two heads) + K 2 tiles (hi, lo) + V 1 tile = 224 KB, so the K and V
// rings have one stage each: the next key tile's K lands while the softmax warps work on the current scores, the next V
// while they work on the next scores.  out_split: output rows are [hi | lo] pairs, 2 * n_q * hd elements apart.
// ---------------------------------------------------------------------------------------------------------
constexpr int SPL_SM_Q = 0, SPL_SM_K = 4 * TILE_BYTES, SPL_SM_V = 6 * TILE_BYTES, SPL_SM_BAR = 7 * TILE_BYTES;
constexpr int SPL_SMEM = SPL_SM_BAR + 256 + 1024;

__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmQlo,
                          const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmKlo,
                          const __grid_constant__ CUtensorMap tmV, AttnParams p, int out_split) {
  const int n_pairs = p.n_q >> 1;
  const int per_tile = p.n_seqs * n_pairs;
  const int qt = p.max_tiles - 1 - (int)(blockIdx.x / per_tile);
  const int rem = blockIdx.x % per_tile;
  const int b = rem / n_pairs, pair = rem % n_pairs;
  const int tok0 = p.cu[b], n = p.cu[b + 1] - tok0;
  if (qt * BQ >= n) return;
  const int k0 = p.k_row0 ? p.k_row0[b] : tok0;
  const int past = p.kv_len ? p.kv_len[b] - n : 0;
  const int h0 = pair * 2;
  const int kvh = h0 / (p.n_q / p.n_kv);
  const int n_kv_tiles = (past + min(n, (qt + 1) * BQ) - 1) / BKV + 1;
  const int q_row0 = tok0 + qt * BQ;

  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SPL_SM_BAR);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 2, *v_full = bars + 3, *v_empty = bars + 4;
  uint64_t *s_full = bars + 5;        // [2]
  uint64_t *p_ready = bars + 7;       // [2]
  uint64_t *p_ready2 = bars + 9;      // [2]
  uint64_t *o_full = bars + 11;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 12);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(q_full), 1);
    tc::mbar_init(tc::smem_u32(k_full), 1);
    tc::mbar_init(tc::smem_u32(k_empty), 1);
    tc::mbar_init(tc::smem_u32(v_full), 1);
    tc::mbar_init(tc::smem_u32(v_empty), 1);
    for (int w = 0; w < 2; ++w) {
      tc::mbar_init(tc::smem_u32(&s_full[w]), 1);
      tc::mbar_init(tc::smem_u32(&p_ready[w]), 4);
      tc::mbar_init(tc::smem_u32(&p_ready2[w]), 4);
    }
    tc::mbar_init(tc::smem_u32(o_full), 1);
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmQ);
    tc::tma_prefetch_desc(&tmQlo);
    tc::tma_prefetch_desc(&tmK);
    tc::tma_prefetch_desc(&tmKlo);
    tc::tma_prefetch_desc(&tmV);
  }
  if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------ TMA producer
      const uint32_t qb = tc::smem_u32(q_full);
      tc::mbar_expect_tx(qb, 4 * TILE_BYTES);
      for (int w = 0; w < 2; ++w)
        for (int c = 0; c < 2; ++c) {
          tc::tma_load_2d(tc::smem_u32(smem + SPL_SM_Q + w * TILE_BYTES + c * CHUNK_BYTES), &tmQ, qb, (h0 + w) * HD + c * 64, q_row0);
          tc::tma_load_2d(tc::smem_u32(smem + SPL_SM_Q + (2 + w) * TILE_BYTES + c * CHUNK_BYTES), &tmQlo, qb, (h0 + w) * HD + c * 64, q_row0);
        }
      for (int j = 0; j < n_kv_tiles; ++j) {
        const uint32_t ph = j & 1;
        const int krow = p.blk ? p.blk[(size_t)b * p.blk_stride + j] * BKV : k0 + j * BKV;
        if (!wait_or_abort(tc::smem_u32(k_empty), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t kb = tc::smem_u32(k_full);
        tc::mbar_expect_tx(kb, 2 * TILE_BYTES);
        for (int c = 0; c < 2; ++c) {
          tc::tma_load_2d(tc::smem_u32(smem + SPL_SM_K + c * CHUNK_BYTES), &tmK, kb, kvh * HD + c * 64, krow);
          tc::tma_load_2d(tc::smem_u32(smem + SPL_SM_K + TILE_BYTES + c * CHUNK_BYTES), &tmKlo, kb, kvh * HD + c * 64, krow);
        }
        if (!wait_or_abort(tc::smem_u32(v_empty), ph ^ 1, abort_flag, p.status)) break;
        const uint32_t vb = tc::smem_u32(v_full);
        tc::mbar_expect_tx(vb, TILE_BYTES);
        for (int c = 0; c < 2; ++c)
          tc::tma_load_2d(tc::smem_u32(smem + SPL_SM_V + c * CHUNK_BYTES), &tmV, vb, kvh * HD + c * 64, krow);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (warp-uniform, one elected lane)
    const bool leader = tc::elect_one();
    constexpr uint32_t idesc_qk = tc::umma_idesc(BQ, BKV, 0, 0, 1, 1);
    constexpr uint32_t idesc_pv = tc::umma_idesc(BQ, HD, 0, 1, 1, 1);
    const uint64_t q_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SPL_SM_Q), 16, 1024);
    const uint64_t k_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SPL_SM_K), 16, 1024);
    const uint64_t v_desc0 = tc::umma_desc_sw128(tc::smem_u32(smem + SPL_SM_V), CHUNK_BYTES, 1024);
    auto issue_qk = [&](int w) {   // S_w = Q_hi K_hi^T + Q_lo K_hi^T + Q_hi K_lo^T, 8 steps of 16 along the head dim each
      const uint64_t qh = q_desc0 + (uint64_t)(w * (TILE_BYTES >> 4)), ql = q_desc0 + (uint64_t)((2 + w) * (TILE_BYTES >> 4));
      const uint64_t kh = k_desc0, kl = k_desc0 + (uint64_t)(TILE_BYTES >> 4);
      const uint32_t d = tmem_base + w * 128;
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const uint32_t off = ((kk >> 2) * CHUNK_BYTES + (kk & 3) * 32) >> 4;
        tc::umma_ss(d, qh + off, kh + off, idesc_qk, kk != 0);
        tc::umma_ss(d, ql + off, kh + off, idesc_qk, 1u);
        tc::umma_ss(d, qh + off, kl + off, idesc_qk, 1u);
      }
    };
    auto issue_pv = [&](int w, bool accumulate, int half) {
      const uint32_t d = tmem_base + 256 + w * 128, a_t = tmem_base + w * 128;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const int kk = half * 4 + k4;
        tc::umma_ts(d, a_t + kk * 8, v_desc0 + (uint64_t)((kk * 16 * 128) >> 4), idesc_pv, (accumulate || kk != 0) ? 1u : 0u);
      }
    };
    const uint32_t b_kf = tc::smem_u32(k_full), b_ke = tc::smem_u32(k_empty), b_vf = tc::smem_u32(v_full), b_ve = tc::smem_u32(v_empty),
                   b_sf = tc::smem_u32(&s_full[0]), b_p1 = tc::smem_u32(&p_ready[0]), b_p2 = tc::smem_u32(&p_ready2[0]);
    auto wait = [&](uint32_t bar, uint32_t parity) {
      const bool ok = wait_or_abort(bar, parity, abort_flag, p.status);
      tc::tc_fence_after_sync();
      return ok;
    };
    bool ok = wait(tc::smem_u32(q_full), 0) && wait(b_kf, 0);
    if (ok && leader) {
      issue_qk(0);
      tc::umma_commit(b_sf);
      issue_qk(1);
      tc::umma_commit(b_sf + 8);
      tc::umma_commit(b_ke);
    }
    for (int j = 0; j < n_kv_tiles && ok; ++j) {
      const uint32_t ph = j & 1;
      const bool more = j + 1 < n_kv_tiles, acc = j > 0;
      if (!wait(b_vf, ph) || !wait(b_p1, ph)) { ok = false; break; }
      if (leader) issue_pv(0, acc, 0);
      if (!wait(b_p2, ph)) { ok = false; break; }
      if (leader) issue_pv(0, acc, 1);
      if (more) {
        if (!wait(b_kf, ph ^ 1)) { ok = false; break; }
        if (leader) {
          issue_qk(0);
          tc::umma_commit(b_sf);
        }
      }
      if (!wait(b_p1 + 8, ph)) { ok = false; break; }
      if (leader) issue_pv(1, acc, 0);
      if (!wait(b_p2 + 8, ph)) { ok = false; break; }
      if (leader) {
        issue_pv(1, acc, 1);
        tc::umma_commit(b_ve);
        if (more) {
          issue_qk(1);
          tc::umma_commit(b_sf + 8);
          tc::umma_commit(b_ke);
        }
      }
    }
    if (ok && leader) tc::umma_commit(tc::smem_u32(o_full));
    __syncwarp();
  } else {
    // -------------------------------------------------------------- softmax warps: head w, one row per thread
    const int w = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t t_s = tmem_base + lane_base + w * 128;
    const uint32_t t_o = tmem_base + lane_base + 256 + w * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv_tiles; ++j) {
      if (!wait_or_abort(tc::smem_u32(&s_full[w]), j & 1, abort_flag, p.status)) { ok = false; break; }
      tc::tc_fence_after_sync();
      const int shift = past + qt * BQ - j * BKV;
      const bool diag = shift < BKV - 1;
      const int lim = row + shift;
      uint32_t s[128];
      tc::tmem_ld_32x32b_x32p(t_s, s);
      tc::tmem_ld_32x32b_x32p(t_s + 32, s + 32);
      tc::tmem_ld_32x32b_x32p(t_s + 64, s + 64);
      tc::tmem_ld_32x32b_x32p(t_s + 96, s + 96);
      tc::tmem_ld_wait();
      if (diag) {
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i > lim) s[i] = 0xff800000u;   // -inf
      }
      float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 128; i += 8) {
        m0 = tc::max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        m1 = tc::max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        m2 = tc::max3(m2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        m3 = tc::max3(m3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
      }
      const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      const bool need = (j == 0) || ((mx - m_ref) * c > RESCALE_THRESHOLD);
      const float m_new = need ? mx : m_ref;
      if (j > 0 && __any_sync(0xffffffffu, need)) {
        const float f = need ? fast_exp2((m_ref - m_new) * c) : 1.f;
        l *= f;
#pragma unroll 1
        for (int ch = 0; ch < 8; ++ch) {
          uint32_t r[16];
          tc::tmem_ld_32x32b_x16(t_o + ch * 16, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
          tc::tmem_st_32x32b_x16(t_o + ch * 16, r);
        }
      }
      m_ref = m_new;
      const float neg_mc = -m_ref * c;
      float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int i = hf * 32; i < hf * 32 + 32; i += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(s[2 * i]), c, neg_mc));
          const float p1 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 1]), c, neg_mc));
          const float p2 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 2]), c, neg_mc));
          const float p3 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 3]), c, neg_mc));
          l0 += p0; l1 += p1; l2 += p2; l3 += p3;
          s[i] = tc::pack_f16x2(p0, p1);
          s[i + 1] = tc::pack_f16x2(p2, p3);
        }
        tc::tmem_st_32x32b_x32(t_s + hf * 32, s + hf * 32);
        tc::tmem_st_wait();
        tc::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(tc::smem_u32(hf == 1 ? &p_ready2[w] : &p_ready[w]));
      }
      l += (l0 + l1) + (l2 + l3);
    }
    // ---- epilogue: O_w / l -> half (and the low halves, if asked for) -> out[token, head, :]
    if (ok && wait_or_abort(tc::smem_u32(o_full), 0, abort_flag, p.status)) {
      tc::tc_fence_after_sync();
      const float inv = 1.f / l;
      const bool valid = qt * BQ + row < n;
      const size_t dq = (size_t)p.n_q * HD;
      const size_t o_off = (size_t)(q_row0 + row) * (out_split ? 2 * dq : dq) + (size_t)(h0 + w) * HD;
      __half *out_lo = out_split ? reinterpret_cast<__half *>(p.out) + dq : nullptr;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tc::tmem_ld_32x32b_x32(t_o + ch * 32, r);
        tc::tmem_ld_wait();
        if (valid) {
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float a = __uint_as_float(r[2 * i]) * inv, bq = __uint_as_float(r[2 * i + 1]) * inv;
            hi[i] = tc::pack_f16x2(a, bq);
            const float2 hf2 = __half22float2(*reinterpret_cast<const __half2 *>(&hi[i]));
            lo[i] = tc::pack_f16x2(a - hf2.x, bq - hf2.y);
          }
          uint4 *d4 = reinterpret_cast<uint4 *>(p.out + o_off + ch * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) d4[i] = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
          if (out_lo) {
            uint4 *l4 = reinterpret_cast<uint4 *>(out_lo + o_off + ch * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) l4[i] = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
          }
        }
      }
    }
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

int attention_schedule(const int32_t *n_new, const int32_t *n_past, int n_seqs, int n_q, int n_ctas, int32_t *off, int32_t *items) {
  const int n_pairs = n_q / 2;
  int max_tiles = 0;
  for (int b = 0; b < n_seqs; ++b) max_tiles = std::max(max_tiles, (n_new[b] + BQ - 1) / BQ);
  const int per_tile = n_seqs * n_pairs;
  // (cost in key tiles, item index); what a CTA pays per item besides its key tiles is worth about 3 of them
  std::vector<std::pair<int, int>> work;
  for (int qt = max_tiles - 1; qt >= 0; --qt)
    for (int b = 0; b < n_seqs; ++b) {
      if (qt * BQ >= n_new[b]) continue;
      const int tiles = (n_past[b] + std::min(n_new[b], (qt + 1) * BQ) - 1) / BKV + 1;
      for (int pr = 0; pr < n_pairs; ++pr) work.emplace_back(tiles + 3, (max_tiles - 1 - qt) * per_tile + b * n_pairs + pr);
    }
  std::stable_sort(work.begin(), work.end(), [](const std::pair<int, int> &x, const std::pair<int, int> &y) { return x.first > y.first; });
  // least loaded CTA first (ties: lowest index)
  std::priority_queue<std::pair<long long, int>, std::vector<std::pair<long long, int>>, std::greater<std::pair<long long, int>>> heap;
  for (int c = 0; c < n_ctas; ++c) heap.emplace(0LL, c);
  std::vector<int> owner(work.size());
  std::vector<int32_t> count(n_ctas, 0);
  for (size_t i = 0; i < work.size(); ++i) {
    auto top = heap.top();
    heap.pop();
    owner[i] = top.second;
    ++count[top.second];
    heap.emplace(top.first + work[i].first, top.second);
  }
  off[0] = 0;
  for (int c = 0; c < n_ctas; ++c) off[c + 1] = off[c] + count[c];
  std::vector<int32_t> fill(off, off + n_ctas);
  for (size_t i = 0; i < work.size(); ++i) items[fill[owner[i]]++] = work[i].second;
  return (int)work.size();
}

bool tc_attention_supported(int n_q, int n_kv, int hd) {
  return hd == HD && n_kv >= 1 && n_q % n_kv == 0 && ((n_q / n_kv) % 2) == 0;
}

int launch_attention_tc(const void *q, bool act_f16, const void *k, const void *v, void *out, const int32_t *cu_seqlens,
                        const int32_t *k_row0, const int32_t *kv_len, const int32_t *blk, int blk_stride, int n_seqs,
                        int n_tokens, int kv_rows, int max_seq_len, int n_q, int n_kv, int hd, unsigned int *status,
                        cudaStream_t st, AttnSchedule sched) {
  if (!tc_attention_supported(n_q, n_kv, hd)) return SWIFTKV_ERR_UNSUPPORTED;
  if (n_tokens < 1 || n_seqs < 1 || max_seq_len < 1 || kv_rows < 1) return SWIFTKV_ERR_INVALID_ARG;
  CUtensorMap tq, tk, tv;
  // row extents = the rows that hold data of this call: rows past them read as zero (never stale memory)
  if (get_tmap(&tq, q, n_tokens, (uint64_t)n_q * hd, (uint64_t)n_q * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tk, k, kv_rows, (uint64_t)n_kv * hd, (uint64_t)n_kv * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tv, v, kv_rows, (uint64_t)n_kv * hd, (uint64_t)n_kv * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_kernel<false, false>), ATT_SMEM) ||
      ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_kernel<true, false>), ATT_SMEM) ||
      ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_kernel<false, true>), ATT_SMEM) ||
      ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_kernel<true, true>), ATT_SMEM))
    return SWIFTKV_ERR_CUDA;
  AttnParams p{};
  p.cu = cu_seqlens; p.k_row0 = k_row0; p.kv_len = kv_len; p.blk = blk; p.blk_stride = blk_stride; p.out = reinterpret_cast<bf16 *>(out); p.n_seqs = n_seqs; p.n_q = n_q; p.n_kv = n_kv;
  p.max_tiles = (max_seq_len + BQ - 1) / BQ;
  p.scale_log2 = (1.0f / sqrtf((float)hd)) * 1.4426950408889634f;
  p.status = status;
  p.store32 = (reinterpret_cast<uintptr_t>(out) & 31) == 0;
  const long long grid = (long long)p.max_tiles * n_seqs * (n_q / 2);
  if (grid > 0x7fffffffLL) return SWIFTKV_ERR_UNSUPPORTED;
  if (sched.off && sched.items && sched.n_ctas > 0) {
    if (ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_persistent_kernel<false>), ATT_SMEM) ||
        ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_persistent_kernel<true>), ATT_SMEM))
      return SWIFTKV_ERR_CUDA;
    if (act_f16) attention_tc_persistent_kernel<true><<<(unsigned)sched.n_ctas, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p, sched.off, sched.items);
    else attention_tc_persistent_kernel<false><<<(unsigned)sched.n_ctas, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p, sched.off, sched.items);
    return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
  }
  static int split = -1;
  if (split < 0) { const char *e = getenv("SWIFTKV_ATT_SPLIT_P"); split = e ? atoi(e) : 1; }
  if (act_f16) {
    if (split) attention_tc_kernel<true, true><<<(unsigned)grid, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p);
    else attention_tc_kernel<true, false><<<(unsigned)grid, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p);
  } else {
    if (split) attention_tc_kernel<false, true><<<(unsigned)grid, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p);
    else attention_tc_kernel<false, false><<<(unsigned)grid, ATT_THREADS, ATT_SMEM, st>>>(tq, tk, tv, p);
  }
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

int launch_attention_tc_split(const void *q_hi, const void *q_lo, const void *k_hi, const void *k_lo, const void *v, void *out,
                              bool out_split, const int32_t *cu_seqlens, int n_seqs, int n_tokens, int max_seq_len, int n_q, int n_kv,
                              int hd, unsigned int *status, cudaStream_t st) {
  if (!tc_attention_supported(n_q, n_kv, hd)) return SWIFTKV_ERR_UNSUPPORTED;
  if (n_tokens < 1 || n_seqs < 1 || max_seq_len < 1) return SWIFTKV_ERR_INVALID_ARG;
  CUtensorMap tq, tql, tk, tkl, tv;
  if (get_tmap(&tq, q_hi, n_tokens, (uint64_t)n_q * hd, (uint64_t)n_q * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tql, q_lo, n_tokens, (uint64_t)n_q * hd, (uint64_t)n_q * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tk, k_hi, n_tokens, (uint64_t)n_kv * hd, (uint64_t)n_kv * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tkl, k_lo, n_tokens, (uint64_t)n_kv * hd, (uint64_t)n_kv * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (get_tmap(&tv, v, n_tokens, (uint64_t)n_kv * hd, (uint64_t)n_kv * hd, 128, 64)) return SWIFTKV_ERR_CUDA;
  if (ensure_dynamic_smem(reinterpret_cast<const void *>(attention_tc_split_kernel), SPL_SMEM)) return SWIFTKV_ERR_CUDA;
  AttnParams p{};
  p.cu = cu_seqlens; p.k_row0 = nullptr; p.kv_len = nullptr; p.blk = nullptr; p.blk_stride = 0;
  p.out = reinterpret_cast<bf16 *>(out); p.n_seqs = n_seqs; p.n_q = n_q; p.n_kv = n_kv;
  p.max_tiles = (max_seq_len + BQ - 1) / BQ;
  p.scale_log2 = (1.0f / sqrtf((float)hd)) * 1.4426950408889634f;
  p.status = status;
  p.store32 = 0;
  const long long grid = (long long)p.max_tiles * n_seqs * (n_q / 2);
  if (grid > 0x7fffffffLL) return SWIFTKV_ERR_UNSUPPORTED;
  attention_tc_split_kernel<<<(unsigned)grid, ATT_THREADS, SPL_SMEM, st>>>(tq, tql, tk, tkl, tv, p, out_split ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? SWIFTKV_OK : SWIFTKV_ERR_CUDA;
}

}  // namespace skv
