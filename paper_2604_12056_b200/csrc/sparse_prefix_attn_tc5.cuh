// Stage 4, bf16, 5th-generation tensor cores: included by sparse_prefix_attn.cu (same namespace;
// the flat work decomposition, the partial-record format and the combine kernel are described there).
//
// A CTA owns up to 128 GQA-grouped query rows of one (sequence, KV head) at a time: the M = 128 rows
// of every MMA, one row per tensor-memory lane.  Pages are taken in groups of 128 tokens (PG pages):
//   S[128 x 128]  = Q . K^T      A = Q from tensor memory (bf16, written there once per piece),
//                                B = the group's K tiles, K-major in shared memory (128-byte swizzle,
//                                as TMA wrote them); D / 16 instructions
//   softmax       eight warps, thread = (query row, half of the columns): the row's scores are read
//                 from tensor memory once, the maximum is exchanged with the partner thread, then
//                 P = 2^(s - m); the reference maximum m only moves when it would grow by more than
//                 2^8 (then O is rescaled in place); P is rounded to bf16 and written over the
//                 scores it came from
//   O[128 x D]   += P . V        A = P from tensor memory, B = the group's V tiles as they lie in
//                                memory (tokens x d: MN-major); 8 instructions
// Issuing one tcgen05.mma costs the issuing thread ~120 cycles whatever its shape (measured), so the
// shapes are as large as the layout allows and the two products have an issuing thread each.
// K and V have a ring of group-sized slots each, filled by one producer warp each (lane = page:
// 32 pages' copies are issued by one instruction); a K slot is free again as soon as its Q K^T has
// run, a V slot after its P V.  S is double-buffered.  Completion is tracked with tcgen05.commit on
// mbarriers; every wait is bounded; tensor memory is returned on every path.
#pragma once

constexpr int kTc5SoftmaxWarps = 8;              // two sets of four: set h takes columns 64h .. 64h+63 of every group
constexpr int kTc5QkWarp = 8, kTc5PvWarp = 9, kTc5KWarp = 10, kTc5VWarp = 11;
constexpr int kTc5Threads = 384;
constexpr int kTc5Tok = 128;                     // tokens per group = N of Q K^T = columns of one S buffer
constexpr int kTc5PgMax = 8;                     // pages per group at the smallest page size (16)
constexpr int kTc5MetaRing = 16;                 // groups whose per-page token counts are kept (producer lead < 16)
constexpr float kTc5Tau = 8.0f;                  // reference maximum moves only when it would grow by more than this (log2 units)
constexpr int kTc5XchgBytes = (2 * 2 + 1) * kRowsPerGroup * 4;   // row maxima [group parity][set][row], row sums [row]
constexpr int kTc5ScaleBytes = 2 * kTc5MetaRing * (kTc5PgMax + 1) * 4;   // FP8 pages: per-page scales and page counts of the groups in flight, K and V
constexpr int kTc5TailBytes = kTailBytes + 512 + kTc5XchgBytes + kTc5ScaleBytes + (kMaxSegments + 1) * 4;  // 1024 bytes of barriers + page meta, the segment prefix and index cache, the exchange arrays, the scales
constexpr int kTc5Stg = 2;                       // FP8 pages: staging slots (bytes as they lie in memory) per tensor

template <int D> constexpr int tc5_slot_bytes() { return kTc5Tok * D * 2; }
template <int D> constexpr int tc5_stg_bytes() { return kTc5Tok * D; }
template <int D, bool FP8> constexpr int tc5_ring_slots() {     // per ring (K and V have one each)
  if (FP8) return 2;                                            // the staging slots take the rest
  const int n = (kSmemBudget - 1024 - kTc5TailBytes) / tc5_slot_bytes<D>() / 2;
  return n > 6 ? 6 : n;
}
template <int D, bool FP8> constexpr int tc5_smem_bytes() {
  return 1024 + 2 * tc5_ring_slots<D, FP8>() * tc5_slot_bytes<D>() + (FP8 ? 2 * kTc5Stg * tc5_stg_bytes<D>() : 0) + kTc5TailBytes;
}

// Shared-memory matrix descriptor: 128-byte swizzle, 8-row groups 1024 bytes apart; lbo = distance
// between 64-element blocks along the MN dimension of an MN-major operand.
__device__ __forceinline__ uint64_t tc5_desc(uint32_t saddr, uint32_t lbo) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16) |
         (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, A and B both bf16 (fmt 1) or both fp16 (fmt 0),
// M x N tile, B optionally MN-major.
__device__ __forceinline__ uint32_t tc5_idesc(int M, int N, int b_mn_major, uint32_t fmt = 1u) {
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
         (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem] . B[smem descriptor]
__device__ __forceinline__ void tc5_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc5_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc5_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc5_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// tcgen05.ld of 32 consecutive 32-bit columns of this thread's lane; the wait is part of the same
// statement so that no use of the registers can be scheduled ahead of it.
__device__ __forceinline__ void tc5_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// The same load without the wait: several can be in flight; tc5_wait_ld() then tc5_pin32() on each
// destination before any use (the empty statement ties the registers to a point after the wait).
__device__ __forceinline__ void tc5_ld32_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc5_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc5_pin32(uint32_t* r) {
#pragma unroll
  for (int i = 0; i < 32; ++i) asm volatile("" : "+r"(r[i]) :: "memory");
}
__device__ __forceinline__ void tc5_st16(uint32_t taddr, const uint32_t* w) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "r"(w[8]),
        "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15])
      : "memory");
}
__device__ __forceinline__ void tc5_st32(uint32_t taddr, const uint32_t* w) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "r"(w[8]),
        "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]), "r"(w[16]), "r"(w[17]),
        "r"(w[18]), "r"(w[19]), "r"(w[20]), "r"(w[21]), "r"(w[22]), "r"(w[23]), "r"(w[24]), "r"(w[25]), "r"(w[26]),
        "r"(w[27]), "r"(w[28]), "r"(w[29]), "r"(w[30]), "r"(w[31])
      : "memory");
}
__device__ __forceinline__ void tc5_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// byte offset of 16-byte chunk c (0..7) of row t in a [rows][128 B] tile with the 128-byte swizzle
__device__ __forceinline__ uint32_t tc5_sw(int t, int c) { return static_cast<uint32_t>(t * 128 + ((c ^ (t & 7)) << 4)); }

// FP8: the K / V pools hold E4M3 bytes with one power-of-two scale per (page, KV head).  The page
// copies land in staging slots as they lie in memory (half the bytes); the producer warp that issued
// them converts a landed group to fp16 times its page's scale (exact) into the ring slot, in the
// layout the tensor maps of the bf16 path produce, and every MMA runs on fp16 operands (Q and P are
// converted to fp16 instead of bf16); nothing else changes.
template <int D, int GP, bool FP8>
__global__ void __launch_bounds__(kTc5Threads, 1)
attn_tc5_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  constexpr int NR = tc5_ring_slots<D, FP8>();  // slots per ring
  constexpr int NSTG = kTc5Stg, STG = tc5_stg_bytes<D>();
  constexpr uint32_t FMT = FP8 ? 0u : 1u;       // operand format of the MMAs: fp16 / bf16
  constexpr int SLOT = tc5_slot_bytes<D>();
  constexpr int PG = kTc5Tok / GP;              // pages per group
  constexpr int HALVES = D / 64;                // 64-column (128-byte) blocks of a K or V row
  constexpr int HS = kTc5Tok * 128;             // bytes of one such block of a whole group
  constexpr int PAGE_BYTES = GP * D * 2;        // of K, and of V
  constexpr uint32_t COL_O = 0, COL_S = 128, COL_Q = 384;   // tensor-memory columns: O[D], S0[128], S1[128], Q[D/2]
  constexpr int TMEM_COLS = 512;
  static_assert(D == 64 || D == 128, "head dimensions of the tensor-core path");
  static_assert(GP == 16 || GP == 32 || GP == 64, "page sizes of the tensor-core path");
  static_assert(NR >= 2 && PG <= kTc5PgMax, "ring too shallow / group too long");
  static_assert(8 * (4 * 6 + 14 + 2 * kTc5Stg) + 4 * kTc5MetaRing * kTc5PgMax + 16 <= 1024, "tail layout");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t kring = base, vring = base + NR * SLOT;
  constexpr int STG_ALL = FP8 ? 2 * NSTG * STG : 0;
  const uint32_t kstg = base + 2 * NR * SLOT, vstg = kstg + NSTG * STG;          // FP8 only
  uint8_t* tail = gen + 2 * NR * SLOT + STG_ALL;
  const uint32_t tail_s = base + 2 * NR * SLOT + STG_ALL;
  const uint32_t kfull = tail_s, kfree = kfull + 8 * NR, vfull = kfree + 8 * NR, vfree = vfull + 8 * NR;
  const uint32_t s_full = vfree + 8 * NR, s_free = s_full + 16, p_full = s_free + 16, q_full = p_full + 16, q_free = q_full + 8, xbar = q_free + 8;
  const uint32_t drain_bar = xbar + 32;            // two barriers: the issuing threads' last commit when the CTA gives up
  const uint32_t kstg_full = drain_bar + 16, vstg_full = kstg_full + 8 * NSTG;   // FP8: a staging slot's copies have landed
  volatile int* meta = reinterpret_cast<volatile int*>(tail + 8 * (4 * 6 + 14 + 2 * kTc5Stg));   // [kTc5MetaRing][kTc5PgMax] valid tokens per page
  volatile int* abort_flag = meta + kTc5MetaRing * kTc5PgMax;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(abort_flag) + 1);
  int* pre = reinterpret_cast<int*>(tail + 1024);
  int* tok_s = pre + kMaxSegments + 2;
  int* na_s = tok_s + kStageIdx;
  int* len_s = na_s + kStageSeq;
  float* xmax = reinterpret_cast<float*>(len_s + kStageSeq);   // [2][2][128]
  float* xsum = xmax + 4 * kRowsPerGroup;                        // [128]
  volatile float* scale_meta = xsum + kRowsPerGroup;             // FP8: [2 (K, V)][kTc5MetaRing][kTc5PgMax] page scales,
  volatile int* ng_meta = reinterpret_cast<volatile int*>(const_cast<float*>(scale_meta) + 2 * kTc5MetaRing * kTc5PgMax);   // [2][kTc5MetaRing] pages per group
  int* vpre = const_cast<int*>(ng_meta) + 2 * kTc5MetaRing;       // prefix of the charged segment lengths (pages + pad)
  const bool staged = p.N * p.B <= kStageIdx && p.N <= kStageSeq;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < NR; ++i) {
      mbar_init(kfull + 8 * i, 1);
      mbar_init(kfree + 8 * i, 1);
      mbar_init(vfull + 8 * i, 1);
      mbar_init(vfree + 8 * i, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s_full + 8 * b, 1);                  // tcgen05.commit after Q K^T
      mbar_init(s_free + 8 * b, 1);                  // tcgen05.commit after P V: the S buffer is free and O holds the group
      mbar_init(p_full + 8 * b, kTc5SoftmaxWarps);
    }
    mbar_init(q_full, kTc5SoftmaxWarps);
    mbar_init(q_free, 1);
    for (int i = 0; i < 4; ++i) mbar_init(xbar + 8 * i, 2);      // the two softmax warps of a scheduler meet here
    mbar_init(drain_bar, 1);
    mbar_init(drain_bar + 8, 1);
    if (FP8)
      for (int i = 0; i < NSTG; ++i) {
        mbar_init(kstg_full + 8 * i, 1);
        mbar_init(vstg_full + 8 * i, 1);
      }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {                                 // tensor memory: taken while the previous kernel drains
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  grid_dep_trigger();
  grid_dep_wait();                                 // nothing above touches global memory
  if (warp == 0) {
    segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane, vpre);
  } else if (staged) {
    for (int i = tid - 32; i < p.N * p.B; i += kTc5Threads - 32) tok_s[i] = p.active_idx[i];
    for (int i = tid - 32; i < p.N; i += kTc5Threads - 32) {
      na_s[i] = clamp_active(p.n_active[i], p.B);
      len_s[i] = p.kv_len[i];
    }
  }
  tc5_fence_before();
  __syncthreads();
  tc5_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (blockIdx.x == 0)                             // the combine kernel reads the prefix instead of recomputing it
    for (int i = tid; i <= p.n_seg; i += kTc5Threads) p.seg_prefix[i] = vpre[i];
  // this CTA's share of the charged list, mapped back to pages: the first page at or after a charged position
  const long long V_all = vpre[p.n_seg];
  auto page_at = [&](long long v) {
    if (v >= V_all) return pre[p.n_seg];
    int a = 0, b = p.n_seg;                          // vpre[a] <= v < vpre[b]
    while (b - a > 1) {
      const int mid = (a + b) >> 1;
      if (vpre[mid] <= v) a = mid; else b = mid;
    }
    const int len = pre[a + 1] - pre[a], pad = vpre[a + 1] - vpre[a] - len;
    const int off = static_cast<int>(v - vpre[a]) - pad;
    return pre[a] + (off < 0 ? 0 : off);
  };
  const int lo = page_at(cta_lo(V_all, blockIdx.x, p.n_ctas));
  const int hi = page_at(cta_lo(V_all, blockIdx.x + 1, p.n_ctas));
  if (lo >= hi) {                                  // nothing to do: give the tensor memory back
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TMEM_COLS) : "memory");
    return;
  }
  int sg0 = 0;
  while (pre[sg0 + 1] <= lo) ++sg0;
  auto n_active_of = [&](int s) { return staged ? na_s[s] : clamp_active(p.n_active[s], p.B); };
  auto kv_len_of = [&](int s) { return staged ? len_s[s] : p.kv_len[s]; };
  auto token_of = [&](int s, int a) { return staged ? tok_s[s * p.B + a] : p.active_idx[s * p.B + a]; };

  int issued = -1;                                   // producer warps: newest group whose copies have been issued
  if (warp == kTc5KWarp || warp == kTc5VWarp) {
    // ------------------------------------------------------------------ producer warps: one for K, one for V
    // Lane j of a batch of 32 consecutive items resolves item -> logical page -> physical page (a
    // three-stage pipeline over batches, the two dependent loads of different batches in flight
    // together) and later issues that page's copies itself.  A piece's items are cut into groups of
    // PG pages; the first lane of a group's run waits for the group's ring slot and announces the
    // group's bytes, then every lane of the run issues its page.
    const bool is_v = warp == kTc5VWarp;
    const unsigned long long policy = l2_evict_first_policy();
    const CUtensorMap* map = is_v ? &tmV : &tmK;
    const uint32_t ring = is_v ? vring : kring, full0 = is_v ? vfull : kfull, free0 = is_v ? vfree : kfree;
    int cursor = sg0, gbase = 0, pstart = lo;       // segment of the lane's newest item, groups before its piece, the piece's first item
    struct Item { int page, sk, grp, j, ng; };
    struct Ready { int phys, kh, valid, grp, j, ng; };
    auto stage_a = [&](int i) {
      Item it{-1, 0, 0, 0, 0};
      if (i < hi) {
        while (pre[cursor + 1] <= i) {
          gbase += (pre[cursor + 1] - pstart + PG - 1) / PG;
          ++cursor;
          pstart = pre[cursor];
        }
        const int q = i - pstart, seg_end = min(hi, pre[cursor + 1]);
        it.sk = cursor % (p.n_seg / p.n_rg);
        it.grp = gbase + q / PG;
        it.j = q % PG;
        it.ng = min(PG, seg_end - (i - it.j));
        it.page = ld_nc_s32(p.union_pages + static_cast<size_t>(it.sk) * p.Pmax + (i - pre[cursor]));
      }
      return it;
    };
    auto stage_b = [&](int i, const Item& it) {
      Ready r{0, 0, 0, it.grp, it.j, it.ng};
      if (i < hi) {
        const int s = it.sk / p.Hkv;
        r.kh = it.sk % p.Hkv;
        const bool ok = it.page >= 0 && it.page < p.Pmax;
        r.phys = ok ? ld_nc_s32(p.page_table + static_cast<size_t>(s) * p.Pmax + it.page) : -1;
        r.valid = ok ? min(GP, kv_len_of(s) - it.page * GP) : 0;
      }
      return r;
    };
    if constexpr (FP8) {
      // ---- FP8 pages.  The copies go to staging slots (NSTG groups in flight); before a staging slot
      // is reused, and at the end, this warp converts the groups that have landed: bytes -> fp16
      // times the page's scale, written where the tensor maps of the bf16 path would have put them
      // (two 128-byte-swizzled blocks per row), then announced to the MMA warps.
      const uint32_t stg = is_v ? vstg : kstg, stg_full0 = is_v ? vstg_full : kstg_full;
      uint8_t* stg_gen = gen + (stg - base);
      uint8_t* ring_gen = gen + (ring - base);
      volatile float* sc_meta = scale_meta + (is_v ? kTc5MetaRing * kTc5PgMax : 0);
      volatile int* ngs = ng_meta + (is_v ? kTc5MetaRing : 0);
      const float* scale_g = is_v ? p.v_scale : p.k_scale;
      constexpr int CPRW = D / 16;                    // 16-byte chunks of a row of bytes
      int conv = 0;                                   // groups converted so far
      bool go = true;
      auto convert = [&](int gc) {
        const int ss = gc % NSTG, sr = gc % NR;
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(stg_full0 + 8 * ss, (gc / NSTG) & 1, abort_flag, p.status, p.wait_cycles);
          if (ok && gc >= NR) ok = mbar_wait(free0 + 8 * sr, (gc / NR - 1) & 1, abort_flag, p.status, p.wait_cycles);
        }
        if (__shfl_sync(0xffffffffu, ok, 0) == 0) return false;
        // Lane = (token within a batch of TPI, 16-byte chunk of the row); U batches are loaded before
        // any is converted, so that the warp - alone with this work - has independent chains in flight.
        // A byte s.eeee.mmm becomes the fp16 s.0eeee.mmm0000000 = its value / 256 (E4M3 subnormals land on
        // fp16 subnormals), then one packed multiply by 256 * scale, exact; the quantiser never writes
        // the NaN code.
        constexpr int TPI = 32 / CPRW, U = (GP / TPI) < 4 ? (GP / TPI) : 4;
        const int npg = ngs[gc % kTc5MetaRing];
        const int tl = lane / CPRW, c8 = lane % CPRW, c = 2 * (c8 & 3);
        const uint8_t* src = stg_gen + ss * STG + tl * D + c8 * 16;
        uint8_t* row = ring_gen + sr * SLOT + (c8 >> 2) * HS;
        for (int pg = 0; pg < npg; ++pg) {
          const __half2 sc2 = __float2half2_rn(256.f * sc_meta[(gc % kTc5MetaRing) * kTc5PgMax + pg]);
          for (int t0 = pg * GP; t0 < (pg + 1) * GP; t0 += TPI * U) {
            uint4 rawb[U];
#pragma unroll
            for (int u = 0; u < U; ++u) rawb[u] = *reinterpret_cast<const uint4*>(src + (t0 + u * TPI) * D);
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const uint32_t w[4] = {rawb[u].x, rawb[u].y, rawb[u].z, rawb[u].w};
              uint32_t h[8];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                  const uint32_t x = __byte_perm(w[e], 0u, hf ? 0x3424u : 0x1404u);      // two bytes, each in the high byte of a half
                  const uint32_t bits = ((x >> 1) & 0x3f803f80u) | (x & 0x80008000u);
                  const __half2 v = __hmul2(*reinterpret_cast<const __half2*>(&bits), sc2);
                  h[2 * e + hf] = *reinterpret_cast<const uint32_t*>(&v);
                }
              }
              const int t = t0 + u * TPI + tl;
              *reinterpret_cast<uint4*>(row + tc5_sw(t, c)) = make_uint4(h[0], h[1], h[2], h[3]);
              *reinterpret_cast<uint4*>(row + tc5_sw(t, c + 1)) = make_uint4(h[4], h[5], h[6], h[7]);
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read the slot through the async proxy; the next copies overwrite the staging slot through it
        __syncwarp();
        if (lane == 0) mbar_arrive(full0 + 8 * sr, 1);
        return true;
      };
      struct Ready8 { int phys, kh, valid, grp, j, ng; float scale; };
      auto stage_b8 = [&](int i, const Item& it) {
        const Ready r = stage_b(i, it);
        return Ready8{r.phys, r.kh, r.valid, r.grp, r.j, r.ng, 1.f};
      };
      auto stage_c = [&](int i, Ready8& r) {          // the page's scale (its address needs the physical page)
        if (i < hi) {
          if (r.phys < 0 || r.phys >= p.n_phys || r.valid <= 0) {
            set_status(p.status, LOSA_ERR_BOUNDS);
            r.phys = 0;
            r.valid = 0;
          }
          r.scale = __ldg(scale_g + static_cast<size_t>(r.phys) * p.Hkv + r.kh);
        }
      };
      Item a = stage_a(lo + lane);
      Ready8 b = stage_b8(lo + lane, a);
      a = stage_a(lo + lane + 32);
      stage_c(lo + lane, b);
      Ready8 b1 = stage_b8(lo + lane + 32, a);
      a = stage_a(lo + lane + 64);
      int n_groups = 0;
      for (int b0 = lo; b0 < hi && go; b0 += 32) {
        const Item a_next = stage_a(b0 + lane + 96);
        const Ready8 b2 = stage_b8(b0 + lane + 64, a);
        stage_c(b0 + lane + 32, b1);
        const int nb = min(32, hi - b0);
        int pos = 0;
        while (pos < nb && go) {
          const int grp = __shfl_sync(0xffffffffu, b.grp, pos), j0 = __shfl_sync(0xffffffffu, b.j, pos);
          const int ng = __shfl_sync(0xffffffffu, b.ng, pos);
          const int cnt = min(ng - j0, nb - pos);
          const int ss = grp % NSTG;
          if (j0 == 0) {
            while (go && conv + NSTG <= grp) go = convert(conv++);          // the staging slot must have been emptied
            if (!go) break;
          }
          const bool mine = lane >= pos && lane < pos + cnt;
          if (mine) {
            if (!is_v) meta[(grp % kTc5MetaRing) * kTc5PgMax + b.j] = b.valid;
            sc_meta[(grp % kTc5MetaRing) * kTc5PgMax + b.j] = b.scale;
          }
          if (j0 == 0 && lane == 0) ngs[grp % kTc5MetaRing] = ng;
          __syncwarp();
          if (j0 == 0 && lane == 0) mbar_expect_tx(stg_full0 + 8 * ss, ng * GP * D);
          __syncwarp();
          if (mine) tma_load_4d(stg + ss * STG + b.j * (GP * D), map, stg_full0 + 8 * ss, 0, 0, b.kh, b.phys, policy);
          issued = grp;
          n_groups = grp + 1;
          pos += cnt;
        }
        a = a_next;
        b = b1;
        b1 = b2;
      }
      while (go && conv < n_groups) go = convert(conv++);
    } else {
    Item a = stage_a(lo + lane);
    Ready b = stage_b(lo + lane, a);
    a = stage_a(lo + lane + 32);
    bool go = true;
    for (int b0 = lo; b0 < hi && go; b0 += 32) {
      const Item a_next = stage_a(b0 + lane + 64);
      const Ready b_next = stage_b(b0 + lane + 32, a);
      if (b0 + lane < hi && (b.phys < 0 || b.phys >= p.n_phys || b.valid <= 0)) {
        set_status(p.status, LOSA_ERR_BOUNDS);
        b.phys = 0;
        b.valid = 0;
      }
      const int nb = min(32, hi - b0);
      int pos = 0;
      while (pos < nb) {
        const int grp = __shfl_sync(0xffffffffu, b.grp, pos), j0 = __shfl_sync(0xffffffffu, b.j, pos);
        const int ng = __shfl_sync(0xffffffffu, b.ng, pos);
        const int cnt = min(ng - j0, nb - pos);
        const int slot = grp % NR, round = grp / NR;
        if (j0 == 0) {
          int ok = 1;
          if (lane == 0 && round > 0) ok = mbar_wait(free0 + 8 * slot, (round - 1) & 1, abort_flag, p.status, p.wait_cycles);
          go = __shfl_sync(0xffffffffu, ok, 0) != 0;
          if (!go) break;
        }
        const bool mine = lane >= pos && lane < pos + cnt;
        if (!is_v && mine) meta[(grp % kTc5MetaRing) * kTc5PgMax + b.j] = b.valid;
        __syncwarp();
        if (j0 == 0 && lane == 0) mbar_expect_tx(full0 + 8 * slot, ng * PAGE_BYTES);
        __syncwarp();
        if (mine) {
          const uint32_t dst = ring + slot * SLOT + b.j * (GP * 128);
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf) tma_load_4d(dst + hf * HS, map, full0 + 8 * slot, hf * 64, 0, b.kh, b.phys, policy);
        }
        issued = grp;
        pos += cnt;
      }
      a = a_next;
      b = b_next;
    }
    }
  } else if (warp == kTc5QkWarp) {
    // ------------------------------------------------------------------ Q K^T issuer (one thread)
    if (lane == 0) {
      int sg = sg0, item = lo, piece = 0, g = 0;
      bool ok = true;
      while (item < hi && ok) {
        const int seg_end = min(hi, pre[sg + 1]);
        ok = mbar_wait(q_full, piece & 1, abort_flag, p.status, p.wait_cycles);
        for (int first = item; first < seg_end && ok; first += PG, ++g) {
          const int ng = min(PG, seg_end - first), b = g & 1, use = g >> 1, slot = g % NR;
          ok = mbar_wait(kfull + 8 * slot, (g / NR) & 1, abort_flag, p.status, p.wait_cycles);
          ok = ok && (use == 0 || mbar_wait(s_free + 8 * b, (use - 1) & 1, abort_flag, p.status, p.wait_cycles));
          if (!ok) break;
          tc5_fence_after();
          const uint32_t idesc = tc5_idesc(kRowsPerGroup, ng * GP, 0, FMT), kt = kring + slot * SLOT;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc5_mma_ts(tmem + COL_S + b * kTc5Tok, tmem + COL_Q + ks * 8, tc5_desc(kt + (ks >> 2) * HS + (ks & 3) * 32, 16),
                       idesc, ks > 0 ? 1u : 0u);
          tc5_commit(s_full + 8 * b);
          tc5_commit(kfree + 8 * slot);
          if (first + PG >= seg_end) tc5_commit(q_free);        // Q may be replaced once the piece's last product has run
        }
        item = seg_end;
        ++sg;
        ++piece;
        while (item < hi && pre[sg + 1] <= item) ++sg;
      }
    }
  } else if (warp == kTc5PvWarp) {
    // ------------------------------------------------------------------ P V issuer (one thread)
    if (lane == 0) {
      const uint32_t idesc = tc5_idesc(kRowsPerGroup, D, 1, FMT);
      int sg = sg0, item = lo, g = 0;
      bool ok = true;
      while (item < hi && ok) {
        const int seg_end = min(hi, pre[sg + 1]);
        for (int first = item; first < seg_end && ok; first += PG, ++g) {
          const int ng = min(PG, seg_end - first), b = g & 1, use = g >> 1, slot = g % NR;
          ok = mbar_wait(vfull + 8 * slot, (g / NR) & 1, abort_flag, p.status, p.wait_cycles);
          ok = ok && mbar_wait(p_full + 8 * b, use & 1, abort_flag, p.status, p.wait_cycles);
          if (!ok) break;
          tc5_fence_after();
          const uint32_t vt = vring + slot * SLOT;
          for (int ks = 0; ks < ng * GP / 16; ++ks)
            tc5_mma_ts(tmem + COL_O, tmem + COL_S + b * kTc5Tok + ks * 8, tc5_desc(vt + ks * 2048, HS), idesc,
                       (first == item && ks == 0) ? 0u : 1u);
          tc5_commit(vfree + 8 * slot);
          tc5_commit(s_free + 8 * b);
        }
        item = seg_end;
        ++sg;
        while (item < hi && pre[sg + 1] <= item) ++sg;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue warps
    // Thread = query row (tensor-memory lane 32 * (warp % 4) + lane) and one half of the columns:
    // set h = warp / 4 takes columns 64h .. 64h+63 of every group (and half of Q, of O when it is
    // rescaled or read out).  The exponentials are the bottleneck of this path (one special-function
    // unit per scheduler); two warps per scheduler keep that unit busy while the partner loads,
    // packs and stores.  The pair meets once per group (named barrier) to exchange the row maxima.
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
    const int quarter = warp & 3, h = warp >> 2;
    const int r = quarter * 32 + lane;                         // row of the tile = tensor-memory lane
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
    const float scale2 = p.sm_scale * kLog2e;
    constexpr int QW = D / 4;                                  // 32-bit words of Q per thread (half a row)
    constexpr int OC = D / 2;                                  // columns of O per thread
    // every wait of these warps ends with one answer for the whole warp: the tensor-memory
    // instructions that follow need all 32 lanes
    auto warp_wait = [&](uint32_t bar, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, p.status, p.wait_cycles)) != 0;
    };
    int n_meet = 0;
    auto pair_sync = [&]() {                                    // bounded like every other wait
      __syncwarp();
      if (lane == 0) mbar_arrive(xbar + 8 * quarter, 1);
      const bool met = warp_wait(xbar + 8 * quarter, n_meet & 1);
      ++n_meet;
      return met;
    };
    int sg = sg0, item = lo, piece = 0, g = 0;
    bool ok = true;
    while (item < hi && ok) {
      const int seg_end = min(hi, pre[sg + 1]);
      const int n_sk = p.n_seg / p.n_rg, rg = sg / n_sk, sk = sg % n_sk, s = sk / p.Hkv, kh = sk % p.Hkv;
      const int rows = rows_in_group(n_active_of(s), p.G, rg);
      const bool warp_has_rows = quarter * 32 < rows;          // the same for both warps of a pair
      // ---- the piece's Q tile: this thread's half row, two bf16 per tensor-memory column
      {
        uint32_t qw[QW];
        const uint4* src = nullptr;
        if (r < rows) {
          const int row = rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
          int tok = token_of(s, a);
          if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
          src = reinterpret_cast<const uint4*>(q + ((static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + gi) * D) + h * (QW / 4);
        }
#pragma unroll
        for (int c = 0; c < QW / 4; ++c) {
          const uint4 v = src ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
          qw[4 * c] = v.x; qw[4 * c + 1] = v.y; qw[4 * c + 2] = v.z; qw[4 * c + 3] = v.w;
        }
        if constexpr (FP8) {                        // the MMAs of this variant take fp16 operands
#pragma unroll
          for (int c = 0; c < QW; ++c) {
            const __half2 hq = __floats2half2_rn(__uint_as_float(qw[c] << 16), __uint_as_float(qw[c] & 0xffff0000u));
            qw[c] = *reinterpret_cast<const uint32_t*>(&hq);
          }
        }
        if (piece > 0) ok = warp_wait(q_free, (piece - 1) & 1);
        if (!ok) break;
        tc5_fence_after();
        if constexpr (QW == 32) tc5_st32(lane_addr + COL_Q + h * QW, qw);
        else tc5_st16(lane_addr + COL_Q + h * QW, qw);
        tc5_wait_st();
        tc5_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(q_full, 1);
      }
      float m_ref = -INFINITY, l = 0.f;                         // l: this thread's columns only
      bool o_valid = false;                                     // O holds at least one group of this piece
      for (int first = item; first < seg_end && ok; first += PG, ++g) {
        const int ng = min(PG, seg_end - first), ncol = ng * GP, b = g & 1, use = g >> 1;
        const uint32_t s_addr = lane_addr + COL_S + b * kTc5Tok;
        volatile int* gmeta = meta + (g % kTc5MetaRing) * kTc5PgMax;
        ok = warp_wait(s_full + 8 * b, use & 1);
        if (!ok) break;
        tc5_fence_after();
        // pages with fewer than GP tokens (the last page of a prefix), or a group that ends inside a
        // 32-column chunk, need per-column masks; everything else takes the plain path
        bool ragged = (ncol & 31) != 0;
        for (int j = 0; j < ng; ++j) ragged |= gmeta[j] < GP;
        auto masked = [&](int col) {
          const int j = col / GP, t = col % GP;
          return j >= ng || t >= gmeta[j];
        };
        const int col0 = 64 * h;                                // this thread's columns: col0 .. col0+63, below ncol
        if (warp_has_rows) {
          // ---- the row's scores: one read of tensor memory into registers, both loads in flight together
          uint32_t sraw[64];
#pragma unroll
          for (int c = 0; c < 2; ++c)
            if (col0 + c * 32 < ncol) tc5_ld32_nowait(s_addr + col0 + 32 * c, sraw + 32 * c);
          tc5_wait_ld();
#pragma unroll
          for (int c = 0; c < 2; ++c)
            if (col0 + c * 32 < ncol) tc5_pin32(sraw + 32 * c);
          if (ragged) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
              if (col0 + c * 32 < ncol) {
#pragma unroll
                for (int e = 0; e < 32; ++e) if (masked(col0 + 32 * c + e)) sraw[32 * c + e] = 0xff800000u;   // -inf
              }
          }
          // ---- pass 1: the row's maximum over the group (own columns, then the partner's)
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 2; ++c)
            if (col0 + c * 32 < ncol) {
#pragma unroll
              for (int e = 0; e < 32; ++e) mx[e & 3] = fmaxf(mx[e & 3], __uint_as_float(sraw[32 * c + e]));
            }
          const float mx_own = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          xmax[(b * 2 + h) * kRowsPerGroup + r] = mx_own;
          ok = pair_sync();
          const float m_new = fmaxf(mx_own, xmax[(b * 2 + (h ^ 1)) * kRowsPerGroup + r]) * scale2;
          float corr = 1.f;
          if (m_new > m_ref + kTc5Tau || (m_ref == -INFINITY && m_new > -INFINITY)) {
            corr = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - m_new);
            m_ref = m_new;
            l *= corr;
          }
          // ---- rescale O (rare): the previous group's P V must have run; all lanes of the warp take
          //      part, each set on its half of the columns
          if (__any_sync(0xffffffffu, o_valid && corr != 1.f)) {
            ok = ok && warp_wait(s_free + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1);
            if (ok) {
              tc5_fence_after();
#pragma unroll
              for (int c0 = 0; c0 < OC; c0 += 32) {
                float t[32];
                uint32_t w[32];
                tc5_ld32(lane_addr + COL_O + h * OC + c0, t);
#pragma unroll
                for (int e = 0; e < 32; ++e) w[e] = __float_as_uint(t[e] * corr);
                tc5_st32(lane_addr + COL_O + h * OC + c0, w);
              }
              tc5_wait_st();
            }
          }
          // ---- pass 2: P = 2^(s - m) as bf16, written over the scores (column c of P takes the
          //      place of columns 2c, 2c+1 of S; every score of the group is in registers by now,
          //      the partner's too: it has passed the pair barrier)
          if (ok) {
            const float ms = (m_ref == -INFINITY) ? 0.f : m_ref;
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              if (col0 + c * 32 < ncol) {
                uint32_t w[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                  const float p0 = ex2(fmaf(__uint_as_float(sraw[32 * c + 2 * e]), scale2, -ms));
                  const float p1 = ex2(fmaf(__uint_as_float(sraw[32 * c + 2 * e + 1]), scale2, -ms));
                  sum[e & 3] += p0 + p1;
                  w[e] = FP8 ? pack_f16(p0, p1) : pack_bf16(p0, p1);
                }
                tc5_st16(s_addr + col0 / 2 + 16 * c, w);
              }
            }
            tc5_wait_st();
            l += (sum[0] + sum[1]) + (sum[2] + sum[3]);
          }
        }
        if (!ok) break;
        if (ragged) {
          // rows of V past the end of the prefix may hold anything (even NaN): clear them once the
          // tile has landed (all softmax warps, whether or not they own rows)
          bool any_short = false;
          for (int j = 0; j < ng; ++j) any_short |= gmeta[j] < GP;
          if (any_short) {
            const int slot = g % NR;
            ok = warp_wait(vfull + 8 * slot, (g / NR) & 1);
            if (!ok) break;
            uint8_t* vg = gen + (NR + slot) * SLOT;
            for (int j = 0; j < ng; ++j) {
              const int valid = gmeta[j];
              for (int idx = tid; idx < (GP - valid) * (D / 8); idx += kTc5SoftmaxWarps * 32) {
                const int t = j * GP + valid + idx / (D / 8), ch = idx % (D / 8);
                *reinterpret_cast<uint4*>(vg + (ch >> 3) * HS + tc5_sw(t, ch & 7)) = make_uint4(0u, 0u, 0u, 0u);
              }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          }
        }
        tc5_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full + 8 * b, 1);
        o_valid = true;
      }
      if (!ok) break;
      // ---- the piece's record: one 16-row tile record per 16 rows, reference maximum in base-2
      //      units; each set writes its half of the columns, set 0 the row's maximum and sum
      ok = warp_wait(s_free + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1);
      if (!ok) break;
      tc5_fence_after();
      if (warp_has_rows) {
        if (h == 1) xsum[r] = l;
        ok = pair_sync();
        if (!ok) break;
        float* rec = record_base(p.partials, blockIdx.x + sg, r / kTileRows, D);
        const int rr = r % kTileRows;
#pragma unroll
        for (int c0 = 0; c0 < OC; c0 += 32) {
          float t[32];
          tc5_ld32(lane_addr + COL_O + h * OC + c0, t);
          if (r < rows) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<float4*>(rec + 2 * kTileRows + rr * D + h * OC + c0 + e) = make_float4(t[e], t[e + 1], t[e + 2], t[e + 3]);
          }
        }
        if (h == 0 && r < rows) { rec[rr] = m_ref; rec[kTileRows + rr] = l + xsum[r]; }
      }
      tc5_fence_before();
      item = seg_end;
      ++sg;
      ++piece;
      while (item < hi && pre[sg + 1] <= item) ++sg;
    }
  }
  // ---- every thread that passed the allocation meets here; tensor memory is returned on all paths
  tc5_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // The CTA has given up (a wait ran out).  Its shared and tensor memory must not be handed on
    // while work it started is still in flight: the producers wait, within a bound, for the newest
    // round of copies of every ring slot (a group that was begun has had all its copies issued: the
    // producer loop only stops between groups), the issuing threads for the products they issued.
    if ((warp == kTc5KWarp || warp == kTc5VWarp) && lane == 0) {
      // (FP8 pages: the copies land in the staging slots)
      const uint32_t full0 = FP8 ? (warp == kTc5VWarp ? vstg_full : kstg_full) : (warp == kTc5VWarp ? vfull : kfull);
      constexpr int NSL = FP8 ? NSTG : NR;
      for (int sl = 0; sl < NSL; ++sl) {
        if (issued < sl) continue;
        const int gl = issued - (issued - sl) % NSL;
        mbar_drain(full0 + 8 * sl, (gl / NSL) & 1);
      }
    }
    if ((warp == kTc5QkWarp || warp == kTc5PvWarp) && lane == 0) {
      const uint32_t bar = drain_bar + (warp == kTc5PvWarp ? 8 : 0);
      tc5_commit(bar);
      mbar_drain(bar, 0);
    }
    __syncthreads();
  }
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TMEM_COLS) : "memory");
}
