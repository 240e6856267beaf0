// Device code of the BSR library (sm_100a): probe, install (verify + scatter), scrub.
//
// Pure data movement and 64-bit integer sums: no tensor cores.  Every byte has exactly one reader,
// so every bulk copy is a plain 1-D copy into the issuing CTA's own shared memory.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#define BSR_K_MAX_GROUPS 8
#define BSR_K_MAX_BATCH 256       // chunk descriptors per install launch
#ifndef BSR_K_TILE_MAX
#define BSR_K_TILE_MAX 16384u     // largest tile in bytes (one bulk-copy stage)
#endif
#ifndef BSR_K_SPAN_RUN_MAX
#define BSR_K_SPAN_RUN_MAX 1024u  // destination runs up to this length travel as spans of several runs
#endif
#define BSR_K_PHI 0x9E3779B97F4A7C15ull

// ---------------------------------------------------------------------------------------------
// shared structs (host fills, device reads)
// ---------------------------------------------------------------------------------------------

// One contiguous span of a chunk, at most BSR_K_TILE_MAX bytes, that is moved as a unit.  Either a
// piece of ONE destination run (n_runs == 1: long runs are cut into pieces), or n_runs > 1 WHOLE
// runs that lie back to back in the chunk: the blocks of one tensor and, where consecutive tensors
// of a group have the same bytes per token, of the tensors that follow it.  Run j of such a span
// belongs to tensor `tensor + (blk + j) / blocks_per_chunk` and logical block
// `(blk + j) % blocks_per_chunk`.  Short runs (256 bytes for 16 B/token in 16-token blocks) thus
// still travel in spans of up to 16 KiB; only their stores are scattered.
// A chunk's tile table is the same for every chunk and rank of a registration: only the source
// base, the block-table row and the tensor base pointers change.
struct __align__(16) BsrTile {
  uint32_t src_off;    // byte offset inside the chunk (multiple of 16)
  uint32_t bytes;      // span length (multiple of 16, <= BSR_K_TILE_MAX)
  uint32_t dst_off;    // byte offset inside the destination block run (0 when n_runs > 1)
  uint32_t word0;      // index of the span's first 32-bit word inside its group segment
  uint32_t run_bytes;  // block_tokens * bytes_per_token of the tensor(s)
  uint16_t tensor;     // registration index l of the first run
  uint8_t group;       // allocator group g
  uint8_t blk;         // logical block of the first run, 0 .. 256/block_tokens - 1
  uint32_t n_runs;     // runs in the span
  uint32_t run_inv;    // ceil(2^32 / run_bytes): byte offset -> run index without a division
};
static_assert(sizeof(BsrTile) == 32, "tile is two 16-byte loads");

// Where vector v (16 bytes) of a span of several whole runs goes.
struct BsrRunMap {
  const int32_t *tab;     // block-table row of the chunk: table(rank, group) + chunk * blocks_per_chunk
  const uint64_t *bases;  // tensor base addresses of the rank: tensor_base + rank * n_tensors
  uint32_t run_bytes, run_inv;
  uint32_t l0, b0;        // tensor and logical block of the span's first run
  uint32_t nb_shift;      // log2(blocks per chunk of the group)
};
__device__ __forceinline__ uint4 *bsr_run_dst(const BsrRunMap &m, uint32_t v) {
  const uint32_t off = v << 4;
  const uint32_t j = __umulhi(off, m.run_inv);  // exact for off < 2^16 and run_bytes >= 256
  const uint32_t within = off - j * m.run_bytes;
  const uint32_t vb = m.b0 + j;
  const uint32_t l = m.l0 + (vb >> m.nb_shift), blk = vb & ((1u << m.nb_shift) - 1u);
  const uint64_t base = __ldg(m.bases + l);
  const int32_t phys = __ldg(m.tab + blk);
  return reinterpret_cast<uint4 *>(base + (uint64_t)phys * m.run_bytes + within);
}

struct BsrChunkDesc {
  const uint8_t *src;  // device address of the staged chunk
  uint32_t chunk;      // index i in the advertised prefix
  uint32_t rank;       // TP rank slice r
  uint64_t expect[BSR_K_MAX_GROUPS];  // stored checksums of the group segments
};

struct BsrInstallParams {
  const BsrTile *tiles;
  uint32_t n_tiles;    // tiles per chunk
  uint32_t n_chunks;   // descriptors in this launch
  uint32_t n_groups;
  uint32_t n_tensors;
  uint32_t n_adv;      // advertised chunks of the request (row length of ck_out / verdict)
  uint32_t scatter;    // 0: checksum only (store path), 1: verify + scatter
  const uint64_t *tensor_base;   // [R][L] device addresses of the paged tensors
  const int32_t *const *tables;  // [R*G] device pointers to the request's block tables
  uint32_t blocks_per_chunk[BSR_K_MAX_GROUPS];
  uint64_t *acc;             // scratch [BSR_K_MAX_BATCH][BSR_K_MAX_GROUPS]; zero on entry, zeroed on exit
  unsigned int *ctas_done;   // scratch counter; zero on entry, zeroed on exit
  unsigned int *err_flag;    // host-mapped word, set to nonzero if a bounded wait gave up (bulk variant)
  uint64_t *ck_out;          // [(r*G + g) * n_adv + i] computed checksum
  uint32_t *verdict;         // same index: 1 verified, 2 mismatch
  uint64_t *span_start;      // scratch word (zero on entry, zeroed on exit) and ...
  uint64_t *span_out;        // ... host-mapped word for the launch's in-kernel span in ns (first CTA's start to
                             // the last CTA's verdict pass); NULL = not measured
  uint64_t wait_ns;          // bound of every wait inside the bulk kernel; 0 = BSR_K_WAIT_NS
  uint32_t stall_tile;       // test hook: work item whose load is never issued; ~0u = none
  uint32_t pad0;
  const BsrChunkDesc *batch; // device array of n_chunks descriptors, or NULL: use `one`
  BsrChunkDesc one;          // the descriptor of a single-chunk launch, carried in the parameters
};

__device__ __forceinline__ const BsrChunkDesc *bsr_desc(const BsrInstallParams &p, uint32_t c) {
  return p.batch ? p.batch + c : &p.one;
}

// ---------------------------------------------------------------------------------------------
// helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t bsr_mix64(uint64_t x) {
  x += BSR_K_PHI;
  x = (x ^ (x >> 32)) * BSR_K_PHI;
  x = (x ^ (x >> 29)) * BSR_K_PHI;
  return x ^ (x >> 32);
}

__device__ __forceinline__ uint64_t bsr_globaltimer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// In-kernel span of a launch, for measurement runs: every CTA notes its start (the earliest wins),
// the last CTA to finish publishes now - earliest.  Costs one atomic per CTA when enabled.
__device__ __forceinline__ void bsr_span_begin(const uint64_t *span_out, uint64_t *span_start) {
  if (span_out && threadIdx.x == 0)
    atomicMax((unsigned long long *)span_start, (unsigned long long)~bsr_globaltimer());
}

__device__ __forceinline__ uint64_t bsr_warp_sum(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Contribution of one 16-byte vector whose first word has index k inside the segment:
// sum_{q<4} w_q * (2(k+q) + 1), each product 32x32 -> 64 bits.
__device__ __forceinline__ uint64_t bsr_ck_vec(uint4 w, uint32_t k) {
  const uint32_t wt = 2u * k + 1u;
  uint64_t s = (uint64_t)w.x * (uint64_t)wt;
  s += (uint64_t)w.y * (uint64_t)(wt + 2u);
  s += (uint64_t)w.z * (uint64_t)(wt + 4u);
  s += (uint64_t)w.w * (uint64_t)(wt + 6u);
  return s;
}

__device__ __forceinline__ uint4 bsr_ld_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void bsr_st_stream(uint4 *p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

// Block-wide sum of per-thread partials, added once into *dst (sums mod 2^64 commute, so the
// order of the atomics cannot change the result).
template <int THREADS>
__device__ __forceinline__ void bsr_block_flush(uint64_t v, uint64_t *dst, uint64_t *smem) {
  v = bsr_warp_sum(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) smem[warp] = v;
  __syncthreads();
  if (warp == 0) {
    uint64_t t = (lane < THREADS / 32) ? smem[lane] : 0ull;
    t = bsr_warp_sum(t);
    if (lane == 0) atomicAdd((unsigned long long *)dst, (unsigned long long)t);
  }
  __syncthreads();
}

// The last CTA to finish compares every (chunk, group) sum of the launch with the stored checksum,
// publishes sum and verdict, and leaves the scratch zeroed for the next launch.
template <int THREADS>
__device__ __forceinline__ void bsr_install_finish(const BsrInstallParams &p) {
  __shared__ int is_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned prev = atomicAdd(p.ctas_done, 1u);
    is_last = (prev == gridDim.x - 1u);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const uint32_t G = p.n_groups;
  for (uint32_t idx = threadIdx.x; idx < p.n_chunks * G; idx += THREADS) {
    const uint32_t c = idx / G, g = idx - c * G;
    uint64_t *a = p.acc + c * BSR_K_MAX_GROUPS + g;
    const uint64_t s = __ldcg((const unsigned long long *)a);
    *a = 0ull;
    const BsrChunkDesc &cd = *bsr_desc(p, c);
    const size_t o = ((size_t)cd.rank * G + g) * p.n_adv + cd.chunk;
    p.ck_out[o] = s;
    p.verdict[o] = (s == cd.expect[g]) ? 1u : 2u;
  }
  if (threadIdx.x == 0) {
    *p.ctas_done = 0u;
    if (p.span_out) {
      const uint64_t first = ~__ldcg((const unsigned long long *)p.span_start);
      *p.span_start = 0ull;
      *reinterpret_cast<volatile uint64_t *>(p.span_out) = bsr_globaltimer() - first;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// install, vector variant: 16-byte streaming loads and stores, UNROLL vectors in flight per thread
// ---------------------------------------------------------------------------------------------
// SPANS: the registration has spans of several runs (their per-vector destination lookup costs
// registers that a registration of long runs alone should not pay for).
template <int THREADS, int UNROLL, bool SPANS>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS)  // full occupancy: 32 registers at 256 threads
bsr_install_vec_kernel(const __grid_constant__ BsrInstallParams p) {
  __shared__ uint64_t red[THREADS / 32];
  bsr_span_begin(p.span_out, p.span_start);
  const uint32_t total = p.n_chunks * p.n_tiles;
  uint64_t sum = 0;
  int cur_c = -1, cur_g = -1;
  for (uint32_t w = blockIdx.x; w < total; w += gridDim.x) {
    const uint32_t c = w / p.n_tiles, t = w - c * p.n_tiles;
    const uint4 *tp = reinterpret_cast<const uint4 *>(p.tiles + t);
    const uint4 t0 = __ldg(tp), t1 = __ldg(tp + 1);
    const uint32_t src_off = t0.x, bytes = t0.y, dst_off = t0.z, word0 = t0.w;
    const uint32_t run_bytes = t1.x, tensor = t1.y & 0xffffu, g = (t1.y >> 16) & 0xffu,
                   blk = t1.y >> 24, n_runs = t1.z;
    if ((int)c != cur_c || (int)g != cur_g) {  // block-uniform
      if (cur_c >= 0) bsr_block_flush<THREADS>(sum, p.acc + cur_c * BSR_K_MAX_GROUPS + cur_g, red);
      sum = 0;
      cur_c = (int)c;
      cur_g = (int)g;
    }
    const BsrChunkDesc &cd = *bsr_desc(p, c);
    const uint4 *src = reinterpret_cast<const uint4 *>(cd.src + src_off);
    uint4 *dst = nullptr;
    BsrRunMap rm;
    const bool several = SPANS && p.scatter && n_runs > 1;  // whole runs, each with its own destination
    if (p.scatter) {
      const uint32_t nb = p.blocks_per_chunk[g];
      const int32_t *row = p.tables[cd.rank * p.n_groups + g] + (size_t)cd.chunk * nb;
      const uint64_t *bases = p.tensor_base + (size_t)cd.rank * p.n_tensors;
      if (several) {
        rm.tab = row;
        rm.bases = bases;
        rm.run_bytes = run_bytes;
        rm.run_inv = t1.w;
        rm.l0 = tensor;
        rm.b0 = blk;
        rm.nb_shift = 31u - __clz(nb);
      } else {
        dst = reinterpret_cast<uint4 *>(__ldg(bases + tensor) + (uint64_t)__ldg(row + blk) * run_bytes + dst_off);
      }
    }
    const uint32_t nvec = bytes >> 4;
    for (uint32_t v0 = threadIdx.x; v0 < nvec; v0 += THREADS * UNROLL) {
      uint4 r[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const uint32_t v = v0 + u * THREADS;
        if (v < nvec) r[u] = bsr_ld_stream(src + v);
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const uint32_t v = v0 + u * THREADS;
        if (v < nvec) {
          if (several)
            bsr_st_stream(bsr_run_dst(rm, v), r[u]);
          else if (dst)
            bsr_st_stream(dst + v, r[u]);
          sum += bsr_ck_vec(r[u], word0 + 4u * v);
        }
      }
    }
  }
  if (cur_c >= 0) bsr_block_flush<THREADS>(sum, p.acc + cur_c * BSR_K_MAX_GROUPS + cur_g, red);
  bsr_install_finish<THREADS>(p);
}

// ---------------------------------------------------------------------------------------------
// install, bulk variant: the copy engine of each SM (1-D bulk async copies, one CTA each) moves the
// spans global -> shared -> global through a ring of shared-memory stages; a producer warp computes
// addresses and issues the loads, a store warp issues the stores, and the sum warps (4 or 8) sum the
// span from shared memory while its store is in flight.
//
//   warp 0, producer:  wait empty[s] -> expect_tx(full[s], bytes) -> bulk load span into stage s
//   warp 1, storer:    wait full[s]  -> bulk store stage s -> dst; once the store issued two spans
//                      earlier has finished reading its stage -> arrive empty[that stage]
//   warps 2.., sums:   wait full[s]  -> checksum from shared memory -> arrive empty[s]
// A span of several short runs has no single destination: the sum warps, which hold every vector
// of the stage in registers anyway, store it to the run it belongs to (16-byte streaming stores,
// a half-warp per 256 bytes), and the storer only hands the stage back.
//
// Every wait is bounded by a wall-clock deadline; a wait that gives up raises *err_flag, the CTA
// stops issuing work, drains what it has in flight and leaves through the common exit.
// ---------------------------------------------------------------------------------------------
#ifndef BSR_K_BULK_STAGES
#define BSR_K_BULK_STAGES 6
#endif
#ifndef BSR_K_BULK_CTAS_PER_SM
#define BSR_K_BULK_CTAS_PER_SM 2  // 2 x 6 stages x 16 KiB = 192 KiB of the SM's shared memory
#endif
#ifndef BSR_K_BULK_TILES_PER_CTA
#define BSR_K_BULK_TILES_PER_CTA 64  // work per CTA; the grid is sized from it in whole waves
#endif
// Sum warps per CTA (the kernel's template parameter): 4 keep up with any stream of long runs and
// give the quickest small launches; a registration whose bytes sit mostly in spans of short runs,
// which the sum warps also store, gets 8 (0.76 -> 0.91 of the copy rate on 256-byte runs).
#define BSR_K_BULK_SUM_WARPS 4
#define BSR_K_BULK_SUM_WARPS_SPANS 8
#define BSR_K_BULK_THREADS(SUM_WARPS) (32 * (2 + (SUM_WARPS)))
#ifndef BSR_K_BULK_STORE_LAG
#define BSR_K_BULK_STORE_LAG 2  // stores whose shared-memory reads may still be pending
#endif
#define BSR_K_BULK_SMEM (BSR_K_BULK_STAGES * BSR_K_TILE_MAX)
// A stage is handed back to the producer only LAG stores after its own store was issued: with as
// many lagging stores as stages the producer would wait for a stage nobody is about to release.
static_assert(BSR_K_BULK_STAGES > BSR_K_BULK_STORE_LAG, "the stage ring must be deeper than the store lag");
static_assert(BSR_K_BULK_STORE_LAG >= 0 && BSR_K_BULK_STORE_LAG <= 5, "the storer packs LAG + 1 stage numbers into 32 bits");
static_assert(BSR_K_TILE_MAX % 128u == 0 && BSR_K_TILE_MAX >= 256u, "tiles are cut on 128-byte boundaries");
#define BSR_K_WAIT_NS 2000000000ull  // 2 s: four orders of magnitude above any legitimate wait

// What the producer tells the other warps about the span it loads into a stage.  One entry per
// span in flight, in a ring indexed by the CTA's span counter: entries are written 32 at a time by
// the lanes that resolve them, and a slot is rewritten only 64 spans later, long after the other
// warps (at most a stage ring behind the producer) are done with it.
#define BSR_K_META_RING 64
struct __align__(16) BsrStageMeta {
  uint64_t src;           // source address of the span
  uint64_t dst;           // one run: destination address of the piece (0 when the launch only sums)
  const int32_t *tab;     // several runs: see BsrRunMap
  const uint64_t *bases;
  uint32_t bytes;         // span length
  uint32_t word0;         // index of the span's first 32-bit word inside its group segment
  uint32_t run_bytes, run_inv;
  uint16_t l0, b0;
  uint16_t nb_shift;
  uint16_t several;       // nonzero: whole runs with their own destinations, stored by the sum warps
  uint32_t cg;            // chunk descriptor index << 8 | group
  uint32_t pad;
};
static_assert(sizeof(BsrStageMeta) == 64, "four 16-byte words per entry");
static_assert(BSR_K_BULK_STAGES <= 32, "the meta ring assumes the other warps trail the producer by < 32 spans");

__device__ __forceinline__ uint32_t bsr_smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void bsr_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void bsr_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bsr_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool bsr_mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the deadline passed (and raises the error flag).
__device__ __forceinline__ bool bsr_mbar_wait(uint32_t bar, uint32_t parity, unsigned int *err_flag,
                                              volatile int *abort_flag, uint64_t wait_ns) {
  if (bsr_mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = bsr_globaltimer();
  for (;;) {
    if (bsr_mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (bsr_globaltimer() - t0 > wait_ns) {
      *abort_flag = 1;
      *reinterpret_cast<volatile unsigned int *>(err_flag) = 1u;  // host-mapped word: a plain store
      __threadfence_system();
      return false;
    }
  }
}
__device__ __forceinline__ uint64_t bsr_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// 1-D bulk copy global -> this CTA's shared memory; completion is counted in bytes on `bar`.
// src, dst and size are multiples of 16 bytes (guaranteed by the tile table).
__device__ __forceinline__ void bsr_bulk_load(uint32_t smem_dst, const void *gsrc, uint32_t bytes,
                                              uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, "
      "[%3], %4;" ::"r"(smem_dst),
      "l"(gsrc), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
// 1-D bulk copy shared -> global, committed as its own bulk group so that its reads of shared
// memory can be waited for individually.
__device__ __forceinline__ void bsr_bulk_store(uint64_t gdst, uint32_t smem_src, uint32_t bytes,
                                               uint64_t pol) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(
                   gdst),
               "r"(smem_src), "r"(bytes), "l"(pol)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int SUM_WARPS>
__global__ void __launch_bounds__(BSR_K_BULK_THREADS(SUM_WARPS))
bsr_install_bulk_kernel(const __grid_constant__ BsrInstallParams p) {
  extern __shared__ __align__(128) uint8_t stage_mem[];
  __shared__ __align__(8) uint64_t full_bar[BSR_K_BULK_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[BSR_K_BULK_STAGES];
  __shared__ BsrStageMeta meta[BSR_K_META_RING];
  __shared__ int last_round[BSR_K_BULK_STAGES];  // last load round issued into each stage, -1 = none
  __shared__ int abort_flag;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  bsr_span_begin(p.span_out, p.span_start);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < BSR_K_BULK_STAGES; ++s) {
      last_round[s] = -1;
      bsr_mbar_init(bsr_smem_u32(&full_bar[s]), 1);
      bsr_mbar_init(bsr_smem_u32(&empty_bar[s]), SUM_WARPS + 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const uint64_t wait_ns = p.wait_ns ? p.wait_ns : BSR_K_WAIT_NS;
  // every byte is read once and written once: mark both streams evict-first in L2
  const uint64_t pol = bsr_policy_evict_first();
  const uint32_t total = p.n_chunks * p.n_tiles;
  const uint32_t my_tiles = (blockIdx.x < total) ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    // ---------------- producer ----------------
    // The address of a span needs a chain of dependent loads (tile entry -> block table -> tensor
    // base).  The 32 lanes resolve 32 consecutive spans of this CTA at once, each into its own
    // entry of the meta ring; lane 0 then issues the loads in order.
    for (uint32_t base = 0; base < my_tiles; base += 32) {
      const uint32_t n_mine = base + lane;
      if (n_mine < my_tiles) {
        const uint32_t w = blockIdx.x + n_mine * gridDim.x;
        const uint32_t c = w / p.n_tiles, t = w - c * p.n_tiles;
        const uint4 *tp = reinterpret_cast<const uint4 *>(p.tiles + t);
        const uint4 t0 = __ldg(tp), t1 = __ldg(tp + 1);
        const uint32_t g = (t1.y >> 16) & 0xffu, tensor = t1.y & 0xffffu, blk = t1.y >> 24;
        const BsrChunkDesc &cd = *bsr_desc(p, c);
        BsrStageMeta m;
        m.src = reinterpret_cast<uint64_t>(cd.src) + t0.x;
        m.dst = 0;
        m.tab = nullptr;
        m.bases = nullptr;
        m.bytes = t0.y;
        m.word0 = t0.w;
        m.run_bytes = t1.x;
        m.run_inv = t1.w;
        m.l0 = (uint16_t)tensor;
        m.b0 = (uint16_t)blk;
        m.nb_shift = 0;
        m.several = 0;
        m.cg = (c << 8) | g;
        m.pad = 0;
        if (p.scatter) {
          const uint32_t nb = p.blocks_per_chunk[g];
          const int32_t *row = p.tables[cd.rank * p.n_groups + g] + (size_t)cd.chunk * nb;
          const uint64_t *bases = p.tensor_base + (size_t)cd.rank * p.n_tensors;
          if (t1.z > 1) {
            m.tab = row;
            m.bases = bases;
            m.nb_shift = (uint16_t)(31u - __clz(nb));
            m.several = 1;
          } else {
            m.dst = __ldg(bases + tensor) + (uint64_t)__ldg(row + blk) * t1.x + t0.z;
          }
        }
        meta[n_mine % BSR_K_META_RING] = m;
      }
      __syncwarp();  // lane 0 publishes the other lanes' entries with its barrier arrivals below
      const uint32_t cnt = min(32u, my_tiles - base);
      int ok = 1;
      if (lane == 0) {
        for (uint32_t j = 0; j < cnt; ++j) {
          const uint32_t n = base + j;
          const uint32_t s = n % BSR_K_BULK_STAGES, round = n / BSR_K_BULK_STAGES;
          if (round > 0 &&
              !bsr_mbar_wait(bsr_smem_u32(&empty_bar[s]), (round - 1) & 1u, p.err_flag, &abort_flag, wait_ns)) {
            ok = 0;
            break;
          }
          if (blockIdx.x + n * gridDim.x == p.stall_tile) continue;  // test hook: never loaded, its waits run out
          const BsrStageMeta &m = meta[n % BSR_K_META_RING];
          const uint32_t bar = bsr_smem_u32(&full_bar[s]);
          bsr_mbar_expect_tx(bar, m.bytes);  // release: the meta entry is visible to whoever sees the stage full
          bsr_bulk_load(bsr_smem_u32(stage_mem + (size_t)s * BSR_K_TILE_MAX),
                        reinterpret_cast<const void *>(m.src), m.bytes, bar, pol);
          last_round[s] = (int)round;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
    }
  } else if (warp == 1) {
    // ---------------- storer ----------------
    if (lane == 0) {
      // stages whose bulk store may still be reading them, oldest in the low bits: at most
      // STORE_LAG + 1 stage numbers of 5 bits each
      uint32_t pending = 0, n_pending = 0;
      for (uint32_t n = 0; n < my_tiles; ++n) {
        const uint32_t s = n % BSR_K_BULK_STAGES, round = n / BSR_K_BULK_STAGES;
        if (!bsr_mbar_wait(bsr_smem_u32(&full_bar[s]), round & 1u, p.err_flag, &abort_flag, wait_ns)) break;
        const BsrStageMeta &m = meta[n % BSR_K_META_RING];
        if (p.scatter && !m.several) {
          bsr_bulk_store(m.dst, bsr_smem_u32(stage_mem + (size_t)s * BSR_K_TILE_MAX), m.bytes, pol);
          pending |= s << (5u * n_pending++);
          if (n_pending > BSR_K_BULK_STORE_LAG) {
            asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(BSR_K_BULK_STORE_LAG) : "memory");
            bsr_mbar_arrive(bsr_smem_u32(&empty_bar[pending & 31u]));
            pending >>= 5;
            --n_pending;
          }
        } else {
          // Nothing of this stage is the storer's to move.  Stages of earlier stores are handed back
          // now: a lagging release waits for the next store, and none may follow for a long time,
          // while the producer already needs those stages.
          if (n_pending) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            for (; n_pending; --n_pending, pending >>= 5)
              bsr_mbar_arrive(bsr_smem_u32(&empty_bar[pending & 31u]));
          }
          bsr_mbar_arrive(bsr_smem_u32(&empty_bar[s]));
        }
      }
      if (p.scatter) {
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        for (; n_pending; --n_pending, pending >>= 5)
          bsr_mbar_arrive(bsr_smem_u32(&empty_bar[pending & 31u]));
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores complete
      }
    }
  } else {
    // ---------------- checksum warps ----------------
    const uint32_t ct = threadIdx.x - 64;  // 0 .. 32 * SUM_WARPS - 1
    uint64_t sum = 0;
    uint32_t cur = ~0u;
    for (uint32_t n = 0; n < my_tiles; ++n) {
      const uint32_t s = n % BSR_K_BULK_STAGES, round = n / BSR_K_BULK_STAGES;
      if (!bsr_mbar_wait(bsr_smem_u32(&full_bar[s]), round & 1u, p.err_flag, &abort_flag, wait_ns)) break;
      const BsrStageMeta &m = meta[n % BSR_K_META_RING];
      const uint32_t cg = m.cg, nvec = m.bytes >> 4, word0 = m.word0;
      if (cg != cur) {  // warp-uniform
        if (cur != ~0u) {
          sum = bsr_warp_sum(sum);
          if (lane == 0)
            atomicAdd((unsigned long long *)(p.acc + (cur >> 8) * BSR_K_MAX_GROUPS + (cur & 0xffu)),
                      (unsigned long long)sum);
        }
        sum = 0;
        cur = cg;
      }
      const uint4 *sv = reinterpret_cast<const uint4 *>(stage_mem + (size_t)s * BSR_K_TILE_MAX);
      if (!m.several) {
#pragma unroll 4
        for (uint32_t v = ct; v < nvec; v += 32 * SUM_WARPS)
          sum += bsr_ck_vec(sv[v], word0 + 4u * v);
      } else {
        BsrRunMap rm;
        rm.tab = m.tab;
        rm.bases = m.bases;
        rm.run_bytes = m.run_bytes;
        rm.run_inv = m.run_inv;
        rm.l0 = m.l0;
        rm.b0 = m.b0;
        rm.nb_shift = m.nb_shift;
#pragma unroll 4
        for (uint32_t v = ct; v < nvec; v += 32 * SUM_WARPS) {
          const uint4 w = sv[v];
          bsr_st_stream(bsr_run_dst(rm, v), w);
          sum += bsr_ck_vec(w, word0 + 4u * v);
        }
      }
      __syncwarp();
      if (lane == 0) bsr_mbar_arrive(bsr_smem_u32(&empty_bar[s]));
    }
    if (cur != ~0u) {
      sum = bsr_warp_sum(sum);
      if (lane == 0)
        atomicAdd((unsigned long long *)(p.acc + (cur >> 8) * BSR_K_MAX_GROUPS + (cur & 0xffu)),
                  (unsigned long long)sum);
    }
  }
  __syncthreads();
  if (abort_flag && threadIdx.x == 0) {
    // A wait gave up.  Loads this CTA issued may still be landing in its shared memory: give each
    // stage one more bounded chance to complete before the CTA exits.
    for (int s = 0; s < BSR_K_BULK_STAGES; ++s) {
      if (last_round[s] < 0) continue;
      const uint64_t t0 = bsr_globaltimer();
      while (!bsr_mbar_try_wait(bsr_smem_u32(&full_bar[s]), (uint32_t)last_round[s] & 1u) &&
             bsr_globaltimer() - t0 < wait_ns) {
      }
    }
  }
  bsr_install_finish<BSR_K_BULK_THREADS(SUM_WARPS)>(p);
}

// ---------------------------------------------------------------------------------------------
// probe: chunk digests (one warp per chunk), then the last block chains the prefix keys
// ---------------------------------------------------------------------------------------------
#define BSR_K_PROBE_THREADS 256
#define BSR_K_CHAIN_TILE 2048

__global__ void __launch_bounds__(BSR_K_PROBE_THREADS)
bsr_probe_kernel(const int32_t *__restrict__ tok, uint32_t n_chunks, uint64_t salt, uint64_t k_init,
                 uint64_t *digests /* scratch [n_chunks] */, unsigned int *blocks_done /* scratch */,
                 uint64_t *keys /* out [n_chunks] */) {
  __shared__ uint64_t tile[BSR_K_CHAIN_TILE];
  __shared__ int is_last;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t chunk = blockIdx.x * (BSR_K_PROBE_THREADS / 32) + (threadIdx.x >> 5);
  if (chunk < n_chunks) {
    const int4 *base = reinterpret_cast<const int4 *>(tok + (size_t)chunk * 256u);
    uint64_t s = 0;
#pragma unroll
    for (uint32_t m = 0; m < 2; ++m) {
      const uint32_t q = m * 32u + lane;  // int4 index inside the chunk: tokens 4q .. 4q+3
      const int4 t = __ldg(base + q);
      const uint32_t j = 4u * q;
      s += bsr_mix64((((uint64_t)(uint32_t)t.x << 32) | (uint64_t)(j + 0u)) ^ salt);
      s += bsr_mix64((((uint64_t)(uint32_t)t.y << 32) | (uint64_t)(j + 1u)) ^ salt);
      s += bsr_mix64((((uint64_t)(uint32_t)t.z << 32) | (uint64_t)(j + 2u)) ^ salt);
      s += bsr_mix64((((uint64_t)(uint32_t)t.w << 32) | (uint64_t)(j + 3u)) ^ salt);
    }
    s = bsr_warp_sum(s);
    if (lane == 0) digests[chunk] = s;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    is_last = (atomicAdd(blocks_done, 1u) == gridDim.x - 1u);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // serial chain k_i = mix64(k_{i-1} ^ d_i), digests staged through shared memory
  uint64_t k = k_init;
  for (uint32_t base_i = 0; base_i < n_chunks; base_i += BSR_K_CHAIN_TILE) {
    const uint32_t n = min((uint32_t)BSR_K_CHAIN_TILE, n_chunks - base_i);
    for (uint32_t i = threadIdx.x; i < n; i += BSR_K_PROBE_THREADS)
      tile[i] = __ldcg((const unsigned long long *)(digests + base_i + i));
    __syncthreads();
    if (threadIdx.x == 0) {
      for (uint32_t i = 0; i < n; ++i) {
        k = bsr_mix64(k ^ tile[i]);
        keys[base_i + i] = k;
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *blocks_done = 0u;
}

// ---------------------------------------------------------------------------------------------
// scrub: zero-fill every destination block run of a request (all ranks, groups, tensors)
// grid.y = r * L + l, grid.x strides over the logical blocks of the tensor's group
// ---------------------------------------------------------------------------------------------
struct BsrScrubParams {
  const uint64_t *tensor_base;   // [R][L]
  const int32_t *const *tables;  // [R*G]
  const uint32_t *tensor_group;  // [L]
  const uint32_t *tensor_run;    // [L] run bytes
  uint32_t n_tensors, n_groups, n_adv;
  uint32_t blocks_per_chunk[BSR_K_MAX_GROUPS];
};

__global__ void __launch_bounds__(256) bsr_scrub_kernel(const __grid_constant__ BsrScrubParams p) {
  const uint32_t r = blockIdx.y / p.n_tensors, l = blockIdx.y - r * p.n_tensors;
  const uint32_t g = p.tensor_group[l], run = p.tensor_run[l];
  const uint32_t n_logical = p.n_adv * p.blocks_per_chunk[g];
  const int32_t *table = p.tables[r * p.n_groups + g];
  const uint64_t base = p.tensor_base[(size_t)r * p.n_tensors + l];
  const uint4 z = make_uint4(0, 0, 0, 0);
  for (uint32_t j = blockIdx.x; j < n_logical; j += gridDim.x) {
    uint4 *dst = reinterpret_cast<uint4 *>(base + (uint64_t)__ldg(table + j) * run);
    for (uint32_t v = threadIdx.x; v < (run >> 4); v += 256) dst[v] = z;
  }
}
