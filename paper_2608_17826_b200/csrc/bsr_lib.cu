// Host side of the BSR library: context, registration, chunk index, probe, the W-slot window
// pipeline (pinned slot pool -> copy stream -> device staging -> install kernel), commit,
// invalidate, request-level recovery.  The C interface is declared in include/bsr.h.
//
// Locks (never nested among the short ones, listed outermost first):
//   req->mu      one call at a time per request object (restore holds it for its whole duration)
//   restore_mu   the paper's bounded-retrieve lock: held by a whole restore unless an admission
//                budget is configured, in which case restores run concurrently and share B slots
//   aux_mu       probe, store-path checksums and scrub: they share context-level scratch and a stream
//   setup_mu     one-time set-up: tile table, slot pool, per-restore device resources
//   fill_mu      the fill task queue;  pool_mu  the slot pool and live/peak accounting
//   mu           tier index, statistics, force-local markers, error text
#include "../../include/bsr.h"

#include <immintrin.h>
#include <pthread.h>
#include <sched.h>
#include <sys/prctl.h>

#include <algorithm>
#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <fstream>
#include <memory>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <unordered_map>
#include <unordered_set>
#include <vector>

#include "bsr_kernels.cuh"

namespace {

using Clock = std::chrono::steady_clock;

constexpr int kInstallThreads = 256;
constexpr int kInstallUnroll = 2;  // 32 registers: 8 CTAs of 256 threads resident per SM
constexpr int kLaunchSlots = 8;  // scratch sets for batched install launches in flight per restore
constexpr uint64_t kPieceBytes = 8ull << 20;  // fill and host-to-device copy granularity
// ... of the last chunks of a prefix.  When the fill threads finish their last pieces at about the same
// time, everything they filled is still to be copied: with 8 threads and 8 MiB pieces up to 64 MiB,
// more than a millisecond of link time after the last byte was fetched.  Small pieces, taken in order,
// let the copies trail the fill closely where the restore ends.
constexpr uint64_t kTailPieceBytes = 2ull << 20;
// ... and of the first chunk of every rank: the copy engine has nothing to do until the first piece has
// been fetched, and a short prefix is over before that millisecond has been made up for.
constexpr uint64_t kHeadPieceBytes = 1ull << 20;
#ifndef BSR_RING_ALLOC_FLAGS
#define BSR_RING_ALLOC_FLAGS cudaHostAllocMapped
#endif

struct TierObj {
  const uint8_t *data;
  size_t len;
  int loc;
  uint64_t ck[BSR_MAX_GROUPS];
};

struct TensorReg {
  uint32_t group;
  uint32_t bytes_per_token;
  uint64_t base[BSR_MAX_RANKS];
};

struct Inject {
  int kind = BSR_INJECT_NONE;
  uint32_t rank = 0, group = 0, chunk = 0;
  uint64_t seed = 0;
};

// Device-side resources of one restore in flight.  Pooled: a finished restore hands them back.
struct JobRes {
  cudaStream_t stream = nullptr;                        // used when the caller passes no stream
  uint8_t *dstage[BSR_MAX_RANKS] = {};                  // D staging buffers per rank
  std::vector<cudaEvent_t> ev_h2d;                      // [n_slots >= R * D]: per staging buffer, the copy of its chunk
  std::vector<cudaEvent_t> ev_inst, ev_start;           // [n_slots]: one pair per install launch in flight
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> ev_pool;  // launch timing, batched launches
  cudaEvent_t ev_done = nullptr;
  uint64_t *d_acc = nullptr;      // [n_slots][BATCH][GROUPS] checksum accumulators, kept zero
  unsigned int *d_cnt = nullptr;  // [n_slots] CTA counters, kept zero
  unsigned int *h_err = nullptr;  // pinned, device-visible: raised by a kernel wait that gave up
  unsigned int *d_err = nullptr;  // device alias of h_err
  uint64_t *d_span_start = nullptr;                  // [n_slots] scratch of the in-kernel span measurement, kept zero
  uint64_t *h_span = nullptr, *d_span = nullptr;     // [n_slots] pinned, device-visible: span of the slot's last launch
  uint32_t n_slots = 0;
  uint64_t seq = 0;
};

// Counters a restore accumulates privately and merges into the context statistics at its end.
struct StatDelta {
  uint64_t bytes_filled[BSR_MAX_RANKS] = {}, bytes_h2d[BSR_MAX_RANKS] = {},
           bytes_installed[BSR_MAX_RANKS] = {};
  uint64_t windows = 0, kernel_launches = 0, h2d_copies = 0, install_launches = 0,
           install_descriptors = 0;
  double install_kernel_ms = 0.0, install_span_ms = 0.0;
};

// One fill task: a piece of one chunk of one rank, bytes [off, off + len) of the tier object.
struct FillTask {
  uint32_t item;  // chunk * R + rank
  uint32_t off, len;
};

// Host-side state of one restore through the slot pool.
struct Job {
  bsr_req *q = nullptr;
  Clock::time_point deadline;
  std::vector<FillTask> tasks;                // every piece of every item, in admission order
  std::vector<uint32_t> task_begin;           // per (chunk, rank) item: index of its first piece; [n] = all pieces
  std::unique_ptr<std::atomic<int>[]> state;  // per piece: 0 pending, 1 ready, <0 error
  std::vector<TierObj> objs;                  // per (chunk, rank)
  std::vector<uint32_t> slot;                 // per (chunk, rank): slot of the rank's pool
  std::vector<uint64_t> t_piece;              // per piece: ns since restore start when its fill ended
  std::vector<bsr_trace_rec> trace;           // per (chunk, rank)
  Clock::time_point t0;
  std::atomic<bool> abort{false};
  uint32_t fill_admitted = 0, fill_next = 0, fill_active = 0;  // guarded by fill_mu
  uint64_t pieces_done = 0;     // guarded by fill_mu: fill tasks finished so far
  std::condition_variable cv;   // with fill_mu: signalled when a fill task of this restore finishes
};

// Where the fill threads and the pinned pool are placed on a host with several NUMA nodes.
struct NumaPlacement {
  int node = -1;      // NUMA node of the context's GPU, -1 unknown
  bool bind = false;  // fill threads and the allocating thread are bound to `cpus`
  cpu_set_t cpus;
};

}  // namespace

struct bsr_req {
  bsr_ctx *ctx = nullptr;
  std::mutex mu;
  uint32_t n_adv = 0;
  std::vector<uint64_t> keys;
  std::vector<std::vector<int32_t>> tables;  // [R*G]
  int32_t *d_tables = nullptr;               // all tables, flat
  const int32_t **d_table_ptrs = nullptr;    // [R*G] device pointers into d_tables
  uint64_t *h_ck = nullptr;                  // pinned, device-visible: [(R*G)][n_adv]
  uint32_t *h_verdict = nullptr;             // pinned, device-visible
  uint64_t *d_ck = nullptr;                  // device aliases of the two arrays above
  uint32_t *d_verdict = nullptr;
  BsrChunkDesc *h_desc = nullptr;            // pinned: one descriptor per (chunk, rank), batch launches
  BsrChunkDesc *d_desc = nullptr;            // device copy, uploaded once per restore
  std::vector<uint64_t> bitmap;              // [R*G][words]
  uint32_t words = 0;
  bool restored = false;
  bool failed = false;
  uint64_t request_id = 0;  // engine's request identity (bsr_req_bind); 0 = unbound
  uint32_t tier = 0;        // the one tier this request is served from
  bool bound = false;
  std::mutex async_mu;       // guards the three fields below
  std::thread async_thread;  // bsr_restore_async: the thread running the restore
  int async_rc = BSR_OK;
  bool async_pending = false;
};

struct bsr_ctx {
  bsr_config cfg{};
  uint32_t budget = 0;  // B: slots per rank shared by all restores (= W without an admission budget)
  NumaPlacement numa;
  uint32_t sm_count = 1;  // multiprocessors of the context's GPU: grids are sized in whole waves of it
  std::mutex mu, restore_mu, aux_mu, setup_mu, fill_mu, pool_mu;
  std::string err;

  // registration
  uint32_t G = 0, L = 0;
  bool rank_registered[BSR_MAX_RANKS] = {};
  std::vector<bsr_group_desc> groups;
  std::vector<TensorReg> tensors;
  uint64_t chunk_bytes = 0, slot_bytes = 0;
  uint64_t seg_begin[BSR_MAX_GROUPS] = {}, seg_bytes[BSR_MAX_GROUPS] = {};
  std::atomic<bool> finalized{false};
  bool use_bulk = true;  // the install kernel chosen for this registration (see finalize_registration)
  bool has_spans = false;     // the tile table holds spans of several runs
  bool mostly_spans = false;  // ... and they carry more than half of a chunk's bytes
  std::vector<BsrTile> h_tiles;
  BsrTile *d_tiles = nullptr;
  uint64_t *d_tensor_base = nullptr;
  uint32_t *d_tensor_group = nullptr, *d_tensor_run = nullptr;

  // tiers + index (mu)
  std::unordered_map<uint64_t, TierObj> tier[BSR_MAX_TIERS][BSR_MAX_RANKS];
  bool tier_available[BSR_MAX_TIERS] = {true, true, true, true};
  bsr_fetch_fn fetch_fn[BSR_MAX_TIERS] = {};  // tier adapters: fill a slot for objects put without data
  void *fetch_user[BSR_MAX_TIERS] = {};
  std::unordered_set<uint64_t> force_local;  // request ids whose next probe must report zero
  Inject inject;
  bsr_stats st{};
  std::vector<bsr_trace_rec> last_trace;  // timeline of the last restore through the slot pool

  // context-level stream and scratch for probe, store-path checksums, scrub (aux_mu)
  cudaStream_t copy_stream = nullptr, own_stream = nullptr;
  JobRes aux;
  uint8_t *d_put_stage = nullptr;
  uint64_t *h_put_ck = nullptr, *d_put_ck = nullptr;  // pinned [G] sums + verdict dump
  uint32_t *h_put_verdict = nullptr, *d_put_verdict = nullptr;
  unsigned int *d_probe_cnt = nullptr;
  int32_t *h_tok = nullptr, *d_tok = nullptr;  // pinned staging for host token ids + its device alias
  uint64_t *d_digests = nullptr, *h_keys = nullptr, *d_keys = nullptr;  // keys: pinned + device alias
  size_t probe_cap_chunks = 0;

  // slot pool (setup_mu to create, pool_mu to use)
  std::atomic<bool> ring_ready{false};
  uint8_t *ring[BSR_MAX_RANKS] = {};
  uint8_t *ring_dev[BSR_MAX_RANKS] = {};  // device-side addresses of the pinned rings
  std::vector<uint32_t> free_slots[BSR_MAX_RANKS];
  uint64_t live_total[BSR_MAX_RANKS] = {};
  std::vector<JobRes *> res_free, res_all;  // setup_mu

  // fill task queue (fill_mu)
  std::vector<std::thread> fillers;
  std::condition_variable fill_cv;
  bool fill_shutdown = false;
  std::vector<Job *> jobs;
  size_t rr = 0;
};

namespace {

int fail(bsr_ctx *c, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) {
    std::lock_guard<std::mutex> g(c->mu);
    c->err = buf;
  }
  return code;
}

#define CU(c, call)                                                                     \
  do {                                                                                  \
    cudaError_t e_ = (call);                                                            \
    if (e_ != cudaSuccess)                                                              \
      return fail((c), BSR_ERR_CUDA, "%s: %s (%s:%d)", #call, cudaGetErrorString(e_),   \
                  __FILE__, __LINE__);                                                  \
  } while (0)

uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

void merge_stats(bsr_ctx *c, const StatDelta &d) {
  std::lock_guard<std::mutex> g(c->mu);
  for (uint32_t r = 0; r < BSR_MAX_RANKS; ++r) {
    c->st.bytes_filled[r] += d.bytes_filled[r];
    c->st.bytes_h2d[r] += d.bytes_h2d[r];
    c->st.bytes_installed[r] += d.bytes_installed[r];
  }
  c->st.windows += d.windows;
  c->st.kernel_launches += d.kernel_launches;
  c->st.h2d_copies += d.h2d_copies;
  c->st.install_launches += d.install_launches;
  c->st.install_descriptors += d.install_descriptors;
  c->st.install_kernel_ms += d.install_kernel_ms;
  c->st.install_span_ms += d.install_span_ms;
}

// ---- registration -> span table -----------------------------------------------------------------
// Cuts one chunk into the spans the install kernels move (see BsrTile).  block_tokens per group;
// group and bytes per token per tensor, group-major.
void plan_spans(const std::vector<uint32_t> &block_tokens, const std::vector<uint32_t> &tensor_group,
                const std::vector<uint32_t> &tensor_bpt, std::vector<BsrTile> &out) {
  const uint32_t L = (uint32_t)tensor_group.size();
  std::vector<uint64_t> seg_begin(block_tokens.size(), 0);
  {
    std::vector<bool> seen(block_tokens.size(), false);
    uint64_t o = 0;
    for (uint32_t l = 0; l < L; ++l) {
      if (!seen[tensor_group[l]]) {
        seen[tensor_group[l]] = true;
        seg_begin[tensor_group[l]] = o;
      }
      o += (uint64_t)BSR_CHUNK_TOKENS * tensor_bpt[l];
    }
  }
  uint64_t off = 0;
  out.clear();
  for (uint32_t l = 0; l < L;) {
    const uint32_t group = tensor_group[l], bpt = tensor_bpt[l];
    const uint32_t B = block_tokens[group];
    const uint32_t nb = BSR_CHUNK_TOKENS / B;
    const uint64_t run = (uint64_t)B * bpt;
    const uint32_t run_inv = (uint32_t)(((1ull << 32) + run - 1) / run);
    // Runs of up to BSR_K_SPAN_RUN_MAX bytes travel several to a span: below that a bulk copy per
    // run costs more in issue and stage turnover (about 150 ns per CTA) than its bytes are worth.
    const bool spans = run <= BSR_K_SPAN_RUN_MAX && 2 * run <= BSR_K_TILE_MAX;
    // a family: this tensor and the ones after it with the same group and bytes per token; their
    // runs have one length and lie back to back in the chunk
    uint32_t l_end = l + 1;
    if (spans)
      while (l_end < L && tensor_group[l_end] == group && tensor_bpt[l_end] == bpt) ++l_end;
    BsrTile tl{};
    tl.run_bytes = (uint32_t)run;
    tl.run_inv = run_inv;
    tl.group = (uint8_t)group;
    if (spans) {
      // short runs: spans of as many whole runs as a stage holds, across the family's tensors
      const uint32_t per_span = (uint32_t)(BSR_K_TILE_MAX / run);
      const uint32_t runs = (l_end - l) * nb;
      for (uint32_t v0 = 0; v0 < runs; v0 += per_span) {
        const uint32_t cnt = runs - v0 < per_span ? runs - v0 : per_span;
        tl.src_off = (uint32_t)(off + (uint64_t)v0 * run);
        tl.bytes = (uint32_t)(cnt * run);
        tl.dst_off = 0;
        tl.word0 = (uint32_t)((tl.src_off - seg_begin[group]) / 4);
        tl.tensor = (uint16_t)(l + v0 / nb);
        tl.blk = (uint8_t)(v0 % nb);
        tl.n_runs = cnt;
        out.push_back(tl);
      }
    } else {
      // long runs: each run on its own, cut into pieces of at most a stage
      const uint32_t nsplit = (uint32_t)((run + BSR_K_TILE_MAX - 1) / BSR_K_TILE_MAX);
      const uint32_t piece = (uint32_t)round_up((run + nsplit - 1) / nsplit, 128);
      for (uint32_t b = 0; b < nb; ++b)
        for (uint64_t s = 0; s < run; s += piece) {
          tl.src_off = (uint32_t)(off + b * run + s);
          tl.bytes = (uint32_t)((run - s < piece) ? run - s : piece);
          tl.dst_off = (uint32_t)s;
          tl.word0 = (uint32_t)((tl.src_off - seg_begin[group]) / 4);
          tl.tensor = (uint16_t)l;
          tl.blk = (uint8_t)b;
          tl.n_runs = 1;
          out.push_back(tl);
        }
    }
    off += (uint64_t)(l_end - l) * BSR_CHUNK_TOKENS * bpt;
    l = l_end;
  }
}

// ---- registration -> tile table (setup_mu held) --------------------------------------------------
int finalize_registration(bsr_ctx *c) {
  if (c->finalized.load(std::memory_order_acquire)) return BSR_OK;
  if (c->L == 0) return fail(c, BSR_ERR_STATE, "no registration");
  for (uint32_t r = 0; r < c->cfg.n_ranks; ++r)
    if (!c->rank_registered[r]) return fail(c, BSR_ERR_STATE, "rank %u is not registered", r);
  CU(c, cudaSetDevice(c->cfg.device));
  std::vector<uint32_t> tgroup(c->L), trun(c->L);
  for (uint32_t l = 0; l < c->L; ++l) {
    tgroup[l] = c->tensors[l].group;
    trun[l] = c->groups[c->tensors[l].group].block_tokens * c->tensors[l].bytes_per_token;
  }
  {
    std::vector<uint32_t> bt(c->G), tg(c->L), te(c->L);
    for (uint32_t g = 0; g < c->G; ++g) bt[g] = c->groups[g].block_tokens;
    for (uint32_t l = 0; l < c->L; ++l) {
      tg[l] = c->tensors[l].group;
      te[l] = c->tensors[l].bytes_per_token;
    }
    plan_spans(bt, tg, te, c->h_tiles);
  }
  // the kernels count the tiles of a launch (up to BSR_K_MAX_BATCH chunks) in 32 bits
  if (c->h_tiles.size() > (1u << 22))
    return fail(c, BSR_ERR_INVALID, "registration needs %zu tiles per chunk (limit %u)",
                c->h_tiles.size(), 1u << 22);
  std::vector<uint64_t> bases((size_t)c->cfg.n_ranks * c->L);
  for (uint32_t r = 0; r < c->cfg.n_ranks; ++r)
    for (uint32_t l = 0; l < c->L; ++l) bases[(size_t)r * c->L + l] = c->tensors[l].base[r];
  CU(c, cudaMalloc(&c->d_tiles, c->h_tiles.size() * sizeof(BsrTile)));
  CU(c, cudaMemcpy(c->d_tiles, c->h_tiles.data(), c->h_tiles.size() * sizeof(BsrTile),
                   cudaMemcpyHostToDevice));
  CU(c, cudaMalloc(&c->d_tensor_base, bases.size() * 8));
  CU(c, cudaMemcpy(c->d_tensor_base, bases.data(), bases.size() * 8, cudaMemcpyHostToDevice));
  CU(c, cudaMalloc(&c->d_tensor_group, c->L * 4));
  CU(c, cudaMemcpy(c->d_tensor_group, tgroup.data(), c->L * 4, cudaMemcpyHostToDevice));
  CU(c, cudaMalloc(&c->d_tensor_run, c->L * 4));
  CU(c, cudaMemcpy(c->d_tensor_run, trun.data(), c->L * 4, cudaMemcpyHostToDevice));
  CU(c, cudaFuncSetAttribute(bsr_install_bulk_kernel<BSR_K_BULK_SUM_WARPS>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, BSR_K_BULK_SMEM));
  CU(c, cudaFuncSetAttribute(bsr_install_bulk_kernel<BSR_K_BULK_SUM_WARPS_SPANS>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, BSR_K_BULK_SMEM));
  {
    std::lock_guard<std::mutex> g(c->mu);
    c->st.dev_aux_bytes += c->h_tiles.size() * sizeof(BsrTile) + bases.size() * 8 + c->L * 8;
  }
  // Kernel choice.  Measured on B200, 256-descriptor launches: the bulk-copy kernel runs at the
  // speed of a device copy where the bytes sit in runs that travel on their own (1.28 ms on the
  // baseline registration) and, with eight sum warps to issue the scattered stores of short-run
  // spans, at 0.91 of it on a registration of 256-byte runs, ahead of the vector kernel on every
  // registration tried (0.89 there, 0.86 on the 170-tensor one).  So BSR_INSTALL_AUTO means the
  // bulk-copy kernel; the vector kernel serves direct_install and an explicit request.
  uint64_t span_bytes = 0;
  for (const BsrTile &tl : c->h_tiles)
    if (tl.n_runs > 1) span_bytes += tl.bytes;
  c->has_spans = span_bytes != 0;
  c->mostly_spans = 2 * span_bytes > c->chunk_bytes;
  c->use_bulk = c->cfg.install_variant != BSR_INSTALL_VECTOR;
  c->finalized.store(true, std::memory_order_release);
  return BSR_OK;
}

int ensure_finalized(bsr_ctx *c) {
  if (c->finalized.load(std::memory_order_acquire)) return BSR_OK;
  std::lock_guard<std::mutex> sl(c->setup_mu);
  return finalize_registration(c);
}

void fill_params(bsr_ctx *c, BsrInstallParams &p, JobRes *res, uint32_t slot) {
  p.tiles = c->d_tiles;
  p.n_tiles = (uint32_t)c->h_tiles.size();
  p.n_groups = c->G;
  p.n_tensors = c->L;
  p.tensor_base = c->d_tensor_base;
  for (uint32_t g = 0; g < c->G; ++g)
    p.blocks_per_chunk[g] = BSR_CHUNK_TOKENS / c->groups[g].block_tokens;
  p.acc = res->d_acc + (size_t)slot * BSR_K_MAX_BATCH * BSR_K_MAX_GROUPS;
  p.ctas_done = res->d_cnt + slot;
  p.err_flag = res->d_err;
  p.stall_tile = ~0u;
  if (c->cfg.time_kernels) {
    p.span_start = res->d_span_start + slot;
    p.span_out = res->d_span + slot;
  }
}

// host_source: the chunk is read from mapped host memory; plain loads are used for that.
int launch_install(bsr_ctx *c, const BsrInstallParams &p, cudaStream_t s, StatDelta &sd,
                   bool host_source = false) {
  const uint64_t total = (uint64_t)p.n_chunks * p.n_tiles;
  if (c->use_bulk && !host_source) {
    // Whole waves of the CTAs an SM holds, each CTA streaming BSR_K_BULK_TILES_PER_CTA tiles through
    // its stage ring: several waves instead of one persistent wave let the hardware scheduler even
    // out the tail (measured on B200: 1.28 ms against 1.35 ms per 256-descriptor launch).
    const uint64_t wave = (uint64_t)c->sm_count * BSR_K_BULK_CTAS_PER_SM;
    uint64_t want = (total / BSR_K_BULK_TILES_PER_CTA + wave - 1) / wave * wave;
    if (want < wave) want = wave;
#ifdef BSR_K_BULK_MAX_GRID  // test builds: few CTAs, so that each one cycles its stage ring many times
    if (want > BSR_K_BULK_MAX_GRID) want = BSR_K_BULK_MAX_GRID;
#endif
    const uint32_t grid = (uint32_t)(total < want ? total : want);
    if (c->mostly_spans)
      bsr_install_bulk_kernel<BSR_K_BULK_SUM_WARPS_SPANS>
          <<<grid, BSR_K_BULK_THREADS(BSR_K_BULK_SUM_WARPS_SPANS), BSR_K_BULK_SMEM, s>>>(p);
    else
      bsr_install_bulk_kernel<BSR_K_BULK_SUM_WARPS>
          <<<grid, BSR_K_BULK_THREADS(BSR_K_BULK_SUM_WARPS), BSR_K_BULK_SMEM, s>>>(p);
  } else {
    // About nine tiles per CTA, in whole waves of the 8 CTAs an SM holds: many more CTAs than are
    // resident let the hardware scheduler even out the tail (measured best on B200; one tile per
    // CTA and a single persistent wave are both slower).
    const uint64_t wave = (uint64_t)c->sm_count * 8;
    uint64_t want = (total / 9 + wave - 1) / wave * wave;
    if (want < 2 * wave) want = 2 * wave;
    const uint32_t grid = (uint32_t)(total < want ? total : want);
    if (c->has_spans)
      bsr_install_vec_kernel<kInstallThreads, kInstallUnroll, true><<<grid, kInstallThreads, 0, s>>>(p);
    else
      bsr_install_vec_kernel<kInstallThreads, kInstallUnroll, false><<<grid, kInstallThreads, 0, s>>>(p);
  }
  CU(c, cudaGetLastError());
  sd.kernel_launches++;
  sd.install_launches++;
  sd.install_descriptors += p.n_chunks;
  return BSR_OK;
}

// ---- per-restore device resources ----------------------------------------------------------------
void destroy_res(JobRes *res) {
  for (uint32_t r = 0; r < BSR_MAX_RANKS; ++r)
    if (res->dstage[r]) cudaFree(res->dstage[r]);
  for (auto e : res->ev_h2d) cudaEventDestroy(e);
  for (auto e : res->ev_inst) cudaEventDestroy(e);
  for (auto e : res->ev_start) cudaEventDestroy(e);
  for (auto &pr : res->ev_pool) {
    cudaEventDestroy(pr.first);
    cudaEventDestroy(pr.second);
  }
  if (res->ev_done) cudaEventDestroy(res->ev_done);
  cudaFree(res->d_acc);
  cudaFree(res->d_cnt);
  cudaFree(res->d_span_start);
  if (res->h_span) cudaFreeHost(res->h_span);
  if (res->h_err) cudaFreeHost(res->h_err);
  if (res->stream) cudaStreamDestroy(res->stream);
}

int init_scratch(bsr_ctx *c, JobRes *res, uint32_t n_slots) {
  res->n_slots = n_slots;
  const size_t acc_bytes = (size_t)n_slots * BSR_K_MAX_BATCH * BSR_K_MAX_GROUPS * 8;
  const size_t cnt_bytes = n_slots * sizeof(unsigned int);
  CU(c, cudaMalloc(&res->d_acc, acc_bytes));
  CU(c, cudaMalloc(&res->d_cnt, cnt_bytes));
  CU(c, cudaMemset(res->d_acc, 0, acc_bytes));
  CU(c, cudaMemset(res->d_cnt, 0, cnt_bytes));
  CU(c, cudaHostAlloc((void **)&res->h_err, sizeof(unsigned int), cudaHostAllocMapped));
  CU(c, cudaHostGetDevicePointer((void **)&res->d_err, res->h_err, 0));
  *res->h_err = 0;
  CU(c, cudaMalloc(&res->d_span_start, n_slots * 8));
  CU(c, cudaMemset(res->d_span_start, 0, n_slots * 8));
  CU(c, cudaHostAlloc((void **)&res->h_span, n_slots * 8, cudaHostAllocMapped));
  CU(c, cudaHostGetDevicePointer((void **)&res->d_span, res->h_span, 0));
  memset(res->h_span, 0, n_slots * 8);
  CU(c, cudaEventCreateWithFlags(&res->ev_done, cudaEventDisableTiming));
  std::lock_guard<std::mutex> g(c->mu);
  c->st.dev_aux_bytes += acc_bytes + cnt_bytes;
  return BSR_OK;
}

// A resource set from the pool, or a new one (setup_mu taken here).
int acquire_res(bsr_ctx *c, JobRes **out) {
  std::lock_guard<std::mutex> sl(c->setup_mu);
  if (!c->res_free.empty()) {
    *out = c->res_free.back();
    c->res_free.pop_back();
    return BSR_OK;
  }
  const uint32_t R = c->cfg.n_ranks, D = c->cfg.dev_staging_depth;
  JobRes *res = new (std::nothrow) JobRes();
  if (!res) return BSR_ERR_NOMEM;
  c->res_all.push_back(res);
  CU(c, cudaStreamCreateWithFlags(&res->stream, cudaStreamNonBlocking));
  int rc = init_scratch(c, res, R * D + kLaunchSlots);
  if (rc != BSR_OK) return rc;
  if (!c->cfg.direct_install) {
    for (uint32_t r = 0; r < R; ++r) {
      if (cudaMalloc((void **)&res->dstage[r], (size_t)D * c->chunk_bytes) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, BSR_ERR_NOMEM, "device staging of %u x %llu bytes", D,
                    (unsigned long long)c->chunk_bytes);
      }
    }
    std::lock_guard<std::mutex> g(c->mu);
    c->st.dev_aux_bytes += (uint64_t)R * D * c->chunk_bytes;
  }
  res->ev_h2d.resize(res->n_slots);
  res->ev_inst.resize(res->n_slots);
  res->ev_start.resize(res->n_slots);
  for (uint32_t k = 0; k < res->n_slots; ++k) {
    CU(c, cudaEventCreateWithFlags(&res->ev_h2d[k], cudaEventDisableTiming));
    CU(c, cudaEventCreate(&res->ev_inst[k]));
    CU(c, cudaEventCreate(&res->ev_start[k]));
  }
  *out = res;
  return BSR_OK;
}

void release_res(bsr_ctx *c, JobRes *res) {
  std::lock_guard<std::mutex> sl(c->setup_mu);
  c->res_free.push_back(res);
}

// ---- filler threads: tier object -> pinned slot -------------------------------------------------
// Streaming copy for the fill: the destination slot will next be read by the copy engine, not by
// this core, so non-temporal stores keep it out of the caches and spare the read-for-ownership.
__attribute__((target("avx2"))) void stream_copy_avx2(uint8_t *dst, const uint8_t *src, size_t n) {
  size_t i = 0;
  while (i < n && (reinterpret_cast<uintptr_t>(dst + i) & 31u)) {
    dst[i] = src[i];
    ++i;
  }
  for (; i + 128 <= n; i += 128) {
    _mm_prefetch(reinterpret_cast<const char *>(src + i + 1024), _MM_HINT_NTA);
    const __m256i a = _mm256_loadu_si256(reinterpret_cast<const __m256i *>(src + i));
    const __m256i b = _mm256_loadu_si256(reinterpret_cast<const __m256i *>(src + i + 32));
    const __m256i c2 = _mm256_loadu_si256(reinterpret_cast<const __m256i *>(src + i + 64));
    const __m256i d = _mm256_loadu_si256(reinterpret_cast<const __m256i *>(src + i + 96));
    _mm256_stream_si256(reinterpret_cast<__m256i *>(dst + i), a);
    _mm256_stream_si256(reinterpret_cast<__m256i *>(dst + i + 32), b);
    _mm256_stream_si256(reinterpret_cast<__m256i *>(dst + i + 64), c2);
    _mm256_stream_si256(reinterpret_cast<__m256i *>(dst + i + 96), d);
  }
  _mm_sfence();
  for (; i < n; ++i) dst[i] = src[i];
}

void fill_copy(uint8_t *dst, const uint8_t *src, size_t n) {
  static const bool avx2 = __builtin_cpu_supports("avx2");
  if (avx2 && n >= 4096)
    stream_copy_avx2(dst, src, n);
  else
    memcpy(dst, src, n);
}

// One fill task = one piece (at most kPieceBytes) of one chunk of one rank of one restore.  Pieces
// let the first device copy start after a fraction of a chunk has been fetched and keep all threads
// busy on the chunks the copy engine needs next.  Restores in flight are served round-robin.
void filler_main(bsr_ctx *c) {
  if (c->numa.bind) pthread_setaffinity_np(pthread_self(), sizeof(cpu_set_t), &c->numa.cpus);
  for (;;) {
    Job *job = nullptr;
    uint32_t t = 0;
    {
      std::unique_lock<std::mutex> lk(c->fill_mu);
      c->fill_cv.wait(lk, [&] {
        if (c->fill_shutdown) return true;
        for (Job *j : c->jobs)
          if (j->fill_next < j->fill_admitted) return true;
        return false;
      });
      if (c->fill_shutdown) return;
      const size_t n = c->jobs.size();
      for (size_t k = 0; k < n; ++k) {
        Job *j = c->jobs[(c->rr + k) % n];
        if (j->fill_next < j->fill_admitted) {
          job = j;
          c->rr = (c->rr + k + 1) % n;
          break;
        }
      }
      t = job->fill_next++;
      job->fill_active++;
    }
    bsr_req *req = job->q;
    const uint32_t R = c->cfg.n_ranks;
    const FillTask ft = job->tasks[t];
    const uint32_t s = ft.item, piece = t - job->task_begin[s];
    const uint32_t i = s / R, r = s % R;
    const uint64_t off = ft.off, len = ft.len;
    int state = 1;
    TierObj obj{};
    if (!job->abort.load(std::memory_order_acquire)) {
      bool found = false, tier_down = false;
      Inject inj;
      bsr_fetch_fn fetch = nullptr;
      void *fetch_user = nullptr;
      {
        std::lock_guard<std::mutex> g(c->mu);
        auto &index = c->tier[req->tier][r];
        auto it = index.find(req->keys[i]);
        if (it != index.end()) {
          obj = it->second;
          found = true;
        }
        if (!c->tier_available[req->tier]) tier_down = true;
        inj = c->inject;
        fetch = c->fetch_fn[req->tier];
        fetch_user = c->fetch_user[req->tier];
      }
      const bool hit = inj.kind != BSR_INJECT_NONE && inj.rank == r && inj.chunk == i;
      if (tier_down) {
        state = BSR_ERR_TRANSFER;  // the tier went away after the probe
      } else if (!found) {
        state = BSR_ERR_MISSING;
      } else if (hit && inj.kind == BSR_INJECT_FILL_ERROR) {
        state = BSR_ERR_TRANSFER;
      } else if (hit && inj.kind == BSR_INJECT_FILL_STALL && piece == 0) {
        while (!job->abort.load(std::memory_order_acquire) &&
               Clock::now() < job->deadline + std::chrono::seconds(5))
          std::this_thread::sleep_for(std::chrono::milliseconds(1));
        state = BSR_ERR_TIMEOUT;
      } else if (obj.loc == BSR_LOC_HOST) {
        uint8_t *slot = c->ring[r] + (size_t)job->slot[s] * c->slot_bytes;
        if (obj.data) {
          fill_copy(slot + off, obj.data + off, len);
        } else if (!fetch ||
                   fetch(fetch_user, req->tier, r, req->keys[i], off, len, slot + off) != 0) {
          state = BSR_ERR_TRANSFER;  // the tier adapter could not deliver the bytes
        }
        if (state == 1 && hit && inj.kind == BSR_INJECT_CORRUPT_SLOT && inj.group < c->G) {
          const uint64_t words = c->seg_bytes[inj.group] / 4;
          const uint64_t at = c->seg_begin[inj.group] + 4 * (inj.seed % words);
          if (at >= off && at < off + len)
            *reinterpret_cast<uint32_t *>(slot + at) ^= (uint32_t)(0x80000000u >> (inj.seed % 31));
        }
      }
    }
    if (piece == 0) job->objs[s] = obj;
    job->t_piece[t] = (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(Clock::now() - job->t0).count();
    job->state[t].store(state, std::memory_order_release);
    {
      // the restore thread sleeps on job->cv; it is signalled under the lock because the Job lives
      // on that thread's stack and may go away as soon as fill_active reaches zero
      std::lock_guard<std::mutex> lk(c->fill_mu);
      job->fill_active--;
      job->pieces_done++;
      job->cv.notify_one();
    }
    c->fill_cv.notify_all();
  }
}

// ---- host placement ---------------------------------------------------------------------------
// "0-3,8,10-11" -> CPU set.  Returns the number of CPUs named, -1 on a malformed list.
int parse_cpulist(const char *s, cpu_set_t *set) {
  CPU_ZERO(set);
  int n = 0;
  const char *p = s;
  while (*p && *p != '\n') {
    char *end = nullptr;
    const long lo = strtol(p, &end, 10);
    if (end == p || lo < 0) return -1;
    long hi = lo;
    p = end;
    if (*p == '-') {
      hi = strtol(p + 1, &end, 10);
      if (end == p + 1 || hi < lo) return -1;
      p = end;
    }
    for (long k = lo; k <= hi; ++k)
      if (k < CPU_SETSIZE) {
        CPU_SET((int)k, set);
        ++n;
      }
    if (*p == ',') ++p;
  }
  return n;
}

bool read_line(const std::string &path, std::string *out) {
  std::ifstream f(path);
  if (!f) return false;
  std::getline(f, *out);
  return true;
}

// Decides where this context's fill threads and pinned pool go (see bsr_config.numa_bind).
void plan_numa(bsr_ctx *c) {
  CPU_ZERO(&c->numa.cpus);
  if (c->cfg.numa_bind == BSR_NUMA_OFF) return;
  char bus[32] = {};
  if (cudaDeviceGetPCIBusId(bus, sizeof bus, c->cfg.device) != cudaSuccess) {
    cudaGetLastError();
    return;
  }
  int node = -1, n_nodes = 0;
  char list[1024] = {};
  if (bsr_numa_of_pci("/sys", bus, &node, list, sizeof list, &n_nodes) != BSR_OK) return;
  c->numa.node = node;
  if (node < 0 || (n_nodes < 2 && c->cfg.numa_bind != BSR_NUMA_ALWAYS)) return;
  cpu_set_t want, have;
  if (parse_cpulist(list, &want) <= 0) return;
  if (sched_getaffinity(0, sizeof have, &have) != 0) return;
  CPU_AND(&c->numa.cpus, &want, &have);  // never widen what the process was given
  c->numa.bind = CPU_COUNT(&c->numa.cpus) > 0;
}

// The pinned slot pool: B slots per rank (B = W unless an admission budget is configured).
int ensure_ring(bsr_ctx *c) {
  if (c->ring_ready.load(std::memory_order_acquire)) return BSR_OK;
  std::lock_guard<std::mutex> sl(c->setup_mu);
  if (c->ring_ready.load(std::memory_order_acquire)) return BSR_OK;
  const uint32_t R = c->cfg.n_ranks, B = c->budget;
  // Pinned pages are placed where the allocating thread runs: on a host with several NUMA nodes
  // the pool is allocated from a thread bound to the GPU's node, so that neither the fill threads
  // (bound to the same node) nor the GPU's DMA reads cross the socket interconnect.
  int alloc_rc = BSR_OK;
  auto alloc = [&] {
    if (c->numa.bind) pthread_setaffinity_np(pthread_self(), sizeof(cpu_set_t), &c->numa.cpus);
    if (cudaSetDevice(c->cfg.device) != cudaSuccess) {
      alloc_rc = BSR_ERR_CUDA;
      return;
    }
    for (uint32_t r = 0; r < R; ++r)
      if (cudaHostAlloc((void **)&c->ring[r], (size_t)B * c->slot_bytes, BSR_RING_ALLOC_FLAGS) !=
              cudaSuccess ||
          cudaHostGetDevicePointer((void **)&c->ring_dev[r], c->ring[r], 0) != cudaSuccess) {
        cudaGetLastError();
        alloc_rc = BSR_ERR_NOMEM;
        return;
      }
  };
  if (c->numa.bind)
    std::thread(alloc).join();
  else
    alloc();
  if (alloc_rc != BSR_OK)
    return fail(c, alloc_rc, "pinned pool of %u x %llu bytes", B, (unsigned long long)c->slot_bytes);
  for (uint32_t r = 0; r < R; ++r) {
    {
      std::lock_guard<std::mutex> g(c->mu);
      c->st.ring_bytes_allocated[r] = (uint64_t)B * c->slot_bytes;
    }
    std::lock_guard<std::mutex> pl(c->pool_mu);
    c->free_slots[r].clear();
    for (uint32_t k = B; k > 0; --k) c->free_slots[r].push_back(k - 1);
  }
  for (uint32_t k = 0; k < c->cfg.load_concurrency; ++k) c->fillers.emplace_back(filler_main, c);
  c->ring_ready.store(true, std::memory_order_release);
  return BSR_OK;
}

// Waits for a restore started with bsr_restore_async (its status stays available to bsr_restore_wait).
void join_async(bsr_req *q) {
  std::lock_guard<std::mutex> al(q->async_mu);
  if (q->async_thread.joinable()) q->async_thread.join();
}

void invalidate_host(bsr_req *q) {
  std::fill(q->bitmap.begin(), q->bitmap.end(), 0ull);
  q->failed = true;
}

// Reads the verdicts of chunk i of rank r after its install event completed.
int harvest(bsr_ctx *c, bsr_req *q, uint32_t r, uint32_t i, StatDelta &sd) {
  int rc = BSR_OK;
  for (uint32_t g = 0; g < c->G; ++g) {
    const size_t o = ((size_t)r * c->G + g) * q->n_adv + i;
    const uint32_t v = reinterpret_cast<volatile uint32_t *>(q->h_verdict)[o];
    if (v == 1u)
      q->bitmap[((size_t)r * c->G + g) * q->words + i / 64] |= 1ull << (i % 64);
    else
      rc = (v == 2u) ? BSR_ERR_CHECKSUM : BSR_ERR_TRANSFER;
  }
  if (rc == BSR_OK) sd.bytes_installed[r] += c->chunk_bytes;
  return rc;
}

int wait_event_deadline(bsr_ctx *c, cudaEvent_t ev, Clock::time_point deadline) {
  for (;;) {
    cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return BSR_OK;
    if (e != cudaErrorNotReady) return fail(c, BSR_ERR_CUDA, "event: %s", cudaGetErrorString(e));
    if (Clock::now() > deadline) return BSR_ERR_TIMEOUT;
    std::this_thread::yield();
  }
}

// ---- fill pieces ---------------------------------------------------------------------------------
// Cuts the n_items (chunk, rank) items of a restore, in admission order (item = chunk * R + rank), into
// the pieces the fill threads fetch and the copy stream moves.  8 MiB in the body of a prefix.  1 MiB
// for the first chunk of every rank, so that the copy engine starts a fraction of a millisecond into
// the restore; from there the pieces grow by 512 KiB each, so that the fill threads, which all start
// at the same instant, finish theirs one after the other instead of in bursts with the link idle in
// between.  2 MiB for the last items of the prefix, as many as the fill threads can have in the air
// at once.  No piece is shorter than 256 KiB unless its chunk is.
void plan_pieces(uint64_t chunk_bytes, uint32_t n_items, uint32_t R, uint32_t fill_threads,
                 std::vector<FillTask> &tasks, std::vector<uint32_t> &task_begin) {
  const uint64_t in_air = (uint64_t)fill_threads * kPieceBytes;
  uint64_t n_tail = (in_air + chunk_bytes - 1) / chunk_bytes;
  n_tail = (n_tail + R - 1) / R * R;
  if (n_tail > n_items) n_tail = n_items;
  tasks.clear();
  task_begin.assign((size_t)n_items + 1, 0);
  uint64_t ramp = kHeadPieceBytes;
  for (uint32_t s = 0; s < n_items; ++s) {
    task_begin[s] = (uint32_t)tasks.size();
    for (uint64_t off = 0; off < chunk_bytes;) {
      uint64_t want;
      if (s < R) {
        want = kHeadPieceBytes;
      } else if (s + n_tail >= n_items) {
        want = kTailPieceBytes;
      } else {
        if (ramp < kPieceBytes) ramp += 512u << 10;
        want = ramp;
      }
      uint64_t len = chunk_bytes - off < want ? chunk_bytes - off : want;
      if (chunk_bytes - off - len < (256u << 10)) len = chunk_bytes - off;  // no sliver at the end
      tasks.push_back(FillTask{s, (uint32_t)off, (uint32_t)len});
      off += len;
    }
  }
  task_begin[n_items] = (uint32_t)tasks.size();
}

// ---- restore when every advertised chunk already lives in device memory --------------------------
int restore_resident(bsr_ctx *c, bsr_req *q, JobRes *res, cudaStream_t stream,
                     Clock::time_point deadline, const std::vector<TierObj> &objs, StatDelta &sd) {
  const uint32_t R = c->cfg.n_ranks, W = c->cfg.window_chunks, N = q->n_adv;
  const uint32_t per_launch = BSR_K_MAX_BATCH / R ? BSR_K_MAX_BATCH / R : 1;
  int rc = BSR_OK;
  size_t n_timed = 0;
  std::vector<uint32_t> span_slots;  // scratch sets of this call's launches (span measurement)
  // one descriptor per (chunk, rank) in launch order, uploaded once, ahead of the first launch
  for (uint32_t i = 0; i < N; ++i)
    for (uint32_t r = 0; r < R; ++r) {
      BsrChunkDesc &d = q->h_desc[(size_t)i * R + r];
      const TierObj &o = objs[(size_t)i * R + r];
      d.src = o.data;
      d.chunk = i;
      d.rank = r;
      for (uint32_t g = 0; g < BSR_MAX_GROUPS; ++g) d.expect[g] = g < c->G ? o.ck[g] : 0;
    }
  CU(c, cudaMemcpyAsync(q->d_desc, q->h_desc, (size_t)N * R * sizeof(BsrChunkDesc),
                        cudaMemcpyHostToDevice, stream));
  sd.h2d_copies++;
  // Nothing is staged for device-resident objects, so a window bounds nothing here: it is counted
  // (K = ceil(N / W)) and the launches take as many chunks as the kernel's scratch allows.
  sd.windows += (N + W - 1) / W;
  for (uint32_t b0 = 0; b0 < N && rc == BSR_OK; b0 += per_launch) {
    const uint32_t b1 = (b0 + per_launch < N) ? b0 + per_launch : N;
    BsrInstallParams p{};
    const uint32_t slot = R * c->cfg.dev_staging_depth + (uint32_t)(res->seq++ % kLaunchSlots);
    fill_params(c, p, res, slot);
    if (c->cfg.time_kernels) span_slots.push_back(slot);
    p.n_adv = N;
    p.scatter = 1;
    p.tables = q->d_table_ptrs;
    p.ck_out = q->d_ck;
    p.verdict = q->d_verdict;
    p.batch = q->d_desc + (size_t)b0 * R;
    p.n_chunks = (b1 - b0) * R;
    if (c->cfg.time_kernels) {
      if (n_timed == res->ev_pool.size()) {
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        CU(c, cudaEventCreate(&e0));
        CU(c, cudaEventCreate(&e1));
        res->ev_pool.emplace_back(e0, e1);
      }
      CU(c, cudaEventRecord(res->ev_pool[n_timed].first, stream));
    }
    rc = launch_install(c, p, stream, sd);
    if (c->cfg.time_kernels) {
      CU(c, cudaEventRecord(res->ev_pool[n_timed].second, stream));
      ++n_timed;
    }
  }
  CU(c, cudaEventRecord(res->ev_done, stream));
  int wrc = wait_event_deadline(c, res->ev_done, deadline);
  if (wrc == BSR_ERR_TIMEOUT) cudaStreamSynchronize(stream);  // kernels are finite: let them finish
  for (size_t k = 0; k < n_timed; ++k) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, res->ev_pool[k].first, res->ev_pool[k].second) == cudaSuccess)
      sd.install_kernel_ms += ms;
  }
  if (span_slots.size() <= kLaunchSlots)  // every launch had a scratch set of its own
    for (size_t k = 0; k < span_slots.size(); ++k)
      sd.install_span_ms += reinterpret_cast<volatile uint64_t *>(res->h_span)[span_slots[k]] * 1e-6;
  if (rc == BSR_OK) rc = wrc;
  if (rc != BSR_OK) return rc;
  for (uint32_t i = 0; i < N; ++i)
    for (uint32_t r = 0; r < R; ++r) {
      const int h = harvest(c, q, r, i, sd);
      if (h != BSR_OK && rc == BSR_OK) rc = h;
    }
  return rc;
}

// ---- restore through the pinned slot pool --------------------------------------------------------
// `stages` selects how much of the pipeline runs: everything (a restore), or, for calibration, only
// the fill (tier -> slot) or the fill plus the copies to device staging.  The calibration forms
// take the same slots in the same order with the same threads but launch no kernel, so they touch
// neither the paged cache nor the request's bitmap.
enum { kStagesAll = 0, kStagesFill = BSR_CAL_FILL, kStagesFillH2d = BSR_CAL_FILL_H2D };

int restore_ring(bsr_ctx *c, bsr_req *q, JobRes *res, cudaStream_t stream,
                 Clock::time_point deadline, StatDelta &sd, int stages = kStagesAll) {
  int rc = ensure_ring(c);
  if (rc != BSR_OK) return rc;
  const uint32_t R = c->cfg.n_ranks, W = c->cfg.window_chunks, D = c->cfg.dev_staging_depth;
  const uint32_t N = q->n_adv, total = N * R;
  const bool direct = c->cfg.direct_install != 0 && stages == kStagesAll;
  const uint32_t n_ev = res->n_slots;  // launch slots: a scratch set and three events each
  // Chunks of each rank that one install launch takes.  A launch costs about 13 us on top of its
  // bytes (read-only ramp, write-only tail, address look-ups, the last CTA's verdicts), so a single
  // 16 MB chunk (5 us of traffic) runs at a third of device-copy speed, 16 chunks at 0.72 and 32 at
  // 0.88.  A launch never needs more staging buffers than a rank has.  A pinned slot goes back to the
  // pool as soon as its copy into device staging has been observed complete, so the size of a launch
  // does not depend on the window: W bounds the pinned slots (Eq. 3), D the device staging (M_aux).
  // A kernel that reads the pinned slots itself (direct_install) holds them until it is done and
  // takes one chunk per launch.
  uint32_t cpl = c->cfg.install_batch / R;
  if (cpl > D) cpl = D;
  if (cpl > BSR_K_MAX_BATCH / R) cpl = BSR_K_MAX_BATCH / R;
  if (cpl == 0) cpl = 1;
  // items (chunk, rank) per launch; a kernel that reads pinned slots over the link takes one
  const uint32_t gsz = direct ? 1 : cpl * R;

  Job job;
  job.q = q;
  job.deadline = deadline;
  plan_pieces(c->chunk_bytes, total, R, c->cfg.load_concurrency, job.tasks, job.task_begin);
  const size_t n_tasks = job.task_begin[total];
  job.state.reset(new std::atomic<int>[n_tasks]);
  for (size_t k = 0; k < n_tasks; ++k) job.state[k].store(0, std::memory_order_relaxed);
  job.objs.resize(total);
  job.slot.assign(total, 0);
  job.t_piece.assign(n_tasks, 0);
  job.trace.assign(total, bsr_trace_rec{});
  job.t0 = Clock::now();
  auto now_ns = [&] {
    return (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(Clock::now() - job.t0).count();
  };
  {
    std::lock_guard<std::mutex> lk(c->fill_mu);
    c->jobs.push_back(&job);
  }
  // items are numbered s = i * R + r in admission order; each counter below is a prefix length
  // admitted >= submitted >= launched >= reaped (install observed), submitted >= released (slot back
  // in the pool) >= reaped
  uint32_t admitted = 0, submitted = 0, launched = 0, reaped = 0, released = 0, cur_piece = 0;
  struct Launch {
    uint32_t first, count;
  };
  std::vector<Launch> launches;                // install launches issued, in order
  size_t launches_reaped = 0;                  // ... of which observed complete
  uint32_t live[BSR_MAX_RANKS] = {};
  uint64_t seen_done = 0;
  Inject inj;
  {
    std::lock_guard<std::mutex> lk(c->mu);
    inj = c->inject;
  }
  bool stop = false;  // a failure was seen: admit and submit nothing more, drain
  // short sleeps while polling events: without this the kernel rounds them up by 50 us
  const int slack_before = prctl(PR_GET_TIMERSLACK);
  prctl(PR_SET_TIMERSLACK, 1000UL);

  auto first_error = [&](int code) {
    if (rc == BSR_OK) rc = code;
    stop = true;
    job.abort.store(true, std::memory_order_release);
  };
  auto release_slot = [&](uint32_t s) {
    const uint32_t r = s % R;
    std::lock_guard<std::mutex> pl(c->pool_mu);
    c->free_slots[r].push_back(job.slot[s]);
    c->live_total[r]--;
  };
  // Hands the slots of the items below `upto` back, in order (their bytes have left the slot).
  auto release_upto = [&](uint32_t upto) {
    for (; released < upto; ++released) {
      job.trace[released].t_done_ns = now_ns();
      release_slot(released);
      live[released % R]--;
    }
  };
  // Closes the open group [launched, submitted): one install launch over all its descriptors.
  auto launch_group = [&]() {
    const uint32_t first = launched, n = submitted - launched;
    const size_t li = launches.size();
    const uint32_t ls = (uint32_t)(li % n_ev);
    cudaError_t e = cudaSuccess;
    if (stages == kStagesFill) {
      // nothing was queued on the GPU: the group counts as complete at once
    } else if (stages == kStagesFillH2d) {
      e = cudaEventRecord(res->ev_inst[ls], c->copy_stream);
    } else {
      // the copy stream is in order: the copy event of the group's last item covers the whole group
      if (!direct) e = cudaStreamWaitEvent(stream, res->ev_h2d[(first + n - 1) % (R * D)], 0);
      BsrInstallParams p{};
      fill_params(c, p, res, ls);
      p.n_adv = N;
      p.scatter = 1;
      p.tables = q->d_table_ptrs;
      p.ck_out = q->d_ck;
      p.verdict = q->d_verdict;
      p.n_chunks = n;
      bool host_source = false;
      if (n == 1) {
        p.one = q->h_desc[first];  // carried in the kernel parameters
        host_source = direct && job.objs[first].loc == BSR_LOC_HOST;
      } else {
        p.batch = q->d_desc + first;
        if (e == cudaSuccess)
          e = cudaMemcpyAsync(q->d_desc + first, q->h_desc + first, (size_t)n * sizeof(BsrChunkDesc),
                              cudaMemcpyHostToDevice, stream);
      }
      for (uint32_t s = first; s < first + n; ++s)
        if (inj.kind == BSR_INJECT_KERNEL_WAIT && inj.rank == s % R && inj.chunk == s / R) {
          p.stall_tile = 0;             // the first tile of this launch is never loaded ...
          p.wait_ns = 50ull * 1000000;  // ... and every wait in the kernel gives up after 50 ms
        }
      if (e == cudaSuccess && c->cfg.time_kernels) e = cudaEventRecord(res->ev_start[ls], stream);
      if (e != cudaSuccess) {
        first_error(fail(c, BSR_ERR_TRANSFER, "install submit: %s", cudaGetErrorString(e)));
        return;
      }
      const int lrc = launch_install(c, p, stream, sd, host_source);
      e = cudaEventRecord(res->ev_inst[ls], stream);
      if (lrc != BSR_OK) {
        first_error(lrc);
        return;
      }
    }
    if (e != cudaSuccess) {
      // a launch without an event to observe it by: wait for it here, nothing may outlive the call
      cudaStreamSynchronize(stream);
      first_error(fail(c, BSR_ERR_CUDA, "record: %s", cudaGetErrorString(e)));
      return;
    }
    launches.push_back(Launch{first, n});
    launched = submitted;
  };

  while (true) {
    bool progress = false;
    // admit: chunk i of rank r enters the window when this restore holds fewer than W slots of the
    // rank (Eq. 3) and the pool, shared with the other restores in flight, has a free one
    if (!stop) {
      uint32_t n_new = 0;
      while (admitted < total) {
        const uint32_t i = admitted / R, r = admitted % R;
        if (live[r] >= W) break;
        {
          std::lock_guard<std::mutex> pl(c->pool_mu);
          if (c->free_slots[r].empty()) break;
          job.slot[admitted] = c->free_slots[r].back();
          c->free_slots[r].pop_back();
          const uint64_t bytes = ++c->live_total[r] * c->slot_bytes;
          if (bytes > c->st.peak_staging_bytes[r]) c->st.peak_staging_bytes[r] = bytes;
        }
        if (i % W == 0 && r == 0) sd.windows++;
        job.trace[admitted].chunk = i;
        job.trace[admitted].rank = r;
        job.trace[admitted].slot = job.slot[admitted];
        job.trace[admitted].t_admit_ns = now_ns();
        live[r]++;
        ++admitted;
        ++n_new;
      }
      if (n_new) {
        {
          std::lock_guard<std::mutex> lk(c->fill_mu);
          job.fill_admitted = job.task_begin[admitted];
        }
        c->fill_cv.notify_all();
        progress = true;
      }
    }
    // reap, in order: observe the oldest install launch in flight, release the slots of its chunks
    while (launches_reaped < launches.size()) {
      const Launch &L = launches[launches_reaped];
      const uint32_t ls = (uint32_t)(launches_reaped % n_ev);
      cudaError_t e = stages == kStagesFill ? cudaSuccess : cudaEventQuery(res->ev_inst[ls]);
      if (e == cudaErrorNotReady) break;
      if (e != cudaSuccess) {
        first_error(fail(c, BSR_ERR_CUDA, "install event: %s", cudaGetErrorString(e)));
        release_upto(submitted);  // the context is unusable; nothing more can be observed
        reaped = launched;
        launches_reaped = launches.size();
        break;
      }
      if (c->cfg.time_kernels && stages == kStagesAll) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, res->ev_start[ls], res->ev_inst[ls]) == cudaSuccess)
          sd.install_kernel_ms += ms;
        sd.install_span_ms += reinterpret_cast<volatile uint64_t *>(res->h_span)[ls] * 1e-6;
      }
      if (stages == kStagesAll)
        for (uint32_t s = L.first; s < L.first + L.count; ++s) {
          const int h = harvest(c, q, s % R, s / R, sd);
          if (h != BSR_OK) first_error(h);
        }
      release_upto(L.first + L.count);  // a finished launch has read its chunks, wherever they lay
      reaped = L.first + L.count;
      ++launches_reaped;
      progress = true;
    }
    // release, in order: a chunk whose copy into device staging has been observed complete no longer
    // needs its pinned slot (the fill-only calibration queues no copy: the slot is free at once)
    if (!direct) {
      const uint32_t before = released;
      while (released < submitted) {
        if (stages != kStagesFill) {
          const cudaError_t e = cudaEventQuery(res->ev_h2d[released % (R * D)]);
          if (e == cudaErrorNotReady) break;
          if (e != cudaSuccess) {
            first_error(fail(c, BSR_ERR_CUDA, "copy event: %s", cudaGetErrorString(e)));
            release_upto(submitted);
            break;
          }
        }
        release_upto(released + 1);
      }
      if (released != before) progress = true;
    }
    // submit, in order: every ready piece slot -> device staging on the copy stream; a chunk whose
    // pieces are all queued joins the open group, and a full group is launched
    while (!stop && submitted < admitted && submitted - reaped < R * D) {
      const uint32_t i = submitted / R, r = submitted % R, d = i % D;
      uint8_t *stage = direct ? nullptr : res->dstage[r] + (size_t)d * c->chunk_bytes;
      uint8_t *slot_host = c->ring[r] + (size_t)job.slot[submitted] * c->slot_bytes;
      cudaError_t e = cudaSuccess;
      bool blocked = false;
      const uint32_t t0 = job.task_begin[submitted], P = job.task_begin[submitted + 1] - t0;
      while (cur_piece < P) {
        const int stt = job.state[(size_t)t0 + cur_piece].load(std::memory_order_acquire);
        if (stt == 0) {
          blocked = true;
          break;
        }
        if (stt < 0) {
          first_error(stt);
          break;
        }
        const TierObj &o = job.objs[submitted];
        const uint64_t off = job.tasks[t0 + cur_piece].off, len = job.tasks[t0 + cur_piece].len;
        const uint8_t *from = (o.loc == BSR_LOC_HOST) ? slot_host + off : o.data + off;
        if (!direct && stages != kStagesFill) {
          // The staging buffer is free: its previous user, item submitted - R * D, lies in the reaped
          // prefix (the loop condition above), so the launch that read it has been observed complete.
          e = cudaMemcpyAsync(stage + off, from, len, cudaMemcpyDefault, c->copy_stream);
          if (e != cudaSuccess) {
            first_error(fail(c, BSR_ERR_TRANSFER, "copy submit: %s", cudaGetErrorString(e)));
            break;
          }
          sd.h2d_copies++;
        }
        sd.bytes_filled[r] += (o.loc == BSR_LOC_HOST) ? len : 0;
        if (stages != kStagesFill)
          sd.bytes_h2d[r] += len;  // bytes that cross the host link, by copy or by kernel loads
        ++cur_piece;
        progress = true;
      }
      if (stop || blocked) break;
      if (!direct && stages != kStagesFill) {
        // Safe to record again: the event's previous item, submitted - R * D, lies in the reaped prefix.
        e = cudaEventRecord(res->ev_h2d[submitted % (R * D)], c->copy_stream);
        if (e != cudaSuccess) {
          cudaStreamSynchronize(c->copy_stream);  // its copies are queued: nothing may outlive the call
          first_error(fail(c, BSR_ERR_CUDA, "record: %s", cudaGetErrorString(e)));
          break;
        }
      }
      const TierObj &o = job.objs[submitted];
      BsrChunkDesc &cd = q->h_desc[submitted];
      // direct mode: the kernel reads the pinned slot (or the device object) itself over the link
      cd.src = !direct ? stage
                       : (o.loc == BSR_LOC_HOST
                              ? c->ring_dev[r] + (size_t)job.slot[submitted] * c->slot_bytes
                              : o.data);
      cd.chunk = i;
      cd.rank = r;
      for (uint32_t g = 0; g < BSR_MAX_GROUPS; ++g) cd.expect[g] = g < c->G ? o.ck[g] : 0;
      for (uint32_t pc = 0; pc < P; ++pc)
        if (job.t_piece[(size_t)t0 + pc] > job.trace[submitted].t_filled_ns)
          job.trace[submitted].t_filled_ns = job.t_piece[(size_t)t0 + pc];
      job.trace[submitted].t_submit_ns = now_ns();
      ++submitted;
      cur_piece = 0;
      progress = true;
      if (submitted - launched == gsz || submitted == total) launch_group();
    }
    if (reaped == launched && launches_reaped == launches.size() && (stop || reaped == total)) break;
    if (!progress) {
      if (Clock::now() > deadline) {
        first_error(BSR_ERR_TIMEOUT);
        // copies and kernels already queued are finite: wait for them, then reap
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamSynchronize(stream);
        continue;
      }
      // A group that cannot grow must not wait to be full: every admitted chunk has been queued,
      // nothing is in flight whose completion would free a slot or a staging buffer, and admission
      // is held up all the same (other restores hold the rest of the pool).
      if (!stop && submitted > launched && submitted == admitted && cur_piece == 0 &&
          released == submitted && launches_reaped == launches.size()) {
        launch_group();
        continue;
      }
      // Sleep until a fill task of this restore finishes, or for a short while when an event decides
      // what happens next: an install launch in flight, or a copy whose slot the fill is waiting for
      // (the fill threads need the cores more than a spinning waiter does).
      std::unique_lock<std::mutex> lk(c->fill_mu);
      const bool fill_waits_for_a_slot = !stop && admitted < total && released < submitted &&
                                         job.fill_next == job.fill_admitted;  // no piece left to hand out
      if (job.pieces_done == seen_done)
        job.cv.wait_for(lk, (launches_reaped < launches.size() || fill_waits_for_a_slot)
                                ? std::chrono::microseconds(20)
                                : std::chrono::microseconds(200));
      seen_done = job.pieces_done;
    }
  }
  prctl(PR_SET_TIMERSLACK, slack_before > 0 ? (unsigned long)slack_before : 0UL);
  // copies of chunks that never reached an install launch may still be queued
  if (submitted > launched || cur_piece != 0) cudaStreamSynchronize(c->copy_stream);
  // quiesce the fillers: nothing of this request may be touched after return
  job.abort.store(true, std::memory_order_release);
  {
    std::unique_lock<std::mutex> lk(c->fill_mu);
    job.fill_admitted = job.fill_next;  // hand out no further task
    c->fill_cv.wait(lk, [&] { return job.fill_active == 0; });
    for (size_t k = 0; k < c->jobs.size(); ++k)
      if (c->jobs[k] == &job) {
        c->jobs.erase(c->jobs.begin() + k);
        break;
      }
    c->rr = 0;
  }
  // slots still held (their chunks never got as far as a finished copy or install) go back to the pool
  for (uint32_t s = released; s < admitted; ++s) release_slot(s);
  {
    std::lock_guard<std::mutex> lk(c->mu);
    job.trace.resize(admitted);
    c->last_trace.swap(job.trace);
  }
  return rc;
}

// Shared by bsr_probe (tier 0, no request identity) and bsr_probe_request (all available tiers,
// force-local marker).  request_scoped selects the second behaviour.
int probe_impl(bsr_ctx *c, bool request_scoped, uint64_t request_id, const int32_t *tok,
               size_t n_tok, int tok_on_device, uint64_t salt, uint64_t *keys_out,
               uint64_t *hit_bitmap_out, uint32_t *n_hit_chunks, int *tier_out) {
  if (!c || (!tok && n_tok) || !n_hit_chunks) return BSR_ERR_INVALID;
  if (tier_out) *tier_out = -1;
  const size_t N = n_tok / BSR_CHUNK_TOKENS;
  if (N > (1u << 24)) return fail(c, BSR_ERR_INVALID, "probe: more than 2^24 chunks");
  if (tok_on_device && (reinterpret_cast<uintptr_t>(tok) & 15u))
    return fail(c, BSR_ERR_ALIGN, "probe: device token ids must be 16-byte aligned");
  if (N == 0) {
    *n_hit_chunks = 0;
    return BSR_OK;
  }
  std::lock_guard<std::mutex> al(c->aux_mu);  // probe scratch is per context
  CU(c, cudaSetDevice(c->cfg.device));
  if (N > c->probe_cap_chunks) {
    if (c->h_tok) cudaFreeHost(c->h_tok);
    cudaFree(c->d_digests);
    if (c->h_keys) cudaFreeHost(c->h_keys);
    c->h_tok = nullptr;
    c->d_digests = c->h_keys = nullptr;
    c->probe_cap_chunks = 0;
    const size_t cap = round_up(N, 1024);
    // Token ids and keys travel through pinned, device-visible host memory: the kernel reads the
    // ids and writes the keys over the host link itself (4 B per token in, 8 B per chunk out), which
    // spares two copy submissions and their latency on a call that takes tens of microseconds.
    CU(c, cudaHostAlloc((void **)&c->h_tok, cap * BSR_CHUNK_TOKENS * 4, cudaHostAllocMapped));
    CU(c, cudaHostGetDevicePointer((void **)&c->d_tok, c->h_tok, 0));
    CU(c, cudaMalloc((void **)&c->d_digests, cap * 8));
    CU(c, cudaHostAlloc((void **)&c->h_keys, cap * 8, cudaHostAllocMapped));
    CU(c, cudaHostGetDevicePointer((void **)&c->d_keys, c->h_keys, 0));
    c->probe_cap_chunks = cap;
  }
  const int32_t *d_tok = tok;
  cudaStream_t s = c->own_stream;
  if (!tok_on_device) {
    memcpy(c->h_tok, tok, N * BSR_CHUNK_TOKENS * 4);
    d_tok = c->d_tok;
  }
  // k_-1 = mix64(salt ^ mix64(reg_id)); a scalar, computed once per call
  auto mix = [](uint64_t x) {
    x += BSR_K_PHI;
    x = (x ^ (x >> 32)) * BSR_K_PHI;
    x = (x ^ (x >> 29)) * BSR_K_PHI;
    return x ^ (x >> 32);
  };
  const uint64_t k_init = mix(salt ^ mix(c->cfg.reg_id));
  const uint32_t per_block = BSR_K_PROBE_THREADS / 32;
  const uint32_t grid = (uint32_t)((N + per_block - 1) / per_block);
  bsr_probe_kernel<<<grid, BSR_K_PROBE_THREADS, 0, s>>>(d_tok, (uint32_t)N, salt, k_init,
                                                        c->d_digests, c->d_probe_cnt, c->d_keys);
  CU(c, cudaGetLastError());
  CU(c, cudaStreamSynchronize(s));
  // index lookup: keys only; no payload byte is read, nothing is pinned or referenced afterwards
  const size_t words = (N + 63) / 64;
  if (hit_bitmap_out) memset(hit_bitmap_out, 0, words * 8);
  uint32_t best_n = 0;
  int best_tier = -1;
  {
    std::lock_guard<std::mutex> lk(c->mu);
    c->st.kernel_launches++;
    const bool forced = request_scoped && c->force_local.count(request_id) != 0;
    std::vector<uint64_t> bm(words), best_bm(words, 0ull);
    for (uint32_t t = 0; t < BSR_MAX_TIERS && !forced; ++t) {
      if (request_scoped ? !c->tier_available[t] : t != 0) continue;
      std::fill(bm.begin(), bm.end(), 0ull);
      uint32_t n_hit = 0;
      bool prefix = true;
      for (size_t i = 0; i < N; ++i) {
        bool hit = true;
        for (uint32_t r = 0; r < c->cfg.n_ranks && hit; ++r)
          hit = c->tier[t][r].find(c->h_keys[i]) != c->tier[t][r].end();
        if (hit) bm[i / 64] |= 1ull << (i % 64);
        if (!hit) prefix = false;
        if (prefix) ++n_hit;
      }
      // one tier serves the request: the longest complete prefix, the higher-priority tier on a tie
      if (n_hit > best_n || (!request_scoped && t == 0)) {
        best_n = n_hit;
        best_tier = n_hit ? (int)t : -1;
        best_bm = bm;
      }
    }
    if (hit_bitmap_out) memcpy(hit_bitmap_out, best_bm.data(), words * 8);
  }
  if (keys_out) memcpy(keys_out, c->h_keys, N * 8);
  *n_hit_chunks = best_n;
  if (tier_out) *tier_out = best_tier;
  return BSR_OK;
}

}  // namespace

// =================================================================================================
// C interface
// =================================================================================================
extern "C" {

int bsr_ctx_create(const bsr_config *cfg, bsr_ctx **out) {
  if (!cfg || !out) return BSR_ERR_INVALID;
  if (cfg->window_chunks == 0 || cfg->n_ranks == 0 || cfg->n_ranks > BSR_MAX_RANKS ||
      cfg->chunk_tokens != BSR_CHUNK_TOKENS)
    return BSR_ERR_INVALID;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) {
    cudaGetLastError();
    return BSR_ERR_CUDA;
  }
  bsr_ctx *c = new (std::nothrow) bsr_ctx();
  if (!c) return BSR_ERR_NOMEM;
  c->cfg = *cfg;
  if (c->cfg.load_concurrency == 0) {  // auto: one copy thread per two hardware threads, 4..16
    const unsigned hw = std::thread::hardware_concurrency() / 2;
    c->cfg.load_concurrency = hw < 4 ? 4 : (hw > 16 ? 16 : hw);
  }
  if (c->cfg.load_concurrency > 64) c->cfg.load_concurrency = 64;
  // Defaults: 64 chunk descriptors per install launch and as many staging buffers as one launch
  // group needs (D = 64 / R per rank: 32 at R = 2), at least 16.  A group that uses every staging buffer makes the
  // copies of the next group wait until its launch has been observed complete (0.35 ms per 19 ms
  // of copying).  Measured on B200, restore from host memory, W = 32: throughput is the same with
  // 32 / D = 16, 64 / D = 32 and 64 / D = 40 (48.6 / 48.5 / 48.5 GB/s: the host-side fill is the
  // bound), the launches run at 0.88 / 0.95 / 0.90 of the HBM copy rate between their events and
  // 0.94 / 0.98 / 0.98 by the kernel's own clock: a launch that meets a busy copy engine waits about
  // 20 us longer for its start and its completion record.
  if (c->cfg.install_batch == 0) c->cfg.install_batch = 64;
  if (c->cfg.dev_staging_depth == 0) {
    const uint32_t per_rank = c->cfg.install_batch / c->cfg.n_ranks;
    // never fewer than 16: with small launch groups and as few buffers, the pauses between groups add
    // up (8 descriptors per launch with D = 4: 41 GB/s instead of 48)
    c->cfg.dev_staging_depth = per_rank < 16 ? 16 : per_rank;
  }
  if (c->cfg.dev_staging_depth > 64) c->cfg.dev_staging_depth = 64;
  if (c->cfg.timeout_ms == 0) c->cfg.timeout_ms = 30000;
  if (c->cfg.slot_align == 0) c->cfg.slot_align = 4096;
  c->budget = c->cfg.budget_slots ? c->cfg.budget_slots : c->cfg.window_chunks;
  int sms = 0;
  bool ok = cudaSetDevice(cfg->device) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess &&
            sms > 0 &&
            cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&c->own_stream, cudaStreamNonBlocking) == cudaSuccess &&
            init_scratch(c, &c->aux, kLaunchSlots) == BSR_OK &&
            cudaMalloc(&c->d_probe_cnt, sizeof(unsigned int)) == cudaSuccess &&
            cudaMemset(c->d_probe_cnt, 0, sizeof(unsigned int)) == cudaSuccess &&
            cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    bsr_ctx_destroy(c);
    return BSR_ERR_CUDA;
  }
  c->sm_count = (uint32_t)sms;
  plan_numa(c);
  c->st.fill_numa_node = c->numa.bind ? c->numa.node : -1;
  *out = c;
  return BSR_OK;
}

int bsr_ctx_destroy(bsr_ctx *c) {
  if (!c) return BSR_ERR_INVALID;
  cudaSetDevice(c->cfg.device);
  {
    std::lock_guard<std::mutex> lk(c->fill_mu);
    c->fill_shutdown = true;
  }
  c->fill_cv.notify_all();
  for (auto &t : c->fillers) t.join();
  cudaDeviceSynchronize();
  for (uint32_t r = 0; r < BSR_MAX_RANKS; ++r)
    if (c->ring[r]) cudaFreeHost(c->ring[r]);
  for (JobRes *res : c->res_all) {
    destroy_res(res);
    delete res;
  }
  destroy_res(&c->aux);
  cudaFree(c->d_tiles);
  cudaFree(c->d_tensor_base);
  cudaFree(c->d_tensor_group);
  cudaFree(c->d_tensor_run);
  cudaFree(c->d_put_stage);
  if (c->h_put_ck) cudaFreeHost(c->h_put_ck);
  if (c->h_put_verdict) cudaFreeHost(c->h_put_verdict);
  cudaFree(c->d_probe_cnt);
  if (c->h_tok) cudaFreeHost(c->h_tok);
  cudaFree(c->d_digests);
  if (c->h_keys) cudaFreeHost(c->h_keys);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->own_stream) cudaStreamDestroy(c->own_stream);
  cudaGetLastError();
  delete c;
  return BSR_OK;
}

const char *bsr_last_error(bsr_ctx *c) {
  // A copy per calling thread: a failing call on another thread may replace the context's text at
  // any time, so the context's own buffer is never handed out.
  static thread_local std::string mine;
  if (!c) return "null context";
  std::lock_guard<std::mutex> lk(c->mu);
  mine = c->err;
  return mine.c_str();
}

int bsr_register(bsr_ctx *c, uint32_t rank, const bsr_group_desc *groups, uint32_t n_groups,
                 const bsr_tensor_desc *tensors, uint32_t n_tensors) {
  if (!c || !groups || !tensors) return BSR_ERR_INVALID;
  if (rank >= c->cfg.n_ranks || n_groups == 0 || n_groups > BSR_MAX_GROUPS || n_tensors == 0 ||
      n_tensors > 65535)
    return fail(c, BSR_ERR_INVALID, "register: rank/groups/tensors out of range");
  if (c->finalized.load()) return fail(c, BSR_ERR_STATE, "register after the registration was used");
  for (uint32_t g = 0; g < n_groups; ++g) {
    const uint32_t B = groups[g].block_tokens;
    if (B == 0 || BSR_CHUNK_TOKENS % B || BSR_CHUNK_TOKENS / B > 255 || groups[g].num_phys_blocks == 0)
      return fail(c, BSR_ERR_INVALID, "group %u: block_tokens must divide 256", g);
  }
  uint32_t prev_group = 0;
  uint64_t per_token = 0;
  for (uint32_t l = 0; l < n_tensors; ++l) {
    const bsr_tensor_desc &t = tensors[l];
    if (t.group >= n_groups || t.group < prev_group)
      return fail(c, BSR_ERR_INVALID, "tensor %u: tensors must be listed group-major", l);
    prev_group = t.group;
    if (t.bytes_per_token == 0 || t.bytes_per_token % 16)
      return fail(c, BSR_ERR_ALIGN, "tensor %u: bytes_per_token must be a multiple of 16", l);
    if (!t.dev_base || (reinterpret_cast<uintptr_t>(t.dev_base) & 15u))
      return fail(c, BSR_ERR_ALIGN, "tensor %u: dev_base must be 16-byte aligned", l);
    per_token += t.bytes_per_token;
  }
  // every group owns at least one tensor: an empty segment would "verify" as 0 == 0 and count
  // toward the commit predicate without any byte behind it
  {
    bool owned[BSR_MAX_GROUPS] = {};
    for (uint32_t l = 0; l < n_tensors; ++l) owned[tensors[l].group] = true;
    for (uint32_t g = 0; g < n_groups; ++g)
      if (!owned[g]) return fail(c, BSR_ERR_INVALID, "group %u has no tensor", g);
  }
  if (per_token * BSR_CHUNK_TOKENS >= (1ull << 32))
    return fail(c, BSR_ERR_INVALID, "chunk larger than 4 GiB");
  std::lock_guard<std::mutex> lk(c->mu);
  const bool first = (c->L == 0);
  if (first) {
    c->G = n_groups;
    c->L = n_tensors;
    c->groups.assign(groups, groups + n_groups);
    c->tensors.resize(n_tensors);
    uint64_t off = 0;
    for (uint32_t g = 0; g < n_groups; ++g) c->seg_begin[g] = c->seg_bytes[g] = 0;
    bool seen[BSR_MAX_GROUPS] = {};
    for (uint32_t l = 0; l < n_tensors; ++l) {
      c->tensors[l].group = tensors[l].group;
      c->tensors[l].bytes_per_token = tensors[l].bytes_per_token;
      const uint64_t sz = (uint64_t)BSR_CHUNK_TOKENS * tensors[l].bytes_per_token;
      if (!seen[tensors[l].group]) {
        seen[tensors[l].group] = true;
        c->seg_begin[tensors[l].group] = off;
      }
      c->seg_bytes[tensors[l].group] += sz;
      off += sz;
    }
    c->chunk_bytes = off;
    c->slot_bytes = round_up(off, c->cfg.slot_align);
    c->st.slot_bytes = c->slot_bytes;
  } else {
    bool same = (n_groups == c->G && n_tensors == c->L);
    for (uint32_t g = 0; same && g < n_groups; ++g)
      same = groups[g].block_tokens == c->groups[g].block_tokens &&
             groups[g].num_phys_blocks == c->groups[g].num_phys_blocks;
    for (uint32_t l = 0; same && l < n_tensors; ++l)
      same = tensors[l].group == c->tensors[l].group &&
             tensors[l].bytes_per_token == c->tensors[l].bytes_per_token;
    if (!same) {
      c->err = "register: every rank must register the same geometry";
      return BSR_ERR_INVALID;
    }
  }
  for (uint32_t l = 0; l < n_tensors; ++l)
    c->tensors[l].base[rank] = reinterpret_cast<uint64_t>(tensors[l].dev_base);
  c->rank_registered[rank] = true;
  return BSR_OK;
}

int bsr_install_kernel_in_use(bsr_ctx *c, int *variant) {
  if (!c || !variant) return BSR_ERR_INVALID;
  CU(c, cudaSetDevice(c->cfg.device));
  const int rc = ensure_finalized(c);
  if (rc != BSR_OK) return rc;
  *variant = c->use_bulk ? BSR_INSTALL_BULK : BSR_INSTALL_VECTOR;
  return BSR_OK;
}

int bsr_chunk_bytes(bsr_ctx *c, uint64_t *chunk_bytes, uint64_t *slot_bytes) {
  if (!c) return BSR_ERR_INVALID;
  if (c->L == 0) return fail(c, BSR_ERR_STATE, "no registration");
  if (chunk_bytes) *chunk_bytes = c->chunk_bytes;
  if (slot_bytes) *slot_bytes = c->slot_bytes;
  return BSR_OK;
}

int bsr_tier_put(bsr_ctx *c, uint32_t rank, uint64_t key, const void *data, size_t len,
                 const uint64_t *group_ck, int location) {
  return bsr_tier_put_at(c, 0, rank, key, data, len, group_ck, location);
}

int bsr_tier_put_at(bsr_ctx *c, uint32_t tier, uint32_t rank, uint64_t key, const void *data,
                    size_t len, const uint64_t *group_ck, int location) {
  if (!c || tier >= BSR_MAX_TIERS) return BSR_ERR_INVALID;
  if (rank >= c->cfg.n_ranks || (location != BSR_LOC_HOST && location != BSR_LOC_DEVICE))
    return fail(c, BSR_ERR_INVALID, "tier_put: bad rank or location");
  if (!data) {
    // an index entry without bytes: the tier's fetch adapter delivers them at restore time
    bool adapter;
    {
      std::lock_guard<std::mutex> lk(c->mu);
      adapter = c->fetch_fn[tier] != nullptr;
    }
    if (!adapter || !group_ck || location != BSR_LOC_HOST)
      return fail(c, BSR_ERR_INVALID,
                  "tier_put: an object without data needs a fetch adapter on its tier, its "
                  "checksums, and BSR_LOC_HOST");
  }
  if (c->L == 0) return fail(c, BSR_ERR_STATE, "tier_put before registration");
  if (len != c->chunk_bytes)
    return fail(c, BSR_ERR_INVALID, "tier_put: len %zu != chunk bytes %llu", len,
                (unsigned long long)c->chunk_bytes);
  if (location == BSR_LOC_DEVICE && (reinterpret_cast<uintptr_t>(data) & 15u))
    return fail(c, BSR_ERR_ALIGN, "tier_put: device object must be 16-byte aligned");
  TierObj o{};
  o.data = static_cast<const uint8_t *>(data);
  o.len = len;
  o.loc = location;
  if (group_ck) {
    for (uint32_t g = 0; g < c->G; ++g) o.ck[g] = group_ck[g];
  } else {
    // store path: compute the group checksums on the GPU with the install kernel's sum stage
    CU(c, cudaSetDevice(c->cfg.device));
    int rc = ensure_finalized(c);
    if (rc != BSR_OK) return rc;
    std::lock_guard<std::mutex> al(c->aux_mu);
    if (!c->h_put_ck) {
      CU(c, cudaHostAlloc((void **)&c->h_put_ck, BSR_MAX_GROUPS * 8, cudaHostAllocMapped));
      CU(c, cudaHostAlloc((void **)&c->h_put_verdict, BSR_MAX_GROUPS * 4, cudaHostAllocMapped));
      CU(c, cudaHostGetDevicePointer((void **)&c->d_put_ck, c->h_put_ck, 0));
      CU(c, cudaHostGetDevicePointer((void **)&c->d_put_verdict, c->h_put_verdict, 0));
    }
    const uint8_t *src = o.data;
    if (location == BSR_LOC_HOST) {
      if (!c->d_put_stage) CU(c, cudaMalloc((void **)&c->d_put_stage, c->chunk_bytes));
      CU(c, cudaMemcpyAsync(c->d_put_stage, data, len, cudaMemcpyHostToDevice, c->own_stream));
      src = c->d_put_stage;
    }
    BsrInstallParams p{};
    fill_params(c, p, &c->aux, (uint32_t)(c->aux.seq++ % kLaunchSlots));
    p.n_adv = 1;
    p.scatter = 0;
    p.ck_out = c->d_put_ck;
    p.verdict = c->d_put_verdict;
    p.n_chunks = 1;
    p.one.src = src;
    StatDelta sd;
    rc = launch_install(c, p, c->own_stream, sd);
    if (rc != BSR_OK) return rc;
    CU(c, cudaStreamSynchronize(c->own_stream));
    merge_stats(c, sd);
    for (uint32_t g = 0; g < c->G; ++g) o.ck[g] = c->h_put_ck[g];
  }
  std::lock_guard<std::mutex> lk(c->mu);
  c->tier[tier][rank][key] = o;
  return BSR_OK;
}

int bsr_tier_remove(bsr_ctx *c, uint32_t rank, uint64_t key) {
  return bsr_tier_remove_at(c, 0, rank, key);
}

int bsr_tier_remove_at(bsr_ctx *c, uint32_t tier, uint32_t rank, uint64_t key) {
  if (!c || rank >= c->cfg.n_ranks || tier >= BSR_MAX_TIERS) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  c->tier[tier][rank].erase(key);
  return BSR_OK;
}

int bsr_tier_set_fetch(bsr_ctx *c, uint32_t tier, bsr_fetch_fn fn, void *user) {
  if (!c || tier >= BSR_MAX_TIERS) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  c->fetch_fn[tier] = fn;
  c->fetch_user[tier] = user;
  return BSR_OK;
}

int bsr_tier_set_available(bsr_ctx *c, uint32_t tier, int available) {
  if (!c || tier >= BSR_MAX_TIERS) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  c->tier_available[tier] = available != 0;
  return BSR_OK;
}

int bsr_tier_checksums(bsr_ctx *c, uint32_t rank, uint64_t key, uint64_t *out) {
  if (!c || !out || rank >= c->cfg.n_ranks) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  auto it = c->tier[0][rank].find(key);
  if (it == c->tier[0][rank].end()) return BSR_ERR_MISSING;
  for (uint32_t g = 0; g < c->G; ++g) out[g] = it->second.ck[g];
  return BSR_OK;
}

int bsr_probe(bsr_ctx *c, const int32_t *tok, size_t n_tok, int tok_on_device, uint64_t salt,
              uint64_t *keys_out, uint64_t *hit_bitmap_out, uint32_t *n_hit_chunks) {
  return probe_impl(c, false, 0, tok, n_tok, tok_on_device, salt, keys_out, hit_bitmap_out,
                    n_hit_chunks, nullptr);
}

int bsr_probe_request(bsr_ctx *c, uint64_t request_id, const int32_t *tok, size_t n_tok,
                      int tok_on_device, uint64_t salt, uint64_t *keys_out, uint64_t *hit_bitmap_out,
                      uint32_t *n_hit_chunks, int *tier_out) {
  return probe_impl(c, true, request_id, tok, n_tok, tok_on_device, salt, keys_out, hit_bitmap_out,
                    n_hit_chunks, tier_out);
}

int bsr_req_bind(bsr_ctx *c, bsr_req *q, uint64_t request_id, uint32_t tier) {
  if (!c || !q || q->ctx != c || tier >= BSR_MAX_TIERS) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> ql(q->mu);
  q->request_id = request_id;
  q->tier = tier;
  q->bound = true;
  return BSR_OK;
}

int bsr_request_done(bsr_ctx *c, uint64_t request_id) {
  if (!c) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  c->force_local.erase(request_id);
  return BSR_OK;
}

int bsr_request_is_force_local(bsr_ctx *c, uint64_t request_id, int *out) {
  if (!c || !out) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  *out = c->force_local.count(request_id) ? 1 : 0;
  return BSR_OK;
}

int bsr_req_create(bsr_ctx *c, const uint64_t *keys, uint32_t n_adv, const int32_t *const *tables,
                   bsr_req **out) {
  if (!c || !out || (n_adv && (!keys || !tables))) return BSR_ERR_INVALID;
  CU(c, cudaSetDevice(c->cfg.device));
  {
    int rc = ensure_finalized(c);
    if (rc != BSR_OK) return rc;
  }
  const uint32_t R = c->cfg.n_ranks, G = c->G;
  bsr_req *q = new (std::nothrow) bsr_req();
  if (!q) return BSR_ERR_NOMEM;
  q->ctx = c;
  q->n_adv = n_adv;
  q->keys.assign(keys, keys + n_adv);
  q->words = (n_adv + 63) / 64;
  q->bitmap.assign((size_t)R * G * q->words, 0ull);
  q->tables.resize((size_t)R * G);
  size_t total_entries = 0;
  for (uint32_t r = 0; r < R; ++r)
    for (uint32_t g = 0; g < G; ++g) {
      const size_t n = (size_t)n_adv * (BSR_CHUNK_TOKENS / c->groups[g].block_tokens);
      const int32_t *t = tables[r * G + g];
      if (n && !t) {
        delete q;
        return fail(c, BSR_ERR_INVALID, "req_create: null block table");
      }
      std::vector<bool> seen(c->groups[g].num_phys_blocks, false);
      for (size_t j = 0; j < n; ++j) {
        if (t[j] < 0 || (uint32_t)t[j] >= c->groups[g].num_phys_blocks || seen[t[j]]) {
          delete q;
          return fail(c, BSR_ERR_INVALID,
                      "req_create: table (rank %u, group %u) entry %zu out of range or repeated", r,
                      g, j);
        }
        seen[t[j]] = true;
      }
      q->tables[r * G + g].assign(t, t + n);
      total_entries += n;
    }
  auto bail = [&](int code, const char *what) {
    bsr_req_release(c, q);
    return fail(c, code, "req_create: %s", what);
  };
  if (n_adv) {
    if (cudaMalloc((void **)&q->d_tables, total_entries * 4) != cudaSuccess ||
        cudaMalloc((void **)&q->d_table_ptrs, (size_t)R * G * sizeof(void *)) != cudaSuccess)
      return bail(BSR_ERR_NOMEM, "device block tables");
    std::vector<const int32_t *> ptrs((size_t)R * G);
    size_t off = 0;
    for (size_t k = 0; k < q->tables.size(); ++k) {
      ptrs[k] = q->d_tables + off;
      if (!q->tables[k].empty() &&
          cudaMemcpy(q->d_tables + off, q->tables[k].data(), q->tables[k].size() * 4,
                     cudaMemcpyHostToDevice) != cudaSuccess)
        return bail(BSR_ERR_CUDA, "table upload");
      off += q->tables[k].size();
    }
    if (cudaMemcpy(q->d_table_ptrs, ptrs.data(), ptrs.size() * sizeof(void *),
                   cudaMemcpyHostToDevice) != cudaSuccess)
      return bail(BSR_ERR_CUDA, "table pointer upload");
    const size_t cells = (size_t)R * G * n_adv;
    if (cudaHostAlloc((void **)&q->h_ck, cells * 8, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostAlloc((void **)&q->h_verdict, cells * 4, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer((void **)&q->d_ck, q->h_ck, 0) != cudaSuccess ||
        cudaHostGetDevicePointer((void **)&q->d_verdict, q->h_verdict, 0) != cudaSuccess)
      return bail(BSR_ERR_NOMEM, "status arrays");
    memset(q->h_ck, 0, cells * 8);
    memset(q->h_verdict, 0, cells * 4);
    const size_t n_desc = (size_t)R * n_adv;
    if (cudaHostAlloc((void **)&q->h_desc, n_desc * sizeof(BsrChunkDesc), cudaHostAllocDefault) !=
            cudaSuccess ||
        cudaMalloc((void **)&q->d_desc, n_desc * sizeof(BsrChunkDesc)) != cudaSuccess)
      return bail(BSR_ERR_NOMEM, "descriptor arrays");
  }
  *out = q;
  return BSR_OK;
}

int bsr_req_release(bsr_ctx *c, bsr_req *q) {
  if (!c || !q || q->ctx != c) return BSR_ERR_INVALID;
  join_async(q);  // an asynchronous restore still running
  { std::lock_guard<std::mutex> ql(q->mu); }  // wait for a call in flight on this request
  cudaSetDevice(c->cfg.device);
  cudaFree(q->d_tables);
  cudaFree(q->d_table_ptrs);
  if (q->h_ck) cudaFreeHost(q->h_ck);
  if (q->h_verdict) cudaFreeHost(q->h_verdict);
  if (q->h_desc) cudaFreeHost(q->h_desc);
  cudaFree(q->d_desc);
  cudaGetLastError();
  delete q;
  return BSR_OK;
}

int bsr_restore(bsr_ctx *c, bsr_req *q, void *cuda_stream) {
  if (!c || !q || q->ctx != c) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> ql(q->mu);
  // the bounded-retrieve lock; with an admission budget restores share the slot pool instead
  std::unique_lock<std::mutex> serial(c->restore_mu, std::defer_lock);
  if (c->cfg.budget_slots == 0) serial.lock();
  const auto t0 = Clock::now();
  const auto deadline = t0 + std::chrono::milliseconds(c->cfg.timeout_ms);
  CU(c, cudaSetDevice(c->cfg.device));
  std::fill(q->bitmap.begin(), q->bitmap.end(), 0ull);
  q->restored = false;
  q->failed = false;
  const uint32_t R = c->cfg.n_ranks, N = q->n_adv;
  if (N) {
    const size_t cells = (size_t)R * c->G * N;
    memset(q->h_ck, 0, cells * 8);
    memset(q->h_verdict, 0, cells * 4);
  }
  StatDelta sd;
  int rc = BSR_OK;
  bool tier_up;
  {
    std::lock_guard<std::mutex> lk(c->mu);
    tier_up = c->tier_available[q->tier];
  }
  if (!tier_up) {
    rc = fail(c, BSR_ERR_TRANSFER, "tier %u is unavailable", q->tier);
  } else if (N) {
    JobRes *res = nullptr;
    rc = acquire_res(c, &res);
    if (rc == BSR_OK) {
      cudaStream_t stream = cuda_stream ? static_cast<cudaStream_t>(cuda_stream) : res->stream;
      // are all advertised chunks already in device memory?  (then no staging is needed at all)
      std::vector<TierObj> objs((size_t)N * R);
      bool all_device = true;
      {
        std::lock_guard<std::mutex> lk(c->mu);
        for (uint32_t i = 0; i < N && all_device; ++i)
          for (uint32_t r = 0; r < R; ++r) {
            auto it = c->tier[q->tier][r].find(q->keys[i]);
            if (it == c->tier[q->tier][r].end() || it->second.loc != BSR_LOC_DEVICE) {
              all_device = false;
              break;
            }
            objs[(size_t)i * R + r] = it->second;
          }
      }
      rc = all_device ? restore_resident(c, q, res, stream, deadline, objs, sd)
                      : restore_ring(c, q, res, stream, deadline, sd);
      // a bounded wait inside the bulk kernel that gave up raised the error word (host-mapped; both
      // restore paths return only after every kernel they launched has been observed complete)
      if (*reinterpret_cast<volatile unsigned int *>(res->h_err)) {
        *res->h_err = 0;
        if (rc == BSR_OK || rc == BSR_ERR_CHECKSUM)
          rc = fail(c, BSR_ERR_TIMEOUT, "a bounded wait inside the install kernel gave up");
      }
      release_res(c, res);
    } else if (res) {
      release_res(c, res);  // partly built: kept in the pool's list for destruction only
    }
  }
  if (rc == BSR_OK)
    q->restored = true;
  else
    invalidate_host(q);
  merge_stats(c, sd);
  {
    std::lock_guard<std::mutex> lk(c->mu);
    if (rc != BSR_OK && q->bound)  // the next admission pass must not re-enter the same fault
      c->force_local.insert(q->request_id);
    for (uint32_t r = 0; r < R; ++r) c->st.bytes_restored_by_tier[q->tier] += sd.bytes_installed[r];
    c->inject.kind = BSR_INJECT_NONE;  // one shot
    c->st.last_restore_ms = std::chrono::duration<double, std::milli>(Clock::now() - t0).count();
  }
  return rc;
}

int bsr_restore_calibrate(bsr_ctx *c, bsr_req *q, int stages, double *seconds) {
  if (!c || !q || q->ctx != c || !seconds || (stages != BSR_CAL_FILL && stages != BSR_CAL_FILL_H2D))
    return BSR_ERR_INVALID;
  join_async(q);
  std::lock_guard<std::mutex> ql(q->mu);
  std::unique_lock<std::mutex> serial(c->restore_mu, std::defer_lock);
  if (c->cfg.budget_slots == 0) serial.lock();
  *seconds = 0.0;
  if (q->n_adv == 0) return BSR_OK;
  if (stages == BSR_CAL_FILL_H2D && c->cfg.direct_install)
    return fail(c, BSR_ERR_STATE, "calibrate: a direct_install context has no device staging to copy into");
  CU(c, cudaSetDevice(c->cfg.device));
  JobRes *res = nullptr;
  int rc = acquire_res(c, &res);
  if (rc != BSR_OK) {
    if (res) release_res(c, res);
    return rc;
  }
  StatDelta sd;  // discarded: a calibration pass is not a restore
  const auto t0 = Clock::now();
  rc = restore_ring(c, q, res, res->stream, t0 + std::chrono::milliseconds(c->cfg.timeout_ms), sd,
                    stages);
  cudaStreamSynchronize(c->copy_stream);
  *seconds = std::chrono::duration<double>(Clock::now() - t0).count();
  release_res(c, res);
  return rc;
}

int bsr_plan_spans(const bsr_group_desc *groups, uint32_t n_groups, const bsr_tensor_desc *tensors,
                   uint32_t n_tensors, bsr_span_info *out, size_t capacity, size_t *count) {
  if (!groups || !tensors || !count || (!out && capacity) || n_groups == 0 || n_groups > BSR_MAX_GROUPS ||
      n_tensors == 0 || n_tensors > 65535)
    return BSR_ERR_INVALID;
  std::vector<uint32_t> bt(n_groups), tg(n_tensors), te(n_tensors);
  for (uint32_t g = 0; g < n_groups; ++g) {
    bt[g] = groups[g].block_tokens;
    if (bt[g] == 0 || BSR_CHUNK_TOKENS % bt[g] || BSR_CHUNK_TOKENS / bt[g] > 255) return BSR_ERR_INVALID;
  }
  uint64_t per_token = 0;
  for (uint32_t l = 0; l < n_tensors; ++l) {
    tg[l] = tensors[l].group;
    te[l] = tensors[l].bytes_per_token;
    if (tg[l] >= n_groups || (l && tg[l] < tg[l - 1])) return BSR_ERR_INVALID;
    if (te[l] == 0 || te[l] % 16) return BSR_ERR_ALIGN;
    per_token += te[l];
  }
  if (per_token * BSR_CHUNK_TOKENS >= (1ull << 32)) return BSR_ERR_INVALID;
  std::vector<BsrTile> tiles;
  plan_spans(bt, tg, te, tiles);
  *count = tiles.size();
  for (size_t k = 0; k < tiles.size() && k < capacity; ++k) {
    out[k].src_off = tiles[k].src_off;
    out[k].bytes = tiles[k].bytes;
    out[k].dst_off = tiles[k].dst_off;
    out[k].run_bytes = tiles[k].run_bytes;
    out[k].tensor = tiles[k].tensor;
    out[k].group = tiles[k].group;
    out[k].block = tiles[k].blk;
    out[k].n_runs = tiles[k].n_runs;
  }
  return BSR_OK;
}

int bsr_plan_pieces(uint64_t chunk_bytes, uint32_t n_chunks, uint32_t n_ranks, uint32_t fill_threads,
                    bsr_piece_info *out, size_t capacity, size_t *count) {
  if (!count || (!out && capacity) || chunk_bytes == 0 || chunk_bytes >= (1ull << 32) || n_ranks == 0 ||
      n_ranks > BSR_MAX_RANKS || fill_threads == 0 || (uint64_t)n_chunks * n_ranks > (1u << 24))
    return BSR_ERR_INVALID;
  std::vector<FillTask> tasks;
  std::vector<uint32_t> begin;
  plan_pieces(chunk_bytes, n_chunks * n_ranks, n_ranks, fill_threads, tasks, begin);
  *count = tasks.size();
  for (size_t k = 0; k < tasks.size() && k < capacity; ++k) {
    out[k].chunk = tasks[k].item / n_ranks;
    out[k].rank = tasks[k].item % n_ranks;
    out[k].offset = tasks[k].off;
    out[k].bytes = tasks[k].len;
  }
  return BSR_OK;
}

int bsr_numa_of_pci(const char *sysfs_root, const char *pci_bus_id, int *node, char *cpulist,
                    size_t cpulist_cap, int *n_nodes) {
  if (!sysfs_root || !pci_bus_id || !node) return BSR_ERR_INVALID;
  std::string id(pci_bus_id);
  for (char &ch : id)
    if (ch >= 'A' && ch <= 'F') ch = (char)(ch - 'A' + 'a');  // sysfs spells bus ids in lower case
  const std::string root(sysfs_root);
  std::string line;
  if (!read_line(root + "/bus/pci/devices/" + id + "/numa_node", &line)) return BSR_ERR_MISSING;
  char *end = nullptr;
  const long v = strtol(line.c_str(), &end, 10);
  if (end == line.c_str()) return BSR_ERR_INVALID;
  *node = (int)v;
  int count = 0;
  for (int k = 0; k < 1024; ++k) {
    std::string dummy;
    if (!read_line(root + "/devices/system/node/node" + std::to_string(k) + "/cpulist", &dummy)) break;
    ++count;
  }
  if (n_nodes) *n_nodes = count;
  if (cpulist && cpulist_cap) {
    cpulist[0] = 0;
    if (v >= 0) {
      if (!read_line(root + "/devices/system/node/node" + std::to_string(v) + "/cpulist", &line))
        return BSR_ERR_MISSING;
      cpu_set_t tmp;
      if (parse_cpulist(line.c_str(), &tmp) < 0) return BSR_ERR_INVALID;
      if (line.size() + 1 > cpulist_cap) return BSR_ERR_INVALID;
      memcpy(cpulist, line.c_str(), line.size() + 1);
    }
  }
  return BSR_OK;
}

int bsr_restore_async(bsr_ctx *c, bsr_req *q, void *cuda_stream) {
  if (!c || !q || q->ctx != c) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> al(q->async_mu);
  if (q->async_pending) return fail(c, BSR_ERR_STATE, "restore_async: a restore of this request is pending");
  if (q->async_thread.joinable()) q->async_thread.join();
  q->async_pending = true;
  q->async_thread = std::thread([c, q, cuda_stream] { q->async_rc = bsr_restore(c, q, cuda_stream); });
  return BSR_OK;
}

int bsr_restore_wait(bsr_ctx *c, bsr_req *q, int *restore_status) {
  if (!c || !q || q->ctx != c) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> al(q->async_mu);
  if (!q->async_pending) return fail(c, BSR_ERR_STATE, "restore_wait: no restore of this request is pending");
  if (q->async_thread.joinable()) q->async_thread.join();
  q->async_pending = false;
  if (restore_status) *restore_status = q->async_rc;
  return BSR_OK;
}

int bsr_commit(bsr_ctx *c, bsr_req *q, uint32_t *exposed) {
  if (!c || !q || q->ctx != c || !exposed) return BSR_ERR_INVALID;
  join_async(q);  // a restore started asynchronously
  std::lock_guard<std::mutex> ql(q->mu);
  bool all = q->restored && !q->failed;
  const uint32_t R = c->cfg.n_ranks;
  for (uint32_t rg = 0; all && rg < R * c->G; ++rg)
    for (uint32_t w = 0; all && w < q->words; ++w) {
      const uint32_t bits = (w + 1 < q->words || q->n_adv % 64 == 0) ? 64 : q->n_adv % 64;
      const uint64_t want = bits == 64 ? ~0ull : ((1ull << bits) - 1);
      all = q->bitmap[(size_t)rg * q->words + w] == want;
    }
  if (all) {
    *exposed = q->n_adv;
  } else {
    invalidate_host(q);
    *exposed = 0;
  }
  return BSR_OK;
}

int bsr_invalidate(bsr_ctx *c, bsr_req *q, unsigned flags) {
  if (!c || !q || q->ctx != c) return BSR_ERR_INVALID;
  join_async(q);  // a restore started asynchronously
  std::lock_guard<std::mutex> ql(q->mu);
  invalidate_host(q);
  if ((flags & BSR_SCRUB) && q->n_adv) {
    std::lock_guard<std::mutex> al(c->aux_mu);
    CU(c, cudaSetDevice(c->cfg.device));
    BsrScrubParams p{};
    p.tensor_base = c->d_tensor_base;
    p.tables = q->d_table_ptrs;
    p.tensor_group = c->d_tensor_group;
    p.tensor_run = c->d_tensor_run;
    p.n_tensors = c->L;
    p.n_groups = c->G;
    p.n_adv = q->n_adv;
    uint32_t max_logical = 0;
    for (uint32_t g = 0; g < c->G; ++g) {
      p.blocks_per_chunk[g] = BSR_CHUNK_TOKENS / c->groups[g].block_tokens;
      const uint32_t n = q->n_adv * p.blocks_per_chunk[g];
      if (n > max_logical) max_logical = n;
    }
    dim3 grid(max_logical < 1024 ? max_logical : 1024, c->cfg.n_ranks * c->L);
    bsr_scrub_kernel<<<grid, 256, 0, c->own_stream>>>(p);
    CU(c, cudaGetLastError());
    CU(c, cudaStreamSynchronize(c->own_stream));
    std::lock_guard<std::mutex> lk(c->mu);
    c->st.kernel_launches++;
  }
  return BSR_OK;
}

int bsr_req_invalid_blocks(bsr_ctx *c, bsr_req *q, uint32_t rank, uint32_t group, int32_t *out,
                           size_t capacity, size_t *count) {
  if (!c || !q || q->ctx != c || !count || (!out && capacity)) return BSR_ERR_INVALID;
  if (rank >= c->cfg.n_ranks || group >= c->G) return fail(c, BSR_ERR_INVALID, "invalid_blocks: rank/group");
  join_async(q);  // a restore started asynchronously
  std::lock_guard<std::mutex> ql(q->mu);
  // a failed retrieve may already have copied a subset of its blocks: all of them are erroneous
  const std::vector<int32_t> &t = q->tables[(size_t)rank * c->G + group];
  *count = q->failed ? t.size() : 0;
  const size_t n = *count < capacity ? *count : capacity;
  if (n) memcpy(out, t.data(), n * sizeof(int32_t));
  return BSR_OK;
}

int bsr_req_bitmap(bsr_ctx *c, bsr_req *q, uint64_t *out, size_t words) {
  if (!c || !q || q->ctx != c || (!out && words)) return BSR_ERR_INVALID;
  join_async(q);  // a restore started asynchronously
  std::lock_guard<std::mutex> ql(q->mu);
  if (words < q->bitmap.size()) return fail(c, BSR_ERR_INVALID, "bitmap buffer too small");
  if (!q->bitmap.empty()) memcpy(out, q->bitmap.data(), q->bitmap.size() * 8);
  return BSR_OK;
}

int bsr_req_checksums(bsr_ctx *c, bsr_req *q, uint64_t *out, size_t count) {
  if (!c || !q || q->ctx != c || (!out && count)) return BSR_ERR_INVALID;
  join_async(q);  // a restore started asynchronously
  std::lock_guard<std::mutex> ql(q->mu);
  const size_t cells = (size_t)c->cfg.n_ranks * c->G * q->n_adv;
  if (count < cells) return fail(c, BSR_ERR_INVALID, "checksum buffer too small");
  if (cells) memcpy(out, q->h_ck, cells * 8);
  return BSR_OK;
}

int bsr_get_stats(bsr_ctx *c, bsr_stats *out) {
  if (!c || !out) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> pl(c->pool_mu);  // peak_staging_bytes is written under pool_mu
  std::lock_guard<std::mutex> lk(c->mu);
  *out = c->st;
  return BSR_OK;
}

int bsr_get_trace(bsr_ctx *c, bsr_trace_rec *out, size_t capacity, size_t *count) {
  if (!c || !count || (!out && capacity)) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  *count = c->last_trace.size();
  const size_t n = *count < capacity ? *count : capacity;
  if (n) memcpy(out, c->last_trace.data(), n * sizeof(bsr_trace_rec));
  return BSR_OK;
}

int bsr_reset_stats(bsr_ctx *c) {
  if (!c) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> pl(c->pool_mu);
  std::lock_guard<std::mutex> lk(c->mu);
  bsr_stats keep = c->st;
  c->st = bsr_stats{};
  c->st.slot_bytes = keep.slot_bytes;
  c->st.dev_aux_bytes = keep.dev_aux_bytes;
  c->st.fill_numa_node = keep.fill_numa_node;
  for (uint32_t r = 0; r < BSR_MAX_RANKS; ++r)
    c->st.ring_bytes_allocated[r] = keep.ring_bytes_allocated[r];
  return BSR_OK;
}

int bsr_test_inject(bsr_ctx *c, int kind, uint32_t rank, uint32_t group, uint32_t chunk,
                    uint64_t seed) {
  if (!c || kind < BSR_INJECT_NONE || kind > BSR_INJECT_KERNEL_WAIT) return BSR_ERR_INVALID;
  std::lock_guard<std::mutex> lk(c->mu);
  c->inject.kind = kind;
  c->inject.rank = rank;
  c->inject.group = group;
  c->inject.chunk = chunk;
  c->inject.seed = seed;
  return BSR_OK;
}

}  // extern "C"

// =================================================================================================
// Allocation-free prefix-key entry point
// =================================================================================================
// Some callers must not allocate.  A serving engine typically hands almost all of HBM to its KV
// block pool at start-up, so a later cudaMalloc can fail outright; and cudaMalloc/cudaFree
// synchronise the whole device, which a scheduler thread sitting between two model steps cannot
// afford.  For them the probe kernel's scratch (the per-chunk digests and the block counter) lives
// in a fixed array inside the library image instead of in memory obtained at run time.
//
// The array is part of the loaded module: every GPU that loads this library carries it
// (BSR_NOALLOC_MAX_CHUNKS * 8 + 256 bytes) until the process exits.
namespace {

constexpr size_t kNoallocCounterWords = 32;  // 256 bytes reserved in front for the block counter
static __device__ __align__(256) unsigned long long
    bsr_noalloc_scratch[kNoallocCounterWords + BSR_NOALLOC_MAX_CHUNKS];

constexpr int kNoallocMaxDevices = 64;
std::mutex g_noalloc_mu;
unsigned long long *g_noalloc_ptr[kNoallocMaxDevices] = {};  // device address of the array, per GPU

}  // namespace

extern "C" int bsr_probe_keys_noalloc(int device, const int32_t *d_tok, size_t n_tok, uint64_t salt,
                                      uint64_t reg_id, uint64_t *d_keys_out, void *cuda_stream) {
  const size_t N = n_tok / BSR_CHUNK_TOKENS;
  if (device < 0 || device >= kNoallocMaxDevices) return BSR_ERR_INVALID;
  if (N > BSR_NOALLOC_MAX_CHUNKS) {
    fprintf(stderr,
            "bsr_probe_keys_noalloc: %zu chunks exceed the fixed scratch of %u chunks "
            "(BSR_NOALLOC_MAX_CHUNKS); use bsr_probe for longer prefixes\n",
            N, (unsigned)BSR_NOALLOC_MAX_CHUNKS);
    return BSR_ERR_INVALID;
  }
  if (N == 0) return BSR_OK;
  if (!d_tok || !d_keys_out) return BSR_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(d_tok) & 15u) || (reinterpret_cast<uintptr_t>(d_keys_out) & 7u))
    return BSR_ERR_ALIGN;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return BSR_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return BSR_ERR_CUDA;
  int rc = BSR_OK;
  unsigned long long *scratch = nullptr;
  {
    // Set-up, once per device, with that device current.  In host code the array's name is only a
    // handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress.
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[device]) {
      void *p = nullptr;
      if (cudaGetSymbolAddress(&p, bsr_noalloc_scratch) != cudaSuccess || !p) {
        cudaGetLastError();
        rc = BSR_ERR_CUDA;
      } else {
        g_noalloc_ptr[device] = static_cast<unsigned long long *>(p);
      }
    }
    scratch = g_noalloc_ptr[device];
  }
  if (rc == BSR_OK) {
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    unsigned int *counter = reinterpret_cast<unsigned int *>(scratch);
    uint64_t *digests = reinterpret_cast<uint64_t *>(scratch + kNoallocCounterWords);
    auto mix = [](uint64_t x) {
      x += BSR_K_PHI;
      x = (x ^ (x >> 32)) * BSR_K_PHI;
      x = (x ^ (x >> 29)) * BSR_K_PHI;
      return x ^ (x >> 32);
    };
    const uint64_t k_init = mix(salt ^ mix(reg_id));
    const uint32_t per_block = BSR_K_PROBE_THREADS / 32;
    const uint32_t grid = (uint32_t)((N + per_block - 1) / per_block);
    // The array keeps whatever the previous call left.  Digests are fully rewritten for the N chunks
    // that are read; the block counter must start at zero, so it is cleared in stream order.
    if (cudaMemsetAsync(counter, 0, kNoallocCounterWords * 8, s) != cudaSuccess) {
      rc = BSR_ERR_CUDA;
    } else {
      bsr_probe_kernel<<<grid, BSR_K_PROBE_THREADS, 0, s>>>(d_tok, (uint32_t)N, salt, k_init, digests,
                                                            counter, d_keys_out);
      if (cudaGetLastError() != cudaSuccess) rc = BSR_ERR_CUDA;
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return rc;
}
