/* A caller of the BSR library written in plain C: no Python, no torch, only include/bsr.h and the
 * CUDA runtime for device memory.  The GPU test writes a seeded case into a directory, runs this
 * program on it and compares what it leaves there with the oracle.
 *
 *   restore_prefix <dir>
 *
 * Reads   <dir>/case.txt          R N W G L salt reg_id, then G lines "block_tokens pool_blocks",
 *                                 then L lines "group bytes_per_token"
 *         <dir>/tokens.bin        int32[N * 256]
 *         <dir>/payload_r<r>.bin  N chunks of rank r, back to back
 *         <dir>/ck_r<r>.bin       uint64[N][G] stored group checksums
 *         <dir>/table_r<r>_g<g>.bin int32[N * 256 / block_tokens]
 * Writes  <dir>/result.txt        "n_hit exposed peak_staging_bytes_rank0"
 *         <dir>/keys.bin          uint64[N]
 *         <dir>/bitmap.bin        uint64[R * G * ceil(N / 64)]
 *         <dir>/paged_r<r>_l<l>.bin  the whole pool of tensor l of rank r after the restore
 */
#include <cuda_runtime_api.h>
#include <inttypes.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "bsr.h"

#define MAX_G 8
#define MAX_L 1024
#define MAX_R 8

static void die(const char *what, int code, bsr_ctx *ctx) {
  fprintf(stderr, "restore_prefix: %s failed with %d (%s)\n", what, code,
          ctx ? bsr_last_error(ctx) : "-");
  exit(1);
}

static void *read_file(const char *dir, const char *name, size_t want) {
  char path[4096];
  snprintf(path, sizeof path, "%s/%s", dir, name);
  FILE *f = fopen(path, "rb");
  if (!f) {
    perror(path);
    exit(1);
  }
  void *buf = malloc(want ? want : 1);
  if (!buf || fread(buf, 1, want, f) != want) {
    fprintf(stderr, "restore_prefix: short read of %s\n", path);
    exit(1);
  }
  fclose(f);
  return buf;
}

static void write_file(const char *dir, const char *name, const void *data, size_t n) {
  char path[4096];
  snprintf(path, sizeof path, "%s/%s", dir, name);
  FILE *f = fopen(path, "wb");
  if (!f || fwrite(data, 1, n, f) != n) {
    perror(path);
    exit(1);
  }
  fclose(f);
}

int main(int argc, char **argv) {
  if (argc != 2) {
    fprintf(stderr, "usage: restore_prefix <dir>\n");
    return 2;
  }
  const char *dir = argv[1];
  char path[4096], name[256];
  snprintf(path, sizeof path, "%s/case.txt", dir);
  FILE *cf = fopen(path, "r");
  if (!cf) {
    perror(path);
    return 1;
  }
  unsigned R, N, W, G, L;
  uint64_t salt, reg_id;
  if (fscanf(cf, "%u %u %u %u %u %" SCNu64 " %" SCNu64, &R, &N, &W, &G, &L, &salt, &reg_id) != 7 ||
      R > MAX_R || G > MAX_G || L > MAX_L)
    return 1;
  bsr_group_desc groups[MAX_G];
  static bsr_tensor_desc tensors[MAX_R][MAX_L];
  static size_t pool_bytes[MAX_L];
  uint64_t bytes_per_token = 0;
  for (unsigned g = 0; g < G; ++g)
    if (fscanf(cf, "%u %u", &groups[g].block_tokens, &groups[g].num_phys_blocks) != 2) return 1;
  for (unsigned l = 0; l < L; ++l) {
    unsigned g, e;
    if (fscanf(cf, "%u %u", &g, &e) != 2 || g >= G) return 1;
    for (unsigned r = 0; r < R; ++r) {
      tensors[r][l].group = g;
      tensors[r][l].bytes_per_token = e;
    }
    pool_bytes[l] = (size_t)groups[g].num_phys_blocks * groups[g].block_tokens * e;
    bytes_per_token += e;
  }
  fclose(cf);
  const size_t chunk_bytes = (size_t)BSR_CHUNK_TOKENS * bytes_per_token;

  /* the engine's paged pools: device memory owned by this program, pre-filled with a canary */
  for (unsigned r = 0; r < R; ++r)
    for (unsigned l = 0; l < L; ++l) {
      void *p = NULL;
      if (cudaMalloc(&p, pool_bytes[l]) != cudaSuccess || cudaMemset(p, 0xA5, pool_bytes[l]) != cudaSuccess)
        die("cudaMalloc/cudaMemset", -1, NULL);
      tensors[r][l].dev_base = p;
    }

  bsr_config cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.window_chunks = W;
  cfg.n_ranks = R;
  cfg.chunk_tokens = BSR_CHUNK_TOKENS;
  cfg.reg_id = reg_id;
  bsr_ctx *ctx = NULL;
  int rc = bsr_ctx_create(&cfg, &ctx);
  if (rc != BSR_OK) die("bsr_ctx_create", rc, NULL);
  for (unsigned r = 0; r < R; ++r)
    if ((rc = bsr_register(ctx, r, groups, G, tensors[r], L)) != BSR_OK) die("bsr_register", rc, ctx);
  uint64_t cb = 0, sb = 0;
  if ((rc = bsr_chunk_bytes(ctx, &cb, &sb)) != BSR_OK || cb != chunk_bytes) die("bsr_chunk_bytes", rc, ctx);

  /* probe first: the keys under which the external tier holds this prefix */
  int32_t *tok = read_file(dir, "tokens.bin", (size_t)N * BSR_CHUNK_TOKENS * 4);
  uint64_t *keys = calloc(N ? N : 1, 8);
  const size_t words = (N + 63) / 64;
  uint64_t *hits = calloc(words ? words : 1, 8);
  uint32_t n_hit = 0;
  rc = bsr_probe(ctx, tok, (size_t)N * BSR_CHUNK_TOKENS, 0, salt, keys, hits, &n_hit);
  if (rc != BSR_OK || n_hit != 0) die("bsr_probe on an empty tier", rc, ctx);

  /* the external tier: host memory owned by this program, borrowed by the library */
  uint8_t *payload[MAX_R];
  for (unsigned r = 0; r < R; ++r) {
    snprintf(name, sizeof name, "payload_r%u.bin", r);
    payload[r] = read_file(dir, name, (size_t)N * chunk_bytes);
    snprintf(name, sizeof name, "ck_r%u.bin", r);
    uint64_t *ck = read_file(dir, name, (size_t)N * G * 8);
    for (unsigned i = 0; i < N; ++i) {
      rc = bsr_tier_put(ctx, r, keys[i], payload[r] + (size_t)i * chunk_bytes, chunk_bytes,
                        ck + (size_t)i * G, BSR_LOC_HOST);
      if (rc != BSR_OK) die("bsr_tier_put", rc, ctx);
    }
    free(ck);
  }
  rc = bsr_probe(ctx, tok, (size_t)N * BSR_CHUNK_TOKENS, 0, salt, keys, hits, &n_hit);
  if (rc != BSR_OK) die("bsr_probe", rc, ctx);

  /* the scheduler allocated the destination blocks: one table per (rank, group) */
  const int32_t *tables[MAX_R * MAX_G];
  for (unsigned r = 0; r < R; ++r)
    for (unsigned g = 0; g < G; ++g) {
      snprintf(name, sizeof name, "table_r%u_g%u.bin", r, g);
      tables[r * G + g] =
          read_file(dir, name, (size_t)N * (BSR_CHUNK_TOKENS / groups[g].block_tokens) * 4);
    }
  bsr_req *req = NULL;
  if ((rc = bsr_req_create(ctx, keys, n_hit, tables, &req)) != BSR_OK) die("bsr_req_create", rc, ctx);
  if ((rc = bsr_restore(ctx, req, NULL)) != BSR_OK) die("bsr_restore", rc, ctx);
  uint32_t exposed = 0;
  if ((rc = bsr_commit(ctx, req, &exposed)) != BSR_OK) die("bsr_commit", rc, ctx);

  bsr_stats st;
  if ((rc = bsr_get_stats(ctx, &st)) != BSR_OK) die("bsr_get_stats", rc, ctx);
  uint64_t *bitmap = calloc((size_t)R * G * words + 1, 8);
  if ((rc = bsr_req_bitmap(ctx, req, bitmap, (size_t)R * G * words)) != BSR_OK)
    die("bsr_req_bitmap", rc, ctx);

  char line[256];
  snprintf(line, sizeof line, "%u %u %" PRIu64 "\n", n_hit, exposed, (uint64_t)st.peak_staging_bytes[0]);
  write_file(dir, "result.txt", line, strlen(line));
  write_file(dir, "keys.bin", keys, (size_t)N * 8);
  write_file(dir, "bitmap.bin", bitmap, (size_t)R * G * words * 8);
  for (unsigned r = 0; r < R; ++r)
    for (unsigned l = 0; l < L; ++l) {
      void *host = malloc(pool_bytes[l]);
      if (!host || cudaMemcpy(host, tensors[r][l].dev_base, pool_bytes[l], cudaMemcpyDeviceToHost) != cudaSuccess)
        die("cudaMemcpy", -1, NULL);
      snprintf(name, sizeof name, "paged_r%u_l%u.bin", r, l);
      write_file(dir, name, host, pool_bytes[l]);
      free(host);
    }
  bsr_req_release(ctx, req);
  bsr_ctx_destroy(ctx);
  printf("restored %u of %u chunks\n", exposed, N);
  return 0;
}
