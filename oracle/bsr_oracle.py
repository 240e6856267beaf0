"""CPU oracle for the bounded-state restore path.  TEST INFRASTRUCTURE ONLY.

A plain, slow numpy restatement of what the path computes, written from the paper and used
only by the tests, the smoke check and the CPU-baseline leg of the benchmark.  It shares no
code with the CUDA library and the library never calls it.

What the paper fixes, and this file follows in the paper's order:
  * probe  -- Section 3 "Probe globally": complete candidate hit H(S) as knowledge, no residency;
  * install -- Section 2 "Bounded installation" and Section 3 "Install locally": ordered windows
    G_1..G_K of at most W chunks, K = ceil(N/W); each window is fetched, required complete,
    verified, mapped onto its destination block slice, installed, then released before the next
    one may reuse the staging (Eq. 3: |L(t)| <= W; Eq. 1: RWS = max_t sum of live c_i);
  * commit -- Section 3 "Commit at request semantics", Eq. 6: Q(S) = AND_r AND_g q_{r,g};
    Q = 0 or any window failure invalidates the whole advertised prefix (Proposition 2).

What the paper leaves open, and is therefore this build's definition: the 64-bit mixer, the chunk
digest, the prefix-key chain, the per-(rank, chunk, group) checksum, the byte layout of a chunk,
the paged layout and the bitmap layout.  Each is stated where it is implemented.  The paper prints
no value for them, so they are pinned by other means: vectors computed independently when the
functions were specified, an explicit inverse of the mixer, closed forms of the checksum,
byte-at-a-time brute force of digest and install, and order / prefix / salt properties.  Every
function in this file has at least one such pin in tests/test_oracle_pins.py or
tests/test_oracle_recovery.py; none is left unpinned.

All arithmetic is on unsigned 64-bit integers modulo 2**64.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

MASK64 = (1 << 64) - 1
PHI = 0x9E3779B97F4A7C15
CHUNK_TOKENS = 256

# status codes of the C interface (interface constants, not arithmetic)
OK, ERR_INVALID, ERR_MISSING, ERR_CHECKSUM, ERR_TIMEOUT, ERR_TRANSFER = 0, -1, -2, -3, -4, -5


# --------------------------------------------------------------------------------------
# build-defined scalar functions
# --------------------------------------------------------------------------------------
def mix64(x: int) -> int:
    """Bijective 64-bit mixer: add PHI, then two xor-shift-multiply rounds (shifts 32, 29),
    then a final xor-shift by 32."""
    x = (x + PHI) & MASK64
    x = ((x ^ (x >> 32)) * PHI) & MASK64
    x = ((x ^ (x >> 29)) * PHI) & MASK64
    return x ^ (x >> 32)


def _mix64_vec(x: np.ndarray) -> np.ndarray:
    """mix64 applied element-wise to a uint64 array (numpy wraps modulo 2**64)."""
    phi = np.uint64(PHI)
    with np.errstate(over="ignore"):
        x = x + phi
        x = (x ^ (x >> np.uint64(32))) * phi
        x = (x ^ (x >> np.uint64(29))) * phi
        return x ^ (x >> np.uint64(32))


def chunk_digests(tok: np.ndarray, salt: int) -> np.ndarray:
    """d_i = sum_{j<256} mix64( ((u32)tok[256 i + j] << 32 | j) XOR salt )  (mod 2**64),
    one digest per full 256-token chunk; a trailing partial chunk is ignored.  The position j
    inside the mixed word makes the digest order-sensitive although the outer sum commutes."""
    n = len(tok) // CHUNK_TOKENS
    t = np.asarray(tok[: n * CHUNK_TOKENS]).astype(np.int64).astype(np.uint64) & np.uint64(0xFFFFFFFF)
    t = t.reshape(n, CHUNK_TOKENS)
    j = np.arange(CHUNK_TOKENS, dtype=np.uint64)[None, :]
    words = ((t << np.uint64(32)) | j) ^ np.uint64(salt)
    return _mix64_vec(words).sum(axis=1, dtype=np.uint64)


def prefix_keys(digests: np.ndarray, salt: int, reg_id: int) -> np.ndarray:
    """k_{-1} = mix64(salt XOR mix64(reg_id));  k_i = mix64(k_{i-1} XOR d_i).
    Key i therefore names the whole token prefix up to and including chunk i under one
    registration and one salt."""
    k = mix64(salt ^ mix64(reg_id))
    out = np.empty(len(digests), dtype=np.uint64)
    for i, d in enumerate(digests):
        k = mix64(k ^ int(d))
        out[i] = k
    return out


def checksum(segment: np.ndarray) -> int:
    """CK = sum_k w_k * (2k + 1) (mod 2**64) over the little-endian u32 words w_k of the
    segment, k counted from the start of the segment.  The weights are odd, so any change to
    a single word changes CK."""
    w = np.ascontiguousarray(segment).view("<u4").astype(np.uint64)
    k = np.arange(w.size, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return int((w * (np.uint64(2) * k + np.uint64(1))).sum(dtype=np.uint64))


# --------------------------------------------------------------------------------------
# registration geometry (Section 4: registered tensors in allocator groups, per TP rank)
# --------------------------------------------------------------------------------------
@dataclass
class Registration:
    """block_tokens[g]: tokens per paged block of group g (divides 256).
    tensors: (group, bytes_per_token) in registration order, group-major.

    Chunk byte layout (build-defined): groups in order; inside a group its tensors in
    registration order; per tensor 256 tokens x bytes_per_token, token-major."""

    block_tokens: list[int]
    tensors: list[tuple[int, int]]
    slot_align: int = 4096

    def __post_init__(self):
        gs = [g for g, _ in self.tensors]
        if gs != sorted(gs):
            raise ValueError("tensors must be registered group-major")
        for b in self.block_tokens:
            if b <= 0 or CHUNK_TOKENS % b:
                raise ValueError("block size must divide the chunk")

    @property
    def n_groups(self) -> int:
        return len(self.block_tokens)

    @property
    def chunk_bytes(self) -> int:
        return CHUNK_TOKENS * sum(e for _, e in self.tensors)

    @property
    def slot_bytes(self) -> int:
        """Staging footprint of one chunk: the payload rounded up to the slot alignment
        (the paper's Eq. 5 coefficient is a multiple of 4 KiB)."""
        a = self.slot_align
        return -(-self.chunk_bytes // a) * a

    def tensor_offset(self, l: int) -> int:
        return CHUNK_TOKENS * sum(e for _, e in self.tensors[:l])

    def segment(self, g: int) -> tuple[int, int]:
        """Byte range [begin, end) of group g inside a chunk."""
        ls = [l for l, (gg, _) in enumerate(self.tensors) if gg == g]
        if not ls:
            return (0, 0)
        b = self.tensor_offset(ls[0])
        return (b, b + CHUNK_TOKENS * sum(self.tensors[l][1] for l in ls))

    def blocks_per_chunk(self, g: int) -> int:
        return CHUNK_TOKENS // self.block_tokens[g]


def group_checksums(reg: Registration, chunk: np.ndarray) -> list[int]:
    """The checksum of every group's segment of one chunk (stored with the chunk at put time)."""
    return [checksum(chunk[slice(*reg.segment(g))]) for g in range(reg.n_groups)]


def new_paged(reg: Registration, pool_blocks: list[int], fill: int) -> list[np.ndarray]:
    """One array [pool_blocks[g], block_tokens[g], bytes_per_token] per tensor, filled with a
    canary byte (paged layout is build-defined: a tensor's block b is one contiguous run)."""
    return [np.full((pool_blocks[g], reg.block_tokens[g], e), fill, dtype=np.uint8)
            for g, e in reg.tensors]


# --------------------------------------------------------------------------------------
# external tier: key -> (payload bytes, per-group checksums), one per rank slice
# --------------------------------------------------------------------------------------
class Tier:
    def __init__(self):
        self.objects: dict[int, tuple[np.ndarray, list[int]]] = {}
        self.bytes_read = 0  # payload bytes handed out; probe must leave this at 0

    def put(self, key: int, payload: np.ndarray, cks: list[int]):
        self.objects[int(key)] = (payload, list(cks))

    def remove(self, key: int):
        self.objects.pop(int(key), None)

    def contains(self, key: int) -> bool:
        return int(key) in self.objects

    def get(self, key: int):
        obj = self.objects.get(int(key))
        if obj is not None:
            self.bytes_read += obj[0].size
        return obj


# --------------------------------------------------------------------------------------
# probe  (Section 3 "Probe globally")
# --------------------------------------------------------------------------------------
def probe(tok: np.ndarray, salt: int, reg_id: int, tiers: list[Tier]):
    """Returns (keys[N], hit[N] bool, n_hit).  hit_i is true iff every rank's tier holds key
    i; n_hit is the length of the longest all-hit prefix.  Only the index is consulted: no
    payload byte is read and nothing stays resident or locked."""
    keys = prefix_keys(chunk_digests(tok, salt), salt, reg_id)
    hit = np.array([all(t.contains(k) for t in tiers) for k in keys], dtype=bool)
    n_hit = int(np.argmin(hit)) if not hit.all() else len(hit)
    return keys, hit, n_hit


def pack_bits(bits: np.ndarray) -> np.ndarray:
    """bool[n] -> uint64[ceil(n/64)], bit i of the array at word i//64, position i%64."""
    words = np.zeros(-(-len(bits) // 64), dtype=np.uint64)
    for i, b in enumerate(bits):
        if b:
            words[i // 64] |= np.uint64(1) << np.uint64(i % 64)
    return words


# --------------------------------------------------------------------------------------
# request: advertised prefix + destination blocks  (Section 3, Fig. 2 second box)
# --------------------------------------------------------------------------------------
@dataclass
class Request:
    keys: np.ndarray                       # first n_adv prefix keys
    block_tables: list[list[np.ndarray]]   # [rank][group] -> int32[n_adv * blocks_per_chunk]
    n_ranks: int
    n_groups: int
    valid: np.ndarray = field(init=False)  # bool [R, G, n_adv]: q_{r,g} per chunk
    restored: bool = False
    failed: bool = False

    def __post_init__(self):
        self.valid = np.zeros((self.n_ranks, self.n_groups, len(self.keys)), dtype=bool)

    @property
    def n_adv(self) -> int:
        return len(self.keys)

    def bitmap(self) -> np.ndarray:
        """uint64 words, bit (r, g, i) at word (r*G + g)*ceil(n_adv/64) + i//64, position i%64."""
        return np.concatenate([pack_bits(self.valid[r, g])
                               for r in range(self.n_ranks) for g in range(self.n_groups)])


@dataclass
class Stats:
    peak_staging_bytes: list[int]
    bytes_filled: list[int]
    bytes_installed: list[int]
    windows: int = 0


# --------------------------------------------------------------------------------------
# install  (Section 2 "Bounded installation", Section 3 "Install locally")
# --------------------------------------------------------------------------------------
def block_of_chunk(reg: Registration, chunk: np.ndarray, l: int, b: int) -> np.ndarray:
    """The rows [B_g, e_l] that a chunk carries for tensor l and the chunk's logical block b:
    tokens b*B_g .. (b+1)*B_g - 1 of the tensor's [256, e_l] slab at byte offset tensor_offset(l)."""
    g, e = reg.tensors[l]
    B = reg.block_tokens[g]
    off = reg.tensor_offset(l) + b * B * e
    return chunk[off: off + B * e].reshape(B, e)


def scatter_chunk_group(reg: Registration, g: int, chunk: np.ndarray, i: int,
                        table: np.ndarray, paged: list[np.ndarray]):
    """Install group g of chunk i: token t of the chunk (global token 256 i + t) of tensor l goes
    to paged[l][ table[(256 i + t) // B_g], (256 i + t) % B_g, : ]."""
    nb = reg.blocks_per_chunk(g)
    for l, (gg, _) in enumerate(reg.tensors):
        if gg != g:
            continue
        for b in range(nb):
            paged[l][table[i * nb + b]] = block_of_chunk(reg, chunk, l, b)


def _verify_and_install_chunk(reg: Registration, data: np.ndarray, cks: list[int], i: int,
                              tables_r: list[np.ndarray], paged_r: list[np.ndarray],
                              valid_r: np.ndarray) -> int:
    """One staged chunk of one rank: per group, verify the checksum of the staged bytes against the
    stored one (a mismatch fails the chunk at that group) and scatter the group."""
    for g in range(reg.n_groups):
        if checksum(data[slice(*reg.segment(g))]) != cks[g]:
            return ERR_CHECKSUM
        scatter_chunk_group(reg, g, data, i, tables_r[g], paged_r)
        valid_r[g, i] = True
    return OK


def restore(reg: Registration, tiers: list[Tier], req: Request, paged: list[list[np.ndarray]],
            W: int, fetch_fault=None, workers: int = 1) -> tuple[int, Stats]:
    """The strict window loop.  For window j (chunks jW .. min((j+1)W, N) - 1), per rank:
    acquire one staging buffer per chunk (live bytes += slot_bytes), fetch every chunk of the
    window (a missing key fails the retrieve), then per chunk and group verify the checksum of
    the staged bytes against the stored one (mismatch fails the retrieve) and scatter; finally
    release the window's buffers.  The first failure stops the retrieve and invalidates the whole
    request (all ranks, all groups).  Returns (status, stats).

    workers > 1 is the same loop with the chunks of a window verified and installed by a plain
    parallel-for (a thread pool; chunks write disjoint blocks), used only to time the oracle on all
    host cores.  The first failure in chunk order is the one reported."""
    if W < 1:
        return ERR_INVALID, Stats([0] * req.n_ranks, [0] * req.n_ranks, [0] * req.n_ranks)
    R, N = req.n_ranks, req.n_adv
    st = Stats([0] * R, [0] * R, [0] * R)
    live = [0] * R
    req.valid[:] = False
    req.restored, req.failed = False, False
    status = OK
    for j in range(-(-N // W)):
        window = range(j * W, min((j + 1) * W, N))
        st.windows += 1
        staged: list[dict[int, tuple[np.ndarray, list[int]]]] = [dict() for _ in range(R)]
        # fetch: L2 -> L1, the window must be completely present
        for r in range(R):
            for i in window:
                live[r] += reg.slot_bytes
                st.peak_staging_bytes[r] = max(st.peak_staging_bytes[r], live[r])
                code = fetch_fault(r, i) if fetch_fault else None
                if code:
                    status = code
                    break
                obj = tiers[r].get(req.keys[i])
                if obj is None:
                    status = ERR_MISSING
                    break
                staged[r][i] = (obj[0].copy(), obj[1])
                st.bytes_filled[r] += obj[0].size
            if status != OK:
                break
        # verify + install
        if status == OK:
            order = [(r, i) for r in range(R) for i in window]

            def one(ri):
                r, i = ri
                return _verify_and_install_chunk(reg, staged[r][i][0], staged[r][i][1], i,
                                                 req.block_tables[r], paged[r], req.valid[r])

            if workers > 1:
                with ThreadPoolExecutor(workers) as pool:
                    codes = list(pool.map(one, order))
            else:
                codes = []
                for ri in order:             # stop at the first failure, as the text says
                    codes.append(one(ri))
                    if codes[-1] != OK:
                        break
            for (r, i), code in zip(order, codes):
                if code != OK:
                    status = code
                    break
                st.bytes_installed[r] += staged[r][i][0].size
        # release before the next window may reuse the staging
        for r in range(R):
            live[r] = 0
        if status != OK:
            break
    if status != OK:
        invalidate(reg, req, paged, scrub=False)
    else:
        req.restored = True
    return status, st


# --------------------------------------------------------------------------------------
# commit / invalidate  (Section 3 "Commit at request semantics", Eq. 6, Proposition 2)
# --------------------------------------------------------------------------------------
def commit(reg: Registration, req: Request, paged) -> int:
    """Exposed chunks: n_adv iff a restore completed and every (rank, group, chunk) bit is set,
    else the request is invalidated and 0 is exposed."""
    if req.restored and not req.failed and bool(req.valid.all()):
        return req.n_adv
    invalidate(reg, req, paged, scrub=False)
    return 0


def invalid_blocks(req: Request, r: int, g: int) -> np.ndarray:
    """Destination blocks the engine must treat as erroneous (Section 4 "vLLM failure integration"):
    a failed retrieve may already have copied a subset of its blocks, so ALL block ids of the
    request's table are reported once it has failed; none while it is healthy."""
    return req.block_tables[r][g].copy() if req.failed else req.block_tables[r][g][:0].copy()


def invalidate(reg: Registration, req: Request, paged, scrub: bool):
    """Whole-prefix invalidation: every bit of every rank and group is cleared, whichever
    component failed.  With scrub, every destination block of the request is zero-filled."""
    req.valid[:] = False
    req.failed = True
    if scrub:
        for r in range(req.n_ranks):
            for l, (g, _) in enumerate(reg.tensors):
                for blk in req.block_tables[r][g]:
                    paged[r][l][blk] = 0


# --------------------------------------------------------------------------------------
# request-level recovery  (Section 3 "Recover without re-entering the same fault";
# Section 6.4 failure outcomes: lower valid tier when available, otherwise zero external reuse)
# --------------------------------------------------------------------------------------
@dataclass
class Engine:
    """The reusable tiers of one engine in priority order (tier 0 first, e.g. remote DRAM, then a
    lower tier such as local SSD), their availability, and the force-local markers."""

    tiers: list[list[Tier]]                 # [tier][rank]
    available: list[bool]
    force_local: set = field(default_factory=set)


def probe_request(eng: Engine, request_id: int, tok: np.ndarray, salt: int, reg_id: int):
    """Request-scoped probe.  Returns (keys, hit, n_hit, tier).
    A request carrying the force-local marker reports zero external tokens without consulting any
    tier (tier = -1).  Otherwise every available tier is probed as in `probe`; the request is
    served by ONE tier, the one with the longest complete prefix, the higher-priority tier on a
    tie.  With no available tier or no hit, n_hit = 0 and tier = -1."""
    keys = prefix_keys(chunk_digests(tok, salt), salt, reg_id)
    none = np.zeros(len(keys), dtype=bool)
    if request_id in eng.force_local:
        return keys, none, 0, -1
    best_tier, best_n, best_hit = -1, 0, none
    for t, ranks in enumerate(eng.tiers):
        if not eng.available[t]:
            continue
        hit = np.array([all(rk.contains(k) for rk in ranks) for k in keys], dtype=bool)
        n = int(np.argmin(hit)) if not hit.all() else len(hit)
        if n > best_n:
            best_tier, best_n, best_hit = t, n, hit
    return keys, best_hit, best_n, best_tier


def restore_request(eng: Engine, request_id: int, tier: int, reg: Registration, req: Request,
                    paged, W: int, fetch_fault=None):
    """Restore of a bound request from the tier the probe chose.  A tier that has become
    unavailable fails the retrieve as a transfer error.  Any failure installs the force-local
    marker for the request, so that its next probe reports zero external tokens."""
    if tier < 0 or tier >= len(eng.tiers):
        return ERR_INVALID, Stats([0] * req.n_ranks, [0] * req.n_ranks, [0] * req.n_ranks)
    if not eng.available[tier]:
        req.valid[:] = False
        req.restored, req.failed = False, True
        eng.force_local.add(request_id)
        return ERR_TRANSFER, Stats([0] * req.n_ranks, [0] * req.n_ranks, [0] * req.n_ranks)
    status, st = restore(reg, eng.tiers[tier], req, paged, W, fetch_fault=fetch_fault)
    if status != OK:
        eng.force_local.add(request_id)
    return status, st


def request_done(eng: Engine, request_id: int):
    """Successful RUNNING admission or request teardown removes the marker."""
    eng.force_local.discard(request_id)


# --------------------------------------------------------------------------------------
# several restores under one admission budget  (Section 7 "Current concurrency is
# conservative": allow several request windows whenever their aggregate RWS stays below B)
# --------------------------------------------------------------------------------------
def restore_concurrent(reg: Registration, tiers: list[Tier], reqs: list[Request],
                       paged: list[list[np.ndarray]], W: int, B: int):
    """Restores several requests into the same paged pools under a budget of B staging slots per
    rank.  The model is synchronous rounds: in every round each unfinished request, in order,
    admits its next window of min(W, chunks left, slots still free in the budget) chunks; all
    admitted windows are fetched, verified and installed as in `restore`; then all are released.
    Every request keeps Eq. 3 (at most W live), all together never exceed B.  A failing request is
    invalidated alone: the others' outcomes do not depend on it.
    Returns (status per request, peak aggregate staging bytes per rank, rounds)."""
    R = reqs[0].n_ranks
    Q = len(reqs)
    done = [0] * Q
    status = [OK] * Q
    for q in reqs:
        q.valid[:] = False
        q.restored, q.failed = False, False
    peak = [0] * R
    rounds = 0
    while any(status[k] == OK and done[k] < reqs[k].n_adv for k in range(Q)):
        rounds += 1
        free = B
        windows = []
        for k in range(Q):
            if status[k] != OK or done[k] >= reqs[k].n_adv:
                continue
            w = min(W, reqs[k].n_adv - done[k], free)
            if w <= 0:
                continue
            free -= w
            windows.append((k, range(done[k], done[k] + w)))
        live = sum(len(win) for _, win in windows) * reg.slot_bytes
        for r in range(R):
            peak[r] = max(peak[r], live)
        for k, win in windows:
            q = reqs[k]
            for r in range(R):
                for i in win:
                    obj = tiers[r].get(q.keys[i])
                    if obj is None:
                        status[k] = ERR_MISSING
                        break
                    data, cks = obj[0].copy(), obj[1]
                    for g in range(reg.n_groups):
                        if checksum(data[slice(*reg.segment(g))]) != cks[g]:
                            status[k] = ERR_CHECKSUM
                            break
                        scatter_chunk_group(reg, g, data, i, q.block_tables[r][g], paged[r])
                        q.valid[r, g, i] = True
                    if status[k] != OK:
                        break
                if status[k] != OK:
                    break
            if status[k] != OK:
                invalidate(reg, q, paged, scrub=False)
            else:
                done[k] += len(win)
    for k in range(Q):
        if status[k] == OK:
            reqs[k].restored = True
    return status, peak, rounds
