"""Test infrastructure (CPU oracle): mobile data chunks and the elastic policies that move them between tasks.

The paper keeps the training data in many small fixed-size chunks that carry the samples together with their
per-sample state (Sec. 3 core concepts; Sec. 4.4 in-memory chunk format: the number of samples in a chunk varies with
their size). Tasks never move; the scheduler moves chunks: when tasks are freed their chunks go to the remaining
tasks in round-robin fashion (Sec. 4.5 elastic scaling policy), when tasks are added each old task hands randomly
picked chunks to the new ones (Sec. 5.3: this is why scaling out reshuffles the samples), and the rebalancing policy
moves chunks from slower to faster tasks (Sec. 4.5). The paper fixes none of the integer rules; the ones below are
this project's reading and are written out in every docstring. Plain loops, no vectorisation: a reader can follow
each rule by eye. Only tests, the smoke check and the CPU baseline may import this module.
"""
import numpy as np

from . import mix64

STATE_BYTES = 8          # per-sample state that travels with a sample: its dual variable and its label, fp32 each
NNZ_BYTES = 8            # one stored entry of a sparse vector: int32 index + fp32 value
SCALE_OUT_STREAM = 0xA0761D6478BD642F


def cut(n_coord, chunk_bytes, indptr=None, dense_dim=0):
    """Chunk boundaries (Sec. 4.4). Coordinates are stored in id order. Coordinate i occupies
    NNZ_BYTES * nnz_i + STATE_BYTES bytes (sparse) or 4 * dense_dim + STATE_BYTES (dense). A chunk is closed in front of
    the coordinate that would take it above chunk_bytes; a chunk holds at least one coordinate. Returns off[C + 1]."""
    off = [0]
    used = 0
    for i in range(n_coord):
        b = (NNZ_BYTES * int(indptr[i + 1] - indptr[i]) if indptr is not None else 4 * dense_dim) + STATE_BYTES
        if i > off[-1] and used + b > chunk_bytes:
            off.append(i)
            used = 0
        used += b
    off.append(n_coord)
    return np.asarray(off, np.int64)


def assign(C, K, seed):
    """First placement (Appendix, baseline comparisons: data is assigned to tasks at random): the chunks, ordered by
    mix64(mix64(seed) ^ chunk), are dealt in consecutive runs, the first C mod K tasks getting one more."""
    if not 1 <= K <= C:
        raise ValueError("need 1 <= K <= number of chunks")
    s = mix64(seed)
    order = sorted(range(C), key=lambda c: (mix64(s ^ c), c))
    task = np.empty(C, np.int32)
    base, extra = divmod(C, K)
    pos = 0
    for k in range(K):
        m = base + (1 if k < extra else 0)
        for c in order[pos:pos + m]:
            task[c] = k
        pos += m
    return task


def scale_in(task, K_old, K_new):
    """Tasks K_new .. K_old - 1 are freed (Sec. 4.5): their chunks, taken in ascending chunk number, go to tasks
    0, 1, ..., K_new - 1, 0, 1, ... in turn. No other chunk moves."""
    if not 1 <= K_new <= K_old:
        raise ValueError("need 1 <= K_new <= K_old")
    out = np.array(task, np.int32, copy=True)
    nxt = 0
    for c in range(out.size):
        if out[c] >= K_new:
            out[c] = nxt
            nxt = (nxt + 1) % K_new
    return out


def scale_out(task, K_old, K_new, seed):
    """Tasks K_old .. K_new - 1 are added (Sec. 4.5, Sec. 5.3): old task j, holding m_j chunks, gives away
    floor(m_j * (K_new - K_old) / K_new) of them, picked at random: its chunks are ordered by
    mix64(mix64(seed ^ SCALE_OUT_STREAM) ^ chunk) and the first ones go. The chunks given away are dealt to the new
    tasks in turn, old tasks in ascending order, the turn carrying over from one old task to the next. No other chunk
    moves."""
    if not 1 <= K_old <= K_new:
        raise ValueError("need 1 <= K_old <= K_new")
    out = np.array(task, np.int32, copy=True)
    add = K_new - K_old
    if add == 0:
        return out
    s = mix64(seed ^ SCALE_OUT_STREAM)
    turn = 0
    for j in range(K_old):
        mine = [c for c in range(out.size) if task[c] == j]
        mine.sort(key=lambda c: (mix64(s ^ c), c))
        give = (len(mine) * add) // K_new
        for c in mine[:give]:
            out[c] = K_old + turn
            turn = (turn + 1) % add
    return out


def rebalance_step(task, chunk_len, K, per_sample_time):
    """One step of the rebalancing policy (Sec. 4.5): tasks are ranked by their time per sample (the caller passes the
    median over its window); the slowest task whose round takes longer than the fastest-finishing task's by more than
    one of its own chunks' processing time gives its highest-numbered chunk to the task that finishes first. Returns
    the new map and whether a chunk moved. Round time of a task = its samples * its time per sample."""
    out = np.array(task, np.int32, copy=True)
    samples = [0] * K
    for c in range(out.size):
        samples[out[c]] += int(chunk_len[c])
    t = [samples[k] * float(per_sample_time[k]) for k in range(K)]
    slow = max(range(K), key=lambda k: (t[k], -k))
    fast = min(range(K), key=lambda k: (t[k], k))
    mine = [c for c in range(out.size) if out[c] == slow]
    if slow == fast or len(mine) <= 1:
        return out, False
    c = mine[-1]
    if t[slow] - t[fast] <= int(chunk_len[c]) * float(per_sample_time[slow]):
        return out, False
    out[c] = fast
    return out, True


def partition_from_chunks(n_coord, K, off, task):
    """The partition a chunk placement induces: coordinate i belongs to the task of the chunk that holds it; inside a
    partition the members are in ascending id order. Returns (owner, part_off, members); every task must hold a chunk."""
    C = len(off) - 1
    if len(task) != C or off[0] != 0 or off[C] != n_coord:
        raise ValueError("chunk offsets must run from 0 to the number of coordinates")
    owner = np.empty(n_coord, np.int32)
    for c in range(C):
        if off[c + 1] <= off[c] or not 0 <= task[c] < K:
            raise ValueError("empty chunk or task out of range")
        owner[off[c]:off[c + 1]] = task[c]
    members = []
    part_off = [0]
    for k in range(K):
        mk = [i for i in range(n_coord) if owner[i] == k] if n_coord <= 4096 else np.nonzero(owner == k)[0].tolist()
        if not mk:
            raise ValueError("task %d holds no chunk" % k)
        members.extend(mk)
        part_off.append(len(members))
    return owner, np.asarray(part_off, np.int64), np.asarray(members, np.int32)
