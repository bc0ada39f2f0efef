"""Eager block rotation, as a plain model.  TEST INFRASTRUCTURE, not product code.

Follows the paper's section 4.3.2 ("Eager block rotation for data race free overlapping"):

* KV generation is incremental.  A block that is completely filled is never written again until
  its request finishes; the last, partly filled block is *dirty*.
* Full blocks are copied to host memory in the background, before any preemption; a full block
  with a valid host copy is *synced*.
* When a request is preempted only the blocks without a valid host copy have to be sent (normally
  the one dirty block); the device blocks of synced blocks are discarded without a transfer, since
  valid copies already exist in host memory.  The host copies are kept while a request runs on the
  GPU (host-side duplication).
* Because discarded device blocks are free at once, requests resuming in the same rotation may take
  them: a resume needs device blocks <= free blocks + blocks discarded in that rotation.

The model works on logical blocks only (no block ids, no bytes).  Every logical block carries a
*version* that goes up whenever tokens are written into it, and each host copy remembers the version
it was taken at; a host copy is valid when the two agree.  That is enough to say, after any sequence
of operations, how many blocks each operation had to move, which copies must exist, and what content
(request, block, version) every copy must hold.

The policy of the background step is part of what is modelled: requests are visited in arrival
order, starting after the last request the previous step looked at; within a request, blocks in
logical order; a request whose blocks cannot get host blocks stops the step and is looked at again
next time.
"""

OK = 0
ERR_INVALID_ARG = -1
ERR_NOMEM = -7


class _Req:
    def __init__(self, tokens, nblocks):
        self.tokens = tokens
        self.on_gpu = True
        self.version = [1] * nblocks          # content version of each logical block
        self.host_version = [None] * nblocks  # version held by the host copy, None = no host block

    def host_valid(self, i):
        return self.host_version[i] == self.version[i]


class BlockTableModel:
    def __init__(self, num_gpu_blocks, num_host_blocks, block_size):
        self.bs = block_size
        self.free_gpu = num_gpu_blocks
        self.free_host = num_host_blocks
        self.reqs = {}
        self.order = []
        self.cursor = 0
        self.eager_blocks = self.preempt_blocks_moved = self.discarded_blocks = self.resume_blocks_moved = 0

    def nblocks(self, tokens):
        return -(-tokens // self.bs)

    def full(self, r, i):
        return (i + 1) * self.bs <= r.tokens

    # ---- requests
    def add(self, rid, tokens):
        if tokens <= 0 or rid in self.reqs:
            return ERR_INVALID_ARG
        n = self.nblocks(tokens)
        if n > self.free_gpu:
            return ERR_NOMEM
        self.free_gpu -= n
        self.reqs[rid] = _Req(tokens, n)
        self.order.append(rid)
        return OK

    def append(self, rid, new_tokens):
        r = self.reqs.get(rid)
        if r is None or not r.on_gpu or new_tokens <= 0:
            return ERR_INVALID_ARG
        have, want = len(r.version), self.nblocks(r.tokens + new_tokens)
        if want - have > self.free_gpu:
            return ERR_NOMEM
        if r.tokens % self.bs != 0:
            r.version[-1] += 1                # tokens land in the dirty block: any host copy of it goes stale
        self.free_gpu -= want - have
        r.version += [1] * (want - have)
        r.host_version += [None] * (want - have)
        r.tokens += new_tokens
        return OK

    def finish(self, rid):
        r = self.reqs.pop(rid, None)
        if r is None:
            return ERR_INVALID_ARG
        if r.on_gpu:
            self.free_gpu += len(r.version)
        self.free_host += sum(1 for v in r.host_version if v is not None)
        pos = self.order.index(rid)
        self.order.remove(rid)
        if self.cursor > pos:
            self.cursor -= 1
        self.cursor = self.cursor % len(self.order) if self.order else 0
        return OK

    # ---- background copies of full blocks
    def eager(self, max_blocks):
        """Returns the list of (request, logical block) copied to host memory in this step."""
        picked, n, visited = [], len(self.order), 0
        while visited < n and len(picked) < max_blocks:
            rid = self.order[(self.cursor + visited) % n]
            r = self.reqs[rid]
            if r.on_gpu:
                idx = [i for i in range(len(r.version)) if self.full(r, i) and not r.host_valid(i)]
                idx = idx[:max_blocks - len(picked)]
                new_host = sum(1 for i in idx if r.host_version[i] is None)
                if new_host > self.free_host:
                    break
                self.free_host -= new_host
                picked += [(rid, i) for i in idx]
            visited += 1
        if n:
            self.cursor = (self.cursor + visited) % n
        for rid, i in picked:
            r = self.reqs[rid]
            r.host_version[i] = r.version[i]
        self.eager_blocks += len(picked)
        return picked

    # ---- rotation of whole requests
    def rotate(self, preempt, resume):
        """Returns (status, blocks sent out, blocks brought in)."""
        if len(set(preempt)) != len(preempt) or len(set(resume)) != len(resume):
            return ERR_INVALID_ARG, 0, 0
        for rid in preempt:
            if rid not in self.reqs or not self.reqs[rid].on_gpu:
                return ERR_INVALID_ARG, 0, 0
        for rid in resume:
            if rid not in self.reqs or self.reqs[rid].on_gpu:
                return ERR_INVALID_ARG, 0, 0
        discard = sum(1 for rid in preempt for i in range(len(self.reqs[rid].version)) if self.reqs[rid].host_valid(i))
        send = sum(1 for rid in preempt for i in range(len(self.reqs[rid].version)) if not self.reqs[rid].host_valid(i))
        new_host = sum(1 for rid in preempt for i, v in enumerate(self.reqs[rid].host_version)
                       if v is None and not self.reqs[rid].host_valid(i))
        bring = sum(len(self.reqs[rid].version) for rid in resume)
        if bring > self.free_gpu + discard or new_host > self.free_host:
            return ERR_NOMEM, 0, 0
        self.free_host -= new_host
        self.free_gpu += discard + send - bring
        for rid in preempt:
            r = self.reqs[rid]
            r.host_version = list(r.version)
            r.on_gpu = False
        for rid in resume:
            self.reqs[rid].on_gpu = True
        self.discarded_blocks += discard
        self.preempt_blocks_moved += send
        self.resume_blocks_moved += bring
        return OK, send, bring

    # ---- what must be true of a request now
    def info(self, rid):
        r = self.reqs[rid]
        n = len(r.version)
        return {"tokens": r.tokens, "num_blocks": n, "on_gpu": int(r.on_gpu),
                "synced_blocks": sum(1 for i in range(n) if r.host_valid(i)),
                "host_blocks": sum(1 for v in r.host_version if v is not None),
                "dirty_blocks": sum(1 for i in range(n) if not self.full(r, i))}
