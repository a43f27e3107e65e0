"""The speculative-decoding iteration as a driver around the C ABI (Section 3.1; Section 4.3, "Rollback").

One iteration: the draft runs L_draft autoregressive steps over its memory-augmented cache (per layer: raw-KV
append + attention in one launch, the whole boundary step in one launch when a memory slot is due), the
target scores the last emitted token and the L_draft proposals in one parallel pass over its full cache, the
accept/reject rule keeps a prefix and emits one target token, and the draft memory is rolled back to the
accepted position.  The driver counts emitted tokens per iteration (Tok./Iter), times the draft step (t_d)
and the target pass (t_t, and the target's one-token pass for the autoregressive baseline) with CUDA events,
and evaluates Eq. 1 from those measurements.

The models here are toys: a one-layer target and a one-layer memory-augmented draft whose dense parts
(embeddings, q/k/v projections, unembedding) are plain torch matmuls with seeded random weights, because the
backbone is outside the library.  Everything the library owns runs in its kernels: draft memory update, draft
attention, slot materialisation, verify attention, accept/reject, rollback.  With temperature 0 the emitted
sequence must equal the target's own greedy decoding, whatever the draft proposes.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding


class ToyTarget:
    """One attention layer between an embedding and an unembedding; K/V cache [1, Hkv, cap, D] bf16."""

    def __init__(self, gen, V=64, Hq=8, Hkv=2, D=128, cap=512, device="cuda"):
        d = 256
        self.V, self.Hq, self.Hkv, self.D, self.cap, self.d, self.dev = V, Hq, Hkv, D, cap, d, device
        r = lambda *s: torch.randn(*s, generator=gen, device=device)
        self.E, self.Pos = r(V, d), r(cap, d) * 0.5
        self.Wq, self.Wk, self.Wv = r(d, Hq * D) / d ** 0.5, r(d, Hkv * D) / d ** 0.5, r(d, Hkv * D) / d ** 0.5
        self.Wu = r(Hq * D, V) * 2.0
        self.K = torch.zeros((1, Hkv, cap, D), dtype=torch.bfloat16, device=device)
        self.Vc = torch.zeros_like(self.K)
        self.n = 0                                      # tokens whose K/V are in the cache
        self.ws = {}

    def logits_rows(self, tokens):
        """Append `tokens` to the cache and return their next-token logits rows (bf16).  A long run of tokens (the
        prompt) goes through in chunks of as many rows as one verification call takes."""
        rows_max = 64 // (self.Hq // self.Hkv)
        if len(tokens) > rows_max:
            return torch.cat([self.logits_rows(tokens[i:i + rows_max]) for i in range(0, len(tokens), rows_max)])
        T = len(tokens)
        pos = torch.arange(self.n, self.n + T, device=self.dev)
        x = self.E[torch.tensor(tokens, device=self.dev)] + self.Pos[pos]
        k = (x @ self.Wk).view(T, self.Hkv, self.D).to(torch.bfloat16)
        v = (x @ self.Wv).view(T, self.Hkv, self.D).to(torch.bfloat16)
        self.K[0, :, self.n:self.n + T] = k.permute(1, 0, 2)
        self.Vc[0, :, self.n:self.n + T] = v.permute(1, 0, 2)
        q = (x @ self.Wq).view(1, T, self.Hq, self.D).to(torch.bfloat16).contiguous()
        kv_len = torch.tensor([self.n + T], dtype=torch.int32, device=self.dev)
        if T not in self.ws:
            self.ws[T] = binding.verify_workspace(self.K, kv_len, self.Hq, T)
        o, _ = binding.verify_attend(self.K, self.Vc, kv_len, q, workspace=self.ws[T])
        self.n += T
        return (o.view(T, -1) @ self.Wu).to(torch.bfloat16)

    def truncate(self, n):
        self.n = n


class ToyDraft:
    """A one-layer draft over the three-part memory: sinks, slots (the adaptor is a copy of the K/V projections
    applied to the mean of the chunk's inputs, standing in for the slot token's hidden state), local window."""

    def __init__(self, gen, V=64, Hq=8, Hkv=2, D=64, S=2, W=8, r=4, max_pos=512, device="cuda"):
        d = Hq * D
        self.V, self.Hq, self.Hkv, self.D, self.S, self.W, self.r, self.d, self.dev = V, Hq, Hkv, D, S, W, r, d, device
        rn = lambda *s: torch.randn(*s, generator=gen, device=device)
        self.E, self.Pos = rn(V, d), rn(max_pos, d) * 0.5
        self.Wq, self.Wk, self.Wv = rn(d, Hq * D) / d ** 0.5, rn(d, Hkv * D) / d ** 0.5, rn(d, Hkv * D) / d ** 0.5
        self.Wkg, self.Wvg = self.Wk.to(torch.bfloat16).contiguous(), self.Wv.to(torch.bfloat16).contiguous()   # copy-init
        self.Wu = rn(Hq * D, V) * 2.0
        cfg = binding.MaswConfig(1, 1, Hq, Hkv, D, d, S, W, r, rollback=8, max_slots=max(128, max_pos // r + 8), gamma_max=8)
        self.mem = binding.DraftMemory(cfg, device)
        self.t = 0                                      # committed tokens (host mirror)
        self.slots = 0

    def step(self, tokens):
        """Feed the pending tokens (their positions are t .. t+n-1), return the arg-max next token after the
        last.  The tokens go in chunks that end at slot boundaries (and hold at most 4 tokens)."""
        nxt = None
        while tokens:
            n = 1
            while n < min(len(tokens), 4) and not self._boundary(self.t + n):
                n += 1
            nxt = self._step_chunk(tokens[:n])
            tokens = tokens[n:]
        return nxt

    def _boundary(self, t_after):
        return t_after > self.S and (t_after - self.S) % self.r == 0

    def _step_chunk(self, tokens):
        n = len(tokens)
        pos = torch.arange(self.t, self.t + n, device=self.dev)
        x = self.E[torch.tensor(tokens, device=self.dev)] + self.Pos[pos]
        k = (x @ self.Wk).view(1, n, self.Hkv, self.D).to(torch.bfloat16).contiguous()
        v = (x @ self.Wv).view(1, n, self.Hkv, self.D).to(torch.bfloat16).contiguous()
        t_after = self.t + n
        boundary = self._boundary(t_after)
        if boundary:      # raw append + slot materialisation + both kinds of rows in one launch
            h_g = x.mean(0, keepdim=True).to(torch.bfloat16).contiguous()
            q = torch.cat([x @ self.Wq, h_g.float() @ self.Wq]).view(1, -1, self.Hq, self.D).to(torch.bfloat16).contiguous()
            o, _ = self.mem.draft_boundary_attend(0, k, v, h_g, self.Wkg, self.Wvg,
                                                  torch.tensor([t_after], dtype=torch.int32, device=self.dev), q)
        else:
            q = (x @ self.Wq).view(1, -1, self.Hq, self.D).to(torch.bfloat16).contiguous()
            o, _ = self.mem.draft_append_attend(0, k, v, q)
        self.mem.mem_advance(n, add_slot=boundary, deferred=True)   # applied by the next rollback (or state read)
        self.t = t_after
        self.slots += int(boundary)
        logits = o[0, n - 1].reshape(-1) @ self.Wu
        return int(torch.argmax(logits))

    def rollback(self, t_keep):
        slots_keep = max(0, t_keep - self.S) // self.r
        self.mem.mem_rollback(torch.tensor([t_keep], dtype=torch.int32, device=self.dev),
                              torch.tensor([slots_keep], dtype=torch.int32, device=self.dev), slots_keep_max=slots_keep)
        self.t, self.slots = t_keep, slots_keep


def greedy_target_only(target, prompt, n, timer=None):
    """The target's own greedy decoding (the sequence speculative decoding must reproduce)."""
    rows = target.logits_rows(prompt)
    out = [int(torch.argmax(rows[-1].float()))]
    while len(out) < n:
        if timer is not None:
            timer.start()
        row = target.logits_rows([out[-1]])
        if timer is not None:
            timer.stop()
        out.append(int(torch.argmax(row[0].float())))
    return out


def sd_speedup(l_acc, l_draft, t_d, t_t):
    """Eq. 1: speedup over standard decoding = (L_acc + 1) / (L_draft t_d / t_t + 1)."""
    return (l_acc + 1.0) / (l_draft * (t_d / t_t) + 1.0)


class EventTimer:
    """Accumulates CUDA-event intervals on the current stream; `mean_us()` synchronises."""

    def __init__(self):
        self.pairs = []

    def start(self):
        self._e0 = torch.cuda.Event(enable_timing=True)
        self._e0.record()

    def stop(self):
        e1 = torch.cuda.Event(enable_timing=True)
        e1.record()
        self.pairs.append((self._e0, e1))

    def mean_us(self):
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in self.pairs) * 1e3 / max(len(self.pairs), 1)


@dataclasses.dataclass
class LoopResult:
    tokens: list            # emitted tokens (the first comes from the prefill pass)
    accepted: list          # accepted proposals per iteration
    tok_per_iter: float     # emitted tokens per iteration = mean accepted + 1
    t_d_us: float           # measured time of one draft step
    t_t_us: float           # measured time of one verification pass (gamma + 1 rows)
    eq1_speedup: float      # Eq. 1 with the measured L_acc, t_d and t_t
    status: int             # the draft memory's device status word


def speculative(target, draft, prompt, n, gamma, spoil=None):
    """Greedy speculative decoding of `n` tokens after `prompt`.  `spoil(iteration, j, token)` may overwrite the
    draft's j-th proposal (tests use it to force every accepted length).  Returns a LoopResult."""
    rows = target.logits_rows(prompt)                       # prefill (all prompt tokens cached)
    emitted = [int(torch.argmax(rows[-1].float()))]
    draft.step(prompt)                                      # draft-side prefill through the same update path, chunked
    pending = [emitted[-1]]                                 # tokens the draft has not processed yet
    iters, accepted_hist = 0, []
    t_draft, t_target = EventTimer(), EventTimer()
    dev = target.dev
    while len(emitted) < n:
        t0 = draft.t
        props = []
        feed = list(pending)
        for j in range(gamma):
            t_draft.start()
            tok = draft.step(feed)
            t_draft.stop()
            if spoil is not None:
                tok = spoil(iters, j, tok)
            props.append(tok)
            feed = [tok]
        n_cached = target.n
        t_target.start()
        rows = target.logits_rows([emitted[-1]] + props)    # gamma + 1 rows: last emitted token + the proposals
        t_target.stop()
        n_acc, out = binding.accept_reject(rows.view(1, gamma + 1, -1).contiguous(), None,
                                           torch.tensor([props], dtype=torch.int32, device=dev), None, 0.0)
        n_acc = int(n_acc.item())
        new = [int(x) for x in out[0, : n_acc + 1].tolist()]
        emitted += new
        accepted_hist.append(n_acc)
        target.truncate(n_cached + 1 + n_acc)               # keep the last emitted token and the accepted proposals
        # the draft keeps the tokens it processed that are still on the accepted path: pending + accepted[:gamma-1]
        keep = t0 + len(pending) + min(n_acc, gamma - 1)
        draft.rollback(keep)
        pending = ([props[-1]] if n_acc == gamma else []) + [new[-1]]
        iters += 1
    _, _, status = draft.mem.mem_get_state()
    l_acc = sum(accepted_hist) / max(len(accepted_hist), 1)
    t_d, t_t = t_draft.mean_us(), t_target.mean_us()
    return LoopResult(emitted[:n], accepted_hist, l_acc + 1.0, t_d, t_t, sd_speedup(l_acc, gamma, t_d, t_t), status)
