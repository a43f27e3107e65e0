"""End-to-end speculative decoding through the C ABI with the packaged loop driver (paper_2608_30252_b200.loop) on
a toy one-layer target and a toy memory-augmented draft: greedy speculative decoding must emit exactly the
target-only greedy sequence (Section 3.1 / Section 4.3: verification keeps the output unchanged), whatever the
draft proposes, including across rejections, rollbacks (Section 4.3, "Rollback"), slot materialisation at
boundaries and window eviction; and the emitted sequence is checked against a host-side copy of the same toy
target built from the oracle's verification attention.

The dense layers around the attention calls (embeddings, q/k/v projections, unembedding) are plain torch
matmuls: the backbone is outside the library.  Everything the library owns — draft memory update, draft
attention, verify attention, accept/reject, rollback — runs in its kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding
from paper_2608_30252_b200.loop import ToyDraft, ToyTarget, greedy_target_only, sd_speedup, speculative

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _oracle_margins(target, prompt, emitted):
    """A host-side copy of the toy target (same weights, fp64, attention = oracle.verify_attend over the bf16 cache
    values) scores every emitted position, teacher-forced on the emitted tokens.  Returns, per emitted token, how far
    the oracle's logit of that token lies below the oracle's best logit (0 where the oracle picks the same token)."""
    f = lambda t: t.double().cpu().numpy()
    E, Pos, Wq, Wk, Wv, Wu = map(f, (target.E, target.Pos, target.Wq, target.Wk, target.Wv, target.Wu))
    toks = list(prompt) + list(emitted[:-1])
    x = E[np.asarray(toks)] + Pos[: len(toks)]
    rb = oracle.round_to_bf16
    # the GPU side forms x W in fp32 and rounds to bf16: fp64 then bf16 differs from that on rare rounding ties only
    K = rb((x @ Wk).astype(np.float32).astype(np.float64)).reshape(1, -1, target.Hkv, target.D).transpose(0, 2, 1, 3)
    V = rb((x @ Wv).astype(np.float32).astype(np.float64)).reshape(1, -1, target.Hkv, target.D).transpose(0, 2, 1, 3)
    margins = []
    for i, tok in enumerate(emitted):
        n = len(prompt) + i                                   # cache entries this row sees: tokens 0 .. n-1
        q = rb((x[n - 1:n] @ Wq).astype(np.float32).astype(np.float64)).reshape(1, 1, target.Hq, target.D)
        o, _ = oracle.verify_attend(q, K[:, :, :n], V[:, :, :n], [n])
        logits = o.reshape(-1) @ Wu
        margins.append(float(logits.max() - logits[tok]))
    return margins


def test_greedy_speculative_decoding_equals_target_only_decoding():
    gen = torch.Generator(device=DEV); gen.manual_seed(2608)
    prompt = [3, 17, 5, 9, 22, 41, 8, 13, 2, 50]
    n = 60
    ref = greedy_target_only(ToyTarget(torch.Generator(device=DEV).manual_seed(1)), prompt, n)
    for gamma in (3, 5):
        # (a) the memory-augmented draft's own proposals (a different random model: mostly rejected)
        res = speculative(ToyTarget(torch.Generator(device=DEV).manual_seed(1)),
                          ToyDraft(torch.Generator(device=DEV).manual_seed(7)), prompt, n, gamma)
        assert res.tokens == ref and res.status == 0, (gamma, "draft")
        assert res.tok_per_iter == sum(res.accepted) / len(res.accepted) + 1
        assert res.t_d_us > 0 and res.t_t_us > 0
        assert abs(res.eq1_speedup - oracle.sd_speedup(res.tok_per_iter - 1, gamma, res.t_d_us, res.t_t_us)) < 1e-9
        # (b) proposals overwritten with the true continuation except every third one: long accepted runs,
        #     full acceptance (bonus token) and mid-block rejections all occur
        res2 = speculative(ToyTarget(torch.Generator(device=DEV).manual_seed(1)),
                           ToyDraft(torch.Generator(device=DEV).manual_seed(7)), prompt, n, gamma,
                           spoil=_make_spoiler(ref, gamma))
        hist2 = res2.accepted
        assert res2.tokens == ref and res2.status == 0, (gamma, "spoiled")
        assert max(hist2) == gamma and min(hist2) < gamma and len(set(hist2)) >= 2
        assert res2.tok_per_iter > res.tok_per_iter          # the better draft emits more tokens per iteration (Eq. 1's numerator)
    # the oracle's copy of the toy target, teacher-forced on the emitted tokens: it picks the same token everywhere
    # except where its two best logits are closer than the bf16 rounding of the logits the decision was taken on
    margins = _oracle_margins(ToyTarget(torch.Generator(device=DEV).manual_seed(1)), prompt, ref)
    assert max(margins) <= 0.25, max(margins)
    assert sum(m == 0.0 for m in margins) >= 0.95 * len(margins)


def _make_spoiler(ref, gamma):
    """Replaces the draft's proposals by the true continuation, except that every (gamma + 2)-th proposal
    overall is wrong: the verifier then sees every accepted length including full acceptance."""
    state = {"emitted": 1, "count": 0, "iter": -1, "base": 1}

    def spoil(it, j, tok):
        if it != state["iter"]:
            state["iter"] = it
            state["base"] = state["emitted"]
        truth = ref[state["base"] + j] if state["base"] + j < len(ref) else 0
        state["count"] += 1
        wrong = state["count"] % (gamma + 2) == 0
        if j == gamma - 1:
            # the block is complete: the number of emitted tokens advances by accepted + 1
            acc = 0
            for jj in range(gamma):
                c = state["count"] - (gamma - 1) + jj
                if c % (gamma + 2) == 0:
                    break
                acc += 1
            state["emitted"] = state["base"] + acc + 1
        return (truth + 1) % 64 if wrong else truth

    return spoil
