"""Several sequences in one pass (a context of batch > 1) against the CPU oracle, sequence by sequence
(needs a B200).  Each sequence has its own prompt length, cache, drafted tree and accepted length."""
import copy

import pytest
import torch

import synth
from helpers import block_for, orc, prompt_tokens
from lockstep import TARGET, BatchLockstep
from test_gpu_parity import FULL_WIDTH_TOL, _write_report

pytestmark = pytest.mark.gpu


def _oracle_continuation(ls, look, depth):
    """The oracle's own greedy continuation from a sequence's current state (one-token passes)."""
    st = copy.deepcopy(ls.st)
    cont = []
    for _ in range(depth):
        cont += orc.bita_step(ls.model, look, st, [])["out_tokens"]
    return cont


def test_batch_lockstep_tiny_ragged():
    """Three sequences with prompts of 64 / 23 / 75 tokens, 10 passes together.  On some passes some
    sequences get the oracle's own continuation planted on a path (so they accept several drafts)
    while the others verify their own drafts: accepted lengths, cache lengths and compaction differ
    per sequence and per pass, and each sequence must match its own oracle run."""
    shape = synth.CONFIGS["tiny"]
    seed = 0x5EED0031
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    B = 3
    prompts = [prompt_tokens(seed + b, n, shape.V) for b, n in enumerate((64, 23, 75))]
    bl = BatchLockstep(shape, seed, tmpl, B, C_max=256)
    bl.prefill(prompts)
    look = block_for(synth.empty_template(), shape.n_mask)
    depth = max(tmpl.depths())
    lens = []
    for step in range(10):
        trees = []
        for b, ls in enumerate(bl.seqs):
            base = list(ls.st.tree)
            if (step + b) % 3 == 1:
                cont = _oracle_continuation(ls, look, depth)
                base = synth.plant_tree(tmpl, base, cont, seed, 16 * step + b, 1.1, shape.V)
            trees.append(base)
        recs = bl.step(trees)
        lens.append(tuple(r["n_out"] for r in recs))
        for r in recs:
            assert r["status"] == 0 and 1 <= r["n_out"] <= depth + 1
    assert len({n for t in lens for n in t}) > 1               # the sequences really accepted different lengths
    assert any(len(set(t)) > 1 for t in lens)                  # ... within one pass too
    assert [ls.st.C for ls in bl.seqs] == [len(p) + sum(t[b] for t in lens) for b, p in enumerate(prompts)]
    for ls in bl.seqs:
        assert ls.max_logit <= TARGET.logit_rms and ls.max_hidden_acc <= TARGET.hidden_rel_l2
        _write_report(ls)
    bl.close()


def test_batch_of_one_sequence_equals_the_single_sequence_calls():
    """A batch context with one sequence is the batch-1 context: same records, bit for bit."""
    from paper_2401_12522_b200 import Bita
    shape = synth.CONFIGS["tiny"]
    w = synth.make_weights(shape, 7, dtype=torch.bfloat16, device="cuda:0")
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    prompt = prompt_tokens(7, 30, shape.V)
    a = Bita(shape, w, tmpl, C_max=256)
    b = Bita(shape, w, tmpl, C_max=256, batch=1)
    ra = [a.prefill(prompt)] + [a.step() for _ in range(4)]
    rb = [b.prefill(prompt, seq=0)] + [b.step_batch()[0] for _ in range(4)]
    assert ra == rb
    a.close()
    b.close()


def test_sequences_do_not_interfere():
    """What a sequence emits does not depend on its neighbours in the block: sequence 0 decoded next
    to two other sequences emits what it emits alone (up to sub-tolerance ties, which the oracle
    lockstep covers; here the tokens are compared directly and must agree on a clear-margin run)."""
    from paper_2401_12522_b200 import Bita
    shape = synth.CONFIGS["tiny"]
    seed = 0x5EED0003
    w = synth.make_weights(shape, seed, dtype=torch.bfloat16, device="cuda:0")
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    prompts = [prompt_tokens(seed + b, n, shape.V) for b, n in enumerate((40, 64, 17))]
    alone = Bita(shape, w, tmpl, C_max=256)
    seq_alone = list(alone.prefill(prompts[0])["out_tokens"])
    for _ in range(6):
        seq_alone += alone.step()["out_tokens"]
    alone.close()
    tog = Bita(shape, w, tmpl, C_max=256, batch=3)
    seqs = [list(tog.prefill(p, seq=b)["out_tokens"]) for b, p in enumerate(prompts)]
    for _ in range(6):
        for b, r in enumerate(tog.step_batch()):
            seqs[b] += r["out_tokens"]
    tog.close()
    n = min(len(seq_alone), len(seqs[0]))
    same = sum(x == y for x, y in zip(seq_alone[:n], seqs[0][:n]))
    assert same >= n - 1, (seq_alone, seqs[0])                 # at most one sub-tolerance tie may flip a token
    assert len({tuple(s) for s in seqs}) == 3                  # and the three sequences are different sequences


def test_batch_errors():
    from paper_2401_12522_b200 import Bita, BitaError
    shape = synth.CONFIGS["tiny"]
    w = synth.make_weights(shape, 5, dtype=torch.bfloat16, device="cuda:0")
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    b = Bita(shape, w, tmpl, C_max=128, batch=2)
    b.prefill(prompt_tokens(5, 20, shape.V), seq=0)
    with pytest.raises(BitaError) as e:
        b.step_batch()
    assert e.value.code == -7                                  # sequence 1 was never prefilled
    with pytest.raises(BitaError) as e:
        b.prefill(prompt_tokens(5, 20, shape.V), seq=2)
    assert e.value.code == -1
    with pytest.raises(BitaError) as e:
        b.step()
    assert e.value.code == -1                                  # the single-sequence call on a batch context
    b.prefill(prompt_tokens(6, 31, shape.V), seq=1)
    recs = b.step_batch()
    assert [r["status"] for r in recs] == [0, 0]
    assert recs[0]["new_len"] == 20 + recs[0]["n_out"] and recs[1]["new_len"] == 31 + recs[1]["n_out"]
    b.reset()
    with pytest.raises(BitaError) as e:
        b.step_batch()
    assert e.value.code == -7
    b.close()


@pytest.mark.parametrize("name,batch,prompt_lens", [("7b", 4, (90, 150, 33, 120)), ("70b", 2, (70, 40))])
def test_batch_full_width_lockstep(name, batch, prompt_lens):
    """The measured model widths with several 69-row sequences in one block (4 x 69 = 276 rows at the
    7B width: two MMA column halves, one CTA per SM; GQA at the 70B width), depth cut to one layer
    so that the fp64 oracle finishes in seconds; sequence 1 gets the oracle's continuation planted."""
    shape = synth.CONFIGS[name].with_layers(1)
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    seed = 0x5EED0032
    prompts = [prompt_tokens(seed + b, n, shape.V) for b, n in enumerate(prompt_lens)]
    bl = BatchLockstep(shape, seed, tmpl, batch, C_max=max(prompt_lens) + 160, lazy_oracle=True,
                       tol=FULL_WIDTH_TOL[shape.name])
    bl.prefill(prompts)
    look = block_for(synth.empty_template(), shape.n_mask)
    bl.step(None)
    trees = [list(ls.st.tree) for ls in bl.seqs]
    cont = _oracle_continuation(bl.seqs[1], look, 2)
    trees[1] = synth.plant_tree(tmpl, trees[1], cont, seed, 1, 1.1, shape.V)
    recs = bl.step(trees)
    assert recs[1]["n_out"] >= 2
    for ls in bl.seqs:
        _write_report(ls)
    bl.close()


def test_rewind_of_one_sequence_leaves_the_others_alone():
    """bita_rewind_seq cuts one sequence back to an earlier state: that sequence then repeats the pass it
    took from there (same drafts, same record), the other one carries on from where it was."""
    from paper_2401_12522_b200 import Bita
    shape = synth.CONFIGS["tiny"]
    w = synth.make_weights(shape, 9, dtype=torch.bfloat16, device="cuda:0")
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    b = Bita(shape, w, tmpl, C_max=256, batch=2)
    first = [b.prefill(prompt_tokens(9 + s, n, shape.V), seq=s) for s, n in enumerate((30, 41))]
    r1 = b.step_batch([first[0]["next_tree"], first[1]["next_tree"]])
    # sequence 1 back to the state after its first pass; sequence 0 stays where the pass left it
    b.rewind(first[1]["new_len"], first[1]["out_tokens"][-1], seq=1)
    r2 = b.step_batch([r1[0]["next_tree"], first[1]["next_tree"]])
    assert r2[1] == r1[1]                                      # the same pass again, bit for bit
    assert r2[0]["new_len"] == r1[0]["new_len"] + r2[0]["n_out"]
    b.close()
