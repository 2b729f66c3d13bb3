"""Host arithmetic of the increasing batch-size schedule (Section 5.2.2) and of the workload tables."""
import pytest

from paper_2108_01624_b200 import synth
from paper_2108_01624_b200.schedule import increasing_batch_size, microbatches_for_step


def test_schedule_matches_the_paper():
    """262,144 -> 1,048,576 over 7,500 steps, +196,608 (~196k) every quarter of the ramp."""
    assert increasing_batch_size(0) == 262_144 and increasing_batch_size(1874) == 262_144
    assert increasing_batch_size(1875) == 262_144 + 196_608
    assert increasing_batch_size(3750) == 262_144 + 2 * 196_608
    assert increasing_batch_size(5625) == 262_144 + 3 * 196_608
    assert increasing_batch_size(7499) == 262_144 + 3 * 196_608
    assert increasing_batch_size(7500) == 1_048_576 == increasing_batch_size(20_000)
    qs = [increasing_batch_size(t) for t in range(0, 20_000, 125)]
    assert qs == sorted(qs)
    assert all(q % 256 == 0 for q in qs)
    assert microbatches_for_step(0, 256) == 1024 and microbatches_for_step(7500, 256) == 4096
    with pytest.raises(ValueError):
        microbatches_for_step(0, 1000)
    # fewer examples than a fixed 1M batch over the 7,500-step ramp
    ramp = sum(increasing_batch_size(t) for t in range(7500))
    assert ramp < 7500 * 1_048_576 and ramp > 7500 * 262_144


def test_workload_parameter_counts():
    assert synth.workload("tiny_linear").n_params() == 64 * 64 + 64
    assert synth.workload("bert_base_layer").n_params() == 7_087_872
    assert synth.workload("bert_large").n_params() == 333_563_904
    wl = synth.workload("bert_large_megabatch")
    assert wl.microbatches * wl.B == 2_097_152          # the paper's largest batch
    emb = synth.workload("bert_large_embeddings")
    assert emb.n_params() == (30522 + 512 + 2) * 1024 + 2 * 1024


def test_synthetic_ids_follow_their_recipes():
    wl = synth.workload("bert_large_embeddings")
    data = synth.generate(wl, seed=0, device="cpu", B=64)
    tok, pos, typ = data[0].ids, data[1].ids, data[2].ids
    assert int(tok.min()) >= 0 and int(tok.max()) < 30522
    assert 0.10 < float((tok == 0).float().mean()) < 0.18          # Zipf(1.1): id 0 carries ~14 % of the tokens
    distinct = sum(len(set(r.tolist())) for r in tok) / 64
    assert 60 < distinct < 105                                      # ~82 distinct ids per 128-token example
    assert (pos == pos[0]).all() and pos[0].tolist() == list(range(128))
    assert set(typ.unique().tolist()) <= {0, 1} and (typ[:, 1:] >= typ[:, :-1]).all()
    # G scaled so that norms straddle C = 1: s_i in [0.1, 10]
    s = synth.example_scales(1000, 0, 0, "cpu")
    assert 0.1 <= float(s.min()) and float(s.max()) <= 10.0 and 0.3 < float((s > 1).float().mean()) < 0.7
