"""Full-size benchmark configurations: CUDA path vs the CPU oracle on the same seeded inputs,
in the launch configuration bench.py times."""
import pytest

from paper_2509_24248_b200 import synth
from tests import harness, parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_chain_config(name):
    wl = synth.workload(name)
    rep = parity.run_chain(harness.build_case(wl, poison_tail=True))
    print(f"{name}: accept_len {rep.accept_len} exit {rep.exit_flag} exempt {rep.exempt} "
          f"signal err {rep.max_signal_err:.2e} hidden rel-L2 {rep.max_hidden_rel:.2e}")
    assert len(rep.exempt) <= max(2, wl.B * (wl.K + 1) // 10)


def test_tree_config4():
    wl = synth.workload("C4")
    rep = parity.run_tree(harness.build_case(wl, poison_tail=True))
    print(f"C4: accept_len {rep.accept_len} exit {rep.exit_flag} exempt {rep.exempt} "
          f"signal err {rep.max_signal_err:.2e} hidden rel-L2 {rep.max_hidden_rel:.2e}")


def test_chain_config1_with_a_32k_draft_vocabulary():
    """C1's shapes with the draft head reduced to 32768 ids (id map + the target's own head)."""
    import dataclasses
    wl = synth.workload("C1")
    wl = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, Vd=32768))
    rep = parity.run_chain(harness.build_case(wl, poison_tail=True))
    print(f"C1/Vd=32768: accept_len {rep.accept_len} exempt {rep.exempt} "
          f"signal err {rep.max_signal_err:.2e} hidden rel-L2 {rep.max_hidden_rel:.2e}")
    assert len(rep.exempt) <= 2


def test_chain_config1_with_the_three_feature_layer_and_a_32k_draft_vocabulary():
    """C1's shapes in the EAGLE-3-like configuration: three-feature fusion, concatenated attention
    input, draft head over 32768 ids."""
    import dataclasses
    wl = synth.workload("C1")
    wl = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, Vd=32768, arch=1))
    rep = parity.run_chain(harness.build_case(wl, poison_tail=True))
    print(f"C1/fused3/Vd=32768: accept_len {rep.accept_len} exempt {rep.exempt} "
          f"signal err {rep.max_signal_err:.2e} hidden rel-L2 {rep.max_hidden_rel:.2e}")
    assert len(rep.exempt) <= 2


@pytest.mark.parametrize("sample_drafts", [False, True])
def test_chain_config1_with_stochastic_acceptance(sample_drafts):
    """C1's shapes with speculative sampling at temperature 1: the verify head's draws over the
    151936-token vocabulary (deterministic drafts), and the accept test with the residual draw
    (sampled drafts)."""
    from oracle import specexit_oracle as orc
    wl = synth.workload("C1")
    rep = parity.run_chain(harness.build_case(wl, poison_tail=True),
                           sample=orc.SampleCfg(1.0, 20250924, 3, sample_drafts))
    print(f"C1/tau=1/sampled drafts {sample_drafts}: accept_len {rep.accept_len} exempt {rep.exempt}")
    assert len(rep.exempt) <= 2
