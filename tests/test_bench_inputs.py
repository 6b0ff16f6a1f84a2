"""The benchmark's synthetic inputs are what the record says: the generator, run here,
reproduces the stored SHA-256 of the smaller tensors of the first benchmark shape."""
import os

from bench import inputs_match_record, tensor_sha256
from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "bench_inputs_sha256.txt")


def test_generator_reproduces_the_recorded_hashes():
    want = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            name, tensor, digest = line.split()
            want[(name, tensor)] = digest
    assert len(want) == 10
    cfg = CONFIGS["cfg3_7b_up"]
    shared = make_inputs(cfg, need=("A", "B"))
    for k in ("A", "B"):
        assert tensor_sha256(shared[k]) == want[("cfg3_7b_up", k)]


def test_a_changed_tensor_is_noticed():
    class S:
        pass
    cfg = CONFIGS["cfg3_7b_up"]
    shared = make_inputs(cfg, need=("A", "B"))
    s = S(); s.cfg = cfg
    s.sha256 = {k: tensor_sha256(v) for k, v in shared.items()}
    assert inputs_match_record([s]) is True
    shared["A"][0, 0] += 1
    s.sha256 = {k: tensor_sha256(v) for k, v in shared.items()}
    assert inputs_match_record([s]) is False
