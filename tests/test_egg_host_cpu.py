"""Host-side logic of the integer training step (no GPU): the update threshold, the step-size schedule and the ids
of the perturbed matrices, against hand-worked values."""
import os

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_update_threshold_matches_the_hand_worked_values():
    from paper_2511_16652_b200 import egg
    rows = 0
    for line in open(os.path.join(GOLD, "int8_update_threshold.txt")):
        if line.startswith("#") or not line.strip():
            continue
        t = line.split()
        alpha, K, zi, ki, thr = float(t[0]), int(t[1]), int(t[3]), int(t[5]), int(t[6])
        assert zi * ki == thr
        assert egg.update_threshold(alpha, K) == thr, (alpha, K)
        rows += 1
    assert rows == 5


def test_alpha_schedule_and_matrix_ids():
    from paper_2511_16652_b200 import egg
    assert egg.alpha_schedule(0) == 1.0
    assert abs(egg.alpha_schedule(200) - 0.25) < 1e-15          # 1 / (0.015 * 200 + 1)
    assert egg.SLOTS == {"Wf": 0, "Uf": 1, "Wh": 2, "Uh": 3, "mlp1": 4, "mlp2": 5}

    class _T:                                                   # stands in for a [layers, ...] tensor
        def __init__(self, n): self.shape = (n,)
        def __getitem__(self, i): return ("view", i)

    params = {k: _T(3) for k in ("ln1", "Wf", "Uf", "Wh", "Uh", "mlp1", "mlp2")}
    params["emb_t"], params["head"] = "E", "H"
    ids = [lid for _, lid in egg.perturbed_matrices(params)]
    assert ids == [0, 1, 2, 3, 4, 5, 16, 17, 18, 19, 20, 21, 32, 33, 34, 35, 36, 37, 1000, 1001]
