"""CPU checks of the synthetic environment generator (the stand-in for the simulators in the closed actor
loop): the SplitMix64 function behind it against its published known-answer vector, and the structure of
what it returns."""
import os

import numpy as np

import gala_inputs as GI

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "splitmix64_seed_1234567.txt")


def test_splitmix64_known_answer_vector():
    want = [int(l) for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    state = np.uint64(1234567)
    got = []
    with np.errstate(over="ignore"):
        for _ in want:
            got.append(int(GI._sm64(state)))     # output k = mix(state + (k + 1) * gamma)
            state = state + np.uint64(0x9E3779B97F4A7C15)
    assert got == want


def test_environment_is_a_function_of_seed_agent_env_step():
    a = GI.synthetic_env(7, 2, 4, 11, 6, False, obs_dim=8, actions=np.array([0, 1, 2, 3]))
    b = GI.synthetic_env(7, 2, 4, 11, 6, False, obs_dim=8, actions=np.array([0, 1, 2, 3]))
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    assert a["obs"].shape == (4, 8) and a["obs"].dtype == np.float32
    assert np.abs(a["obs"]).max() <= np.float32(1.7320508)
    assert (a["uniforms"] >= 0).all() and (a["uniforms"] < 1).all()
    c = GI.synthetic_env(7, 2, 4, 12, 6, False, obs_dim=8)
    assert not np.array_equal(a["obs"], c["obs"])            # another step, another observation
    d = GI.synthetic_env(7, 3, 4, 11, 6, False, obs_dim=8)
    assert not np.array_equal(a["obs"], d["obs"])            # another agent likewise
    # environment e of a batch is the same whatever the batch size
    np.testing.assert_array_equal(GI.synthetic_env(7, 2, 2, 11, 6, False, obs_dim=8)["obs"], a["obs"][:2])


def test_environment_statistics():
    fr = GI.synthetic_env(1, 0, 2, 0, 6, True)["obs"]
    assert fr.shape == (2, 84, 84, 4) and fr.dtype == np.uint8
    assert abs(fr.mean() - 127.5) < 1.0                       # bytes uniform over 0..255
    steps = 4000
    acts = np.zeros(8, np.int64)
    r = np.concatenate([GI.synthetic_env(3, 0, 8, s, 4, False, actions=acts)["rewards"] for s in range(steps)])
    d = np.concatenate([GI.synthetic_env(3, 0, 8, s, 4, False, actions=acts)["dones"] for s in range(steps)])
    n = r.size
    assert abs(r.mean() - 0.25) < 4 * np.sqrt(0.25 * 0.75 / n)     # a fixed action hits the target 1 time in A
    assert abs(d.mean() - 0.01) < 4 * np.sqrt(0.01 * 0.99 / n)
    assert set(np.unique(r)) <= {0.0, 1.0}
