"""The stored values under tests/golden/ (written by tests/golden/make_config1_step0.py from the
oracle alone) still come out of the oracle and the input generators as they stand."""
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _stored():
    rows, counts = [], None
    for line in open(os.path.join(HERE, "golden", "config1_step0.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if len(f) == 3 and "." in f[1]:
            rows.append((float(f[1]), float(f[2])))
        else:
            counts = [int(x) for x in f]
    return np.array(rows), counts


def test_oracle_reproduces_the_stored_configuration_1_values():
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_config1_step0",
                                                  os.path.join(HERE, "golden", "make_config1_step0.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    loss, psum, d = mod.compute()
    rows, counts = _stored()
    assert rows.shape == (8, 2)
    np.testing.assert_allclose(loss, rows[:, 0], rtol=1e-10)
    np.testing.assert_allclose(psum, rows[:, 1], rtol=1e-10)
    assert counts == [d["set_size"], d["intra_viol"], d["boundary_viol"]]
