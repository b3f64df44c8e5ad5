"""CPU-side checks of the CUDA library: it loads, exports what the header declares, its host
control plane (iteration times, Algorithm 3, validation) agrees with the oracle.  No kernel runs."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import policy as opolicy
from paper_2009_05766_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "netmax.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(netmax_[a-z_]+)\s*\(", header)))
    assert len(declared) >= 20
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTS) == declared


def test_binding_config_matches_the_header_field_by_field(tmp_path):
    """The ctypes mirror of netmax_config must have the C compiler's layout: a small C program that
    includes the header prints the size of the struct and the offset of every field."""
    import subprocess
    fields = [name for name, _ in binding.Config._fields_]
    src = tmp_path / "layout.c"
    lines = ['#include <stddef.h>', '#include <stdio.h>', f'#include "{os.path.join(ROOT, "include", "netmax.h")}"',
             'int main(void) {', '  printf("%zu\\n", sizeof(netmax_config));']
    lines += [f'  printf("%zu\\n", offsetof(netmax_config, {f}));' for f in fields]
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-o", str(exe), str(src)], check=True)
    out = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert out[0] == C.sizeof(binding.Config)
    assert out[1:] == [getattr(binding.Config, f).offset for f in fields]
    header = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "netmax.h")).read(), flags=re.S)
    body = re.search(r"typedef struct netmax_config \{(.*?)\} netmax_config;", header, flags=re.S).group(1)
    declared = re.findall(r"\b([A-Za-z_0-9]+)\s*(?:,|;)", body)
    assert declared == fields      # every field of the header is mirrored, in order


def test_iteration_times_match_oracle():
    for idx in (1, 2, 3, 4):
        w = workloads.config(idx)
        s = w.link_speeds(0)
        t, adj = binding.netmax_iteration_times(s, w.d)
        t0, adj0 = opolicy.iteration_times(s, w.d)
        np.testing.assert_allclose(t, t0, rtol=1e-15)
        assert (adj == adj0).all()


def _policy_case(name):
    if name.startswith("cfg"):
        w = workloads.config(int(name[3]))
        K, R = {1: (20, 20), 2: (10, 10), 3: (6, 6), 4: (3, 3)}[w.index]
        return opolicy.iteration_times(w.link_speeds(1 if w.index == 3 else 0), w.d) + (w.lr, K, R)
    rng = np.random.default_rng(5)
    M = 7
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(50.0), (M, M))), 1)
    s[0, 4] = s[1, 5] = s[2, 6] = 0.0
    return opolicy.iteration_times(s + s.T, 1_000_000) + (0.05, 8, 8)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "sparse7"])
def test_policy_generator_matches_oracle(name):
    t, adj, lr, K, R = _policy_case(name)
    P, rho, info = binding.netmax_policy_generate(t, adj, lr, K, R)
    P0, rho0, info0 = opolicy.generate_policy(t, adj, lr, K, R)
    assert (info["k"], info["r"]) == (info0["k"], info0["r"])
    assert rho == pytest.approx(rho0, rel=1e-14)
    np.testing.assert_allclose(P, P0, atol=1e-9)
    assert info["lam2"] == pytest.approx(info0["lam2"], abs=1e-9)
    assert info["t_conv"] == pytest.approx(info0["t_conv"], rel=1e-6)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-12)


def test_lanczos_path_of_the_library_agrees_with_dense_eigenvalues():
    """M > 96 switches the library's lambda_2 to Lanczos; the oracle uses a dense solver."""
    M = 128
    rng = np.random.default_rng(9)
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(100.0), (M, M))), 1)
    t, adj = opolicy.iteration_times(s + s.T, 1_000_000)
    P, rho, info = binding.netmax_policy_generate(t, adj, 0.05, 2, 2)
    Y = opolicy.y_matrix(P, opolicy.node_probabilities(P, t, adj), adj, 0.05, rho)
    assert info["lam2"] == pytest.approx(np.linalg.eigvalsh(Y)[-2], abs=1e-9)


def test_policy_generate_rejects_bad_arguments():
    t, adj = opolicy.iteration_times(np.ones((3, 3)) - np.eye(3), 100)
    with pytest.raises(binding.NetmaxError) as e:
        binding.netmax_policy_generate(t, adj, -0.1, 4, 4)
    assert e.value.code == -1
    lone = adj.copy()
    lone[0, :] = lone[:, 0] = 0
    with pytest.raises(binding.NetmaxError) as e:
        binding.netmax_policy_generate(t, lone, 0.1, 4, 4)
    assert e.value.code == -6
    with pytest.raises(binding.NetmaxError) as e:
        binding.netmax_iteration_times(np.zeros((3, 3)), 10)
    assert e.value.code == -6


def test_create_validates_before_touching_the_gpu():
    M = 3
    good = np.array([[0, .5, .5], [.5, 0, .5], [.5, .5, 0]])
    cases = [
        (dict(M=1, d=8, lr=0.1, prob=None), -1),
        (dict(M=M, d=0, lr=0.1, prob=good), -1),
        (dict(M=M, d=8, lr=0.0, prob=good), -1),
        (dict(M=M, d=8, lr=0.1, prob=good, sigma=-1.0), -1),
        (dict(M=M, d=8, lr=0.1, prob=good, objective=2), -1),
        (dict(M=M, d=8, lr=0.1, prob=good, trace_rounds=0), -1),
        (dict(M=M, d=8, lr=0.1, prob=good, rho=2.6), -1),        # Eq. 11: alpha rho (d_im + d_mi) = 0.52 > p_im = 0.5
        (dict(M=M, d=8, lr=0.1, prob=good * 0.9), -2),
        (dict(M=M, d=8, lr=0.1, prob=np.array([[0, 1.5, -.5], [.5, 0, .5], [.5, .5, 0]])), -2),
        (dict(M=M, d=8, lr=0.1, prob=good, link_speed_gbps=np.array([[0, 1, 0], [1, 0, 1], [0, 1, 0.]])), -2),
        (dict(M=M, d=8, lr=0.1, prob=None, link_speed_gbps=np.array([[0, 1, 0], [1, 0, 0], [0, 0, 0.]])), -6),
    ]
    for kw, code in cases:
        with pytest.raises(binding.NetmaxError) as e:
            binding.Netmax(**kw)
        assert e.value.code == code, (kw, str(e.value))


def test_rho_beyond_eq_11_is_named_and_a_fixed_weight_or_the_floor_itself_passes(gpu_available):
    good = np.array([[0, .5, .5], [.5, 0, .5], [.5, .5, 0]])
    with pytest.raises(binding.NetmaxError) as e:
        binding.Netmax(M=3, d=8, lr=0.1, prob=good, rho=2.6)
    assert e.value.code == -1 and "Eq. 11" in str(e.value) and "(0,1)" in str(e.value)
    # on the floor (w = 1/2, Eq. 11 taken closed) and with a fixed pull weight (rho unused) validation
    # passes: without a GPU the call then fails later, at the device
    for kw in (dict(rho=2.5), dict(rho=50.0, pull_weight=0.5)):
        try:
            binding.Netmax(M=3, d=8, lr=0.1, prob=good, **kw).close()
        except binding.NetmaxError as err:
            assert not gpu_available and err.code == -4, str(err)


def test_null_context_calls_return_errors_not_crashes():
    L = binding.lib()
    assert L.netmax_round(None, 1) == -1
    assert L.netmax_read_replicas(None, None) == -1
    assert L.netmax_rounds_done(None) == -1
    assert L.netmax_create_ex(None, None) == -1
    L.netmax_destroy(None)
    size = binding.Netmax.workspace_size(8, 1000, 16)
    assert size >= 3 * 8 * 1024 * 4 and size % 256 == 0


def test_product_path_fails_loudly_without_a_gpu(gpu_available):
    if gpu_available:
        pytest.skip("a GPU is present")
    good = np.array([[0, 1.0], [1.0, 0]])
    with pytest.raises(binding.NetmaxError) as e:
        binding.Netmax(M=2, d=8, lr=0.1, prob=good)
    assert e.value.code == -4


def test_explicit_rho_grid_matches_oracle_and_is_more_adaptive():
    """The printed U_rho = 0.5/alpha with a coarse K leaves one feasible rho, smaller than the default
    grid's choice, and a policy that prefers the fast links more."""
    w = workloads.config(2)
    t, adj = opolicy.iteration_times(w.link_speeds(0), w.d)
    P, rho, info = binding.netmax_policy_generate(t, adj, w.lr, 10, 10, rho_upper=0.5 / w.lr)
    P0, rho0, info0 = opolicy.generate_policy(t, adj, w.lr, 10, 10, rho_upper=0.5 / w.lr)
    assert (info["k"], info["r"]) == (info0["k"], info0["r"]) and rho == pytest.approx(rho0, rel=1e-14)
    np.testing.assert_allclose(P, P0, atol=1e-9)
    Pd, rhod, _ = binding.netmax_policy_generate(t, adj, w.lr, 10, 10)
    assert rho < rhod
    fast, slow = P[0, 1], P[0, 5]
    assert fast / slow > Pd[0, 1] / Pd[0, 5] > 1.0


def test_the_allocation_free_entry_point_names_no_allocating_call():
    """netmax_read_columns_static promises to call no cudaMalloc / cudaFree: its body and the
    helper that looks up the static array's address must not name one."""
    src = open(os.path.join(ROOT, "paper_2009_05766_b200", "csrc", "netmax.cu")).read()
    for start in ("int netmax_read_columns_static(", "static int gather_scratch_address("):
        at = src.index(start)
        body = src[at:src.index("\n}\n", at)]
        assert "cudaGetSymbolAddress" in body or "gather_scratch_address" in body
        for banned in ("cudaMalloc", "cudaFree", "cudaHostAlloc", "cudaMallocAsync", "new ", "std::vector"):
            assert banned not in body, (start, banned)


# ---- constant pull weight (the paper's extension section)
def _fixed_case(name):
    if name.startswith("cfg"):
        w = workloads.config(int(name[3]))
        return opolicy.iteration_times(w.link_speeds(0), w.d)
    rng = np.random.default_rng(5)
    M = 7
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(50.0), (M, M))), 1)
    s[0, 4] = s[1, 5] = s[2, 6] = 0.0
    return opolicy.iteration_times(s + s.T, 1_000_000)


@pytest.mark.parametrize("name,floor_upper,K,R", [("cfg1", 0.0, 6, 6), ("cfg1", 0.1, 4, 4), ("cfg2", 0.0, 6, 6),
                                                  ("cfg2", 0.3 / 7, 6, 6), ("cfg3", 0.0, 3, 4), ("cfg3", 0.02, 4, 4),
                                                  ("sparse7", 0.0, 3, 3), ("sparse7", 0.05, 3, 3)])
def test_fixed_weight_generator_matches_oracle(name, floor_upper, K, R):
    t, adj = _fixed_case(name)
    P, phi, info = binding.netmax_policy_generate_fixed_weight(t, adj, 0.5, K, R, floor_upper)
    P0, phi0, info0 = opolicy.generate_policy_fixed_weight(t, adj, 0.5, K, R, floor_upper=floor_upper)
    assert (info["k"], info["r"]) == (info0["k"], info0["r"]) and phi == pytest.approx(phi0, rel=1e-14)
    np.testing.assert_allclose(P, P0, atol=1e-8)
    assert info["lam2"] == pytest.approx(info0["lam2"], abs=1e-9)
    assert info["t_conv"] == pytest.approx(info0["t_conv"], rel=1e-6)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-9)
    np.testing.assert_allclose(P.sum(axis=0), 1.0, atol=1e-9)


def test_fixed_weight_grid_points_match_oracle_and_report_infeasibility():
    t, adj = _fixed_case("cfg2")
    M = t.shape[0]
    mean_time = float(t[0][adj[0] == 1].mean())
    for phi, frac in ((0.02, 0.6), (0.05, 0.9), (0.1, 1.0), (1.0 / 7, 1.0)):
        P = binding.netmax_policy_fixed_weight_at(t, adj, phi, frac * mean_time / M)
        P0 = opolicy.solve_fixed_weight(t, adj, phi, frac * mean_time)
        np.testing.assert_allclose(P, P0, atol=1e-8)
    with pytest.raises(binding.NetmaxError) as e:           # faster than the intra-machine links allow
        binding.netmax_policy_fixed_weight_at(t, adj, 0.02, 0.5 * float(t[0, 1]) / M)
    assert e.value.code == -7
    assert opolicy.solve_fixed_weight(t, adj, 0.02, 0.5 * float(t[0, 1])) is None
    with pytest.raises(binding.NetmaxError) as e:           # floors beyond a row sum of one
        binding.netmax_policy_fixed_weight_at(t, adj, 0.2, mean_time / M)
    assert e.value.code == -7
    with pytest.raises(binding.NetmaxError) as e:
        binding.netmax_policy_generate_fixed_weight(t, adj, 1.0, 4, 4)
    assert e.value.code == -1
    one_way = adj.copy()
    one_way[0, 1] = 0
    with pytest.raises(binding.NetmaxError) as e:
        binding.netmax_policy_generate_fixed_weight(t, one_way, 0.5, 4, 4)
    assert e.value.code == -1
