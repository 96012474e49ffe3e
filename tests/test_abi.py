"""The C-ABI library builds, loads and exports every entry point the header declares
(no compute: runs without a GPU)."""
import ctypes
import os
import re


def declared(repo_root):
    text = open(os.path.join(repo_root, "include", "gto.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gto_[a-z_]+)\s*\(", text)))


def struct_body(text, name):
    end = text.index("} %s;" % name)
    return text[text.rindex("typedef struct {", 0, end):end]


def test_library_exports_every_declared_symbol(repo_root):
    from paper_2509_22134_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared(repo_root)
    assert {"gto_build_tree", "gto_tree_reward", "gto_group_surrogate_grad", "gto_create",
            "gto_destroy", "gto_device_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in gto.h but not exported"


def test_binding_has_the_same_names_and_status_strings(repo_root):
    from paper_2509_22134_b200 import binding
    for n in declared(repo_root):
        assert hasattr(binding, n), n
    assert binding.gto_status_string(0) == "ok"
    assert "non-finite" in binding.gto_status_string(5)


def test_config_struct_matches_header_layout(repo_root):
    from paper_2509_22134_b200 import binding
    text = open(os.path.join(repo_root, "include", "gto.h")).read()
    body = struct_body(text, "gto_config")
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b(?:int32_t|float|uint32_t)\s+(\w+);", body)
    assert fields == [f[0] for f in binding.gto_config._fields_]
    for struct, cname in ((binding.gto_tree, "gto_tree"), (binding.gto_reward, "gto_reward"),
                          (binding.gto_grad_stats, "gto_grad_stats")):
        body = struct_body(text, cname)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        fields = re.findall(r"\*\s*(\w+);", body)
        assert fields == [f[0] for f in struct._fields_], cname


def test_invalid_arguments_are_refused_without_a_device(repo_root):
    from paper_2509_22134_b200 import binding as gto
    import pytest
    for kw in (dict(m=3), dict(g=10 ** 6), dict(k=0)):
        args = dict(B=8, D=3, k=4, g=12, m=8, V_draft=512, V_target=512, dtype="f32")
        args.update(kw)
        with pytest.raises(gto.GtoError) as e:
            gto.gto_create(gto.make_config(**args), 0)
        assert e.value.code == 1
    with pytest.raises(gto.GtoError) as e:
        gto.gto_create(gto.make_config(8, 3, 12, 12, 8, 512, 512, "f32"), 0)   # k*k > 128
    assert e.value.code == 2


def test_sample_groups_matches_the_oracle_on_the_host(repo_root):
    """Host logic of SampleGroups (Algorithm 1, Eq. 6-7): the library against the oracle."""
    import numpy as np
    import pytest
    from oracle import gto_oracle as orc
    from paper_2509_22134_b200 import binding as gto
    rng = np.random.default_rng(3)
    for _ in range(300):
        s, m = int(rng.integers(1, 400)), int(rng.integers(1, 33))
        K = int(rng.integers(0, s // m + 1))
        u = rng.random(K)
        assert gto.gto_sample_groups(s, m, K, u) == orc.sample_groups(s, m, K, u)
    assert gto.gto_sample_groups(2048, 8, 16, [0.999999] * 16) == [2048 - 128 + 1 + 8 * i for i in range(16)]
    with pytest.raises(gto.GtoError):
        gto.gto_sample_groups(10, 4, 3, [0.1, 0.2, 0.3])          # K*m > s
    with pytest.raises(gto.GtoError):
        gto.gto_sample_groups(10, 4, 1, [1.0])                    # not in [0, 1)
