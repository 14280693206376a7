"""Host-side checks of the C ABI: the library builds, loads, exports every function include/gear.h
declares, and its host-only entry points validate their arguments.  No GPU needed."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gb():
    from paper_1806_03925_b200 import build
    build.build()
    from paper_1806_03925_b200 import binding
    binding.load()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gear_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(gb):
    names = declared_functions()
    assert len(names) >= 10
    lib = C.CDLL(gb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(gb.EXPORTS)


def test_workspace_bytes_and_config_validation(gb):
    cfg = gb.make_config(10_000, 10_000, 5_000, 16, 64, gb.GEAR_F32, gb.GEAR_F32, [64], 4, 1000, 256, 1024)
    n = gb.gear_workspace_bytes(cfg)
    assert n > 0 and n % 256 == 0
    bigger = gb.make_config(10_000, 10_000, 5_000, 16, 64, gb.GEAR_F32, gb.GEAR_F32, [64], 4, 1000, 512, 2048)
    assert gb.gear_workspace_bytes(bigger) > n
    for bad in (dict(emb_dim=15), dict(dfv_dim=4), dict(M=0), dict(expire=-1), dict(max_batch=0), dict(hidden=[63]),
                dict(img_vocab=2**31), dict(hidden=[64, 64, 64][:0])):
        kw = dict(user_vocab=100, url_vocab=100, img_vocab=100, emb_dim=16, dfv_dim=64, dfv_dtype=0, head_dtype=0,
                  hidden=[64], M=4, expire=0, max_batch=8, max_nnz=32)
        kw.update(bad)
        with pytest.raises(gb.GearError) as e:
            gb.gear_workspace_bytes(gb.make_config(**kw))
        assert e.value.code == gb.GEAR_ERR_ARG
        assert gb.load().gear_last_error()


def test_bf16_head_wants_wider_alignment(gb):
    ok = gb.make_config(100, 100, 100, 32, 128, gb.GEAR_BF16, gb.GEAR_BF16, [256, 128], 16, 0, 64, 512)
    assert gb.gear_workspace_bytes(ok) > 0
    with pytest.raises(gb.GearError):
        gb.gear_workspace_bytes(gb.make_config(100, 100, 100, 32, 128, gb.GEAR_BF16, gb.GEAR_BF16, [40], 16, 0, 64, 512))


def test_null_ctx_is_a_state_error(gb):
    assert gb.load().gear_status(None, None, None) == gb.GEAR_ERR_STATE
    assert gb.load().gear_destroy(None) == gb.GEAR_OK


def test_binding_refuses_host_tensors(gb):
    import torch
    with pytest.raises(TypeError):
        gb.gear_fill_uniform(torch.zeros((4, 4)), 0, 1)


def test_struct_layouts_of_the_binding_match_the_header(gb, tmp_path):
    """The ctypes structures of the binding against the C compiler's view of include/gear.h: same size, and every
    field at the same offset (a field added to the header and not to the binding would shift everything behind it)."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    structs = {"gear_config": gb.gear_config, "gear_buffers": gb.gear_buffers, "gear_batch": gb.gear_batch,
               "gear_adam": gb.gear_adam, "gear_step_out": gb.gear_step_out}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "gear.h"', 'int main(void) {']
    for name, st in structs.items():
        lines.append('  printf("%s %%zu\\n", sizeof(%s));' % (name, name))
        for field, _ in st._fields_:
            lines.append('  printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (name, field, name, field))
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines) + "\n")
    exe = tmp_path / "layout"
    subprocess.check_call([cc, "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    seen = dict(line.split() for line in subprocess.check_output([str(exe)], text=True).splitlines())
    for name, st in structs.items():
        assert int(seen[name]) == C.sizeof(st), name
        for field, _ in st._fields_:
            assert int(seen["%s.%s" % (name, field)]) == getattr(st, field).offset, "%s.%s" % (name, field)
    # every field of the header's structures is known to the binding
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "gear.h")).read(), flags=re.S)
    for name, st in structs.items():
        body = re.search(r"typedef struct \{([^}]*)\}\s*%s;" % name, text).group(1)
        fields = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            names = decl.split(",")
            names[0] = names[0].split()[-1]                      # drop the type of the first declarator
            fields += [re.sub(r"\[.*\]", "", n).strip().lstrip("*").strip() for n in names]
        assert fields == [f for f, _ in st._fields_], (name, fields)
