"""The checked build of the library (compiled with PREBA_CHECKED): every kernel tests its
shared-memory offsets, table indices and global addresses against their ranges before use and
reports a violation in the status word instead of making the access.  A few small cases per
kernel run under it in a process of their own (the binding loads one library per process): the
status word must stay 0 and the results must be the oracle's."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

CASES = r'''
import sys
import numpy as np
import torch
sys.path.insert(0, "{root}")
sys.path.insert(0, "{root}/tests")
import oracle
from oracle import antialias as oaa, audio as oa
from paper_2411_19114_b200 import binding as pb, workloads as wl
from helpers import MEAN, STD, run_gpu, oracle_f64, assert_parity

assert pb._LIB_PATH.name == "libpreba_checked.so"
rng = np.random.default_rng(5)
u = lambda h, w: wl.uniform_image(rng, h, w)
dev = torch.device("cuda:0")

# fused kernel: staged path (ragged sizes, partial column block, one row), direct path (wide)
imgs = wl.mixed_smooth(9, seed=31) + [u(1, 1), u(300, 7), u(5, 4000), u(64, 20000)]
for dt in (pb.F32, pb.F16):
    assert_parity(run_gpu(imgs, 224, 256, out_dtype=dt), oracle_f64(imgs, 224, 256), dt)
assert_parity(run_gpu(imgs[:5], 300, 301), oracle_f64(imgs[:5], 300, 301), pb.F32)
assert_parity(run_gpu(imgs[:5], 17, 40, dynamic=False), oracle_f64(imgs[:5], 17, 40), pb.F32)

# rounded uint8 variant with crop windows
n = 6
packed, table = pb.preba_pack(imgs[:n])
pix = torch.from_numpy(packed).to(dev)
tab = torch.from_numpy(table.view(np.uint8)).to(dev)
status = torch.zeros(1, dtype=torch.int32, device=dev)
origins = np.asarray([(i % 3, (5 * i) % 7) for i in range(n)], dtype=np.uint32)
crop = torch.from_numpy(origins.astype(np.int64)).to(dev).to(torch.int32).reshape(-1)
out8 = torch.empty((n, 224, 224, 3), dtype=torch.uint8, device=dev)
pb.preba_preprocess_ex(pix, tab, n, out8, 224, 256, MEAN, STD, pb.U8, round_u8=True,
                       crop_origin=crop, crop_origin_host=origins, table_host=table, status=status)
torch.cuda.synchronize()
assert int(status.item()) == 0, pb.preba_strerror(int(status.item()))
want8 = oracle.preprocess_ex(imgs[:n], 224, 256, MEAN, STD, oracle.OUT_U8_HWC, crop_origin=origins,
                             round_u8=True)
assert np.array_equal(out8.cpu().numpy(), want8)

# antialiased Resize: all its kernels (both passes on the tensor cores with windows of three and
# of four steps, the horizontal pass on them, the general one: widths that are and are not
# multiples of 4)
aa_imgs = [u(1080, 1920), u(1600, 1600), u(600, 808), u(700, 901), u(241, 499), u(100, 150),
           u(64, 2000)]
pk, tb = pb.preba_pack(aa_imgs)
out = torch.empty((len(aa_imgs), 3, 224, 224), dtype=torch.float32, device=dev)
for host in (tb, None):
    pb.preba_preprocess_antialias(torch.from_numpy(pk).to(dev), torch.from_numpy(tb.view(np.uint8)).to(dev),
                                  len(aa_imgs), out, 224, 256, MEAN, STD, pb.F32, table_host=host,
                                  status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, pb.preba_strerror(int(status.item()))
    err = float(np.max(np.abs(out.cpu().numpy() - oaa.preprocess(aa_imgs, 224, 256, MEAN, STD))))
    assert err <= 1e-5, err

# audio path
utts = wl.utterances(5, seed=6, min_s=0.2, max_s=2.0) + [np.zeros(399, dtype=np.float32),
                                                          rng.uniform(-1, 1, 561).astype(np.float32)]
pa, ta = pb.preba_audio_pack(utts)
t_max = int(ta["frames"].max())
feat = torch.empty((len(utts), 80, t_max), dtype=torch.float32, device=dev)
pb.preba_audio_logmel(torch.from_numpy(pa).to(dev), torch.from_numpy(ta.view(np.uint8)).to(dev),
                      len(utts), t_max, feat, True, table_host=ta, status=status)
torch.cuda.synchronize()
assert int(status.item()) == 0, pb.preba_strerror(int(status.item()))
err = float(np.max(np.abs(feat.cpu().numpy().astype(np.float64) - oa.preprocess(utts))))
assert err <= 3e-4, err
print("checked build: all cases clean")
'''


@pytest.mark.gpu
def test_small_cases_run_clean_under_the_checked_build():
    from paper_2411_19114_b200 import build as pbuild

    pbuild.build(checked=True)
    env = dict(os.environ, PREBA_CHECKED_BUILD="1")
    done = subprocess.run([sys.executable, "-c", CASES.replace("{root}", str(ROOT))], env=env,
                          capture_output=True, text=True, timeout=900)
    assert done.returncode == 0, done.stdout[-2000:] + done.stderr[-4000:]
    assert "all cases clean" in done.stdout


def test_range_code_has_a_text():
    from paper_2411_19114_b200 import binding as pb

    assert "checked build" in pb.preba_strerror(pb.ERR_RANGE)
