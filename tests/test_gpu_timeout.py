"""The bounded device-side wait, made to run out on purpose - without hanging or
faulting anything.  The library's self-test kernel waits, through the very
routine every kernel of the engine uses, on a barrier that nothing arrives on,
with a limit of a millisecond; it must give up, set the workspace's status
word, and leave the context usable."""
import pytest
import torch

from paper_2405_16528_b200 import binding as L

pytestmark = pytest.mark.gpu


def test_wait_runs_out_and_is_reported():
    ws = L.new_workspace(256)
    L.loqt_device_status(ws)                       # clean to begin with
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    L.loqt_selftest_wait_timeout(ws, limit_us=1000)
    t1.record()
    with pytest.raises(L.LoqtError, match="timed out"):
        L.loqt_device_status(ws)
    words = ws.view(torch.int32)[:4].cpu().tolist()
    assert words[0] == 1                           # the status word the host maps to LOQT_ERR_TIMEOUT
    assert words[2] == 0, "a wait on a barrier without arrivals reported completion"
    assert words[3] == 1, "the CTA-wide abort flag was not raised"
    ms = t0.elapsed_time(t1)
    assert 0.9 <= ms < 100.0, f"the wait gave up after {ms:.2f} ms (limit 1 ms)"
    # the status word is sticky until the caller clears it; the context still works
    ws.zero_()
    L.loqt_device_status(ws)
    a = torch.ones(1024, device="cuda")
    assert float(a.sum()) == 1024.0


def test_selftest_argument_checks():
    ws = L.new_workspace(256)
    with pytest.raises(L.LoqtError, match="invalid"):
        L.loqt_selftest_wait_timeout(ws, limit_us=0)
    with pytest.raises(L.LoqtError, match="invalid"):
        L.loqt_selftest_wait_timeout(ws, limit_us=10_000_000)
