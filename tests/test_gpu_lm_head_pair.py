"""The optional two-SM shape of the fused LM-head consensus (ORTHRUS_LM_HEAD_PAIR=1: CTA pairs
sharing 256-row items through tcgen05.mma.cta_group::2) is chosen when the library is first
used in a process, so its parity run happens in a child process: the cases of
test_gpu_lm_head_consensus.py with more than 128 rows, full size included, plus the rest
(which must be unaffected) with the variable set."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_parity_with_cta_pairs():
    env = dict(os.environ, ORTHRUS_LM_HEAD_PAIR="1")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(HERE, "test_gpu_lm_head_consensus.py"),
                        "-x", "-q"], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
