"""The package's usage example runs and passes its own checks."""
import pytest

pytestmark = pytest.mark.gpu


def test_the_usage_example_runs(capsys):
    from paper_2511_16138_b200 import example
    example.main()
    assert "chunks restored and compared" in capsys.readouterr().out
